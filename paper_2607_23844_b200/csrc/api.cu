// The C-ABI layer: argument validation, context, launch bookkeeping, Layered Cache store, and the
// host-buffer convenience call.  No kernel lives here.
#include <math.h>
#include <string.h>

#include <new>

#include <algorithm>
#include <cmath>
#include "common.cuh"

namespace oc {

// ---- launch bookkeeping ------------------------------------------------------------------------
static cudaEvent_t take_event(oc_ctx* c) {
    if (!c->free_events.empty()) { cudaEvent_t e = c->free_events.back(); c->free_events.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
    return e;
}

LaunchScope::LaunchScope(oc_ctx* c, int kernel, cudaStream_t stream) : ctx(c), k(kernel), s(stream) {
    ctx->prof[k].launches += 1;
    if (ctx->profile_on) {
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(s, &cap) != cudaSuccess) { cudaGetLastError(); cap = cudaStreamCaptureStatusNone; }
        capturing = cap == cudaStreamCaptureStatusActive;
        e0 = take_event(ctx); e1 = take_event(ctx);
        // in a capture the records become event-record nodes of the graph (external events), so that the
        // bracket is taken again on every replay
        if (e0 && e1) cudaEventRecordWithFlags(e0, s, capturing ? cudaEventRecordExternal : cudaEventRecordDefault);
    }
}
LaunchScope::~LaunchScope() {
    if (e0 && e1) {
        cudaEventRecordWithFlags(e1, s, capturing ? cudaEventRecordExternal : cudaEventRecordDefault);
        if (capturing) ctx->prof[k].captured.emplace_back(e0, e1);
        else ctx->prof[k].pending.emplace_back(e0, e1);
    } else {
        if (e0) ctx->free_events.push_back(e0);
        if (e1) ctx->free_events.push_back(e1);
    }
}

// ---- geometry ----------------------------------------------------------------------------------
oc_status make_geo(const oc_layout* L, Geo* g) {
    if (!L || !g) return OC_ERR_INVALID_ARG;
    if (L->kind < OC_KIND_TOKEN || L->kind > OC_KIND_BLOCK) return OC_ERR_INVALID_ARG;
    if (L->dtype != OC_DTYPE_F32 && L->dtype != OC_DTYPE_BF16) return OC_ERR_INVALID_ARG;
    if (L->B <= 0 || L->T <= 0 || L->H <= 0 || L->W <= 0 || L->C <= 0) return OC_ERR_INVALID_ARG;
    if (!(L->eps >= 0.0f) || !isfinite(L->eps)) return OC_ERR_INVALID_ARG;
    g->kind = L->kind; g->dtype = L->dtype; g->B = L->B; g->T = L->T; g->H = L->H; g->W = L->W; g->C = L->C;
    g->sy = L->sy; g->sx = L->sx; g->oy = L->oy; g->ox = L->ox; g->gy = L->gy; g->gx = L->gx;
    g->self_match = L->self_match ? 1 : 0; g->frame_stat = L->frame_stat; g->eps = L->eps;
    g->elem_bytes = L->dtype == OC_DTYPE_F32 ? 4 : 2;
    if (((int64_t)L->C * g->elem_bytes) % 16 != 0) return OC_ERR_ALIGNMENT;
    const int64_t n_tok = (int64_t)L->B * L->T * L->H * L->W;
    if (n_tok > 0x7FFFFFFFll) return OC_ERR_UNSUPPORTED;
    if (L->kind == OC_KIND_FRAME) {
        if (L->frame_stat != OC_FRAME_MEAN_POS_COS && L->frame_stat != OC_FRAME_FLAT_COS) return OC_ERR_INVALID_ARG;
        // patch-local Frame Cache (Section 3.3): gy x gx equal patches per frame, one group per
        // patch position of a batch element; a layout that leaves gy = gx = 0 means whole frames
        g->gy = L->gy > 0 ? L->gy : 1; g->gx = L->gx > 0 ? L->gx : 1;
        if (L->gy < 0 || L->gx < 0 || L->H % g->gy != 0 || L->W % g->gx != 0) return OC_ERR_INVALID_ARG;
        g->sy = g->sx = 1; g->oy = g->ox = 0; g->self_match = 0;
        g->Hp = L->H / g->gy; g->Wp = L->W / g->gx; g->Hs = g->Hp; g->Ws = g->Wp;
        g->n_groups = (int64_t)L->B * g->gy * g->gx; g->units_per_group = L->T; g->reps_per_group = (L->T + 1) / 2;
        g->n_units = g->n_groups * L->T;
        if (g->n_units > 0x7FFFFFFFll) return OC_ERR_UNSUPPORTED;
        return OC_OK;
    }
    if (L->gy <= 0 || L->gx <= 0) return OC_ERR_INVALID_ARG;
    if (L->kind == OC_KIND_BLOCK && L->self_match) return OC_ERR_INVALID_ARG;
    if (L->H % L->gy != 0 || L->W % L->gx != 0) return OC_ERR_INVALID_ARG;
    g->Hp = L->H / L->gy; g->Wp = L->W / L->gx;
    if (g->self_match) {
        if (L->gy != 1 || L->gx != 1) return OC_ERR_UNSUPPORTED;
        g->sy = g->sx = 1; g->oy = g->ox = 0;
        g->Hs = g->Hp; g->Ws = g->Wp;
    } else {
        if (L->sy <= 0 || L->sx <= 0 || (int64_t)L->sy * L->sx < 2) return OC_ERR_INVALID_ARG;
        if (L->oy < 0 || L->oy >= L->sy || L->ox < 0 || L->ox >= L->sx) return OC_ERR_INVALID_ARG;
        if (g->Hp % L->sy != 0 || g->Wp % L->sx != 0) return OC_ERR_INVALID_ARG;
        g->Hs = g->Hp / L->sy; g->Ws = g->Wp / L->sx;
    }
    if (L->kind == OC_KIND_TOKEN) {
        g->n_groups = (int64_t)L->B * L->T * L->gy * L->gx;
        g->units_per_group = (int64_t)g->Hp * g->Wp;
        g->reps_per_group = (int64_t)g->Hs * g->Ws;
    } else {
        // a patch confines the selection; matching stays inside the sy x sx neighbourhood, which a
        // patch never cuts (Hp % sy == 0, Wp % sx == 0 above)
        g->n_groups = (int64_t)L->B * L->gy * L->gx;
        g->units_per_group = (int64_t)g->Hp * g->Wp;
        g->reps_per_group = (int64_t)g->Hs * g->Ws;
        if ((int64_t)L->H * L->W * L->B > 0x7FFFFFFFll) return OC_ERR_UNSUPPORTED;
    }
    g->n_units = g->n_groups * g->units_per_group;
    return OC_OK;
}

GroupMap make_group_map(const Geo& g) {
    GroupMap m;
    m.kind = g.kind; m.self_match = g.self_match; m.H = g.H; m.W = g.W; m.gy = g.gy; m.gx = g.gx;
    m.Hp = g.Hp; m.Wp = g.Wp; m.sy = g.sy; m.sx = g.sx; m.oy = g.oy; m.ox = g.ox;
    m.units_per_group = (int)g.units_per_group;
    m.frames = nullptr; m.n_reuse_single = 0;
    return m;
}

static oc_status check_rows(const oc_rows* r) {
    if (!r) return OC_ERR_INVALID_ARG;
    if (r->seg_bytes <= 0 || r->n_seg <= 0 || r->unit_pitch <= 0 || r->units_per_outer <= 0) return OC_ERR_INVALID_ARG;
    if (r->seg_stride < 0 || r->outer_pitch < 0) return OC_ERR_INVALID_ARG;
    if ((r->seg_bytes | r->seg_stride | r->unit_pitch | r->outer_pitch) & 15) return OC_ERR_ALIGNMENT;
    if (r->n_seg > 65535 || r->seg_bytes * r->n_seg > (1ll << 34)) return OC_ERR_UNSUPPORTED;
    return OC_OK;
}

static inline bool misaligned(const void* p) { return ((uintptr_t)p & 15u) != 0; }

}  // namespace oc

using namespace oc;

extern "C" {

const char* oc_status_str(oc_status s) {
    switch (s) {
        case OC_OK: return "OC_OK";
        case OC_ERR_INVALID_ARG: return "OC_ERR_INVALID_ARG";
        case OC_ERR_ALIGNMENT: return "OC_ERR_ALIGNMENT";
        case OC_ERR_UNSUPPORTED: return "OC_ERR_UNSUPPORTED";
        case OC_ERR_WORKSPACE: return "OC_ERR_WORKSPACE";
        case OC_ERR_CUDA: return "OC_ERR_CUDA";
        case OC_ERR_TIMEOUT: return "OC_ERR_TIMEOUT";
        case OC_ERR_OOM: return "OC_ERR_OOM";
        case OC_CACHE_MISS: return "OC_CACHE_MISS";
        default: return "OC_UNKNOWN_STATUS";
    }
}

const char* oc_kernel_name(int k) {
    static const char* names[OC_K_COUNT] = {"norms", "match_tc", "match_simt", "match_finalize", "frame_pair",
                                            "frame_finalize", "block_partial", "block_finalize", "select",
                                            "gather", "restore", "copy", "linear"};
    return (k >= 0 && k < OC_K_COUNT) ? names[k] : "unknown";
}

oc_status oc_layout_check(const oc_layout* layout) {
    Geo g;
    return make_geo(layout, &g);
}

oc_status oc_layout_counts(const oc_layout* layout, int64_t* n_groups, int64_t* units_per_group,
                           int64_t* reps_per_group) {
    Geo g;
    oc_status st = make_geo(layout, &g);
    if (st != OC_OK) return st;
    if (n_groups) *n_groups = g.n_groups;
    if (units_per_group) *units_per_group = g.units_per_group;
    if (reps_per_group) *reps_per_group = g.reps_per_group;
    return OC_OK;
}

oc_status oc_match_workspace_bytes(const oc_layout* layout, size_t* bytes) {
    if (!bytes) return OC_ERR_INVALID_ARG;
    Geo g;
    oc_status st = make_geo(layout, &g);
    if (st != OC_OK) return st;
    *bytes = match_workspace_bytes(g);
    return OC_OK;
}

oc_status oc_rows_from_layout(const oc_layout* layout, int channels, int elem_bytes, oc_rows* rows) {
    if (!rows || channels <= 0 || (elem_bytes != 1 && elem_bytes != 2 && elem_bytes != 4 && elem_bytes != 8))
        return OC_ERR_INVALID_ARG;
    Geo g;
    oc_status st = make_geo(layout, &g);
    if (st != OC_OK) return st;
    const int64_t cb = (int64_t)channels * elem_bytes;
    if (cb % 16 != 0) return OC_ERR_ALIGNMENT;
    const int64_t P = (int64_t)g.H * g.W;
    if (g.kind == OC_KIND_TOKEN) {
        *rows = oc_rows{cb, 1, 0, cb, (int64_t)1 << 40, 0};
    } else if (g.kind == OC_KIND_FRAME) {
        if (g.gy * g.gx == 1) *rows = oc_rows{P * cb, 1, 0, P * cb, (int64_t)1 << 40, 0};
        // a patch of a frame: Hp segments of Wp*C' elements; the gx patches of a patch row sit side by
        // side and patch rows follow one another at one pitch through frames and batch elements
        else *rows = oc_rows{g.Wp * cb, g.Hp, (int64_t)g.W * cb, g.Wp * cb, g.gx, (int64_t)g.Hp * g.W * cb};
    } else {
        *rows = oc_rows{cb, g.T, P * cb, cb, P, (int64_t)g.T * P * cb};
    }
    return OC_OK;
}

int oc_layer_cache_would_hit(int stored_step, int step, int interval) {
    const long long d = (long long)step - (long long)stored_step;
    return d >= 0 && d < (long long)interval;
}

// ---- context -----------------------------------------------------------------------------------
oc_status oc_create(oc_ctx** out, int device, size_t workspace_bytes) {
    if (!out || device < 0) return OC_ERR_INVALID_ARG;
    *out = nullptr;
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || device >= n) { cudaGetLastError(); return OC_ERR_CUDA; }
    DeviceGuard guard(device);
    if (!guard.ok) return OC_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return OC_ERR_CUDA;
    if (prop.major != 10) return OC_ERR_UNSUPPORTED;      // the kernels are built for sm_100a only
    oc_ctx* c = new (std::nothrow) oc_ctx();
    if (!c) return OC_ERR_OOM;
    c->device = device; c->sm_count = prop.multiProcessorCount;
    if (cudaMalloc(&c->d_status, 256) != cudaSuccess) { delete c; cudaGetLastError(); return OC_ERR_OOM; }
    cudaMemset(c->d_status, 0, 256);
    if (cudaMalloc(&c->d_span, 512 * sizeof(unsigned long long)) != cudaSuccess) {
        cudaFree(c->d_status); delete c; cudaGetLastError(); return OC_ERR_OOM;
    }
    cudaMemset(c->d_span, 0, 512 * sizeof(unsigned long long));
    if (workspace_bytes) {
        if (cudaMalloc(&c->workspace, workspace_bytes) != cudaSuccess) {
            cudaGetLastError();
            cudaFree(c->d_span); cudaFree(c->d_status); delete c;
            return OC_ERR_OOM;
        }
        c->workspace_bytes = workspace_bytes;
    }
    *out = c;
    return OC_OK;
}

oc_status oc_destroy(oc_ctx* c) {
    if (!c) return OC_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    cudaDeviceSynchronize();
    for (auto& kv : c->layers) cudaFree(kv.second.ptr);
    for (int k = 0; k < OC_K_COUNT; ++k) {
        for (auto& p : c->prof[k].pending) { cudaEventDestroy(p.first); cudaEventDestroy(p.second); }
        for (auto& p : c->prof[k].captured) { cudaEventDestroy(p.first); cudaEventDestroy(p.second); }
    }
    for (auto e : c->free_events) cudaEventDestroy(e);
    cudaFree(c->stage);
    cudaFree(c->workspace);
    for (auto e : c->chunk_events) cudaEventDestroy(e);
    if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
    cudaFree(c->d_span);
    cudaFree(c->d_status);
    delete c;
    return cuda_ok(cudaGetLastError());
}

oc_status oc_device_status(oc_ctx* c, int* code) {
    if (!c || !code) return OC_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    int v = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return OC_ERR_CUDA;
    if (cudaMemcpy(&v, c->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return OC_ERR_CUDA;
    if (v != 0) cudaMemset(c->d_status, 0, sizeof(int));
    *code = v;
    return OC_OK;
}

oc_status oc_selftest_per_device_once(int n_devices, int n_rounds, int fail_dev, int* runs, int* ok) {
    if (n_devices < 1 || n_devices > oc::PerDeviceOnce::MAX_DEV || n_rounds < 1 || !runs || !ok) return OC_ERR_INVALID_ARG;
    oc::PerDeviceOnce once;
    for (int d = 0; d < n_devices; ++d) { runs[d] = 0; ok[d] = 0; }
    for (int r = 0; r < n_rounds; ++r)
        for (int d = 0; d < n_devices; ++d)
            if (once.ensure(d, [&] { ++runs[d]; return d != fail_dev; })) ++ok[d];
    return OC_OK;
}

oc_status oc_selftest_bounded_wait(oc_ctx* c, unsigned int limit_us, void* stream) {
    if (!c || limit_us == 0 || limit_us > 1000000u) return OC_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return OC_ERR_CUDA;
    return launch_bounded_wait_selftest(c, (unsigned long long)limit_us * 1000ull, (cudaStream_t)stream);
}

oc_status oc_tc_plan_override(oc_ctx* c, int on, int pair, int tiles_per_cta, int pieces_per_row, int single_accumulator,
                              int candidates_resident) {
    if (!c) return OC_ERR_INVALID_ARG;
    if (on && ((pair != 0 && pair != 1) || (tiles_per_cta != 1 && tiles_per_cta != 2) || pieces_per_row < 1))
        return OC_ERR_INVALID_ARG;
    c->tc_plan_forced = on != 0;
    c->tc_plan_pair = pair; c->tc_plan_tiles = tiles_per_cta; c->tc_plan_pieces = pieces_per_row;
    c->tc_plan_no_narrow = single_accumulator ? 1 : 0;
    c->tc_plan_a_res = candidates_resident < 0 ? -1 : (candidates_resident ? 1 : 0);
    return OC_OK;
}

oc_status oc_tc_plan_describe(oc_ctx* c, const oc_layout* layout, int32_t* out) {
    if (!c || !out) return OC_ERR_INVALID_ARG;
    Geo g;
    oc_status st = make_geo(layout, &g);
    if (st != OC_OK) return st;
    DeviceGuard guard(c->device);
    if (!guard.ok) return OC_ERR_CUDA;
    return tc_plan_describe(c, g, out);
}

oc_status oc_profile_enable(oc_ctx* c, int on) {
    if (!c) return OC_ERR_INVALID_ARG;
    c->profile_on = on == 1;
    c->span_on = on == 2;
    return OC_OK;
}

static void drain(oc_ctx* c, int k) {
    for (auto& p : c->prof[k].pending) {
        float ms = 0.f;
        if (cudaEventSynchronize(p.second) == cudaSuccess && cudaEventElapsedTime(&ms, p.first, p.second) == cudaSuccess)
            c->prof[k].total_ms += ms;
        c->free_events.push_back(p.first); c->free_events.push_back(p.second);
    }
    c->prof[k].pending.clear();
}

oc_status oc_profile_reset(oc_ctx* c) {
    if (!c) return OC_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    for (int k = 0; k < OC_K_COUNT; ++k) { drain(c, k); c->prof[k].launches = 0; c->prof[k].total_ms = 0.0; }
    c->span_count = 0;
    return OC_OK;
}

oc_status oc_profile_read(oc_ctx* c, int k, int64_t* launches, double* total_ms) {
    if (!c || k < 0 || k >= OC_K_COUNT) return OC_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    drain(c, k);
    if (launches) *launches = c->prof[k].launches;
    if (total_ms) *total_ms = c->prof[k].total_ms;
    return OC_OK;
}

oc_status oc_profile_captured_read(oc_ctx* c, int k, int64_t* launches, double* total_ms) {
    if (!c || k < 0 || k >= OC_K_COUNT) return OC_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    double sum = 0.0;
    int64_t n = 0;
    for (auto& p : c->prof[k].captured) {
        float ms = 0.f;
        if (cudaEventSynchronize(p.second) == cudaSuccess && cudaEventElapsedTime(&ms, p.first, p.second) == cudaSuccess) {
            sum += ms; ++n;
        } else {
            cudaGetLastError();                  // captured but its graph has not run yet
        }
    }
    if (launches) *launches = n;
    if (total_ms) *total_ms = sum;
    return OC_OK;
}

oc_status oc_profile_span_read(oc_ctx* c, int k, int64_t* launches, double* total_ms) {
    if (!c || k < 0 || k >= OC_K_COUNT) return OC_ERR_INVALID_ARG;
    if (k != OC_K_MATCH_TC) return OC_ERR_UNSUPPORTED;
    DeviceGuard guard(c->device);
    if (!guard.ok || cudaDeviceSynchronize() != cudaSuccess) return OC_ERR_CUDA;
    const long long n = c->span_count < 256 ? c->span_count : 256;
    std::vector<unsigned long long> h(512);
    if (cudaMemcpy(h.data(), c->d_span, 512 * sizeof(unsigned long long), cudaMemcpyDeviceToHost) != cudaSuccess)
        return OC_ERR_CUDA;
    double ns = 0.0;
    long long counted = 0;
    for (long long i = 0; i < n; ++i) {
        const long long slot = (c->span_count - 1 - i) & 255;
        const unsigned long long entry = ~h[2 * slot], exit = h[2 * slot + 1];
        if (h[2 * slot] != 0 && exit >= entry) { ns += (double)(exit - entry); ++counted; }
    }
    if (launches) *launches = counted;
    if (total_ms) *total_ms = ns * 1e-6;
    return OC_OK;
}

// ---- hot path ----------------------------------------------------------------------------------
oc_status oc_match(oc_ctx* c, const oc_layout* layout, const void* x, float* best_sim, int32_t* best_idx,
                   float* aux_sim, float* pair_sim, void* stream) {
    if (!c || !x || !best_sim || !best_idx) return OC_ERR_INVALID_ARG;
    Geo g;
    oc_status st = make_geo(layout, &g);
    if (st != OC_OK) return st;
    if (misaligned(x)) return OC_ERR_ALIGNMENT;
    if (pair_sim && g.kind != OC_KIND_FRAME) return OC_ERR_INVALID_ARG;
    if (aux_sim && g.kind == OC_KIND_BLOCK) return OC_ERR_INVALID_ARG;
    if (match_workspace_bytes(g) > c->workspace_bytes) return OC_ERR_WORKSPACE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return OC_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    if (g.kind == OC_KIND_TOKEN) return launch_match_token(c, g, x, best_sim, best_idx, aux_sim, s);
    if (g.kind == OC_KIND_FRAME) return launch_match_frame(c, g, x, best_sim, best_idx, aux_sim, pair_sim, s);
    return launch_match_block(c, g, x, best_sim, best_idx, s);
}

oc_status oc_match_frame_levels(oc_ctx* c, const oc_layout* layout, const void* x, int n_levels,
                                const int32_t* grids, float* best_sim, int32_t* best_idx, float* pos_sim,
                                float* pair_sim, void* stream) {
    if (!c || !x || !best_sim || !best_idx || !grids || n_levels < 1 || n_levels > OC_MAX_FRAME_LEVELS)
        return OC_ERR_INVALID_ARG;
    Geo g;
    oc_status st = make_geo(layout, &g);
    if (st != OC_OK) return st;
    if (g.kind != OC_KIND_FRAME) return OC_ERR_INVALID_ARG;
    long long units = 0;
    for (int l = 0; l < n_levels; ++l) {
        const int gy = grids[2 * l], gx = grids[2 * l + 1];
        if (gy <= 0 || gx <= 0 || g.gy % gy != 0 || g.gx % gx != 0) return OC_ERR_INVALID_ARG;
        units += (long long)g.B * g.T * gy * gx;
    }
    if (units > 0x7FFFFFFFll) return OC_ERR_UNSUPPORTED;
    if (misaligned(x)) return OC_ERR_ALIGNMENT;
    if (match_workspace_bytes(g) > c->workspace_bytes) return OC_ERR_WORKSPACE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return OC_ERR_CUDA;
    return launch_match_frame_levels(c, g, x, n_levels, grids, best_sim, best_idx, pos_sim, pair_sim, (cudaStream_t)stream);
}

oc_status oc_linear_gather_scatter(oc_ctx* c, const void* a, int64_t a_rows, int64_t K, const int32_t* a_idx,
                                   int64_t n_rows, const void* w, int64_t N, void* out, int64_t out_rows,
                                   const int32_t* out_idx, void* stream) {
    if (!c || !a || !w || !out || a_rows <= 0 || K <= 0 || N <= 0 || n_rows < 0 || out_rows <= 0) return OC_ERR_INVALID_ARG;
    if (K % 8 != 0 || N % 8 != 0) return OC_ERR_ALIGNMENT;
    if (misaligned(a) || misaligned(w) || misaligned(out)) return OC_ERR_ALIGNMENT;
    if (!a_idx && n_rows > a_rows) return OC_ERR_INVALID_ARG;
    if (N < 128 || a_rows > 0x7FFFFFFFll || out_rows > 0x7FFFFFFFll || K > 0x7FFFFFFFll || N > 0x7FFFFFFFll) return OC_ERR_UNSUPPORTED;
    DeviceGuard guard(c->device);
    if (!guard.ok) return OC_ERR_CUDA;
    return launch_linear_gs(c, a, a_rows, K, a_idx, n_rows, w, N, out, out_rows, out_idx, (cudaStream_t)stream);
}

// ---- Token Cache on the frame pairs of Frame Cache (Section 3.2.3) ---------------------------------
static oc_status joint_geo(const oc_layout* layout, Geo* g) {
    oc_status st = make_geo(layout, g);
    if (st != OC_OK) return st;
    if (g->kind != OC_KIND_TOKEN || g->self_match) return OC_ERR_INVALID_ARG;
    if (g->gy != 1 || g->gx != 1 || g->dtype != OC_DTYPE_BF16) return OC_ERR_UNSUPPORTED;
    return OC_OK;
}

oc_status oc_joint_workspace_bytes(const oc_layout* layout, size_t* bytes) {
    if (!bytes) return OC_ERR_INVALID_ARG;
    Geo g;
    oc_status st = joint_geo(layout, &g);
    if (st != OC_OK) return st;
    *bytes = joint_workspace_bytes(g);
    return OC_OK;
}

oc_status oc_joint_groups(oc_ctx* c, const oc_layout* layout, const float* frame_best_sim,
                          const int32_t* frame_best_idx, const int32_t* frame_slot_of, int32_t* frames, void* stream) {
    if (!c || !frame_best_sim || !frame_best_idx || !frame_slot_of || !frames) return OC_ERR_INVALID_ARG;
    Geo g;
    oc_status st = joint_geo(layout, &g);
    if (st != OC_OK) return st;
    if (((uintptr_t)frames & 7u) != 0) return OC_ERR_ALIGNMENT;
    DeviceGuard guard(c->device);
    if (!guard.ok) return OC_ERR_CUDA;
    return launch_joint_groups(c, g.B, g.T, frame_best_sim, frame_best_idx, frame_slot_of, (int2*)frames, (cudaStream_t)stream);
}

oc_status oc_match_joint(oc_ctx* c, const oc_layout* layout, const void* x, const int32_t* frames, float* best_sim,
                         int32_t* best_idx, void* stream) {
    if (!c || !x || !frames || !best_sim || !best_idx) return OC_ERR_INVALID_ARG;
    Geo g;
    oc_status st = joint_geo(layout, &g);
    if (st != OC_OK) return st;
    if (misaligned(x) || ((uintptr_t)frames & 7u) != 0) return OC_ERR_ALIGNMENT;
    if (joint_workspace_bytes(g) > c->workspace_bytes) return OC_ERR_WORKSPACE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return OC_ERR_CUDA;
    return launch_match_joint(c, g, x, (const int2*)frames, best_sim, best_idx, (cudaStream_t)stream);
}

oc_status oc_select_joint(oc_ctx* c, const oc_layout* layout, const int32_t* frames, const float* best_sim,
                          const int32_t* best_idx, int mode, float thr, int64_t n_reuse_pair, int64_t n_reuse_single,
                          int64_t y_stride, int32_t* kept_idx, int32_t* kept_count, int32_t* match_map,
                          int32_t* slot_of, void* stream) {
    if (!c || !frames || !best_sim || !best_idx || !kept_idx || !kept_count || !match_map || !slot_of)
        return OC_ERR_INVALID_ARG;
    if (mode != OC_SELECT_THRESHOLD && mode != OC_SELECT_COUNT) return OC_ERR_INVALID_ARG;
    Geo g;
    oc_status st = joint_geo(layout, &g);
    if (st != OC_OK) return st;
    const int64_t P = (int64_t)g.H * g.W;
    if (n_reuse_pair < 0 || n_reuse_single < 0 || y_stride <= 0 || y_stride > 2 * P) return OC_ERR_INVALID_ARG;
    // capacity: a pair keeps at least 2P - min(n_reuse_pair, 7P/4-ish candidates), a single frame P - ...
    const int64_t cand_single = P - g.reps_per_group, cand_pair = 2 * P - g.reps_per_group;
    const int64_t keep_pair = mode == OC_SELECT_COUNT ? 2 * P - (n_reuse_pair < cand_pair ? n_reuse_pair : cand_pair) : 2 * P;
    const int64_t keep_single = mode == OC_SELECT_COUNT ? P - (n_reuse_single < cand_single ? n_reuse_single : cand_single) : P;
    if (y_stride < keep_pair || y_stride < keep_single) return OC_ERR_INVALID_ARG;
    if ((int64_t)g.B * g.T * y_stride > 0x7FFFFFFFll) return OC_ERR_UNSUPPORTED;
    if (((uintptr_t)frames & 7u) != 0) return OC_ERR_ALIGNMENT;
    DeviceGuard guard(c->device);
    if (!guard.ok) return OC_ERR_CUDA;
    return launch_select_joint(c, g, (const int2*)frames, best_sim, best_idx, mode, thr, n_reuse_pair, n_reuse_single,
                               y_stride, kept_idx, kept_count, match_map, slot_of, (cudaStream_t)stream);
}

oc_status oc_select(oc_ctx* c, const oc_layout* layout, const float* best_sim, const int32_t* best_idx, int mode,
                    float thr, int64_t n_reuse, int64_t y_stride, int32_t* kept_idx, int32_t* kept_count,
                    int32_t* match_map, int32_t* slot_of, void* stream) {
    if (!c || !best_sim || !best_idx || !kept_idx || !kept_count || !match_map || !slot_of) return OC_ERR_INVALID_ARG;
    if (mode != OC_SELECT_THRESHOLD && mode != OC_SELECT_COUNT) return OC_ERR_INVALID_ARG;
    Geo g;
    oc_status st = make_geo(layout, &g);
    if (st != OC_OK) return st;
    if (n_reuse < 0 || y_stride <= 0 || y_stride > g.units_per_group) return OC_ERR_INVALID_ARG;
    if (mode == OC_SELECT_THRESHOLD && isnan(thr)) return OC_ERR_INVALID_ARG;
    if (mode == OC_SELECT_COUNT && g.self_match) return OC_ERR_UNSUPPORTED;
    const int64_t n_cand = g.self_match ? g.units_per_group : g.units_per_group - g.reps_per_group;
    const int64_t min_keep = mode == OC_SELECT_COUNT ? g.units_per_group - (n_reuse < n_cand ? n_reuse : n_cand)
                                                     : g.units_per_group;
    if (y_stride < min_keep) return OC_ERR_INVALID_ARG;   // the dense buffer could overflow
    if (g.n_groups * y_stride > 0x7FFFFFFFll) return OC_ERR_UNSUPPORTED;
    DeviceGuard guard(c->device);
    if (!guard.ok) return OC_ERR_CUDA;
    return launch_select(c, g, best_sim, best_idx, mode, thr, n_reuse, y_stride, kept_idx, kept_count, match_map,
                         slot_of, (cudaStream_t)stream);
}

oc_status oc_gather(oc_ctx* c, const oc_rows* rows, const void* x, const int32_t* kept_idx, int64_t n_slots, void* y,
                    void* stream) {
    if (!c || !x || !kept_idx || !y || n_slots < 0) return OC_ERR_INVALID_ARG;
    oc_status st = check_rows(rows);
    if (st != OC_OK) return st;
    if (misaligned(x) || misaligned(y)) return OC_ERR_ALIGNMENT;
    DeviceGuard guard(c->device);
    if (!guard.ok) return OC_ERR_CUDA;
    return launch_gather(c, *rows, x, kept_idx, n_slots, y, (cudaStream_t)stream);
}

oc_status oc_restore(oc_ctx* c, const oc_rows* rows, const void* z, const void* cache, int64_t n_units,
                     const int32_t* slot_of, const int32_t* match_map, void* out, int src_mode, void* stream) {
    if (!c || !z || !slot_of || !out || n_units < 0) return OC_ERR_INVALID_ARG;
    if (src_mode != OC_RESTORE_FROM_CACHE && src_mode != OC_RESTORE_FROM_REPRESENTATIVE) return OC_ERR_INVALID_ARG;
    if (src_mode == OC_RESTORE_FROM_CACHE && !cache) return OC_ERR_INVALID_ARG;
    if (src_mode == OC_RESTORE_FROM_REPRESENTATIVE && !match_map) return OC_ERR_INVALID_ARG;
    if (n_units > 0x7FFFFFFFll) return OC_ERR_UNSUPPORTED;
    oc_status st = check_rows(rows);
    if (st != OC_OK) return st;
    if (misaligned(z) || misaligned(out) || (cache && misaligned(cache))) return OC_ERR_ALIGNMENT;
    if (out == z) return OC_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return OC_ERR_CUDA;
    return launch_restore(c, *rows, z, cache, n_units, slot_of, match_map ? match_map : slot_of, out, src_mode,
                          (cudaStream_t)stream);
}

// ---- Layered Cache -----------------------------------------------------------------------------
oc_status oc_layer_cache_put(oc_ctx* c, int layer, int step, const void* src, size_t bytes, void* stream) {
    if (!c || !src || bytes == 0) return OC_ERR_INVALID_ARG;
    if (misaligned(src)) return OC_ERR_ALIGNMENT;
    DeviceGuard guard(c->device);
    if (!guard.ok) return OC_ERR_CUDA;
    LayerEntry& e = c->layers[layer];
    if (e.capacity < bytes) {
        // stream-ordered users of the old buffer must finish before it is released
        if (e.ptr) { cudaStreamSynchronize((cudaStream_t)stream); cudaFree(e.ptr); e.ptr = nullptr; e.capacity = 0; e.bytes = 0; }
        void* p = nullptr;
        if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); c->layers.erase(layer); return OC_ERR_OOM; }
        e.ptr = p; e.capacity = bytes;
    }
    oc_status st = launch_copy(c, src, e.ptr, bytes, (cudaStream_t)stream);
    if (st != OC_OK) return st;
    e.bytes = bytes; e.step = step;
    return OC_OK;
}

oc_status oc_layer_cache_get(oc_ctx* c, int layer, int step, int interval, void* dst, const void** view,
                             size_t* bytes, void* stream) {
    if (!c) return OC_ERR_INVALID_ARG;
    if (dst && misaligned(dst)) return OC_ERR_ALIGNMENT;
    auto it = c->layers.find(layer);
    if (it == c->layers.end() || it->second.bytes == 0) return OC_CACHE_MISS;
    const LayerEntry& e = it->second;
    if (!oc_layer_cache_would_hit(e.step, step, interval)) return OC_CACHE_MISS;
    if (view) *view = e.ptr;
    if (bytes) *bytes = e.bytes;
    if (dst) {
        DeviceGuard guard(c->device);
        if (!guard.ok) return OC_ERR_CUDA;
        return launch_copy(c, e.ptr, dst, e.bytes, (cudaStream_t)stream);
    }
    return OC_OK;
}

oc_status oc_layer_cache_clear(oc_ctx* c) {
    if (!c) return OC_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    cudaDeviceSynchronize();
    for (auto& kv : c->layers) cudaFree(kv.second.ptr);
    c->layers.clear();
    return cuda_ok(cudaGetLastError());
}

// ---- Layered Cache schedule proposal (host only) -------------------------------------------------
oc_status oc_schedule_propose(const double* latency, const double* quality_loss, int64_t n, double target_speedup,
                              int32_t* chosen, int64_t* n_chosen, double* saved) {
    if (!latency || !quality_loss || !chosen || !n_chosen || n < 0 || n > 0x7FFFFFFF) return OC_ERR_INVALID_ARG;
    if (!(target_speedup >= 1.0)) return OC_ERR_INVALID_ARG;
    for (int64_t i = 0; i < n; ++i)
        if (!(latency[i] > 0.0) || !std::isfinite(latency[i]) || !std::isfinite(quality_loss[i])) return OC_ERR_INVALID_ARG;
    // Algorithm 1 as a prefix-sum problem: rank the candidates by quality loss per unit of latency
    // (a stable ranking keeps equal scores in candidate order), accumulate their latencies along the
    // ranking, and the answer is the shortest prefix whose sum reaches the latency budget -- the
    // whole ranking when even that does not.
    std::vector<int32_t> ranking((size_t)n);
    std::vector<double> score((size_t)n);
    for (int64_t i = 0; i < n; ++i) { ranking[(size_t)i] = (int32_t)i; score[(size_t)i] = quality_loss[i] / latency[i]; }
    std::stable_sort(ranking.begin(), ranking.end(), [&score](int32_t a, int32_t b) { return score[(size_t)a] < score[(size_t)b]; });
    std::vector<double> prefix((size_t)n + 1);
    double total = 0.0;                                   // (summed in candidate order, like the budget's definition)
    for (int64_t i = 0; i < n; ++i) total += latency[i];
    prefix[0] = 0.0;
    for (int64_t r = 0; r < n; ++r) prefix[(size_t)r + 1] = prefix[(size_t)r] + latency[ranking[(size_t)r]];
    const double budget = (1.0 - 1.0 / target_speedup) * total;
    // first prefix length whose sum is >= budget (prefix sums of positive terms ascend)
    const int64_t len = std::lower_bound(prefix.begin(), prefix.end(), budget) - prefix.begin();
    const int64_t k = len > n ? n : len;
    for (int64_t r = 0; r < k; ++r) chosen[r] = ranking[(size_t)r];
    *n_chosen = k;
    if (saved) *saved = prefix[(size_t)k];
    return OC_OK;
}

// ---- host-buffer call --------------------------------------------------------------------------
oc_status oc_cache_step_host(oc_ctx* c, const oc_layout* layout, int mode, float thr, int64_t n_reuse,
                             const void* x_host, const void* cache_host, void* out_host, int32_t* kept_count_host,
                             void* stream) {
    if (!c || !x_host || !cache_host || !out_host) return OC_ERR_INVALID_ARG;
    if (mode != OC_SELECT_THRESHOLD && mode != OC_SELECT_COUNT) return OC_ERR_INVALID_ARG;
    Geo g;
    oc_status st = make_geo(layout, &g);
    if (st != OC_OK) return st;
    if (match_workspace_bytes(g) > c->workspace_bytes) return OC_ERR_WORKSPACE;
    oc_rows rows;
    st = oc_rows_from_layout(layout, g.C, g.elem_bytes, &rows);
    if (st != OC_OK) return st;
    DeviceGuard guard(c->device);
    if (!guard.ok) return OC_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;

    const size_t tensor_bytes = (size_t)g.B * g.T * g.H * g.W * g.C * g.elem_bytes;
    const size_t nu = (size_t)g.n_units, ng = (size_t)g.n_groups;
    auto up = [](size_t v) { return (v + 255) / 256 * 256; };
    // staging: x | cache | out | y | best_sim | best_idx | kept_idx | match_map | slot_of | kept_count
    const size_t need = 4 * up(tensor_bytes) + 5 * up(nu * 4) + up(ng * 4);
    if (c->stage_bytes < need) {
        cudaStreamSynchronize(s);
        cudaFree(c->stage); c->stage = nullptr; c->stage_bytes = 0;
        if (cudaMalloc(&c->stage, need) != cudaSuccess) { cudaGetLastError(); return OC_ERR_OOM; }
        c->stage_bytes = need;
    }
    uint8_t* p = (uint8_t*)c->stage;
    void* dx = p; p += up(tensor_bytes);
    void* dcache = p; p += up(tensor_bytes);
    void* dout = p; p += up(tensor_bytes);
    void* dy = p; p += up(tensor_bytes);
    float* dsim = (float*)p; p += up(nu * 4);
    int32_t* didx = (int32_t*)p; p += up(nu * 4);
    int32_t* dkept = (int32_t*)p; p += up(nu * 4);
    int32_t* dmap = (int32_t*)p; p += up(nu * 4);
    int32_t* dslot = (int32_t*)p; p += up(nu * 4);
    int32_t* dcount = (int32_t*)p;

    // Pinned (page-locked, device-mapped) host buffers are read and written by the restore kernel
    // itself: of the cache only the rows of reused units then cross the bus, and the output streams
    // to the host while those rows stream in (the link is full duplex).  Pageable buffers go through
    // staging copies.
    auto mapped = [](const void* h) -> void* {
        cudaPointerAttributes a;
        if (cudaPointerGetAttributes(&a, h) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        return (a.type == cudaMemoryTypeHost && ((uintptr_t)a.devicePointer & 15) == 0) ? a.devicePointer : nullptr;
    };
    void* cache_dev = mapped(cache_host);
    void* out_dev = mapped(out_host);

    // Token Cache groups never span frames, so the call is cut into up to 8 chunks of whole frames:
    // all host->device copies of x are queued at once on a second stream, and chunk k is matched,
    // selected, gathered and restored (its output streaming back to the host) while the copies of the
    // chunks after it are still arriving.  Other kinds, and single frames, are one chunk.
    const int64_t frames = (int64_t)g.B * g.T;
    int n_chunks = (g.kind == OC_KIND_TOKEN && frames > 1) ? (int)(frames < 8 ? frames : 8) : 1;
    if (n_chunks > 1) {
        if (!c->copy_stream && cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) != cudaSuccess) {
            cudaGetLastError(); n_chunks = 1;
        }
        while (n_chunks > 1 && (int)c->chunk_events.size() < n_chunks + 1) {
            cudaEvent_t e;
            if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) { cudaGetLastError(); n_chunks = 1; break; }
            c->chunk_events.push_back(e);
        }
    }
    if (n_chunks == 1) {
        if (cudaMemcpyAsync(dx, x_host, tensor_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return OC_ERR_CUDA;
        if (!cache_dev && cudaMemcpyAsync(dcache, cache_host, tensor_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess)
            return OC_ERR_CUDA;
        st = oc_match(c, layout, dx, dsim, didx, nullptr, nullptr, stream);
        if (st != OC_OK) return st;
        st = oc_select(c, layout, dsim, didx, mode, thr, n_reuse, g.units_per_group, dkept, dcount, dmap, dslot, stream);
        if (st != OC_OK) return st;
        st = oc_gather(c, &rows, dx, dkept, (int64_t)nu, dy, stream);
        if (st != OC_OK) return st;
        st = oc_restore(c, &rows, dy, cache_dev ? cache_dev : dcache, (int64_t)nu, dslot, dmap, out_dev ? out_dev : dout,
                        OC_RESTORE_FROM_CACHE, stream);
        if (st != OC_OK) return st;
        if (!out_dev && cudaMemcpyAsync(out_host, dout, tensor_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess)
            return OC_ERR_CUDA;
    } else {
        const int64_t fpc = (frames + n_chunks - 1) / n_chunks;              // frames per chunk
        const size_t frame_bytes = tensor_bytes / (size_t)frames;
        const size_t units_pf = nu / (size_t)frames, groups_pf = ng / (size_t)frames;
        cudaStream_t cs = c->copy_stream;
        // the copies may not overtake earlier work of the caller's stream on the staging buffers
        if (cudaEventRecord(c->chunk_events[n_chunks], s) != cudaSuccess ||
            cudaStreamWaitEvent(cs, c->chunk_events[n_chunks], 0) != cudaSuccess) return OC_ERR_CUDA;
        for (int k = 0; k < n_chunks; ++k) {
            const int64_t f0 = k * fpc, f1 = (f0 + fpc < frames) ? f0 + fpc : frames;
            if (f0 >= f1) { n_chunks = k; break; }
            const size_t off = (size_t)f0 * frame_bytes, len = (size_t)(f1 - f0) * frame_bytes;
            if (cudaMemcpyAsync((uint8_t*)dx + off, (const uint8_t*)x_host + off, len, cudaMemcpyHostToDevice, cs) != cudaSuccess)
                return OC_ERR_CUDA;
            if (!cache_dev && cudaMemcpyAsync((uint8_t*)dcache + off, (const uint8_t*)cache_host + off, len,
                                              cudaMemcpyHostToDevice, cs) != cudaSuccess) return OC_ERR_CUDA;
            if (cudaEventRecord(c->chunk_events[k], cs) != cudaSuccess) return OC_ERR_CUDA;
        }
        for (int k = 0; k < n_chunks; ++k) {
            const int64_t f0 = k * fpc, f1 = (f0 + fpc < frames) ? f0 + fpc : frames;
            oc_layout sub = *layout;
            sub.B = (int)(f1 - f0); sub.T = 1;
            oc_rows sub_rows;
            st = oc_rows_from_layout(&sub, g.C, g.elem_bytes, &sub_rows);
            if (st != OC_OK) return st;
            const size_t off = (size_t)f0 * frame_bytes, uoff = (size_t)f0 * units_pf, goff = (size_t)f0 * groups_pf;
            const int64_t sub_units = (int64_t)((size_t)(f1 - f0) * units_pf);
            if (cudaStreamWaitEvent(s, c->chunk_events[k], 0) != cudaSuccess) return OC_ERR_CUDA;
            st = oc_match(c, &sub, (uint8_t*)dx + off, dsim + uoff, didx + uoff, nullptr, nullptr, stream);
            if (st != OC_OK) return st;
            st = oc_select(c, &sub, dsim + uoff, didx + uoff, mode, thr, n_reuse, g.units_per_group, dkept + uoff,
                           dcount + goff, dmap + uoff, dslot + uoff, stream);
            if (st != OC_OK) return st;
            st = oc_gather(c, &sub_rows, (uint8_t*)dx + off, dkept + uoff, sub_units, (uint8_t*)dy + off, stream);
            if (st != OC_OK) return st;
            st = oc_restore(c, &sub_rows, (uint8_t*)dy + off, (uint8_t*)(cache_dev ? cache_dev : dcache) + off, sub_units,
                            dslot + uoff, dmap + uoff, (uint8_t*)(out_dev ? out_dev : dout) + off, OC_RESTORE_FROM_CACHE, stream);
            if (st != OC_OK) return st;
            if (!out_dev && cudaMemcpyAsync((uint8_t*)out_host + off, (uint8_t*)dout + off, (size_t)(f1 - f0) * frame_bytes,
                                            cudaMemcpyDeviceToHost, s) != cudaSuccess) return OC_ERR_CUDA;
        }
    }
    if (kept_count_host &&
        cudaMemcpyAsync(kept_count_host, dcount, ng * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return OC_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return OC_ERR_CUDA;
    return OC_OK;
}

}  // extern "C"
