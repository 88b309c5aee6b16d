// Shared internals of the OmniCache sm_100a library: context, launch bookkeeping, small device helpers.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <map>
#include <mutex>
#include <vector>

#include "omnicache.h"

namespace oc {

struct KernelProf {
    int64_t launches = 0;
    double total_ms = 0.0;
    std::vector<std::pair<cudaEvent_t, cudaEvent_t>> pending;
    // brackets recorded while the stream was being captured: event-record nodes of that graph, recorded
    // anew on every replay (never recycled while the context lives)
    std::vector<std::pair<cudaEvent_t, cudaEvent_t>> captured;
};

struct LayerEntry {
    void* ptr = nullptr;
    size_t bytes = 0;
    size_t capacity = 0;
    int step = 0;
};

}  // namespace oc

struct oc_ctx {
    int device = 0;
    int sm_count = 0;
    void* workspace = nullptr;
    size_t workspace_bytes = 0;
    int* d_status = nullptr;                 // device status word (first device-side error)
    bool profile_on = false;                 // event brackets around every launch
    bool span_on = false;                    // device-side spans of the tensor-core matcher instead
    unsigned long long* d_span = nullptr;    // 256 slots of {~first entry, last exit} in GPU-timer ns
    long long span_count = 0;                // launches stamped since the last reset
    oc::KernelProf prof[OC_K_COUNT];
    std::vector<cudaEvent_t> free_events;
    std::map<int, oc::LayerEntry> layers;    // Layered Cache store
    // staging for oc_cache_step_host
    void* stage = nullptr;
    size_t stage_bytes = 0;
    cudaStream_t copy_stream = nullptr;      // host->device copies of the chunks of oc_cache_step_host
    std::vector<cudaEvent_t> chunk_events;
    // test hook (oc_tc_plan_override): forces the tensor-core matcher's work split
    bool tc_plan_forced = false;
    int tc_plan_pair = 0, tc_plan_tiles = 0, tc_plan_pieces = 0, tc_plan_no_narrow = 0, tc_plan_a_res = -1;
};

namespace oc {

// RAII: makes ctx->device current for the duration of a call and restores the caller's device.
struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

// Work that has to be done once per DEVICE rather than once per process: function attributes such as
// the opt-in to more than 48 KB of dynamic shared memory belong to the device's context, and one
// process may hold contexts on several GPUs.  ensure(dev, f) runs f() the first time it is called for
// `dev` (with that device current: every launcher runs under a DeviceGuard) and remembers whether it
// succeeded; device ids beyond the table run f() every time.
struct PerDeviceOnce {
    static constexpr int MAX_DEV = 64;
    std::mutex m;
    unsigned char state[MAX_DEV] = {};           // 0 = not yet, 1 = done, 2 = failed
    template <class F>
    bool ensure(int dev, F&& f) {
        if (dev < 0 || dev >= MAX_DEV) return f();
        std::lock_guard<std::mutex> lock(m);
        if (state[dev] == 0) state[dev] = f() ? 1 : 2;
        return state[dev] == 1;
    }
};

// Counts a kernel launch and, if timers are on, brackets it with events on the launching stream.
struct LaunchScope {
    oc_ctx* ctx; int k; cudaStream_t s; cudaEvent_t e0 = nullptr, e1 = nullptr; bool capturing = false;
    LaunchScope(oc_ctx* c, int kernel, cudaStream_t stream);
    ~LaunchScope();
};

// Launch with programmatic stream serialization: the grid may be scheduled while the kernel before it
// in the stream is still running, once every CTA of that kernel has executed
// griddepcontrol.launch_dependents (or exited), which hides the launch latency between the kernels of
// a step.  Kernels launched this way execute griddepcontrol.wait (pdl_wait) before they touch
// anything the earlier kernel reads or writes, and only then let their own dependents go, so a grid
// never runs ahead of more than the one kernel before it.  Use as
//     OC_LAUNCH((kernel<T, N>), grid, block, smem_bytes, stream, args...);
struct PdlLaunch {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    PdlLaunch(dim3 grid, dim3 block, size_t smem, cudaStream_t s, unsigned cluster_x = 0) {
        cfg = cudaLaunchConfig_t{};
        cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.numAttrs = 1;
        if (cluster_x > 1) {
            attr[1].id = cudaLaunchAttributeClusterDimension;
            attr[1].val.clusterDim.x = cluster_x; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
            cfg.numAttrs = 2;
        }
        cfg.attrs = attr;
    }
};
#define OC_LAUNCH(kernel, grid, block, smem, stream, ...)                      \
    do {                                                                       \
        ::oc::PdlLaunch oc_l_((grid), (block), (smem), (stream));              \
        cudaLaunchKernelEx(&oc_l_.cfg, kernel, __VA_ARGS__);                   \
    } while (0)

inline oc_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? OC_OK : OC_ERR_CUDA; }
inline oc_status last_launch_status() { return cuda_ok(cudaGetLastError()); }

// Host-side geometry derived from a layout (validated before use).
struct Geo {
    int kind, dtype, B, T, H, W, C, sy, sx, oy, ox, gy, gx, self_match, frame_stat;
    float eps;
    int Hp, Wp;          // patch size (TOKEN) or frame size
    int Hs, Ws;          // representative lattice size inside a patch
    int64_t n_groups, units_per_group, reps_per_group, n_units;
    int elem_bytes;
};
oc_status make_geo(const oc_layout* L, Geo* g);

// Device-side description of the select / match group structure.
struct GroupMap {
    int kind, self_match;
    int H, W, gy, gx, Hp, Wp, sy, sx, oy, ox;
    int units_per_group;
    // Joint form (Token Cache on frame pairs, Section 3.2.3): group g is slot g of this table,
    // {representative frame, partner frame or -1}, {-1, -1} for a frame absorbed into its partner's
    // group; a pair's units are the tokens of its two frames in time order.  Null otherwise.
    const int2* frames;
    int n_reuse_single;                  // count-mode budget of a single-frame group (pairs take n_reuse)
};
GroupMap make_group_map(const Geo& g);

__host__ __device__ inline int64_t gm_unit_index(const GroupMap& m, int64_t g, int u) {
    if (m.kind != OC_KIND_FRAME) {                     // TOKEN: bt = frame; BLOCK: bt = batch element
        int px = (int)(g % m.gx);
        int py = (int)((g / m.gx) % m.gy);
        int64_t bt = g / ((int64_t)m.gx * m.gy);
        int ly = u / m.Wp, lx = u - ly * m.Wp;
        return (bt * m.H + (int64_t)py * m.Hp + ly) * m.W + (int64_t)px * m.Wp + lx;
    }
    // FRAME group (b, patch): its frames are n_patches apart
    const int64_t np = (int64_t)m.gy * m.gx, b = g / np, patch = g - b * np;
    return (b * m.units_per_group + u) * np + patch;
}
__host__ __device__ inline bool gm_is_rep(const GroupMap& m, int u) {
    if (m.kind == OC_KIND_FRAME) return (u & 1) == 0;
    if (m.self_match) return true;
    int ly = u / m.Wp, lx = u - ly * m.Wp;
    return (ly % m.sy) == m.oy && (lx % m.sx) == m.ox;
}
__host__ __device__ inline bool gm_is_cand(const GroupMap& m, int u) {
    if (m.kind == OC_KIND_TOKEN && m.self_match) return true;
    return !gm_is_rep(m, u);
}

// ---- internal launchers (each validates nothing: the C-ABI layer in api.cu has done so) --------
oc_status launch_gather(oc_ctx*, const oc_rows&, const void* x, const int32_t* kept_idx, int64_t n_slots,
                        void* y, cudaStream_t);
oc_status launch_restore(oc_ctx*, const oc_rows&, const void* z, const void* cache, int64_t n_units,
                         const int32_t* slot_of, const int32_t* match_map, void* out, int src_mode,
                         cudaStream_t);
oc_status launch_copy(oc_ctx*, const void* src, void* dst, size_t bytes, cudaStream_t);
oc_status launch_select(oc_ctx*, const Geo&, const float* best_sim, const int32_t* best_idx, int mode,
                        float thr, int64_t n_reuse, int64_t y_stride, int32_t* kept_idx,
                        int32_t* kept_count, int32_t* match_map, int32_t* slot_of, cudaStream_t);
oc_status launch_match_frame(oc_ctx*, const Geo&, const void* x, float* best_sim, int32_t* best_idx,
                             float* pos_sim, float* pair_sim, cudaStream_t);
oc_status launch_match_frame_levels(oc_ctx*, const Geo&, const void* x, int n_levels, const int32_t* levels,
                                    float* best_sim, int32_t* best_idx, float* pos_sim, float* pair_sim, cudaStream_t);
oc_status launch_match_block(oc_ctx*, const Geo&, const void* x, float* best_sim, int32_t* best_idx,
                             cudaStream_t);
oc_status launch_match_token(oc_ctx*, const Geo&, const void* x, float* best_sim, int32_t* best_idx,
                             float* aux_sim, cudaStream_t);
// tcgen05 path of launch_match_token; returns OC_ERR_UNSUPPORTED if the shape is not covered.
bool tc_match_supported(const Geo&);
oc_status launch_linear_gs(oc_ctx*, const void* a, int64_t a_rows, int64_t K, const int32_t* a_idx, int64_t n_rows,
                           const void* w, int64_t N, void* out, int64_t out_rows, const int32_t* out_idx, cudaStream_t);
size_t joint_workspace_bytes(const Geo&);
oc_status launch_joint_groups(oc_ctx*, int B, int T, const float* frame_best_sim, const int32_t* frame_best_idx,
                              const int32_t* frame_slot_of, int2* frames, cudaStream_t);
oc_status launch_match_joint(oc_ctx*, const Geo&, const void* x, const int2* frames, float* best_sim, int32_t* best_idx,
                             cudaStream_t);
oc_status launch_select_joint(oc_ctx*, const Geo&, const int2* frames, const float* best_sim, const int32_t* best_idx,
                              int mode, float thr, int64_t n_reuse_pair, int64_t n_reuse_single, int64_t y_stride,
                              int32_t* kept_idx, int32_t* kept_count, int32_t* match_map, int32_t* slot_of, cudaStream_t);
bool tc_match_supported(const Geo&);
oc_status launch_match_joint_tc(oc_ctx*, const Geo&, const void* x, const float* inv_norm, unsigned long long* keys,
                                const int4* units, const int* n_units_dev, long long max_units, cudaStream_t);
oc_status launch_match_token_tc(oc_ctx*, const Geo&, const void* x, const float* inv_norm,
                                unsigned long long* keys, float* aux_sim, cudaStream_t);
oc_status tc_plan_describe(oc_ctx*, const Geo&, int32_t* out12);
oc_status launch_bounded_wait_selftest(oc_ctx*, unsigned long long limit_ns, cudaStream_t);

size_t match_workspace_bytes(const Geo&);

// ---- device helpers ---------------------------------------------------------------------------
#ifdef __CUDACC__
// See PdlLaunch: wait for the kernel before this one in the stream (all of it, memory included), and
// let the kernel after this one be scheduled.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_enter() { pdl_wait(); pdl_launch_dependents(); }

// ---- shared-memory barriers (mbarrier) with bounded waits ----------------------------------------
// Every wait in this library gives up after WAIT_LIMIT_NS, so that a lost copy shows up as
// OC_ERR_TIMEOUT in the context's status word instead of a hung device.
static constexpr unsigned long long WAIT_LIMIT_NS = 1000000000ull;   // 1 s per wait
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: false if the phase did not complete within WAIT_LIMIT_NS or another role gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    // (the clock is first read after 256 failed tries: reading %globaltimer is slow, and nearly every wait
    //  of the hot loops ends long before that)
    unsigned long long t0 = 0;
    unsigned spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 255u) == 0) {
            if (*abort_flag) return false;
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > WAIT_LIMIT_NS) return false;
        }
    }
    return true;
}
__device__ __forceinline__ uint4 ld_nc_v4(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_v4(void* p, uint4 v) {
    asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

// Order-preserving map float -> uint32 (larger float <=> larger key) and back.
__device__ __forceinline__ uint32_t f32_to_ordered(float f) {
    uint32_t b = __float_as_uint(f);
    if (b == 0x80000000u) b = 0u;                           // -0.0 and +0.0 compare equal: one key
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float ordered_to_f32(uint32_t k) {
    uint32_t b = (k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k;
    return __uint_as_float(b);
}
// (value, index) -> 64-bit key whose maximum is the largest value, then the lowest index.
__device__ __forceinline__ unsigned long long pack_key(float v, uint32_t idx) {
    return ((unsigned long long)f32_to_ordered(v) << 32) | (unsigned long long)(0xFFFFFFFFu - idx);
}

// fp32 partial products of one 16-byte chunk of two rows: dot, |a|^2, |b|^2.
template <int DT> struct Chunk;
// bf16 operands go straight into the fp32 FMA (fma.rn.f32.bf16: bf16 x bf16 + fp32, one rounding), so a
// pair of packed elements costs its FMAs and nothing else -- no shift/mask to widen them first.  The
// product of two bf16 values is exact in fp32, so the result equals that of widening and fmaf().
template <> struct Chunk<OC_DTYPE_BF16> {
    static __device__ __forceinline__ void word3(uint32_t a, uint32_t b, float& dot, float& na, float& nb) {
        asm("{\n\t.reg .b16 al, ah, bl, bh;\n\t"
            "mov.b32 {al, ah}, %3;\n\tmov.b32 {bl, bh}, %4;\n\t"
            "fma.rn.f32.bf16 %0, al, bl, %0;\n\tfma.rn.f32.bf16 %0, ah, bh, %0;\n\t"
            "fma.rn.f32.bf16 %1, al, al, %1;\n\tfma.rn.f32.bf16 %1, ah, ah, %1;\n\t"
            "fma.rn.f32.bf16 %2, bl, bl, %2;\n\tfma.rn.f32.bf16 %2, bh, bh, %2;\n\t}"
            : "+f"(dot), "+f"(na), "+f"(nb) : "r"(a), "r"(b));
    }
    static __device__ __forceinline__ void word2(uint32_t a, uint32_t b, float& dot, float& na) {
        asm("{\n\t.reg .b16 al, ah, bl, bh;\n\t"
            "mov.b32 {al, ah}, %2;\n\tmov.b32 {bl, bh}, %3;\n\t"
            "fma.rn.f32.bf16 %0, al, bl, %0;\n\tfma.rn.f32.bf16 %0, ah, bh, %0;\n\t"
            "fma.rn.f32.bf16 %1, al, al, %1;\n\tfma.rn.f32.bf16 %1, ah, ah, %1;\n\t}"
            : "+f"(dot), "+f"(na) : "r"(a), "r"(b));
    }
    static __device__ __forceinline__ void word1(uint32_t a, float& na) {
        asm("{\n\t.reg .b16 al, ah;\n\t"
            "mov.b32 {al, ah}, %1;\n\t"
            "fma.rn.f32.bf16 %0, al, al, %0;\n\tfma.rn.f32.bf16 %0, ah, ah, %0;\n\t}"
            : "+f"(na) : "r"(a));
    }
    static __device__ __forceinline__ void acc3(const uint4& a, const uint4& b, float& dot, float& na, float& nb) {
        word3(a.x, b.x, dot, na, nb); word3(a.y, b.y, dot, na, nb);
        word3(a.z, b.z, dot, na, nb); word3(a.w, b.w, dot, na, nb);
    }
    static __device__ __forceinline__ void acc2(const uint4& a, const uint4& b, float& dot, float& na) {
        word2(a.x, b.x, dot, na); word2(a.y, b.y, dot, na);
        word2(a.z, b.z, dot, na); word2(a.w, b.w, dot, na);
    }
    static __device__ __forceinline__ void sq(const uint4& a, float& na) {
        word1(a.x, na); word1(a.y, na); word1(a.z, na); word1(a.w, na);
    }
};
template <> struct Chunk<OC_DTYPE_F32> {
    static __device__ __forceinline__ void acc3(const uint4& a, const uint4& b, float& dot, float& na, float& nb) {
        const float av[4] = {__uint_as_float(a.x), __uint_as_float(a.y), __uint_as_float(a.z), __uint_as_float(a.w)};
        const float bv[4] = {__uint_as_float(b.x), __uint_as_float(b.y), __uint_as_float(b.z), __uint_as_float(b.w)};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            dot = fmaf(av[i], bv[i], dot); na = fmaf(av[i], av[i], na); nb = fmaf(bv[i], bv[i], nb);
        }
    }
    static __device__ __forceinline__ void acc2(const uint4& a, const uint4& b, float& dot, float& na) {
        const float av[4] = {__uint_as_float(a.x), __uint_as_float(a.y), __uint_as_float(a.z), __uint_as_float(a.w)};
        const float bv[4] = {__uint_as_float(b.x), __uint_as_float(b.y), __uint_as_float(b.z), __uint_as_float(b.w)};
#pragma unroll
        for (int i = 0; i < 4; ++i) { dot = fmaf(av[i], bv[i], dot); na = fmaf(av[i], av[i], na); }
    }
    static __device__ __forceinline__ void sq(const uint4& a, float& na) {
        const float av[4] = {__uint_as_float(a.x), __uint_as_float(a.y), __uint_as_float(a.z), __uint_as_float(a.w)};
#pragma unroll
        for (int i = 0; i < 4; ++i) na = fmaf(av[i], av[i], na);
    }
};

__device__ __forceinline__ float clamp_unit(float v) { return fminf(1.0f, fmaxf(-1.0f, v)); }
#endif  // __CUDACC__

}  // namespace oc
