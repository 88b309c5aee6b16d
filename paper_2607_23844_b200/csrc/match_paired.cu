// Frame Cache and Block Cache matching: a handful of cosine comparisons over very long descriptors
// (Sections 3.2.1, 3.2.2).  About 3 FMA per element read, so both are HBM-bound streaming
// reductions: 16-byte loads, fp32 accumulators for <a,b>, |a|^2, |b|^2, sub-warp shuffle
// reductions, and a fixed-order two-level sum (no floating-point atomics) so results are
// reproducible run to run.
#include <mutex>

#include "common.cuh"

namespace oc {

static constexpr int PAIR_THREADS = 256;

// lanes cooperating on one row: power of two, about 4 chunks per lane
static int lanes_per_row(int64_t chunks_per_row) {
    int l = 1;
    while (l < 32 && (int64_t)l * 4 < chunks_per_row) l <<= 1;
    return l;
}

template <int LPR>
__device__ __forceinline__ float group_sum(float v) {
#pragma unroll
    for (int d = LPR / 2; d >= 1; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    return v;
}

// fixed-order CTA reduction of one value per thread-group; result valid in thread 0
__device__ __forceinline__ float cta_sum_fixed(float v, float* sh /*[PAIR_THREADS]*/) {
    sh[threadIdx.x] = v;
    __syncthreads();
    for (int w = PAIR_THREADS / 2; w >= 1; w >>= 1) {
        if ((int)threadIdx.x < w) sh[threadIdx.x] += sh[threadIdx.x + w];
        __syncthreads();
    }
    float r = sh[0];
    __syncthreads();
    return r;
}

// ------------------------------------------------------------------------------------------------
// Patch-local Frame Cache (Section 3.3): the frame is cut into gy x gx equal patches and every
// patch position is a matching problem of its own.  The position tiles of the kernels below never
// straddle a patch: tile i covers local positions of patch i / tiles_per_patch, so a partial record
// belongs to one (pair, patch) and the per-patch statistics are sums of whole records.  With one
// patch the local position IS the frame position and no index arithmetic is added.
// ------------------------------------------------------------------------------------------------
struct PatchGrid {
    int n_patches, gx, Hp, Wp, W;
    int Pp;                 // positions per patch
    int tiles_per_patch;
};
static PatchGrid make_patch_grid(const Geo& g, int pos_per_tile) {
    PatchGrid pg;
    pg.n_patches = g.gy * g.gx; pg.gx = g.gx; pg.Hp = g.Hp; pg.Wp = g.Wp; pg.W = g.W;
    pg.Pp = g.Hp * g.Wp;
    pg.tiles_per_patch = (pg.Pp + pos_per_tile - 1) / pos_per_tile;
    return pg;
}
// frame position of local position lp of a patch
__device__ __forceinline__ int patch_position(const PatchGrid& pg, int patch, int lp) {
    if (pg.n_patches == 1) return lp;
    const int py = patch / pg.gx, px = patch - py * pg.gx;
    const int ly = lp / pg.Wp, lx = lp - ly * pg.Wp;
    return (py * pg.Hp + ly) * pg.W + px * pg.Wp + lx;
}

// ------------------------------------------------------------------------------------------------
// Frame Cache: for every adjacent pair (t, t-1) and position p, cos(x[t,p,:], x[t-1,p,:]).
// grid = (position tiles, B*(T-1)).  A CTA covers POS_PER_CTA consecutive positions of one patch of
// one pair and writes one partial record {sum cos, sum dot, sum |a|^2, sum |b|^2}.  Frame t is read
// from HBM by pair (t, t-1) and again, out of L2, by pair (t+1, t).
// ------------------------------------------------------------------------------------------------
template <int DT, int LPR>
__global__ void __launch_bounds__(PAIR_THREADS)
frame_pair_kernel(const uint8_t* __restrict__ x, int T, int P, int cpr, float eps,
                  float* __restrict__ pos_sim, float4* __restrict__ partial, int pos_per_cta, PatchGrid pg) {
    pdl_enter();
    __shared__ float sh[PAIR_THREADS];
    const int q = blockIdx.y;                       // pair index b*(T-1) + (t-1)
    const int b = q / (T - 1), t = q - b * (T - 1) + 1;
    const int groups = PAIR_THREADS / LPR;
    const int grp = threadIdx.x / LPR, lane = threadIdx.x % LPR;
    const long long row_bytes = (long long)cpr * 16;
    const uint8_t* cur = x + ((long long)(b * T + t) * P) * row_bytes;
    const uint8_t* prv = cur - (long long)P * row_bytes;
    int patch = 0, tile = blockIdx.x;
    if (pg.n_patches > 1) { patch = tile / pg.tiles_per_patch; tile -= patch * pg.tiles_per_patch; }
    const int p_begin = tile * pos_per_cta;
    const int p_end = min(pg.Pp, p_begin + pos_per_cta);

    float s_cos = 0.f, s_dot = 0.f, s_na = 0.f, s_nb = 0.f;
    // the trip count is the same for every thread of the CTA: the shuffles below name all 32 lanes
    for (int p0 = p_begin; p0 < p_end; p0 += groups) {
        const bool valid = p0 + grp < p_end;
        const int p = valid ? patch_position(pg, patch, p0 + grp) : 0;
        float dot = 0.f, na = 0.f, nb = 0.f;
        if (valid) {
            const uint8_t* a = cur + (long long)p * row_bytes;
            const uint8_t* bb = prv + (long long)p * row_bytes;
            int c = lane;
            for (; c + LPR < cpr; c += 2 * LPR) {                   // two chunks in flight per row
                uint4 a0 = ld_nc_v4(a + (long long)c * 16), b0 = ld_nc_v4(bb + (long long)c * 16);
                uint4 a1 = ld_nc_v4(a + (long long)(c + LPR) * 16), b1 = ld_nc_v4(bb + (long long)(c + LPR) * 16);
                Chunk<DT>::acc3(a0, b0, dot, na, nb);
                Chunk<DT>::acc3(a1, b1, dot, na, nb);
            }
            if (c < cpr) {
                uint4 a0 = ld_nc_v4(a + (long long)c * 16), b0 = ld_nc_v4(bb + (long long)c * 16);
                Chunk<DT>::acc3(a0, b0, dot, na, nb);
            }
        }
        dot = group_sum<LPR>(dot); na = group_sum<LPR>(na); nb = group_sum<LPR>(nb);
        if (valid && lane == 0) {
            float cs = clamp_unit(dot / (fmaxf(sqrtf(na), eps) * fmaxf(sqrtf(nb), eps)));
            if (pos_sim) pos_sim[(long long)q * P + p] = cs;
            s_cos += cs; s_dot += dot; s_na += na; s_nb += nb;
        }
    }
    float r0 = cta_sum_fixed(s_cos, sh), r1 = cta_sum_fixed(s_dot, sh);
    float r2 = cta_sum_fixed(s_na, sh), r3 = cta_sum_fixed(s_nb, sh);
    if (threadIdx.x == 0) partial[(long long)q * gridDim.x + blockIdx.x] = make_float4(r0, r1, r2, r3);
}

// Time-marching variant: a thread-group owns ONE position and walks a segment of frames, keeping the
// previous frame's row in registers and prefetching the next one, so every row is read exactly once
// (the pair kernel above reads each row twice, the second time out of L2).  Segments overlap by one
// frame.  Inside the frame loop a thread-group only leaves {dot, norm} of its position in shared memory;
// the cosines and, per pair, the tile's sums (a fixed-order shuffle tree) are taken once at the end,
// written as one partial record per (pair, position tile).
static constexpr int MARCH_CPL = 8;      // most 16-byte chunks a lane may hold per row (instantiated for 5 and 8)

template <int DT, int LPR, int CPL>
__global__ void __launch_bounds__(PAIR_THREADS, CPL <= 5 ? 3 : 2)
frame_march_kernel(const uint8_t* __restrict__ x, int T, int P, int cpr, float eps, int seg_len, int n_seg,
                   float* __restrict__ pos_sim, float4* __restrict__ partial, PatchGrid pg) {
    pdl_enter();
    // per (pair of the segment, position of the tile): {dot, |frame t|^2}; and |frame t0|^2 per position.  The
    // cosines and the per-pair sums are taken from these at the end, with every lane busy, instead of by one
    // lane per thread-group inside the frame loop (the kernel is bound by instruction issue as much as by HBM).
    extern __shared__ float2 pair_dn[];                    // [seg_len][GROUPS], then float n0[GROUPS]
    constexpr int GROUPS = PAIR_THREADS / LPR, WARPS = PAIR_THREADS / 32;
    float* n0 = (float*)(pair_dn + (size_t)seg_len * GROUPS);
    const int b = blockIdx.y / n_seg, seg = blockIdx.y - b * n_seg;
    const int t0 = seg * seg_len;                         // first frame of the segment (as "previous")
    const int t1 = min(T - 1, t0 + seg_len);              // last frame of the segment
    const int grp = threadIdx.x / LPR, lane = threadIdx.x % LPR, warp = threadIdx.x >> 5, wl = threadIdx.x & 31;
    int patch = 0, tile = blockIdx.x;
    if (pg.n_patches > 1) { patch = tile / pg.tiles_per_patch; tile -= patch * pg.tiles_per_patch; }
    const bool valid = tile * GROUPS + grp < pg.Pp;
    const int p = valid ? patch_position(pg, patch, tile * GROUPS + grp) : 0;
    const long long row_bytes = (long long)cpr * 16;
    const long long frame_bytes = (long long)P * row_bytes;
    const uint8_t* base = x + ((long long)b * T * P + (valid ? p : 0)) * row_bytes;

    uint4 prev[CPL], cur[CPL], nxt[CPL];
    auto load_row = [&](uint4* dst, int t) {
#pragma unroll
        for (int k = 0; k < CPL; ++k)
            if (lane + k * LPR < cpr) dst[k] = ld_nc_v4(base + (long long)t * frame_bytes + (long long)(lane + k * LPR) * 16);
    };
    load_row(prev, t0);
    if (t0 + 1 <= t1) load_row(cur, t0 + 1);
    {
        float n_first = 0.f;
#pragma unroll
        for (int k = 0; k < CPL; ++k)
            if (lane + k * LPR < cpr) Chunk<DT>::sq(prev[k], n_first);
        n_first = group_sum<LPR>(n_first);
        if (lane == 0) n0[grp] = n_first;
    }
    for (int t = t0 + 1; t <= t1; ++t) {
        if (t + 1 <= t1) load_row(nxt, t + 1);            // in flight while frame t is reduced
        float dot = 0.f, n_cur = 0.f;
#pragma unroll
        for (int k = 0; k < CPL; ++k)
            if (lane + k * LPR < cpr) Chunk<DT>::acc2(cur[k], prev[k], dot, n_cur);
        dot = group_sum<LPR>(dot); n_cur = group_sum<LPR>(n_cur);
        if (lane == 0) pair_dn[(t - t0 - 1) * GROUPS + grp] = make_float2(dot, n_cur);
#pragma unroll
        for (int k = 0; k < CPL; ++k) { prev[k] = cur[k]; cur[k] = nxt[k]; }
    }
    __syncthreads();
    // one warp per pair of the segment: lanes take the tile's positions (two each when a tile has 64), the
    // cosine of every position, then a fixed-order sum of {cos, dot, |a|^2, |b|^2} over the tile
    const int n_here = min(GROUPS, pg.Pp - tile * GROUPS);            // positions of this tile
    for (int i = warp; i < t1 - t0; i += WARPS) {
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int gq = wl; gq < n_here; gq += 32) {
            const float2 dn = pair_dn[i * GROUPS + gq];
            const float n_prev = i == 0 ? n0[gq] : pair_dn[(i - 1) * GROUPS + gq].y;
            const float cs = clamp_unit(dn.x / (fmaxf(sqrtf(dn.y), eps) * fmaxf(sqrtf(n_prev), eps)));
            if (pos_sim) pos_sim[((long long)b * (T - 1) + t0 + i) * P + patch_position(pg, patch, tile * GROUPS + gq)] = cs;
            v.x += cs; v.y += dn.x; v.z += dn.y; v.w += n_prev;
        }
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) {
            v.x += __shfl_xor_sync(0xFFFFFFFFu, v.x, d); v.y += __shfl_xor_sync(0xFFFFFFFFu, v.y, d);
            v.z += __shfl_xor_sync(0xFFFFFFFFu, v.z, d); v.w += __shfl_xor_sync(0xFFFFFFFFu, v.w, d);
        }
        const int q = b * (T - 1) + t0 + i;               // pair (t0+i+1, t0+i)
        if (wl == 0) partial[(long long)q * gridDim.x + blockIdx.x] = v;
    }
}

// One warp per unit (a frame, or one patch of a frame): it sums, in a fixed order, the CTA partials
// of the pair (t, t-1) and of the pair (t+1, t) that belong to its patch, publishes the first as
// pair_sim[t-1][patch] and, for an odd (candidate) frame, picks the better of its two adjacent
// representatives.  Every warp is independent, so units run in parallel.
//
// The partial records are laid out for the FINEST patch grid; a coarser level of the hierarchy
// (Section 3.3: larger patches, up to whole frames, after the patch-level pass) whose patches are
// unions of ry x rx fine patches is finalized from the same records, so one pass over the tensor
// serves every level.
struct FinLevel {
    int gy, gx;             // this level's patch grid
    int ry, rx;             // fine patches per patch of this level, per axis
    int gx_fine, np_fine;   // finest grid: patches per row, patches per frame
    int tiles_per_patch;    // records per (pair, fine patch)
    int n_pos;              // positions per patch of this level
};

// record j (0 <= j < ry*rx*tiles_per_patch, a fixed enumeration) of patch `patch` of pair q at this level
__device__ __forceinline__ float4 level_record(const float4* __restrict__ partial, long long q, int patch,
                                               const FinLevel& lv, int j) {
    if (lv.ry * lv.rx == 1) return partial[(q * lv.np_fine + patch) * lv.tiles_per_patch + j];
    const int py = patch / lv.gx, px = patch - py * lv.gx;
    const int per_row = lv.rx * lv.tiles_per_patch;
    const int fy = j / per_row, r = j - fy * per_row;
    const int fx = r / lv.tiles_per_patch, k = r - fx * lv.tiles_per_patch;
    const int fine = (py * lv.ry + fy) * lv.gx_fine + px * lv.rx + fx;
    return partial[(q * lv.np_fine + fine) * lv.tiles_per_patch + k];
}

// The statistics of pair q0 (if has0) and pair q1 (if has1) for one patch, by one warp.  The kernel is
// pure latency (a few hundred records out of L2), so a lane issues the loads of eight rounds of both
// pairs before it adds anything; the order of the additions is fixed.
__device__ __forceinline__ void frame_pair_values(const float4* __restrict__ partial, long long q0, bool has0,
                                                  long long q1, bool has1, int patch, const FinLevel& lv, int stat,
                                                  float eps, float& out0, float& out1) {
    const int lane = threadIdx.x & 31;
    const int n_rec = lv.ry * lv.rx * lv.tiles_per_patch;
    float4 s0 = make_float4(0.f, 0.f, 0.f, 0.f), s1 = s0;
    constexpr int BATCH = 8;
    for (int j0 = lane; j0 < n_rec; j0 += 32 * BATCH) {
        float4 v0[BATCH], v1[BATCH];
#pragma unroll
        for (int k = 0; k < BATCH; ++k) {
            const int j = j0 + 32 * k;
            v0[k] = (has0 && j < n_rec) ? level_record(partial, q0, patch, lv, j) : make_float4(0.f, 0.f, 0.f, 0.f);
            v1[k] = (has1 && j < n_rec) ? level_record(partial, q1, patch, lv, j) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int k = 0; k < BATCH; ++k) {
            s0.x += v0[k].x; s0.y += v0[k].y; s0.z += v0[k].z; s0.w += v0[k].w;
            s1.x += v1[k].x; s1.y += v1[k].y; s1.z += v1[k].z; s1.w += v1[k].w;
        }
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        s0.x += __shfl_xor_sync(0xFFFFFFFFu, s0.x, d); s0.y += __shfl_xor_sync(0xFFFFFFFFu, s0.y, d);
        s0.z += __shfl_xor_sync(0xFFFFFFFFu, s0.z, d); s0.w += __shfl_xor_sync(0xFFFFFFFFu, s0.w, d);
        s1.x += __shfl_xor_sync(0xFFFFFFFFu, s1.x, d); s1.y += __shfl_xor_sync(0xFFFFFFFFu, s1.y, d);
        s1.z += __shfl_xor_sync(0xFFFFFFFFu, s1.z, d); s1.w += __shfl_xor_sync(0xFFFFFFFFu, s1.w, d);
    }
    if (stat == OC_FRAME_FLAT_COS) {
        out0 = clamp_unit(s0.y / (fmaxf(sqrtf(s0.z), eps) * fmaxf(sqrtf(s0.w), eps)));
        out1 = clamp_unit(s1.y / (fmaxf(sqrtf(s1.z), eps) * fmaxf(sqrtf(s1.w), eps)));
    } else {
        out0 = s0.x / (float)lv.n_pos;
        out1 = s1.x / (float)lv.n_pos;
    }
}

struct FinLevels {
    int n;
    FinLevel lv[OC_MAX_FRAME_LEVELS];
    int unit_off[OC_MAX_FRAME_LEVELS + 1];      // first output unit of each level (levels are stored one after another)
    int pair_off[OC_MAX_FRAME_LEVELS + 1];      // first pair_sim entry of each level
};

__global__ void __launch_bounds__(PAIR_THREADS)
frame_finalize_kernel(const float4* __restrict__ partial, const __grid_constant__ FinLevels F, int B, int T, int stat,
                      float eps, float* __restrict__ pair_sim, float* __restrict__ best_sim,
                      int32_t* __restrict__ best_idx) {
    pdl_enter();
    const int w = blockIdx.x * (PAIR_THREADS / 32) + (threadIdx.x >> 5);     // output unit over all levels
    const int lane = threadIdx.x & 31;
    if (w >= F.unit_off[F.n]) return;                                         // whole warps leave together
    int l = 0;
    while (l + 1 < F.n && w >= F.unit_off[l + 1]) ++l;
    const FinLevel& lv = F.lv[l];
    const int n_patches = lv.gy * lv.gx;
    const int i = w - F.unit_off[l];                                          // unit index (b*T + t)*n_patches + patch
    const int bt = i / n_patches, patch = i - bt * n_patches;
    const int b = bt / T, t = bt - b * T;
    const long long q_prev = (long long)b * (T - 1) + t - 1;                  // pair (t, t-1)
    const bool has_prev = t >= 1, has_next = (t & 1) && t + 1 < T;
    float with_prev, with_next;
    frame_pair_values(partial, q_prev, has_prev, q_prev + 1, has_next, patch, lv, stat, eps, with_prev, with_next);
    if (!has_prev) with_prev = -INFINITY;
    if (!has_next) with_next = -INFINITY;
    if (lane == 0 && has_prev && pair_sim) pair_sim[F.pair_off[l] + q_prev * n_patches + patch] = with_prev;
    if (lane == 0) {
        if ((t & 1) == 0) { best_sim[w] = -INFINITY; best_idx[w] = i; }
        else if (with_next > with_prev) { best_sim[w] = with_next; best_idx[w] = i + n_patches; }
        else { best_sim[w] = with_prev; best_idx[w] = i - n_patches; }
    }
}

template <int DT>
static void frame_dispatch(int lpr, dim3 grid, cudaStream_t s, const uint8_t* x, int T, int P, int cpr, float eps,
                           float* pos_sim, float4* partial, int ppc, const PatchGrid& pg) {
    switch (lpr) {
        case 1:  OC_LAUNCH((frame_pair_kernel<DT, 1>), grid, PAIR_THREADS, 0, s, x, T, P, cpr, eps, pos_sim, partial, ppc, pg); break;
        case 2:  OC_LAUNCH((frame_pair_kernel<DT, 2>), grid, PAIR_THREADS, 0, s, x, T, P, cpr, eps, pos_sim, partial, ppc, pg); break;
        case 4:  OC_LAUNCH((frame_pair_kernel<DT, 4>), grid, PAIR_THREADS, 0, s, x, T, P, cpr, eps, pos_sim, partial, ppc, pg); break;
        case 8:  OC_LAUNCH((frame_pair_kernel<DT, 8>), grid, PAIR_THREADS, 0, s, x, T, P, cpr, eps, pos_sim, partial, ppc, pg); break;
        case 16: OC_LAUNCH((frame_pair_kernel<DT, 16>), grid, PAIR_THREADS, 0, s, x, T, P, cpr, eps, pos_sim, partial, ppc, pg); break;
        default: OC_LAUNCH((frame_pair_kernel<DT, 32>), grid, PAIR_THREADS, 0, s, x, T, P, cpr, eps, pos_sim, partial, ppc, pg); break;
    }
}

struct FramePlan {
    bool march;          // time-marching kernel (rows short enough to keep in registers) or pair kernel
    int lpr, n_tiles, ppc, seg_len, n_seg;     // n_tiles = patches * tiles per patch
    PatchGrid pg;
};
// sm_count only steers how a clip is cut into segments (never the number of partial records, so the
// workspace size does not depend on it)
static FramePlan frame_plan(const Geo& g, int sm_count) {
    FramePlan f;
    const int cpr = g.C * g.elem_bytes / 16, P = g.H * g.W;
    int l = 4;
    while (l < 32 && l * 5 < cpr) l <<= 1;               // about 5 chunks per lane
    f.march = g.T >= 2 && cpr <= l * MARCH_CPL;
    if (f.march) {
        f.lpr = l;
        f.ppc = PAIR_THREADS / l;
        f.pg = make_patch_grid(g, f.ppc);
        f.n_tiles = f.pg.n_patches * f.pg.tiles_per_patch;
        // segments: enough CTAs for a few waves, but at least 6 pairs per segment (one frame re-read each)
        int n_seg = 1;
        while ((long long)f.n_tiles * g.B * n_seg < (long long)sm_count * 4 && (g.T - 1) / (n_seg + 1) >= 6) ++n_seg;
        f.seg_len = (g.T - 1 + n_seg - 1) / n_seg;
        const int seg_cap = 40960 / ((PAIR_THREADS / l) * (int)sizeof(float2));   // per-pair, per-position values live in shared memory
        if (f.seg_len > seg_cap) f.seg_len = seg_cap;
        f.n_seg = (g.T - 1 + f.seg_len - 1) / f.seg_len;
    } else {
        f.lpr = lanes_per_row(cpr);
        f.ppc = (PAIR_THREADS / f.lpr) * 4;              // every thread-group takes about 4 positions
        f.pg = make_patch_grid(g, f.ppc);
        f.n_tiles = f.pg.n_patches * f.pg.tiles_per_patch;
        f.seg_len = f.n_seg = 0;
    }
    return f;
}

size_t frame_workspace_bytes(const Geo& g) {
    size_t pairs = (size_t)g.B * (size_t)(g.T > 1 ? g.T - 1 : 0);
    return pairs * (size_t)frame_plan(g, 1).n_tiles * sizeof(float4) + 256;
}

template <int DT>
static void march_dispatch(int lpr, dim3 grid, size_t smem, cudaStream_t s, const uint8_t* x, int T, int P, int cpr,
                           float eps, int seg_len, int n_seg, float* pos_sim, float4* partial, const PatchGrid& pg) {
#define OC_MARCH(L) do { if (cpr <= 5 * L) OC_LAUNCH((frame_march_kernel<DT, L, 5>), grid, PAIR_THREADS, smem, s, x, T, P, cpr, eps, seg_len, n_seg, pos_sim, partial, pg); \
                         else OC_LAUNCH((frame_march_kernel<DT, L, 8>), grid, PAIR_THREADS, smem, s, x, T, P, cpr, eps, seg_len, n_seg, pos_sim, partial, pg); } while (0)
    switch (lpr) {
        case 4: OC_MARCH(4); break; case 8: OC_MARCH(8); break; case 16: OC_MARCH(16); break; default: OC_MARCH(32); break;
    }
#undef OC_MARCH
}

// Every frame entry point runs this: `scratch` holds the partial records.  ctx may be null (no launch
// counters then).  levels == nullptr: one level, the layout's own grid; otherwise n_levels grids
// (gy_l, gx_l), each dividing the layout's, whose outputs follow one another in best_sim / best_idx
// (B*T*gy_l*gx_l entries each) and pair_sim (B*(T-1)*gy_l*gx_l each).
static oc_status run_frame_match(oc_ctx* ctx, int sm_count, uint8_t* scratch, const Geo& g, const void* x, float* best_sim,
                                 int32_t* best_idx, float* pos_sim, float* pair_sim, cudaStream_t s,
                                 int n_levels = 1, const int32_t* levels = nullptr) {
    const int P = g.H * g.W, cpr = g.C * g.elem_bytes / 16;
    const int n_pairs = g.B * (g.T - 1);
    const FramePlan f = frame_plan(g, sm_count);
    float4* partial = (float4*)scratch;
    if (n_pairs > 65535 || (long long)g.B * (f.march ? f.n_seg : 1) > 65535) return OC_ERR_UNSUPPORTED;
    struct Scope { oc_ctx* c; int k; cudaStream_t s; LaunchScope* l; 
                   Scope(oc_ctx* c_, int k_, cudaStream_t s_) : c(c_), k(k_), s(s_), l(c_ ? new LaunchScope(c_, k_, s_) : nullptr) {}
                   ~Scope() { delete l; } };
    if (n_pairs > 0) {
        Scope scope(ctx, OC_K_FRAME, s);
        if (f.march) {
            dim3 grid((unsigned)f.n_tiles, (unsigned)(g.B * f.n_seg));
            const size_t smem = ((size_t)f.seg_len * sizeof(float2) + sizeof(float)) * (size_t)(PAIR_THREADS / f.lpr);
            if (g.dtype == OC_DTYPE_BF16)
                march_dispatch<OC_DTYPE_BF16>(f.lpr, grid, smem, s, (const uint8_t*)x, g.T, P, cpr, g.eps, f.seg_len, f.n_seg, pos_sim, partial, f.pg);
            else
                march_dispatch<OC_DTYPE_F32>(f.lpr, grid, smem, s, (const uint8_t*)x, g.T, P, cpr, g.eps, f.seg_len, f.n_seg, pos_sim, partial, f.pg);
        } else {
            dim3 grid((unsigned)f.n_tiles, (unsigned)n_pairs);
            if (g.dtype == OC_DTYPE_BF16)
                frame_dispatch<OC_DTYPE_BF16>(f.lpr, grid, s, (const uint8_t*)x, g.T, P, cpr, g.eps, pos_sim, partial, f.ppc, f.pg);
            else
                frame_dispatch<OC_DTYPE_F32>(f.lpr, grid, s, (const uint8_t*)x, g.T, P, cpr, g.eps, pos_sim, partial, f.ppc, f.pg);
        }
    }
    FinLevels F;
    F.n = n_levels;
    F.unit_off[0] = F.pair_off[0] = 0;
    for (int l = 0; l < n_levels; ++l) {
        FinLevel& lv = F.lv[l];
        lv.gy = levels ? levels[2 * l] : g.gy; lv.gx = levels ? levels[2 * l + 1] : g.gx;
        lv.ry = g.gy / lv.gy; lv.rx = g.gx / lv.gx;
        lv.gx_fine = g.gx; lv.np_fine = g.gy * g.gx;
        lv.tiles_per_patch = f.pg.tiles_per_patch;
        lv.n_pos = f.pg.Pp * lv.ry * lv.rx;
        F.unit_off[l + 1] = F.unit_off[l] + g.B * g.T * lv.gy * lv.gx;
        F.pair_off[l + 1] = F.pair_off[l] + n_pairs * lv.gy * lv.gx;
    }
    {
        Scope scope(ctx, OC_K_FRAME_FIN, s);
        const int warps = PAIR_THREADS / 32;
        OC_LAUNCH((frame_finalize_kernel), (unsigned)((F.unit_off[n_levels] + warps - 1) / warps), PAIR_THREADS, 0, s,
            partial, F, g.B, g.T, g.frame_stat, g.eps, pair_sim, best_sim, best_idx);
    }
    return last_launch_status();
}

oc_status launch_match_frame(oc_ctx* ctx, const Geo& g, const void* x, float* best_sim, int32_t* best_idx,
                             float* pos_sim, float* pair_sim, cudaStream_t s) {
    return run_frame_match(ctx, ctx->sm_count, (uint8_t*)ctx->workspace, g, x, best_sim, best_idx, pos_sim, pair_sim, s);
}

oc_status launch_match_frame_levels(oc_ctx* ctx, const Geo& g, const void* x, int n_levels, const int32_t* levels,
                                    float* best_sim, int32_t* best_idx, float* pos_sim, float* pair_sim, cudaStream_t s) {
    return run_frame_match(ctx, ctx->sm_count, (uint8_t*)ctx->workspace, g, x, best_sim, best_idx, pos_sim, pair_sim, s, n_levels, levels);
}

// ------------------------------------------------------------------------------------------------
// Block Cache: inside every sy x sx neighbourhood, each non-representative position's T*C
// descriptor against the representative's.  grid = (cell tiles, B*T): a thread-group handles one
// (cell, t) and writes the C-long partial sums {|rep|^2, then (dot, |cand|^2) per member}; the
// finalize kernel adds the T partials of a cell in order of t.
// ------------------------------------------------------------------------------------------------
static constexpr int MAX_MEMBERS = 16;

template <int DT, int LPR, int NCMAX>
__global__ void __launch_bounds__(PAIR_THREADS)
block_partial_kernel(const uint8_t* __restrict__ x, int T, int H, int W, int cpr, int sy, int sx, int oy, int ox,
                     float* __restrict__ partial, int rec /*floats per (cell,t)*/) {
    pdl_enter();
    const int bt = blockIdx.y;
    const int cells_x = W / sx, cells = (H / sy) * cells_x;
    const int groups = PAIR_THREADS / LPR;
    const int grp = threadIdx.x / LPR, lane = threadIdx.x % LPR;
    const int cell_raw = blockIdx.x * groups + grp;
    const bool valid = cell_raw < cells;             // out-of-range groups redo cell 0 and write nothing,
    const int cell = valid ? cell_raw : 0;           // so that every lane takes part in the shuffles
    const int cy = cell / cells_x, cx = cell - cy * cells_x;
    const long long row_bytes = (long long)cpr * 16;
    const uint8_t* frame = x + (long long)bt * H * W * row_bytes;
    const uint8_t* rep = frame + ((long long)(cy * sy + oy) * W + (cx * sx + ox)) * row_bytes;
    const int b = bt / T, t = bt - b * T;
    float* out = partial + (((long long)b * T + t) * cells + cell) * rec;     // [b][t][cell][rec]

    // the neighbourhood's other members, in (my, mx) order
    const int nc = sy * sx - 1;
    const uint8_t* cand[NCMAX];
    const int rep_m = oy * sx + ox;
#pragma unroll
    for (int k = 0; k < NCMAX; ++k) {
        const int m = k + (k >= rep_m ? 1 : 0);      // k-th non-representative member
        const int my = m / sx, mx = m - my * sx;
        cand[k] = k < nc ? frame + ((long long)(cy * sy + my) * W + (cx * sx + mx)) * row_bytes : rep;
    }
    // one pass over the channels: the representative's chunk and every member's chunk are loaded
    // together, so up to 1 + nc loads are in flight per lane and step
    float rn = 0.f, dot[NCMAX], na[NCMAX];
#pragma unroll
    for (int k = 0; k < NCMAX; ++k) { dot[k] = 0.f; na[k] = 0.f; }
    for (int c = lane; c < cpr; c += LPR) {
        const uint4 r = ld_nc_v4(rep + (long long)c * 16);
        uint4 a[NCMAX];
#pragma unroll
        for (int k = 0; k < NCMAX; ++k)
            if (k < nc) a[k] = ld_nc_v4(cand[k] + (long long)c * 16);
        Chunk<DT>::sq(r, rn);
#pragma unroll
        for (int k = 0; k < NCMAX; ++k)
            if (k < nc) Chunk<DT>::acc2(a[k], r, dot[k], na[k]);
    }
    rn = group_sum<LPR>(rn);
    if (valid && lane == 0) out[0] = rn;
#pragma unroll
    for (int k = 0; k < NCMAX; ++k) {
        if (k < nc) {                                 // nc is uniform over the grid
            const float d = group_sum<LPR>(dot[k]), n = group_sum<LPR>(na[k]);
            if (valid && lane == 0) { out[1 + 2 * k] = d; out[2 + 2 * k] = n; }
        }
    }
}

// Variant for neighbourhoods with at most three candidates and rows short enough to hold in
// registers (CPL chunks per lane): every load of the item - the representative's row and all
// candidates' rows - is issued before the first one is used.
template <int DT, int LPR, int CPL>
__global__ void __launch_bounds__(PAIR_THREADS)
block_partial_reg_kernel(const uint8_t* __restrict__ x, int T, int H, int W, int cpr, int sy, int sx, int oy, int ox,
                         float* __restrict__ partial, int rec) {
    pdl_enter();
    constexpr int NC = 3;
    const int bt = blockIdx.y;
    const int cells_x = W / sx, cells = (H / sy) * cells_x;
    const int groups = PAIR_THREADS / LPR;
    const int grp = threadIdx.x / LPR, lane = threadIdx.x % LPR;
    const int cell_raw = blockIdx.x * groups + grp;
    const bool valid = cell_raw < cells;
    const int cell = valid ? cell_raw : 0;
    const int cy = cell / cells_x, cx = cell - cy * cells_x;
    const long long row_bytes = (long long)cpr * 16;
    const uint8_t* frame = x + (long long)bt * H * W * row_bytes;
    const uint8_t* rep = frame + ((long long)(cy * sy + oy) * W + (cx * sx + ox)) * row_bytes;
    const int b = bt / T, t = bt - b * T;
    float* out = partial + (((long long)b * T + t) * cells + cell) * rec;     // [b][t][cell][rec]
    const int nc = sy * sx - 1, rep_m = oy * sx + ox;
    const uint8_t* cand[NC];
#pragma unroll
    for (int k = 0; k < NC; ++k) {
        const int m = k + (k >= rep_m ? 1 : 0);
        const int my = m / sx, mx = m - my * sx;
        cand[k] = k < nc ? frame + ((long long)(cy * sy + my) * W + (cx * sx + mx)) * row_bytes : rep;
    }
    uint4 r[CPL], a[NC][CPL];
#pragma unroll
    for (int j = 0; j < CPL; ++j) {
        const int c = lane + j * LPR;
        if (c < cpr) {
            r[j] = ld_nc_v4(rep + (long long)c * 16);
#pragma unroll
            for (int k = 0; k < NC; ++k)
                if (k < nc) a[k][j] = ld_nc_v4(cand[k] + (long long)c * 16);
        }
    }
    float rn = 0.f, dot[NC] = {0.f, 0.f, 0.f}, na[NC] = {0.f, 0.f, 0.f};
#pragma unroll
    for (int j = 0; j < CPL; ++j) {
        if (lane + j * LPR < cpr) {
            Chunk<DT>::sq(r[j], rn);
#pragma unroll
            for (int k = 0; k < NC; ++k)
                if (k < nc) Chunk<DT>::acc2(a[k][j], r[j], dot[k], na[k]);
        }
    }
    rn = group_sum<LPR>(rn);
    if (valid && lane == 0) out[0] = rn;
#pragma unroll
    for (int k = 0; k < NC; ++k) {
        if (k < nc) {
            const float d = group_sum<LPR>(dot[k]), n = group_sum<LPR>(na[k]);
            if (valid && lane == 0) { out[1 + 2 * k] = d; out[2 + 2 * k] = n; }
        }
    }
}

// Fused variant of the two kernels around it, for clips whose T frames fit the thread-groups of one CTA
// (T <= threads / LPR): a thread-group still handles one (cell, t) with every load issued up front, but
// all T groups of a cell sit in the same CTA, leave their partial sums in shared memory, and the cell's
// candidates are finished right there -- the T partials never travel through global memory and the
// finalize launch disappears (what matters on small tensors, where a launch costs more than the work).
// The sums over t are taken in the same order as block_finalize_kernel takes them: same bits.
template <int DT, int LPR, int CPL, int THREADS>
__global__ void __launch_bounds__(THREADS)
block_fused_kernel(const uint8_t* __restrict__ x, int T, int H, int W, int cpr, int sy, int sx, int oy, int ox,
                   int cells_per_cta, float eps, float* __restrict__ best_sim, int32_t* __restrict__ best_idx) {
    pdl_enter();
    constexpr int NC = 3, REC = 1 + 2 * NC, GROUPS = THREADS / LPR;
    __shared__ float rec[GROUPS][REC];
    const int b = blockIdx.y;
    const int cells_x = W / sx, cells = (H / sy) * cells_x;
    const int grp = threadIdx.x / LPR, lane = threadIdx.x % LPR;
    const int lc = grp / T, t = grp - lc * T;                       // local cell, frame
    const int cell_raw = blockIdx.x * cells_per_cta + lc;
    const bool valid = lc < cells_per_cta && cell_raw < cells;      // idle groups redo cell 0 and publish nothing
    const int cell = valid ? cell_raw : 0;
    const int cy = cell / cells_x, cx = cell - cy * cells_x;
    const long long row_bytes = (long long)cpr * 16;
    const uint8_t* frame = x + ((long long)b * T + (valid ? t : 0)) * H * W * row_bytes;
    const uint8_t* rep = frame + ((long long)(cy * sy + oy) * W + (cx * sx + ox)) * row_bytes;
    const int nc = sy * sx - 1, rep_m = oy * sx + ox;
    const uint8_t* cand[NC];
#pragma unroll
    for (int k = 0; k < NC; ++k) {
        const int m = k + (k >= rep_m ? 1 : 0);
        const int my = m / sx, mx = m - my * sx;
        cand[k] = k < nc ? frame + ((long long)(cy * sy + my) * W + (cx * sx + mx)) * row_bytes : rep;
    }
    uint4 r[CPL], a[NC][CPL];
#pragma unroll
    for (int j = 0; j < CPL; ++j) {
        const int c = lane + j * LPR;
        if (c < cpr) {
            r[j] = ld_nc_v4(rep + (long long)c * 16);
#pragma unroll
            for (int k = 0; k < NC; ++k)
                if (k < nc) a[k][j] = ld_nc_v4(cand[k] + (long long)c * 16);
        }
    }
    float rn = 0.f, dot[NC] = {0.f, 0.f, 0.f}, na[NC] = {0.f, 0.f, 0.f};
#pragma unroll
    for (int j = 0; j < CPL; ++j) {
        if (lane + j * LPR < cpr) {
            Chunk<DT>::sq(r[j], rn);
#pragma unroll
            for (int k = 0; k < NC; ++k)
                if (k < nc) Chunk<DT>::acc2(a[k][j], r[j], dot[k], na[k]);
        }
    }
    rn = group_sum<LPR>(rn);
    if (lane == 0) rec[grp][0] = rn;
#pragma unroll
    for (int k = 0; k < NC; ++k) {
        const float d = group_sum<LPR>(dot[k]), n = group_sum<LPR>(na[k]);
        if (lane == 0) { rec[grp][1 + 2 * k] = d; rec[grp][2 + 2 * k] = n; }
    }
    __syncthreads();
    // one thread per (local cell, member of the neighbourhood): the representative's own entry, or a
    // candidate's cosine from the T partials added in order of t
    const int members = sy * sx;
    for (int i = threadIdx.x; i < cells_per_cta * members; i += THREADS) {
        const int c_l = i / members, m = i - c_l * members;
        const int c_g = blockIdx.x * cells_per_cta + c_l;
        if (c_g >= cells) continue;
        const int gy = c_g / cells_x, gx = c_g - gy * cells_x;
        const int my = m / sx, mx = m - my * sx;
        const long long P = (long long)H * W;
        const long long pos = (long long)b * P + (long long)(gy * sy + my) * W + (gx * sx + mx);
        const long long rep_pos = (long long)b * P + (long long)(gy * sy + oy) * W + (gx * sx + ox);
        if (m == rep_m) { best_sim[pos] = -INFINITY; best_idx[pos] = (int32_t)pos; continue; }
        const int k = m > rep_m ? m - 1 : m;
        float s_rn = 0.f, s_dot = 0.f, s_na = 0.f;
        for (int tt = 0; tt < T; ++tt) {
            const float* q = rec[c_l * T + tt];
            s_rn += q[0]; s_dot += q[1 + 2 * k]; s_na += q[2 + 2 * k];
        }
        best_sim[pos] = clamp_unit(s_dot / (fmaxf(sqrtf(s_na), eps) * fmaxf(sqrtf(s_rn), eps)));
        best_idx[pos] = (int32_t)rep_pos;
    }
}

__global__ void __launch_bounds__(PAIR_THREADS)
block_finalize_kernel(const float* __restrict__ partial, int B, int T, int H, int W, int sy, int sx, int oy, int ox,
                      int rec, float eps, float* __restrict__ best_sim, int32_t* __restrict__ best_idx) {
    pdl_enter();
    const long long n = (long long)B * H * W;
    const long long i = (long long)blockIdx.x * PAIR_THREADS + threadIdx.x;
    if (i >= n) return;
    const int P = H * W;
    const int b = (int)(i / P), p = (int)(i - (long long)b * P);
    const int y = p / W, xx = p - y * W;
    const int my = y % sy, mx = xx % sx;
    if (my == oy && mx == ox) { best_sim[i] = -INFINITY; best_idx[i] = (int32_t)i; return; }
    const int cells_x = W / sx, cells = (H / sy) * cells_x;
    const int cell = (y / sy) * cells_x + xx / sx;
    int k = my * sx + mx;                        // rank among the neighbourhood's non-representatives
    if (k > oy * sx + ox) --k;
    // records are laid out [b][t][cell][rec]: neighbouring threads (cells) read neighbouring records
    const float* recs = partial + ((long long)b * T * cells + cell) * rec;
    const long long t_stride = (long long)cells * rec;
    float rn = 0.f, dot = 0.f, na = 0.f;
    for (int t = 0; t < T; ++t) {
        rn += recs[t * t_stride]; dot += recs[t * t_stride + 1 + 2 * k]; na += recs[t * t_stride + 2 + 2 * k];
    }
    best_sim[i] = clamp_unit(dot / (fmaxf(sqrtf(na), eps) * fmaxf(sqrtf(rn), eps)));
    best_idx[i] = (int32_t)((long long)b * P + (y - my + oy) * W + (xx - mx + ox));
}

size_t block_workspace_bytes(const Geo& g) {
    size_t cells = (size_t)(g.H / g.sy) * (size_t)(g.W / g.sx);
    size_t rec = 1 + 2 * (size_t)(g.sy * g.sx - 1);
    return (size_t)g.B * cells * (size_t)g.T * rec * sizeof(float) + 256;
}

template <int DT>
static void block_dispatch(int lpr, dim3 grid, cudaStream_t s, const uint8_t* x, const Geo& g, int cpr, float* partial, int rec) {
#define OC_BLK(L) do { if (g.sy * g.sx - 1 <= 3) OC_LAUNCH((block_partial_kernel<DT, L, 3>), grid, PAIR_THREADS, 0, s, x, g.T, g.H, g.W, cpr, g.sy, g.sx, g.oy, g.ox, partial, rec); \
                       else OC_LAUNCH((block_partial_kernel<DT, L, 15>), grid, PAIR_THREADS, 0, s, x, g.T, g.H, g.W, cpr, g.sy, g.sx, g.oy, g.ox, partial, rec); } while (0)
    switch (lpr) {
        case 1: OC_BLK(1); break; case 2: OC_BLK(2); break; case 4: OC_BLK(4); break;
        case 8: OC_BLK(8); break; case 16: OC_BLK(16); break; default: OC_BLK(32); break;
    }
#undef OC_BLK
}

oc_status launch_match_block(oc_ctx* ctx, const Geo& g, const void* x, float* best_sim, int32_t* best_idx,
                             cudaStream_t s) {
    if (g.sy * g.sx > MAX_MEMBERS) return OC_ERR_UNSUPPORTED;
    const int cpr = g.C * g.elem_bytes / 16;
    const int cells = (g.H / g.sy) * (g.W / g.sx);
    const int rec = 1 + 2 * (g.sy * g.sx - 1);
    float* partial = (float*)ctx->workspace;
    if ((int64_t)g.B * g.T > 65535) return OC_ERR_UNSUPPORTED;
    // register-resident variant: about five chunks per lane, at most three candidates
    int lr = 4;
    while (lr < 32 && lr * 5 < cpr) lr <<= 1;
    const bool reg_variant = g.sy * g.sx - 1 <= 3 && cpr <= 5 * lr;
    const int lpr = reg_variant ? lr : lanes_per_row(cpr);
    // one launch instead of two when a cell's T frames fit one CTA's thread-groups and the whole grid is
    // small enough that the second launch would cost more than it saves (large tensors keep the two-kernel
    // form: its first kernel has no CTA-wide barrier and more CTAs in flight)
    const int fused_threads = g.T * lpr <= PAIR_THREADS ? PAIR_THREADS : 512;
    const bool fused = reg_variant && g.T * lpr <= 512 && (long long)cells * g.B * g.T * lpr <= 512ll * 4 * ctx->sm_count;
    if (fused) {
        const int groups = fused_threads / lpr, cells_per_cta = groups / g.T;
        dim3 grid((unsigned)((cells + cells_per_cta - 1) / cells_per_cta), (unsigned)g.B);
        LaunchScope scope(ctx, OC_K_BLOCK, s);
        const uint8_t* xb = (const uint8_t*)x;
#define OC_BLKF(DTV, L, TH) OC_LAUNCH((block_fused_kernel<DTV, L, 5, TH>), grid, TH, 0, s, xb, g.T, g.H, g.W, cpr, g.sy, g.sx, g.oy, g.ox, cells_per_cta, g.eps, best_sim, best_idx)
#define OC_BLKF_L(DTV, TH) switch (lpr) { case 4: OC_BLKF(DTV, 4, TH); break; case 8: OC_BLKF(DTV, 8, TH); break; case 16: OC_BLKF(DTV, 16, TH); break; default: OC_BLKF(DTV, 32, TH); break; }
        if (g.dtype == OC_DTYPE_BF16) { if (fused_threads == 256) { OC_BLKF_L(OC_DTYPE_BF16, 256) } else { OC_BLKF_L(OC_DTYPE_BF16, 512) } }
        else { if (fused_threads == 256) { OC_BLKF_L(OC_DTYPE_F32, 256) } else { OC_BLKF_L(OC_DTYPE_F32, 512) } }
#undef OC_BLKF_L
#undef OC_BLKF
        return last_launch_status();
    }
    {
        const int groups = PAIR_THREADS / lpr;
        dim3 grid((unsigned)((cells + groups - 1) / groups), (unsigned)(g.B * g.T));
        LaunchScope scope(ctx, OC_K_BLOCK, s);
        const uint8_t* xb = (const uint8_t*)x;
        if (reg_variant) {
#define OC_BLKR(DTV, L) OC_LAUNCH((block_partial_reg_kernel<DTV, L, 5>), grid, PAIR_THREADS, 0, s, xb, g.T, g.H, g.W, cpr, g.sy, g.sx, g.oy, g.ox, partial, rec)
            if (g.dtype == OC_DTYPE_BF16) {
                switch (lpr) { case 4: OC_BLKR(OC_DTYPE_BF16, 4); break; case 8: OC_BLKR(OC_DTYPE_BF16, 8); break;
                               case 16: OC_BLKR(OC_DTYPE_BF16, 16); break; default: OC_BLKR(OC_DTYPE_BF16, 32); break; }
            } else {
                switch (lpr) { case 4: OC_BLKR(OC_DTYPE_F32, 4); break; case 8: OC_BLKR(OC_DTYPE_F32, 8); break;
                               case 16: OC_BLKR(OC_DTYPE_F32, 16); break; default: OC_BLKR(OC_DTYPE_F32, 32); break; }
            }
#undef OC_BLKR
        } else if (g.dtype == OC_DTYPE_BF16) {
            block_dispatch<OC_DTYPE_BF16>(lpr, grid, s, xb, g, cpr, partial, rec);
        } else {
            block_dispatch<OC_DTYPE_F32>(lpr, grid, s, xb, g, cpr, partial, rec);
        }
    }
    {
        const long long n = (long long)g.B * g.H * g.W;
        LaunchScope scope(ctx, OC_K_BLOCK_FIN, s);
        OC_LAUNCH((block_finalize_kernel), (unsigned)((n + PAIR_THREADS - 1) / PAIR_THREADS), PAIR_THREADS, 0, s, 
            partial, g.B, g.T, g.H, g.W, g.sy, g.sx, g.oy, g.ox, rec, g.eps, best_sim, best_idx);
    }
    return last_launch_status();
}

}  // namespace oc


// ------------------------------------------------------------------------------------------------
// Allocation-free Frame Cache match (see oc_match_frame_noalloc in omnicache.h).
//
// Same two kernels as launch_match_frame, but the partial sums live in a fixed array that is part
// of the library image, so the call never asks the driver (or anybody's allocator) for memory.
// ------------------------------------------------------------------------------------------------
namespace oc {

static constexpr size_t NOALLOC_SCRATCH_BYTES = OC_NOALLOC_SCRATCH_BYTES;
static constexpr int NOALLOC_MAX_DEVICES = 64;

// Every GPU that loads this library carries this array until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_SCRATCH_BYTES];

// In host code `g_noalloc_scratch` is only a handle for the runtime, not a device address.  The
// address each device gave the array is looked up once per device and kept here, together with the
// device's SM count (which steers the segment split of the streaming kernel).
static void* g_noalloc_dev_ptr[NOALLOC_MAX_DEVICES] = {};
static int g_noalloc_sm_count[NOALLOC_MAX_DEVICES] = {};
static std::mutex g_noalloc_mutex;

// Makes the driver load every kernel instance the frame path can launch (a query of its attributes
// does that), so that later calls find all code resident and have no reason to touch the loader.
template <int DT>
static bool noalloc_touch_kernels() {
    cudaFuncAttributes fa;
    bool ok = true;
#define OC_TOUCH(k) ok = ok && cudaFuncGetAttributes(&fa, k) == cudaSuccess
#define OC_TOUCH_L(L)                                                                                  \
    OC_TOUCH((frame_march_kernel<DT, L, 5>)); OC_TOUCH((frame_march_kernel<DT, L, 8>)); OC_TOUCH((frame_pair_kernel<DT, L>))
    OC_TOUCH_L(4); OC_TOUCH_L(8); OC_TOUCH_L(16); OC_TOUCH_L(32);
    OC_TOUCH((frame_pair_kernel<DT, 1>)); OC_TOUCH((frame_pair_kernel<DT, 2>));
#undef OC_TOUCH_L
#undef OC_TOUCH
    return ok;
}

}  // namespace oc

extern "C" oc_status oc_match_frame_noalloc(int device, const oc_layout* layout, const void* x, float* best_sim,
                                            int32_t* best_idx, float* pair_sim, void* stream) {
    using namespace oc;
    if (device < 0 || device >= NOALLOC_MAX_DEVICES || !x || !best_sim || !best_idx) return OC_ERR_INVALID_ARG;
    Geo g;
    oc_status st = make_geo(layout, &g);
    if (st != OC_OK) return st;
    if (g.kind != OC_KIND_FRAME) return OC_ERR_INVALID_ARG;
    if (((uintptr_t)x & 15u) != 0) return OC_ERR_ALIGNMENT;
    const int n_pairs = g.B * (g.T - 1);
    if (n_pairs > 65535) return OC_ERR_UNSUPPORTED;
    // the fixed array must hold what the context workspace would hold for this layout
    if (frame_workspace_bytes(g) > NOALLOC_SCRATCH_BYTES) return OC_ERR_WORKSPACE;

    DeviceGuard guard(device);
    if (!guard.ok) return OC_ERR_CUDA;
    uint8_t* scratch = nullptr;
    int sm_count = 0;
    {
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!g_noalloc_dev_ptr[device]) {
            // set-up, once per device, with that device current
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) { cudaGetLastError(); return OC_ERR_CUDA; }
            int n_sm = 0;
            if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || n_sm <= 0) {
                cudaGetLastError(); return OC_ERR_CUDA;
            }
            cudaFuncAttributes fa;
            if (!noalloc_touch_kernels<OC_DTYPE_BF16>() || !noalloc_touch_kernels<OC_DTYPE_F32>() ||
                cudaFuncGetAttributes(&fa, frame_finalize_kernel) != cudaSuccess) { cudaGetLastError(); return OC_ERR_CUDA; }
            g_noalloc_sm_count[device] = n_sm;
            g_noalloc_dev_ptr[device] = p;
        }
        scratch = (uint8_t*)g_noalloc_dev_ptr[device];
        sm_count = g_noalloc_sm_count[device];
    }
    // nothing in the array has to start at zero: every partial record and every pair value that
    // the kernels read is written first by this call's own kernels
    return run_frame_match(nullptr, sm_count, scratch, g, x, best_sim, best_idx, nullptr, pair_sim, (cudaStream_t)stream);
}
