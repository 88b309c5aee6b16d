// Dense (Token Cache) matching, the parts that are not the tensor-core kernel:
//   norms_kernel     inverse row norms in fp32 + reset of the packed arg-max keys (pre-pass)
//   dense_simt_kernel  fp32-FMA all-pairs matcher for fp32 inputs, self-match and shapes the tcgen05
//                      kernel does not cover (fp32 inputs must hold 1e-5, which rules out tf32)
//   finalize_kernel  packed key -> best_sim / best_idx
// Both matchers merge their per-tile row maxima with one 64-bit atomicMax per (row, tile) on
// (ordered(value) << 32 | ~index): largest value, then lowest index, independent of arrival order.
#include "common.cuh"

namespace oc {

// ---- pre-pass ----------------------------------------------------------------------------------
// A thread-group of LPR lanes owns a row (about five 16-byte chunks per lane), so a
// warp has 32/LPR rows in flight and every lane keeps several independent loads outstanding.
template <int DT, int LPR>
__global__ void __launch_bounds__(256)
norms_kernel(const uint8_t* __restrict__ x, long long n_tok, int cpr, float eps,
             float* __restrict__ inv_norm, unsigned long long* __restrict__ keys) {
    pdl_enter();
    constexpr int CPL = 8;                                   // chunks a lane holds at once
    const int lane = threadIdx.x % LPR;
    const long long groups_total = (long long)gridDim.x * (256 / LPR);
    const long long grp0 = (long long)blockIdx.x * (256 / LPR) + threadIdx.x / LPR;
    const long long n_iter = (n_tok + groups_total - 1) / groups_total;   // same trip count for every thread
    for (long long it = 0; it < n_iter; ++it) {
        const long long row = grp0 + it * groups_total;
        const bool valid = row < n_tok;
        const uint8_t* r = x + (valid ? row : 0) * (long long)cpr * 16;
        float s = 0.f;
        for (int c0 = 0; c0 < cpr; c0 += CPL * LPR) {
            uint4 v[CPL];
#pragma unroll
            for (int k = 0; k < CPL; ++k)
                if (c0 + lane + k * LPR < cpr) v[k] = ld_nc_v4(r + (long long)(c0 + lane + k * LPR) * 16);
#pragma unroll
            for (int k = 0; k < CPL; ++k)
                if (c0 + lane + k * LPR < cpr) Chunk<DT>::sq(v[k], s);
        }
#pragma unroll
        for (int d = LPR / 2; d >= 1; d >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, d);
        if (valid && lane == 0) {
            inv_norm[row] = 1.0f / fmaxf(sqrtf(s), eps);
            keys[row] = 0ull;
        }
    }
}

template <int DT>
static void norms_dispatch(int sm_count, cudaStream_t s, const uint8_t* x, long long n_tok, int cpr, float eps,
                           float* inv_norm, unsigned long long* keys) {
    int lpr = 4;
    while (lpr < 32 && lpr * 5 < cpr) lpr <<= 1;
    const long long rows_per_block = 256 / lpr;
    long long blocks = (n_tok + rows_per_block - 1) / rows_per_block;
    // one pass per CTA: short CTAs that retire and are replaced keep more loads in flight than a
    // persistent grid does (measured: 0.75 against 0.71 of the copy bandwidth on a 147 MB tensor)
    const long long cap = 0x7FFFFFFFll;
    (void)sm_count;
    if (blocks > cap) blocks = cap;
    switch (lpr) {
        case 4:  OC_LAUNCH((norms_kernel<DT, 4>), (unsigned)blocks, 256, 0, s, x, n_tok, cpr, eps, inv_norm, keys); break;
        case 8:  OC_LAUNCH((norms_kernel<DT, 8>), (unsigned)blocks, 256, 0, s, x, n_tok, cpr, eps, inv_norm, keys); break;
        case 16: OC_LAUNCH((norms_kernel<DT, 16>), (unsigned)blocks, 256, 0, s, x, n_tok, cpr, eps, inv_norm, keys); break;
        default: OC_LAUNCH((norms_kernel<DT, 32>), (unsigned)blocks, 256, 0, s, x, n_tok, cpr, eps, inv_norm, keys); break;
    }
}

// ---- fp32-FMA matcher --------------------------------------------------------------------------
static constexpr int ST = 64;        // tile: 64 candidate rows x 64 representative columns
static constexpr int SK = 32;        // K elements staged per step

struct SimtGeo {
    GroupMap gm;
    int C, reps_per_group, Ws;       // Ws: representative lattice width inside a patch
};

__device__ __forceinline__ int rep_local_unit(const SimtGeo& sg, int r) {
    if (sg.gm.self_match) return r;
    int rh = r / sg.Ws, rw = r - rh * sg.Ws;
    return (rh * sg.gm.sy + sg.gm.oy) * sg.gm.Wp + rw * sg.gm.sx + sg.gm.ox;
}

template <int DT>
__device__ __forceinline__ void load8(const uint8_t* row, int k0, int C, float* dst) {
    // 8 consecutive elements starting at k0 (k0 % 8 == 0); zeros beyond C
    if (DT == OC_DTYPE_BF16) {
        if (k0 < C) {                                   // C % 8 == 0
            uint4 v = ld_nc_v4(row + (long long)k0 * 2);
            dst[0] = bf16_lo(v.x); dst[1] = bf16_hi(v.x); dst[2] = bf16_lo(v.y); dst[3] = bf16_hi(v.y);
            dst[4] = bf16_lo(v.z); dst[5] = bf16_hi(v.z); dst[6] = bf16_lo(v.w); dst[7] = bf16_hi(v.w);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) dst[i] = 0.f;
        }
    } else {
#pragma unroll
        for (int h = 0; h < 2; ++h) {                   // C % 4 == 0
            if (k0 + 4 * h < C) {
                uint4 v = ld_nc_v4(row + (long long)(k0 + 4 * h) * 4);
                dst[4 * h] = __uint_as_float(v.x); dst[4 * h + 1] = __uint_as_float(v.y);
                dst[4 * h + 2] = __uint_as_float(v.z); dst[4 * h + 3] = __uint_as_float(v.w);
            } else {
                dst[4 * h] = dst[4 * h + 1] = dst[4 * h + 2] = dst[4 * h + 3] = 0.f;
            }
        }
    }
}

template <int DT>
__global__ void __launch_bounds__(256)
dense_simt_kernel(const uint8_t* __restrict__ x, SimtGeo sg, const float* __restrict__ inv_norm,
                  unsigned long long* __restrict__ keys, float* __restrict__ aux_sim) {
    pdl_enter();
    __shared__ __align__(16) float As[SK][ST + 4];
    __shared__ __align__(16) float Bs[SK][ST + 4];
    __shared__ long long a_tok[ST], b_tok[ST];          // global token index, -1 = masked
    const int U = sg.gm.units_per_group, R = sg.reps_per_group, C = sg.C;
    const long long g = blockIdx.z;
    const int u0 = blockIdx.y * ST, r0 = blockIdx.x * ST;
    const int tid = threadIdx.x;
    const long long row_bytes = (long long)C * (DT == OC_DTYPE_BF16 ? 2 : 4);

    if (tid < ST) {
        int u = u0 + tid;
        a_tok[tid] = (u < U && gm_is_cand(sg.gm, u)) ? gm_unit_index(sg.gm, g, u) : -1;
    } else if (tid < 2 * ST) {
        int r = r0 + tid - ST;
        b_tok[tid - ST] = (r < R) ? gm_unit_index(sg.gm, g, rep_local_unit(sg, r)) : -1;
    }
    __syncthreads();

    const int ty = tid >> 4, tx = tid & 15;              // 4x4 outputs per thread
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    const int lrow = tid >> 2, lk = (tid & 3) * 8;       // loader: 64 rows x 4 threads x 8 elements
    for (int k0 = 0; k0 < C; k0 += SK) {
        float va[8], vb[8];
        long long ta = a_tok[lrow], tb = b_tok[lrow];
        if (ta >= 0) load8<DT>(x + ta * row_bytes, k0 + lk, C, va);
        else {
#pragma unroll
            for (int i = 0; i < 8; ++i) va[i] = 0.f;
        }
        if (tb >= 0) load8<DT>(x + tb * row_bytes, k0 + lk, C, vb);
        else {
#pragma unroll
            for (int i = 0; i < 8; ++i) vb[i] = 0.f;
        }
        __syncthreads();                                  // previous step's reads are done
#pragma unroll
        for (int i = 0; i < 8; ++i) { As[lk + i][lrow] = va[i]; Bs[lk + i][lrow] = vb[i]; }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < SK; ++k) {
            float4 a = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            float4 b = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
    }

    // epilogue: scale by the representative's inverse norm, row arg-max over the tile, merge
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const long long ti = a_tok[ty * 4 + i];
        float best = -INFINITY; long long arg = 0x7FFFFFFF;
        const float inv_i = ti >= 0 ? inv_norm[ti] : 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const long long tj = b_tok[tx * 4 + j];
            if (ti < 0 || tj < 0 || tj == ti) continue;
            const float v = acc[i][j] * inv_norm[tj];
            if (aux_sim) {
                const int u = u0 + ty * 4 + i, r = r0 + tx * 4 + j;
                aux_sim[((long long)g * U + u) * R + r] = clamp_unit(v * inv_i);
            }
            if (v > best) { best = v; arg = tj; }         // columns ascend: strict > keeps the lowest
        }
        // reduce over the 16 threads (tx) that share this row: lanes of one half-warp
#pragma unroll
        for (int d = 8; d >= 1; d >>= 1) {
            float ob = __shfl_xor_sync(0xFFFFFFFFu, best, d);
            long long oa = __shfl_xor_sync(0xFFFFFFFFu, arg, d);
            if (ob > best || (ob == best && oa < arg)) { best = ob; arg = oa; }
        }
        if (tx == 0 && ti >= 0 && arg != 0x7FFFFFFF) atomicMax(keys + ti, pack_key(best, (uint32_t)arg));
    }
}

// ---- key unpack --------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
finalize_kernel(GroupMap gm, long long n_groups, const float* __restrict__ inv_norm,
                const unsigned long long* __restrict__ keys, float* __restrict__ best_sim,
                int32_t* __restrict__ best_idx) {
    pdl_enter();
    const long long w = (long long)blockIdx.x * 256 + threadIdx.x;
    const int U = gm.units_per_group;
    if (w >= n_groups * U) return;
    const long long g = w / U;
    const int u = (int)(w - g * U);
    const long long i = gm_unit_index(gm, g, u);
    const unsigned long long key = keys[i];
    if (!gm_is_cand(gm, u) || key == 0ull) {
        best_sim[i] = -INFINITY; best_idx[i] = (int32_t)i;
        return;
    }
    const float v = ordered_to_f32((uint32_t)(key >> 32));
    best_sim[i] = clamp_unit(v * inv_norm[i]);
    best_idx[i] = (int32_t)(0xFFFFFFFFu - (uint32_t)(key & 0xFFFFFFFFull));
}

size_t frame_workspace_bytes(const Geo&);
size_t block_workspace_bytes(const Geo&);

size_t match_workspace_bytes(const Geo& g) {
    if (g.kind == OC_KIND_FRAME) return frame_workspace_bytes(g);
    if (g.kind == OC_KIND_BLOCK) return block_workspace_bytes(g);
    size_t n = (size_t)g.n_units;
    return n * sizeof(unsigned long long) + ((n * sizeof(float) + 255) / 256) * 256 + 256;
}

// the pre-pass alone (also used by the joint frame-pair matcher)
void launch_norms(oc_ctx* ctx, const Geo& g, const void* x, float* inv_norm, unsigned long long* keys, cudaStream_t s) {
    const int cpr = g.C * g.elem_bytes / 16;
    LaunchScope scope(ctx, OC_K_NORMS, s);
    if (g.dtype == OC_DTYPE_BF16)
        norms_dispatch<OC_DTYPE_BF16>(ctx->sm_count, s, (const uint8_t*)x, g.n_units, cpr, g.eps, inv_norm, keys);
    else
        norms_dispatch<OC_DTYPE_F32>(ctx->sm_count, s, (const uint8_t*)x, g.n_units, cpr, g.eps, inv_norm, keys);
}

oc_status launch_match_token(oc_ctx* ctx, const Geo& g, const void* x, float* best_sim, int32_t* best_idx,
                             float* aux_sim, cudaStream_t s) {
    const long long n_tok = g.n_units;
    if (n_tok == 0) return OC_OK;
    unsigned long long* keys = (unsigned long long*)ctx->workspace;
    float* inv_norm = (float*)((uint8_t*)ctx->workspace + (size_t)n_tok * sizeof(unsigned long long));
    const int cpr = g.C * g.elem_bytes / 16;
    {
        LaunchScope scope(ctx, OC_K_NORMS, s);
        if (g.dtype == OC_DTYPE_BF16)
            norms_dispatch<OC_DTYPE_BF16>(ctx->sm_count, s, (const uint8_t*)x, n_tok, cpr, g.eps, inv_norm, keys);
        else
            norms_dispatch<OC_DTYPE_F32>(ctx->sm_count, s, (const uint8_t*)x, n_tok, cpr, g.eps, inv_norm, keys);
    }
    oc_status st = OC_ERR_UNSUPPORTED;
    if (tc_match_supported(g)) st = launch_match_token_tc(ctx, g, x, inv_norm, keys, aux_sim, s);
    if (st == OC_ERR_UNSUPPORTED) {
        SimtGeo sg;
        sg.gm = make_group_map(g); sg.C = g.C; sg.reps_per_group = (int)g.reps_per_group; sg.Ws = g.Ws;
        if (g.n_groups > 65535) return OC_ERR_UNSUPPORTED;
        dim3 grid((unsigned)((g.reps_per_group + ST - 1) / ST), (unsigned)((g.units_per_group + ST - 1) / ST),
                  (unsigned)g.n_groups);
        if (grid.y > 65535) return OC_ERR_UNSUPPORTED;
        LaunchScope scope(ctx, OC_K_MATCH_SIMT, s);
        if (g.dtype == OC_DTYPE_BF16)
            OC_LAUNCH(dense_simt_kernel<OC_DTYPE_BF16>, grid, 256, 0, s, (const uint8_t*)x, sg, inv_norm, keys, aux_sim);
        else
            OC_LAUNCH(dense_simt_kernel<OC_DTYPE_F32>, grid, 256, 0, s, (const uint8_t*)x, sg, inv_norm, keys, aux_sim);
        st = last_launch_status();
    }
    if (st != OC_OK) return st;
    {
        LaunchScope scope(ctx, OC_K_MATCH_FIN, s);
        OC_LAUNCH(finalize_kernel, (unsigned)((n_tok + 255) / 256), 256, 0, s, make_group_map(g), g.n_groups, inv_norm, keys,
                  best_sim, best_idx);
    }
    return last_launch_status();
}

}  // namespace oc
