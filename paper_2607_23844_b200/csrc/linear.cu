// The wrapped layer's projection with the gather folded into its A-operand load and the restore folded
// into its store (Appendix A's token compaction and its permutation/scatter on the way back, taken one
// step further: the dense buffer between gather and the layer, and between the layer and restore, is
// never written):
//     out[dst(r), :] = bf16( sum_k a[src(r), k] * w[n, k] ),     r = 0 .. n_rows-1
// src(r) = a_idx[r] (the kept-index list of select), dst(r) = out_idx[r] (the same list: computed rows
// go straight to their positions in the restored tensor, which already holds the cached rows).
//
// One CTA per (128 or 256) x N_TILE output tile: two 128-row tiles share the weight tile whenever that
// still leaves enough CTAs (the kernel is bound by the turnaround of its 3-4 stage ring -- copy latency,
// proxy fence, hand-over, MMA, commit -- and 256 rows per CTA put twice the MMA work into a stage).
// Rows that are not gathered (a_idx null: only the restore is folded in) travel as plain TMA boxes.
// Warp-specialised like the matcher:
//   warps 0..3  A producers: the gathered rows arrive by 16-byte asynchronous copies (cp.async), eight
//               threads per row, written straight into the K-major, 128-byte-swizzled tile (chunk c of
//               row r goes to r*128 + ((c ^ (r & 7)) << 4), which is where a TMA box would have put it);
//               three stages of copies are in flight per thread, and a stage is handed to the tensor cores
//               with a proxy fence per thread and one mbarrier arrival per warp.  (One single-row TMA box per
//               gathered row was tried first: correct, but the SM's TMA unit takes ~60 cycles per box
//               whatever its size, and 128 boxes per stage made the kernel ten times slower.)
//   warp 4      W producer: ONE TMA box per stage for the weight tile
//   warp 5      tcgen05.mma kind::f16, fp32 accumulator in TMEM; owns alloc / dealloc
//   warps 6..9  epilogue: thread = output row; tcgen05.ld 32 columns at a time, round to bf16, 64-byte
//               stores into the row out_idx names
// K and N tails are zero-filled by TMA and not stored.  Every wait is bounded (OC_ERR_TIMEOUT in the
// status word).  No cluster features are used.
#include <mutex>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace oc {

static constexpr int LIN_BM = 128, LIN_BK = 64;
static constexpr int LIN_THREADS = 320;
static constexpr int LIN_A_PRODUCERS = 128;      // threads of warps 0..3
static constexpr int LIN_A_BYTES = LIN_BM * LIN_BK * 2;          // 16 KB
static constexpr int LIN_MAX_STAGES = 6;

struct LinParams {
    CUtensorMap mapW;            // {K, N},      box {64, n_tile}
    CUtensorMap mapA;            // {K, a_rows}, box {64, 128}: used when the rows are not gathered (a_idx null)
    const int32_t* a_idx;        // nullable
    const int32_t* out_idx;      // nullable
    const uint16_t* a;
    uint16_t* out;
    long long n_rows, N, K, a_rows, out_rows;
    int kblocks, n_tile, n_stages, stage_bytes, depth;
    int* status;
};

template <int N_TILE, int M_TILES>
__global__ void __launch_bounds__(LIN_THREADS, 1)
linear_gs_kernel(const __grid_constant__ LinParams P) {
    // the operand ring starts at the base of dynamic shared memory (1024-byte aligned for the 128-byte
    // swizzle: no static shared memory in front of it; checked below); barriers and flags follow it
    extern __shared__ __align__(1024) uint8_t lin_smem[];
    uint64_t* bars = (uint64_t*)(lin_smem + (size_t)P.n_stages * P.stage_bytes);      // [2 * MAX_STAGES + 1]
    uint32_t* tmem_slot_p = (uint32_t*)(bars + 2 * LIN_MAX_STAGES + 1);
    volatile int* abort_flag = (volatile int*)(tmem_slot_p + 1);
    const uint32_t tiles = smem_u32(lin_smem);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * LIN_MAX_STAGES, bar_acc = bar_empty + 8 * LIN_MAX_STAGES;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long m0 = (long long)blockIdx.x * (LIN_BM * M_TILES);
    const int n0 = blockIdx.y * N_TILE;
    const int STAGES = P.n_stages;
    constexpr uint32_t W_BYTES = N_TILE * LIN_BK * 2;

    if ((tiles & 1023u) != 0) {                                   // never expected; refuse rather than compute garbage
        if (threadIdx.x == 0) atomicCAS(P.status, 0, OC_ERR_ALIGNMENT);
        return;
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < LIN_MAX_STAGES; ++s) { mbar_init(bar_full + 8 * s, P.a_idx ? LIN_A_PRODUCERS / 32 + 1 : 1); mbar_init(bar_empty + 8 * s, 1); }
        mbar_init(bar_acc, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        tma_prefetch_map(&P.mapW);
        if (!P.a_idx) tma_prefetch_map(&P.mapA);
    }
    if (warp == 5) tmem_alloc_cta1(smem_u32(tmem_slot_p), (uint32_t)(N_TILE * M_TILES));
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_p;
    // everything read below (the index lists, the operands) may come from the kernel before this one
    pdl_wait();
    if (threadIdx.x == 0) pdl_launch_dependents();

    if (warp < 4 && P.a_idx) {
        // ================================ A producers ===========================================
        const int t = threadIdx.x, sub = t & 7, rbase = t >> 3;       // chunk of the row; rows rbase + 16 p
        constexpr int RPT = 8 * M_TILES;                               // rows per thread and stage
        long long src_off[RPT];                                        // element offset of the row in `a`, or -1
#pragma unroll
        for (int p = 0; p < RPT; ++p) {
            const long long r = m0 + rbase + 16 * p;
            src_off[p] = -1;
            if (r < P.n_rows) {
                const int v = P.a_idx ? __ldg(P.a_idx + r) : (int)r;
                if (v >= 0 && v < P.a_rows) src_off[p] = (long long)v * P.K;
            }
        }
        const int DEPTH = P.depth;                                     // stages of copies in flight per thread (1..3)
        int stage = 0; uint32_t phase = 0;
        bool ok = true;
        int kb = 0;
        for (; kb < P.kblocks; ++kb) {
            bool go = true;
            if (lane == 0) go = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag);
            go = __shfl_sync(0xFFFFFFFFu, (int)go, 0) != 0;
            if (!go) { ok = false; break; }
            const uint32_t a_dst = tiles + (uint32_t)(stage * P.stage_bytes);
            const long long k_el = (long long)kb * LIN_BK + sub * 8;
            const uint32_t src_size = k_el < P.K ? 16u : 0u;          // past K: zero fill (K % 8 == 0: whole chunks)
#pragma unroll
            for (int p = 0; p < RPT; ++p) {
                if (src_off[p] >= 0) {
                    const int r = rbase + 16 * p;                      // (tiles of 128 rows follow one another: r * 128)
                    const uint32_t dst = a_dst + (uint32_t)(r * 128 + ((sub ^ (r & 7)) << 4));
                    const uint16_t* src = P.a + src_off[p] + (src_size ? k_el : 0);
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(dst), "l"(src), "r"(src_size) : "memory");
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            if (kb >= DEPTH) {                                          // the copies of stage kb - DEPTH have landed
                if (DEPTH == 1) asm volatile("cp.async.wait_group 1;" ::: "memory");
                else if (DEPTH == 2) asm volatile("cp.async.wait_group 2;" ::: "memory");
                else asm volatile("cp.async.wait_group 3;" ::: "memory");
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();                                           // every lane's copies landed and are fenced
                if (lane == 0) mbar_arrive(bar_full + 8 * ((kb - DEPTH) % STAGES));
            }
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        // hand over what is still in flight (on a give-up too: the arrivals are harmless and nothing is left
        // writing this CTA's shared memory when it retires)
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0)
            for (int j = (kb > DEPTH ? kb - DEPTH : 0); j < kb; ++j) mbar_arrive(bar_full + 8 * (j % STAGES));
        if (!ok && lane == 0) { atomicCAS(P.status, 0, OC_ERR_TIMEOUT); *abort_flag = 1; }
    } else if (warp == 4) {
        // ================================ W producer ============================================
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            for (int kb = 0; kb < P.kblocks; ++kb) {
                if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                // rows that are not gathered travel as plain 128-row boxes (rows past the end read as zeros)
                mbar_arrive_expect_tx(bar_full + 8 * stage, W_BYTES + (P.a_idx ? 0u : (uint32_t)(M_TILES * LIN_A_BYTES)));
                tma_load_2d(tiles + (uint32_t)(stage * P.stage_bytes) + M_TILES * LIN_A_BYTES, &P.mapW, kb * LIN_BK, n0, bar_full + 8 * stage);
                if (!P.a_idx)
                    for (int mt = 0; mt < M_TILES; ++mt)
                        tma_load_2d(tiles + (uint32_t)(stage * P.stage_bytes) + mt * LIN_A_BYTES, &P.mapA, kb * LIN_BK,
                                    (int)(m0 + mt * LIN_BM), bar_full + 8 * stage);
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
            if (!ok) {
                atomicCAS(P.status, 0, OC_ERR_TIMEOUT);
                *abort_flag = 1;
                const unsigned long long t0 = global_ns();             // boxes already issued: a bounded chance to land
                while (global_ns() - t0 < 2000000ull) {}
            }
        }
    } else if (warp == 5) {
        // ================================ MMA issuer ============================================
        constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N_TILE >> 3) << 17) |
                                   ((uint32_t)(LIN_BM >> 4) << 24);        // D=f32, A=B=bf16, K-major, N, M=128
        const uint32_t issue = elect_one();
        int stage = 0; uint32_t phase = 0;
        bool ok = true;
        for (int kb = 0; kb < P.kblocks; ++kb) {
            if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) ok = false;
            if (!__all_sync(0xFFFFFFFFu, ok)) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_addr = tiles + (uint32_t)(stage * P.stage_bytes);
            const uint64_t a_desc = make_smem_desc(a_addr), a1_desc = make_smem_desc(a_addr + LIN_A_BYTES);
            const uint64_t b_desc = make_smem_desc(a_addr + M_TILES * LIN_A_BYTES);
#pragma unroll
            for (int k4 = 0; k4 < 4; ++k4) {                           // UMMA K = 16: +32 bytes along the swizzled row
                tc_mma_bf16<false>(tmem_base, a_desc + 2 * k4, b_desc + 2 * k4, IDESC, (uint32_t)((kb | k4) != 0), issue);
                if (M_TILES == 2)                                      // the second 128 rows share the weight tile
                    tc_mma_bf16<false>(tmem_base + N_TILE, a1_desc + 2 * k4, b_desc + 2 * k4, IDESC, (uint32_t)((kb | k4) != 0), issue);
            }
            tc_commit<false>(bar_empty + 8 * stage, issue);            // frees the stage when the MMAs retire
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit<false>(bar_acc, issue);
        else if (lane == 0) { atomicCAS(P.status, 0, OC_ERR_TIMEOUT); *abort_flag = 1; }
    } else if (warp >= 6) {
        // ================================ epilogue ==============================================
        const int quarter = warp & 3;                                  // TMEM lanes this warp may read
        long long dst[M_TILES];
#pragma unroll
        for (int mt = 0; mt < M_TILES; ++mt) {
            const long long r = m0 + mt * LIN_BM + quarter * 32 + lane;
            dst[mt] = -1;
            if (r < P.n_rows) {
                const bool src_ok = !P.a_idx || __ldg(P.a_idx + r) >= 0;
                const long long d = P.out_idx ? (long long)__ldg(P.out_idx + r) : r;
                if (src_ok && d >= 0 && d < P.out_rows) dst[mt] = d;
            }
        }
        const bool ready = __all_sync(0xFFFFFFFFu, mbar_wait(bar_acc, 0, abort_flag));
        if (ready) {
            tc_fence_after();
#pragma unroll
            for (int mt = 0; mt < M_TILES; ++mt) {
                const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(mt * N_TILE);
                uint16_t* orow = P.out + (dst[mt] >= 0 ? dst[mt] : 0) * P.N + n0;
#pragma unroll 1
                for (int ch = 0; ch < N_TILE / 32; ++ch) {
                    uint32_t v[32];
                    tmem_ld32(t_row + (uint32_t)(ch * 32), v);
                    tmem_ld_wait();
                    if (dst[mt] >= 0) {
#pragma unroll
                        for (int j = 0; j < 32; j += 8) {
                            const int col = n0 + ch * 32 + j;
                            if (col < P.N) {                           // N % 8 == 0: whole 16-byte groups
                                uint4 o;
                                asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o.x) : "f"(__uint_as_float(v[j + 1])), "f"(__uint_as_float(v[j])));
                                asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o.y) : "f"(__uint_as_float(v[j + 3])), "f"(__uint_as_float(v[j + 2])));
                                asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o.z) : "f"(__uint_as_float(v[j + 5])), "f"(__uint_as_float(v[j + 4])));
                                asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o.w) : "f"(__uint_as_float(v[j + 7])), "f"(__uint_as_float(v[j + 6])));
                                st_v4(orow + ch * 32 + j, o);
                            }
                        }
                    }
                }
            }
            tc_fence_before();
        } else if (lane == 0) {
            atomicCAS(P.status, 0, OC_ERR_TIMEOUT);
            *abort_flag = 1;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 5) tmem_dealloc_cta1(tmem_base, (uint32_t)(N_TILE * M_TILES));
}

typedef CUresult (*LinEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static LinEncodeFn lin_encode_fn() {
    static LinEncodeFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (LinEncodeFn)p;
        else
            cudaGetLastError();
    });
    return fn;
}

oc_status launch_linear_gs(oc_ctx* ctx, const void* a, int64_t a_rows, int64_t K, const int32_t* a_idx, int64_t n_rows,
                           const void* w, int64_t N, void* out, int64_t out_rows, const int32_t* out_idx, cudaStream_t s) {
    if (n_rows == 0) return OC_OK;
    LinEncodeFn enc = lin_encode_fn();
    if (!enc) return OC_ERR_UNSUPPORTED;
    const int n_tile = N >= 256 ? 256 : 128;
    LinParams P;
    memset(&P, 0, sizeof(P));
    const cuuint32_t estr[2] = {1, 1};
    if (!a_idx) {
        const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)a_rows};
        const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
        const cuuint32_t box[2] = {(cuuint32_t)LIN_BK, (cuuint32_t)LIN_BM};
        if (enc(&P.mapA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void*)a, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return OC_ERR_UNSUPPORTED;
    }
    {
        const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)N};
        const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
        const cuuint32_t box[2] = {(cuuint32_t)LIN_BK, (cuuint32_t)n_tile};
        if (enc(&P.mapW, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void*)w, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return OC_ERR_UNSUPPORTED;
    }
    P.a_idx = a_idx; P.out_idx = out_idx; P.a = (const uint16_t*)a; P.out = (uint16_t*)out;
    P.n_rows = n_rows; P.N = N; P.K = K; P.a_rows = a_rows; P.out_rows = out_rows;
    P.kblocks = (int)((K + LIN_BK - 1) / LIN_BK);
    P.n_tile = n_tile;
    // two 128-row tiles per CTA share the weight tile (twice the MMA work per ring stage, whose turnaround
    // bounds the kernel) whenever that still leaves enough CTAs for the device
    const int m_tiles_per_cta = (n_tile == 256 && ((n_rows + 255) / 256) * ((N + n_tile - 1) / n_tile) >= (ctx->sm_count * 3) / 4) ? 2 : 1;
    P.stage_bytes = m_tiles_per_cta * LIN_A_BYTES + n_tile * LIN_BK * 2;
    const int smem_budget = 200 * 1024;
    P.n_stages = smem_budget / P.stage_bytes;
    if (P.n_stages > LIN_MAX_STAGES) P.n_stages = LIN_MAX_STAGES;
    if (P.n_stages > P.kblocks) P.n_stages = P.kblocks < 2 ? 2 : P.kblocks;
    P.depth = P.n_stages >= 5 ? 3 : (P.n_stages >= 4 ? 2 : 1);
    P.status = ctx->d_status;
    const size_t smem = (size_t)P.n_stages * P.stage_bytes + (2 * LIN_MAX_STAGES + 1) * 8 + 64;
    static PerDeviceOnce attr_once;                 // (the context's device is current here)
    const bool attr_ok = attr_once.ensure(ctx->device, [] {
        const bool ok =
            cudaFuncSetAttribute(linear_gs_kernel<256, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 201 * 1024) == cudaSuccess &&
            cudaFuncSetAttribute(linear_gs_kernel<256, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 201 * 1024) == cudaSuccess &&
            cudaFuncSetAttribute(linear_gs_kernel<128, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 201 * 1024) == cudaSuccess;
        if (!ok) cudaGetLastError();
        return ok;
    });
    if (!attr_ok) return OC_ERR_CUDA;
    const long long rows_per_cta = (long long)LIN_BM * m_tiles_per_cta;
    const long long m_tiles = (n_rows + rows_per_cta - 1) / rows_per_cta, n_tiles = (N + n_tile - 1) / n_tile;
    if (m_tiles > 0x7FFFFFFFll || n_tiles > 65535) return OC_ERR_UNSUPPORTED;
    dim3 grid((unsigned)m_tiles, (unsigned)n_tiles);
    LaunchScope scope(ctx, OC_K_LINEAR, s);
    if (n_tile == 256 && m_tiles_per_cta == 2) OC_LAUNCH((linear_gs_kernel<256, 2>), grid, LIN_THREADS, smem, s, P);
    else if (n_tile == 256) OC_LAUNCH((linear_gs_kernel<256, 1>), grid, LIN_THREADS, smem, s, P);
    else OC_LAUNCH((linear_gs_kernel<128, 1>), grid, LIN_THREADS, smem, s, P);
    return last_launch_status();
}

}  // namespace oc
