// Dense (Token Cache) matcher on the 5th-generation tensor cores.
//
// For every token group the candidates x representatives similarity matrix is a dense contraction
// over the channel axis, S = A * B^T with A = candidate rows, B = representative rows, both read IN
// PLACE from the channel-last feature tensor: each sub-lattice of the (sy, sx)-strided grid is one
// 4-D TMA tensor map {C, W/sx, H/sy, B*T}, so a box {64 channels, bw, bh, 1} lands in shared memory
// as a canonical K-major, 128-byte-swizzled tile of bw*bh rows.  No operand is gathered or copied.
//
// One persistent CTA per SM, warp specialised:
//   warp 0      TMA producer   (one lane): global -> smem ring, mbarrier complete_tx
//   warp 1      MMA issuer     (one lane): tcgen05.mma kind::f16 (bf16 x bf16 -> fp32 in TMEM),
//               128 x BN accumulator, double buffered in TMEM so the next tile's MMAs overlap the
//               epilogue; also owns tcgen05.alloc / dealloc
//   warps 2..5  epilogue: thread r owns candidate row r (= TMEM lane r): tcgen05.ld 32 columns at a
//               time, scale by the representative's inverse norm, running (max, arg max) in
//               registers - no cross-thread reduction - then ONE 64-bit atomicMax per row merges the
//               tile into the packed key array (largest value, then lowest index: order independent).
// Rows / columns of a box that fall outside the patch are masked in the epilogue (bias -inf), so
// ragged lattices need no padding.  Every mbarrier wait is bounded: on expiry the CTA records
// OC_ERR_TIMEOUT in the context's status word, drains its outstanding copies, frees TMEM and exits.
#include <cuda.h>

#include <mutex>

#include "common.cuh"

namespace oc {

static constexpr int BM = 128;           // candidate rows per tile (UMMA M)
static constexpr int BK = 64;            // channels per stage: 128 bytes of bf16 = one swizzle row
static constexpr int TC_THREADS = 192;
static constexpr int MAX_LATTICES = 9;
static constexpr unsigned long long WAIT_LIMIT_NS = 1000000000ull;   // 1 s per wait

struct TcParams {
    CUtensorMap maps[MAX_LATTICES];      // one per sub-lattice member (my*sx + mx)
    int H, W, sy, sx, gy, gx;
    int Hp, Wp, Hs, Ws;                  // patch size; representative-lattice size per patch
    int rep_member;                      // oy*sx + ox
    int n_cand_lat;                      // sy*sx - 1
    int kblocks;
    int bwA_log2, bhA, n_wtA, n_htA;     // A box: (1<<bwA_log2) x bhA lattice points = 128 rows
    int bwB_log2, bhB, n_wtB, n_htB;     // B box: BN rows
    int total_units;
    int units_per_group, reps_per_group;
    const float* inv_norm;
    unsigned long long* keys;
    float* aux;
    int* status;
};

// ---- PTX wrappers ------------------------------------------------------------------------------
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
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    unsigned spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 255u) == 0) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > WAIT_LIMIT_NS) return false;
        }
    }
    return true;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        :: "r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* v) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
// Barrier over the 128 epilogue threads that also ANDs a flag: every thread learns whether any
// thread has given up, so they all leave the unit loop together.
__device__ __forceinline__ bool epilogue_barrier_all(bool ok) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "bar.red.and.pred p, 1, 128, q;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(r) : "r"((uint32_t)ok) : "memory");
    return r != 0;
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// K-major, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr) {
    const uint32_t lo = ((addr >> 4) & 0x3FFFu) | (1u << 16);           // start address, LBO = 16 B (unused)
    const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);         // SBO = 1024 B, version 1, SWIZZLE_128B
    return ((uint64_t)hi << 32) | lo;
}

struct UnitCoord {
    int bt, py, px, member;              // frame, patch, candidate sub-lattice member
    int htA, wtA, htB, wtB;
    long long g;
};
__device__ __forceinline__ UnitCoord decode_unit(const TcParams& P, int u) {
    UnitCoord c;
    const int nB = P.n_htB * P.n_wtB, nA = P.n_htA * P.n_wtA;
    int tb = u % nB; u /= nB;
    int ta = u % nA; u /= nA;
    int k = u % P.n_cand_lat; u /= P.n_cand_lat;
    c.g = u;
    c.px = u % P.gx; u /= P.gx;
    c.py = u % P.gy; c.bt = u / P.gy;
    c.member = k < P.rep_member ? k : k + 1;
    c.htA = ta / P.n_wtA; c.wtA = ta - c.htA * P.n_wtA;
    c.htB = tb / P.n_wtB; c.wtB = tb - c.htB * P.n_wtB;
    return c;
}

template <int BN, int STAGES>
struct TcSmem {
    static constexpr int A_BYTES = BM * BK * 2;
    static constexpr int B_BYTES = BN * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int TILE_BYTES = STAGES * STAGE_BYTES;
    static constexpr int COL_BYTES = 2 * BN * 8;                        // {scale, bias} x 2 buffers
    static constexpr int BAR_BYTES = (2 * STAGES + 4 + 1) * 8 + 16;
    static constexpr int TOTAL = 1024 + TILE_BYTES + COL_BYTES + BAR_BYTES;
};

template <int BN, int STAGES>
__global__ void __launch_bounds__(TC_THREADS, 1)
match_tc_kernel(const __grid_constant__ TcParams P) {
    using S = TcSmem<BN, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    float2* colsb = (float2*)(smem + S::TILE_BYTES);                    // [2][BN]
    uint64_t* bars = (uint64_t*)(smem + S::TILE_BYTES + S::COL_BYTES);
    // barrier layout: full[STAGES], empty[STAGES], acc_full[2], acc_empty[2], drain
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_acc_full = bar_empty + 8 * STAGES, bar_acc_empty = bar_acc_full + 16;
    const uint32_t bar_drain = bar_acc_empty + 16;
    uint32_t* tmem_slot = (uint32_t*)(bars + 2 * STAGES + 5);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
    const uint32_t tiles_base = smem_u32(smem);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t TMEM_COLS = 2 * BN;                              // 256 or 512: a power of two

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        mbar_init(bar_acc_full, 1); mbar_init(bar_acc_full + 8, 1);
        mbar_init(bar_acc_empty, 128); mbar_init(bar_acc_empty + 8, 128);
        mbar_init(bar_drain, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int bwA = 1 << P.bwA_log2, bwB = 1 << P.bwB_log2;

    if (warp == 0) {
        // ================================ TMA producer ==========================================
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            uint32_t armed = 0;                       // stages with a copy possibly still in flight
            bool ok = true;
            for (int u = blockIdx.x; u < P.total_units && ok; u += gridDim.x) {
                const UnitCoord c = decode_unit(P, u);
                const CUtensorMap* mapA = &P.maps[c.member];
                const CUtensorMap* mapB = &P.maps[P.rep_member];
                const int wA = c.px * P.Ws + c.wtA * bwA, hA = c.py * P.Hs + c.htA * P.bhA;
                const int wB = c.px * P.Ws + c.wtB * bwB, hB = c.py * P.Hs + c.htB * P.bhB;
                for (int kb = 0; kb < P.kblocks; ++kb) {
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t full = bar_full + 8 * stage;
                    const uint32_t a_dst = tiles_base + stage * S::STAGE_BYTES;
                    mbar_arrive_expect_tx(full, S::STAGE_BYTES);
                    tma_load_4d(a_dst, mapA, kb * BK, wA, hA, c.bt, full);
                    tma_load_4d(a_dst + S::A_BYTES, mapB, kb * BK, wB, hB, c.bt, full);
                    armed |= 1u << stage;
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                atomicCAS(P.status, 0, OC_ERR_TIMEOUT);
                *abort_flag = 1;
                // copies already issued still write this CTA's shared memory: give each a bounded
                // chance to land before the CTA retires (the parity armed last is phase or phase^1)
                for (int s = 0; s < STAGES; ++s) {
                    if (!(armed & (1u << s))) continue;
                    const uint32_t par = (s < stage) ? phase : (phase ^ 1u);
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar_full + 8 * s, par) && global_ns() - t0 < 20000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        // ================================ MMA issuer ============================================
        if (lane == 0) {
            constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) |
                                       ((uint32_t)(BM >> 4) << 24);   // D=f32, A=B=bf16, K-major both
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            int it = 0;
            for (int u = blockIdx.x; u < P.total_units && ok; u += gridDim.x, ++it) {
                const int buf = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                if (!mbar_wait(bar_acc_empty + 8 * buf, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                for (int kb = 0; kb < P.kblocks; ++kb) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = tiles_base + stage * S::STAGE_BYTES;
                    const uint64_t a_desc = make_smem_desc(a_addr);
                    const uint64_t b_desc = make_smem_desc(a_addr + S::A_BYTES);
#pragma unroll
                    for (int k4 = 0; k4 < BK / 16; ++k4)              // UMMA K = 16: 32 bytes along the row
                        tc_mma_bf16(d_tmem, a_desc + (uint64_t)(2 * k4), b_desc + (uint64_t)(2 * k4), IDESC,
                                    (uint32_t)((kb | k4) != 0));
                    tc_commit(bar_empty + 8 * stage);                  // frees the stage when the MMAs retire
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) tc_commit(bar_acc_full + 8 * buf);
            }
            if (!ok) { atomicCAS(P.status, 0, OC_ERR_TIMEOUT); *abort_flag = 1; }
            // all MMAs issued by this thread must retire before TMEM is released
            tc_commit(bar_drain);
            const unsigned long long t0 = global_ns();
            while (!mbar_try_wait(bar_drain, 0) && global_ns() - t0 < WAIT_LIMIT_NS) {}
        }
    } else {
        // ================================ epilogue ==============================================
        const int et = threadIdx.x - 64;                               // 0..127
        const int lane_group = warp & 3;                               // TMEM lanes this warp may read
        const int row = lane_group * 32 + lane;                        // tile row owned by this thread
        bool ok = true;
        int it = 0;
        for (int u = blockIdx.x; u < P.total_units; u += gridDim.x, ++it) {
            const int buf = it & 1;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
            const UnitCoord c = decode_unit(P, u);
            const int my_rep = P.rep_member / P.sx, mx_rep = P.rep_member - my_rep * P.sx;
            // ---- column table: inverse norm and validity of every representative of the B box ----
            float2* cs = colsb + buf * BN;
            for (int n = et; n < BN; n += 128) {
                const int hl = n >> P.bwB_log2, wl = n & (bwB - 1);
                const int hs = c.htB * P.bhB + hl, ws = c.wtB * bwB + wl;
                float2 v = make_float2(0.f, -INFINITY);
                if (hs < P.Hs && ws < P.Ws) {
                    const int y = (c.py * P.Hs + hs) * P.sy + my_rep, x = (c.px * P.Ws + ws) * P.sx + mx_rep;
                    v = make_float2(__ldg(P.inv_norm + ((long long)c.bt * P.H + y) * P.W + x), 0.f);
                }
                cs[n] = v;
            }
            if (!epilogue_barrier_all(ok)) { ok = false; break; }     // also orders the table writes
            // ---- this thread's candidate row ------------------------------------------------------
            const int my = c.member / P.sx, mx = c.member - my * P.sx;
            const int hlA = row >> P.bwA_log2, wlA = row & (bwA - 1);
            const int hsA = c.htA * P.bhA + hlA, wsA = c.wtA * bwA + wlA;
            const bool row_ok = hsA < P.Hs && wsA < P.Ws;
            const int yA = (c.py * P.Hs + hsA) * P.sy + my, xA = (c.px * P.Ws + wsA) * P.sx + mx;
            const long long tokA = ((long long)c.bt * P.H + yA) * P.W + xA;
            float inv_a = 0.f;
            float* aux_row = nullptr;
            if (P.aux && row_ok) {
                inv_a = __ldg(P.inv_norm + tokA);
                const int u_local = (hsA * P.sy + my) * P.Wp + wsA * P.sx + mx;
                aux_row = P.aux + ((long long)c.g * P.units_per_group + u_local) * P.reps_per_group;
            }
            // warp-uniform outcome: the TMEM loads below are warp-collective
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(bar_acc_full + 8 * buf, acc_phase, abort_flag))) { ok = false; continue; }
            tc_fence_after();
            float best = -INFINITY; int best_n = -1;
            const uint32_t t_row = tmem_base + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)(buf * BN);
#pragma unroll 1
            for (int ch = 0; ch < BN / 32; ++ch) {
                uint32_t v[32];
                tmem_ld32(t_row + (uint32_t)(ch * 32), v);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float2 sb = cs[ch * 32 + j];
                    const float val = fmaf(__uint_as_float(v[j]), sb.x, sb.y);
                    if (val > best) { best = val; best_n = ch * 32 + j; }   // ascending columns: lowest index wins
                }
                if (aux_row) {
                    for (int j = 0; j < 32; ++j) {
                        const int n = ch * 32 + j;
                        const float2 sb = cs[n];
                        if (sb.y == 0.f) {
                            const int hs = c.htB * P.bhB + (n >> P.bwB_log2), ws = c.wtB * bwB + (n & (bwB - 1));
                            aux_row[hs * P.Ws + ws] = clamp_unit(__uint_as_float(v[j]) * sb.x * inv_a);
                        }
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(bar_acc_empty + 8 * buf);                      // accumulator may be overwritten
            if (row_ok && best_n >= 0) {
                const int hs = c.htB * P.bhB + (best_n >> P.bwB_log2), ws = c.wtB * bwB + (best_n & (bwB - 1));
                const int y = (c.py * P.Hs + hs) * P.sy + my_rep, x = (c.px * P.Ws + ws) * P.sx + mx_rep;
                const long long tokB = ((long long)c.bt * P.H + y) * P.W + x;
                atomicMax(P.keys + tokA, pack_key(best, (uint32_t)tokB));
            }
        }
        if (!ok) { atomicCAS(P.status, 0, OC_ERR_TIMEOUT); *abort_flag = 1; }
    }

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---- host side ---------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
        else
            cudaGetLastError();
    });
    return fn;
}

static int pow2_ceil_log2(int v) { int l = 0; while ((1 << l) < v) ++l; return l; }

struct TcPlan { int bn; int bwA_log2, bhA, bwB_log2, bhB; int n_wtA, n_htA, n_wtB, n_htB; long long units; };

static TcPlan make_plan(const Geo& g, int bn) {
    TcPlan p; p.bn = bn;
    int la = pow2_ceil_log2(g.Ws); if ((1 << la) > BM) la = pow2_ceil_log2(BM);
    p.bwA_log2 = la; p.bhA = BM >> la;
    int lb = pow2_ceil_log2(g.Ws); if ((1 << lb) > bn) lb = pow2_ceil_log2(bn);
    p.bwB_log2 = lb; p.bhB = bn >> lb;
    p.n_wtA = (g.Ws + (1 << la) - 1) >> la; p.n_htA = (g.Hs + p.bhA - 1) / p.bhA;
    p.n_wtB = (g.Ws + (1 << lb) - 1) >> lb; p.n_htB = (g.Hs + p.bhB - 1) / p.bhB;
    p.units = g.n_groups * (long long)(g.sy * g.sx - 1) * p.n_wtA * p.n_htA * p.n_wtB * p.n_htB;
    return p;
}

bool tc_match_supported(const Geo& g) {
    if (g.kind != OC_KIND_TOKEN || g.dtype != OC_DTYPE_BF16 || g.self_match) return false;
    if (g.sy * g.sx > MAX_LATTICES) return false;
    if (g.C % 8 != 0) return false;
    if ((long long)g.B * g.T > 0x7FFFFFFFll) return false;
    TcPlan p = make_plan(g, 128);
    if (p.bhA > 256 || p.bhB > 256) return false;
    return p.units < 0x7FFFFFFFll && encode_fn() != nullptr;
}

template <int BN, int STAGES>
static oc_status launch_tc(oc_ctx* ctx, const TcParams& P, cudaStream_t s) {
    using S = TcSmem<BN, STAGES>;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(match_tc_kernel<BN, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::TOTAL) != cudaSuccess)
            return OC_ERR_CUDA;
        attr_set = true;
    }
    int grid = P.total_units < ctx->sm_count ? P.total_units : ctx->sm_count;
    LaunchScope scope(ctx, OC_K_MATCH_TC, s);
    match_tc_kernel<BN, STAGES><<<grid, TC_THREADS, S::TOTAL, s>>>(P);
    return last_launch_status();
}

void tc_cache_free(oc_ctx*) {}

oc_status launch_match_token_tc(oc_ctx* ctx, const Geo& g, const void* x, const float* inv_norm,
                                unsigned long long* keys, float* aux_sim, cudaStream_t s) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return OC_ERR_UNSUPPORTED;
    // tile width: the variant that wastes fewer SM-waves on this problem
    TcPlan p128 = make_plan(g, 128), p256 = make_plan(g, 256);
    auto cost = [&](const TcPlan& p) {
        long long waves = (p.units + ctx->sm_count - 1) / ctx->sm_count;
        return (double)waves * (double)p.bn;
    };
    const TcPlan& p = (p256.bhB <= 256 && cost(p256) <= cost(p128)) ? p256 : p128;

    TcParams P;
    memset(&P, 0, sizeof(P));
    const int bwA = 1 << p.bwA_log2, bwB = 1 << p.bwB_log2;
    const cuuint64_t dims[4] = {(cuuint64_t)g.C, (cuuint64_t)(g.W / g.sx), (cuuint64_t)(g.H / g.sy),
                                (cuuint64_t)g.B * g.T};
    const cuuint64_t strides[3] = {(cuuint64_t)g.sx * g.C * 2, (cuuint64_t)g.sy * g.W * g.C * 2,
                                   (cuuint64_t)g.H * g.W * g.C * 2};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const int rep_member = g.oy * g.sx + g.ox;
    for (int m = 0; m < g.sy * g.sx; ++m) {
        const int my = m / g.sx, mx = m - my * g.sx;
        const bool is_rep = m == rep_member;
        const cuuint32_t box[4] = {(cuuint32_t)BK, (cuuint32_t)(is_rep ? bwB : bwA),
                                   (cuuint32_t)(is_rep ? p.bhB : p.bhA), 1};
        void* base = (uint8_t*)x + ((size_t)my * g.W + mx) * g.C * 2;
        CUresult r = enc(&P.maps[m], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return OC_ERR_UNSUPPORTED;     // the FMA matcher takes over
    }
    P.H = g.H; P.W = g.W; P.sy = g.sy; P.sx = g.sx; P.gy = g.gy; P.gx = g.gx;
    P.Hp = g.Hp; P.Wp = g.Wp; P.Hs = g.Hs; P.Ws = g.Ws;
    P.rep_member = rep_member; P.n_cand_lat = g.sy * g.sx - 1;
    P.kblocks = (g.C + BK - 1) / BK;
    P.bwA_log2 = p.bwA_log2; P.bhA = p.bhA; P.n_wtA = p.n_wtA; P.n_htA = p.n_htA;
    P.bwB_log2 = p.bwB_log2; P.bhB = p.bhB; P.n_wtB = p.n_wtB; P.n_htB = p.n_htB;
    P.total_units = (int)p.units;
    P.units_per_group = (int)g.units_per_group; P.reps_per_group = (int)g.reps_per_group;
    P.inv_norm = inv_norm; P.keys = keys; P.aux = aux_sim; P.status = ctx->d_status;
    if (p.bn == 256) return launch_tc<256, 4>(ctx, P, s);
    return launch_tc<128, 6>(ctx, P, s);
}

}  // namespace oc
