// Dense (Token Cache) matcher on the 5th-generation tensor cores.
//
// For every token group the candidates x representatives similarity matrix is a dense contraction
// over the channel axis, S = A * B^T with A = candidate rows, B = representative rows, both read IN
// PLACE from the channel-last feature tensor: each sub-lattice of the (sy, sx)-strided grid is one
// 4-D TMA tensor map {C, W/sx, H/sy, B*T}, so a box {64 channels, bw, bh, 1} lands in shared memory
// as a canonical K-major, 128-byte-swizzled tile.  No operand is gathered or copied beforehand.
//
// What bounds it.  Measured on B200, this loop is limited by operand traffic L2 -> shared memory
// (every variant tried settled at 8-10 TB/s over all SMs, with ~3000 cycles from "stage free" to
// "stage full"), not by the tensor pipe.  So the tile is chosen for FLOP per fetched byte:
// one CTA multiplies TWO 128-row candidate tiles by the same N <= 256 representatives
// (M = 256 per CTA: 128 FLOP/B at N = 256, twice what a 128 x 128 tile gets), using all 512 TMEM
// columns as two accumulators.
//
// Work split.  The representatives of a group are cut into "quanta" of 32 lattice points (one 4 KB
// box per 64 channels).  A row of the problem is one pair of candidate tiles against all
// representatives of its group; it is cut into P pieces of nearly equal width (<= 8 quanta), and the
// pieces are dealt out evenly to one persistent CTA per SM.  The host picks P with a small cost
// model (bytes fetched per piece x number of waves).
//
// Warp specialised:
//   warp 0      TMA producer   (one lane per box): global -> smem ring (as many stages as fit in
//               192 KB for this launch's piece width), mbarrier complete_tx
//   warp 1      MMA issuer     (one lane): tcgen05.mma kind::f16 (bf16 x bf16 -> fp32 in TMEM), two
//               MMAs per 16 channels (one per candidate tile); owns tcgen05.alloc / dealloc
//   warps 2..9  epilogue: thread r of warps 2..5 / 6..9 owns row r (= TMEM lane r) of both candidate
//               tiles for the first / second half of the piece's columns: tcgen05.ld 32 columns at a
//               time (double buffered), scale by the representative's inverse norm, running
//               (max, arg max) in two independent register chains - no cross-thread reduction - then
//               ONE 64-bit atomicMax per row merges the piece into the packed key array (largest
//               value, then lowest index: independent of arrival order, hence deterministic).
// Rows / columns of a box that fall outside the patch are masked in the epilogue (bias -inf), so
// ragged lattices need no padding.  Every mbarrier wait is bounded: on expiry the CTA records
// OC_ERR_TIMEOUT in the context's status word, lets its outstanding copies land, frees TMEM and exits.
#include <cuda.h>

#include <mutex>

#include "common.cuh"

namespace oc {

static constexpr int BM = 128;           // rows per candidate tile (UMMA M)
static constexpr int QN = 32;            // representatives per quantum
static constexpr int MAXQ = 8;           // quanta per piece -> N <= 256
static constexpr int BK = 64;            // channels per stage: 128 bytes of bf16 = one swizzle row
static constexpr int A_BYTES = BM * BK * 2;
static constexpr int Q_BYTES = QN * BK * 2;
static constexpr int MAX_STAGES = 8;
static constexpr int SMEM_LIMIT = 232448;         // 227 KB: the most dynamic shared memory a CTA may have
static constexpr int TC_THREADS = 320;   // producer warp, MMA warp, 8 epilogue warps
static constexpr int EPI_THREADS = 256;
static constexpr int MAX_LATTICES = 9;
static constexpr uint32_t TMEM_COLS = 512;
static constexpr unsigned long long WAIT_LIMIT_NS = 1000000000ull;   // 1 s per wait

struct TcParams {
    CUtensorMap mapsA[MAX_LATTICES];     // 128-row boxes, one map per sub-lattice member (my*sx + mx)
    CUtensorMap mapQ;                    // 32-row boxes of the representative lattice
    int H, W, sy, sx, gy, gx;
    int Hp, Wp, Hs, Ws;                  // patch size; lattice size per patch (same for every member)
    int rep_member;                      // oy*sx + ox
    int n_cand_lat;                      // sy*sx - 1
    int kblocks;
    int bwA_log2, bhA, n_wtA, n_tilesA;  // candidate box: (1 << bwA_log2) x bhA lattice points = 128 rows
    int tpp;                             // candidate tiles per piece: 2 (M = 256), or 1 for small problems
    int n_apairs;                        // tile rows per lattice member = ceil(n_tilesA / tpp)
    int bwQ_log2, bhQ, n_wq, n_quanta;   // quantum box:   (1 << bwQ_log2) x bhQ lattice points = 32 rows
    int pieces_per_row, total_items;     // a row = one pair of candidate tiles against all representatives
    int n_stages, stage_bytes;           // operand ring of this launch
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
__device__ __forceinline__ void tma_prefetch_map(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" :: "l"(map) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        :: "r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// arrive on `bar` once every MMA issued so far by this thread has retired
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
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// Barrier over the 256 epilogue threads that also ANDs a flag: every thread learns whether any
// thread has given up, so they all leave the piece loop together.
__device__ __forceinline__ bool epilogue_barrier_all(bool ok) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "bar.red.and.pred p, 1, 256, q;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(r) : "r"((uint32_t)ok) : "memory");
    return r != 0;
}

// K-major, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr) {
    const uint32_t lo = ((addr >> 4) & 0x3FFFu) | (1u << 16);           // start address, LBO = 16 B (unused)
    const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);         // SBO = 1024 B, version 1, SWIZZLE_128B
    return ((uint64_t)hi << 32) | lo;
}

// ---- the walk over this CTA's share of the piece list ----------------------------------------------
struct Piece {
    int bt, py, px, member;              // frame, patch, candidate sub-lattice member
    int a_pair;                          // candidate tiles 2*a_pair and 2*a_pair + 1 of the member's lattice
    int q0, nq;                          // quanta [q0, q0 + nq) of the group's representatives
    long long g;
};
struct Walk {
    int i, i_end;
    __device__ Walk(const TcParams& P) {
        const long long n = gridDim.x, c = blockIdx.x;
        i = (int)((long long)P.total_items * c / n); i_end = (int)((long long)P.total_items * (c + 1) / n);
    }
    __device__ bool next(const TcParams& P, Piece& p) {
        if (i >= i_end) return false;
        int row = i / P.pieces_per_row;
        const int j = i - row * P.pieces_per_row;
        ++i;
        p.q0 = j * P.n_quanta / P.pieces_per_row;
        p.nq = (j + 1) * P.n_quanta / P.pieces_per_row - p.q0;
        p.a_pair = row % P.n_apairs; row /= P.n_apairs;
        const int k = row % P.n_cand_lat; row /= P.n_cand_lat;
        p.g = row;
        p.px = row % P.gx; row /= P.gx;
        p.py = row % P.gy; p.bt = row / P.gy;
        p.member = k < P.rep_member ? k : k + 1;
        return true;
    }
};

static constexpr int COL_BYTES = 256 * 8;                               // {scale, bias} per column of a piece
static constexpr int N_BARS = 2 * MAX_STAGES + 3;                       // full[], empty[], acc_full, acc_empty, drain
static constexpr int TAIL_BYTES = COL_BYTES + N_BARS * 8 + 32;        // column table, barriers, TMEM slot, flags
static constexpr int TILE_BYTES = (SMEM_LIMIT - TAIL_BYTES) / 1024 * 1024;   // operand ring: everything else
static constexpr int SMEM_TOTAL = TILE_BYTES + TAIL_BYTES;

__global__ void __launch_bounds__(TC_THREADS, 1)
match_tc_kernel(const __grid_constant__ TcParams P) {
    // The operand ring starts at the base of dynamic shared memory, which must be 1024-byte aligned
    // for the 128-byte swizzle (this kernel has no static shared memory in front of it; checked below).
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = smem_raw;
    float4* colsb = (float4*)(smem + TILE_BYTES);                      // 128 pairs of {scale, bias}
    uint64_t* bars = (uint64_t*)(smem + TILE_BYTES + COL_BYTES);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * MAX_STAGES;
    const uint32_t bar_acc_full = bar_empty + 8 * MAX_STAGES, bar_acc_empty = bar_acc_full + 8;
    const uint32_t bar_drain = bar_acc_empty + 8;
    uint32_t* tmem_slot = (uint32_t*)(bars + N_BARS);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
    const uint32_t tiles_base = smem_u32(smem);
    const int STAGES = P.n_stages, STAGE_BYTES = P.stage_bytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if ((tiles_base & 1023u) != 0) {                                   // never expected; refuse rather than compute garbage
        if (threadIdx.x == 0) atomicCAS(P.status, 0, OC_ERR_ALIGNMENT);
        return;
    }

    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        mbar_init(bar_acc_full, 1);
        mbar_init(bar_acc_empty, 8);                                    // one arrival per epilogue warp
        mbar_init(bar_drain, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 0 && lane == 0) {
        tma_prefetch_map(&P.mapQ);
        for (int m = 0; m <= P.n_cand_lat; ++m)
            if (m != P.rep_member) tma_prefetch_map(&P.mapsA[m]);
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

    const int bwA = 1 << P.bwA_log2, bwQ = 1 << P.bwQ_log2;
    const int my_rep = P.rep_member / P.sx, mx_rep = P.rep_member - my_rep * P.sx;

    if (warp == 0) {
        // ================================ TMA producer ==========================================
        // One lane per box: lanes 0 and 1 fetch the two candidate tiles, lanes 2..nq+1 one quantum
        // each, so a stage costs one barrier wait plus one copy instruction per lane.
        int stage = 0; uint32_t phase = 0;
        uint32_t armed = 0;                           // stages with a copy possibly still in flight
        bool ok = true;
        Walk walk(P); Piece c;
        while (ok && walk.next(P, c)) {
            const CUtensorMap* map = &P.mapQ;
            int w, h;
            if (lane < P.tpp) {
                map = &P.mapsA[c.member];
                const int ta = P.tpp * c.a_pair + lane;   // may lie past the lattice: the box is then masked
                const int htA = ta / P.n_wtA, wtA = ta - htA * P.n_wtA;
                w = c.px * P.Ws + wtA * bwA; h = c.py * P.Hs + htA * P.bhA;
            } else {
                const int qi = c.q0 + lane - P.tpp;
                const int hq = qi / P.n_wq, wq = qi - hq * P.n_wq;
                w = c.px * P.Ws + wq * bwQ; h = c.py * P.Hs + hq * P.bhQ;
            }
            const bool active = lane < c.nq + P.tpp;
            const uint32_t dst_off = lane < P.tpp ? (uint32_t)(lane * A_BYTES)
                                                  : (uint32_t)(P.tpp * A_BYTES + (lane - P.tpp) * Q_BYTES);
            const uint32_t bytes = (uint32_t)(P.tpp * A_BYTES + c.nq * Q_BYTES);
            for (int kb = 0; kb < P.kblocks; ++kb) {
                const uint32_t full = bar_full + 8 * stage;
                bool go = true;
                if (lane == 0) {
                    go = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag);
                    if (go) mbar_arrive_expect_tx(full, bytes);
                }
                go = __shfl_sync(0xFFFFFFFFu, (int)go, 0) != 0;
                if (!go) { ok = false; break; }
                if (active) tma_load_4d(tiles_base + stage * STAGE_BYTES + dst_off, map, kb * BK, w, h, c.bt, full);
                armed |= 1u << stage;
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
        if (!ok && lane == 0) {
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
    } else if (warp == 1) {
        // ================================ MMA issuer ============================================
        if (lane == 0) {
            constexpr uint32_t IDESC_BASE = (1u << 4) | (1u << 7) | (1u << 10) |
                                            ((uint32_t)(BM >> 4) << 24);   // D=f32, A=B=bf16, K-major both, M=128
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            uint32_t it = 0;
            Walk walk(P); Piece c;
            while (ok && walk.next(P, c)) {
                const uint32_t acc_phase = it & 1u;
                ++it;
                if (!mbar_wait(bar_acc_empty, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t idesc = IDESC_BASE | ((uint32_t)((c.nq * QN) >> 3) << 17);
                for (int kb = 0; kb < P.kblocks; ++kb) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = tiles_base + stage * STAGE_BYTES;
                    const uint64_t a0_desc = make_smem_desc(a_addr);
                    const uint64_t a1_desc = make_smem_desc(a_addr + A_BYTES);
                    const uint64_t b_desc = make_smem_desc(a_addr + P.tpp * A_BYTES);
#pragma unroll
                    for (int k4 = 0; k4 < BK / 16; ++k4) {            // UMMA K = 16: 32 bytes along the row
                        const uint32_t acc = (uint32_t)((kb | k4) != 0);
                        tc_mma_bf16(tmem_base, a0_desc + (uint64_t)(2 * k4), b_desc + (uint64_t)(2 * k4), idesc, acc);
                        if (P.tpp == 2)
                            tc_mma_bf16(tmem_base + 256u, a1_desc + (uint64_t)(2 * k4), b_desc + (uint64_t)(2 * k4), idesc, acc);
                    }
                    tc_commit(bar_empty + 8 * stage);                  // frees the stage when the MMAs retire
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) tc_commit(bar_acc_full);
            }
            if (!ok) { atomicCAS(P.status, 0, OC_ERR_TIMEOUT); *abort_flag = 1; }
            // all MMAs issued by this thread must retire before TMEM is released
            tc_commit(bar_drain);
            const unsigned long long t0 = global_ns();
            while (!mbar_try_wait(bar_drain, 0) && global_ns() - t0 < WAIT_LIMIT_NS) {}
        }
    } else {
        // ================================ epilogue ==============================================
        const int et = threadIdx.x - 64;                               // 0..255
        const int half = et >> 7;                                      // which half of the piece's columns
        const int lane_group = warp & 3;                               // TMEM lanes this warp may read
        const int row = lane_group * 32 + lane;                        // tile row owned by this thread
        bool ok = true;
        uint32_t it = 0;
        Walk walk(P); Piece c;
        float2* cs = (float2*)colsb;
        const float4* cs4 = colsb;
        while (walk.next(P, c)) {
            const uint32_t acc_phase = it & 1u;
            ++it;
            const int ncol = c.nq * QN;
            // ---- column table: inverse norm and validity of every representative of the piece -------
            // (safe to overwrite: every epilogue thread passed the previous piece's loop before the
            //  barrier below was completed for that piece ... see the trailing barrier)
            for (int n = et; n < ncol; n += EPI_THREADS) {
                const int qi = c.q0 + (n >> 5), r = n & 31;
                const int hq = qi / P.n_wq, wq = qi - hq * P.n_wq;
                const int hs = hq * P.bhQ + (r >> P.bwQ_log2), ws = wq * bwQ + (r & (bwQ - 1));
                float2 v = make_float2(0.f, -INFINITY);
                if (hs < P.Hs && ws < P.Ws) {
                    const int y = (c.py * P.Hs + hs) * P.sy + my_rep, x = (c.px * P.Ws + ws) * P.sx + mx_rep;
                    v = make_float2(__ldg(P.inv_norm + ((long long)c.bt * P.H + y) * P.W + x), 0.f);
                }
                cs[n] = v;
            }
            if (!epilogue_barrier_all(ok)) { ok = false; break; }     // also orders the table writes
            // warp-uniform outcome: the TMEM loads below are warp-collective
            const bool ready = __all_sync(0xFFFFFFFFu, mbar_wait(bar_acc_full, acc_phase, abort_flag));
            if (ready) {
                tc_fence_after();
                const int my = c.member / P.sx, mx = c.member - my * P.sx;
                // chunks of 32 columns: the first half of them to warps 2..5, the rest to warps 6..9
                const int ch_split = (c.nq + 1) >> 1;
                const int ch_begin = half ? ch_split : 0, ch_end = half ? c.nq : ch_split;
#pragma unroll 1
                for (int t = 0; t < P.tpp; ++t) {                      // the piece's candidate tiles
                    const int ta = P.tpp * c.a_pair + t;
                    const int htA = ta / P.n_wtA, wtA = ta - htA * P.n_wtA;
                    const int hsA = htA * P.bhA + (row >> P.bwA_log2), wsA = wtA * bwA + (row & (bwA - 1));
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
                    float best0 = -INFINITY, best1 = -INFINITY; int n0 = -1, n1 = -1;
                    const uint32_t t_row = tmem_base + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)(t * 256);
                    // two register buffers: the TMEM load of the next chunk is in flight while this one is reduced
                    uint32_t va[32], vb[32];
                    auto reduce_chunk = [&](const uint32_t* v, int ch) {
#pragma unroll
                        for (int j = 0; j < 32; j += 2) {              // two independent (max, arg max) chains
                            const float4 sb = cs4[ch * 16 + (j >> 1)];
                            const float x0 = fmaf(__uint_as_float(v[j]), sb.x, sb.y);
                            const float x1 = fmaf(__uint_as_float(v[j + 1]), sb.z, sb.w);
                            if (x0 > best0) { best0 = x0; n0 = ch * 32 + j; }      // ascending columns: lowest index wins
                            if (x1 > best1) { best1 = x1; n1 = ch * 32 + j + 1; }
                        }
                        if (aux_row) {
                            for (int j = 0; j < 32; ++j) {
                                const float2 sb = cs[ch * 32 + j];
                                if (sb.y == 0.f) {
                                    const int qi = c.q0 + ch;
                                    const int hq = qi / P.n_wq, wq = qi - hq * P.n_wq;
                                    const int hs = hq * P.bhQ + (j >> P.bwQ_log2), ws = wq * bwQ + (j & (bwQ - 1));
                                    aux_row[hs * P.Ws + ws] = clamp_unit(__uint_as_float(v[j]) * sb.x * inv_a);
                                }
                            }
                        }
                    };
                    if (ch_begin < ch_end) tmem_ld32(t_row + (uint32_t)(ch_begin * 32), va);
#pragma unroll 1
                    for (int ch = ch_begin; ch < ch_end; ch += 2) {
                        tmem_ld_wait();
                        if (ch + 1 < ch_end) tmem_ld32(t_row + (uint32_t)((ch + 1) * 32), vb);
                        reduce_chunk(va, ch);
                        if (ch + 1 < ch_end) {
                            tmem_ld_wait();
                            if (ch + 2 < ch_end) tmem_ld32(t_row + (uint32_t)((ch + 2) * 32), va);
                            reduce_chunk(vb, ch + 1);
                        }
                    }
                    if (best1 > best0 || (best1 == best0 && n1 >= 0 && (n0 < 0 || n1 < n0))) { best0 = best1; n0 = n1; }
                    if (row_ok && n0 >= 0) {
                        const int qi = c.q0 + (n0 >> 5), r = n0 & 31;
                        const int hq = qi / P.n_wq, wq = qi - hq * P.n_wq;
                        const int hs = hq * P.bhQ + (r >> P.bwQ_log2), ws = wq * bwQ + (r & (bwQ - 1));
                        const int y = (c.py * P.Hs + hs) * P.sy + my_rep, x = (c.px * P.Ws + ws) * P.sx + mx_rep;
                        const long long tokB = ((long long)c.bt * P.H + y) * P.W + x;
                        atomicMax(P.keys + tokA, pack_key(best0, (uint32_t)tokB));
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_acc_empty);              // both accumulators may be overwritten
            } else {
                ok = false;
            }
            // the column table is rewritten for the next piece: everyone must be done reading it
            if (!epilogue_barrier_all(ok)) { ok = false; break; }
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

// ---- self-test of the bounded wait ---------------------------------------------------------------
// One warp waits on an mbarrier that nothing ever completes, with the same try_wait / %globaltimer
// loop the matcher uses but a caller-chosen limit.  The wait runs out, the kernel records
// OC_ERR_TIMEOUT in the status word and returns normally: the context stays usable.
__global__ void bounded_wait_selftest_kernel(unsigned long long limit_ns, int* status) {
    __shared__ uint64_t bar;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        const unsigned long long t0 = global_ns();
        bool done = false;
        unsigned spins = 0;
        while (!(done = mbar_try_wait(b, 0))) {
            if ((++spins & 63u) == 0 && global_ns() - t0 > limit_ns) break;
        }
        if (!done) atomicCAS(status, 0, OC_ERR_TIMEOUT);
    }
}

oc_status launch_bounded_wait_selftest(oc_ctx* ctx, unsigned long long limit_ns, cudaStream_t s) {
    bounded_wait_selftest_kernel<<<1, 32, 0, s>>>(limit_ns, ctx->d_status);
    return last_launch_status();
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

struct TcPlan {
    int bwA_log2, bhA, n_wtA, n_tilesA, tpp, n_apairs, bwQ_log2, bhQ, n_wq, n_quanta;
    int pieces_per_row, qmax, n_stages, stage_bytes;
    long long rows, items;
};

static TcPlan make_plan(const Geo& g, int sm_count) {
    TcPlan p;
    int la = pow2_ceil_log2(g.Ws); if ((1 << la) > BM) la = pow2_ceil_log2(BM);
    p.bwA_log2 = la; p.bhA = BM >> la;
    p.n_wtA = (g.Ws + (1 << la) - 1) >> la;
    p.n_tilesA = p.n_wtA * ((g.Hs + p.bhA - 1) / p.bhA);
    int lq = pow2_ceil_log2(g.Ws); if ((1 << lq) > QN) lq = pow2_ceil_log2(QN);
    p.bwQ_log2 = lq; p.bhQ = QN >> lq;
    p.n_wq = (g.Ws + (1 << lq) - 1) >> lq;
    p.n_quanta = p.n_wq * ((g.Hs + p.bhQ - 1) / p.bhQ);
    // Tiles per piece (1 or 2) and pieces per row: estimated cycles = waves x per-piece cycles.  Per
    // 64-channel step a piece fetches tpp*16 + 4q KB; the step takes the longest of: that fetch at
    // ~48 B/clk/SM (measured L2 -> shared-memory feed), the fetch round trip (~3000 cycles) divided
    // by the stages that fit in the ring, and tpp*64q tensor cycles.  The epilogue (~200 cycles per
    // quantum and tile) is not overlapped.
    const int kblocks = (g.C + BK - 1) / BK;
    double best_cost = 0; int best_P = 0, best_tpp = 2;
    for (int tpp = 1; tpp <= 2; ++tpp) {
        const long long rows = g.n_groups * (long long)(g.sy * g.sx - 1) * ((p.n_tilesA + tpp - 1) / tpp);
        for (int P = (p.n_quanta + MAXQ - 1) / MAXQ; P <= p.n_quanta; ++P) {
            const int q = (p.n_quanta + P - 1) / P;
            const double stage_kb = tpp * 16.0 + 4.0 * q;
            int stages = (int)(TILE_BYTES / 1024 / stage_kb); if (stages > MAX_STAGES) stages = MAX_STAGES;
            const long long waves = (rows * P + sm_count - 1) / sm_count;
            const double fetch = stage_kb * 1024.0 / 48.0, lat = 3000.0 / stages, mma = tpp * 64.0 * q;
            double step = fetch > lat ? fetch : lat; if (mma > step) step = mma;
            const double piece = kblocks * step + 200.0 * q * tpp + 1500.0;
            const double cost = waves * piece;
            if (best_P == 0 || cost < best_cost) { best_cost = cost; best_P = P; best_tpp = tpp; }
        }
    }
    p.tpp = best_tpp;
    p.n_apairs = (p.n_tilesA + p.tpp - 1) / p.tpp;
    p.rows = g.n_groups * (long long)(g.sy * g.sx - 1) * p.n_apairs;
    p.pieces_per_row = best_P;
    p.qmax = (p.n_quanta + best_P - 1) / best_P;
    p.stage_bytes = p.tpp * A_BYTES + p.qmax * Q_BYTES;
    p.n_stages = TILE_BYTES / p.stage_bytes;
    if (p.n_stages > MAX_STAGES) p.n_stages = MAX_STAGES;
    p.items = p.rows * p.pieces_per_row;
    return p;
}

bool tc_match_supported(const Geo& g) {
    if (g.kind != OC_KIND_TOKEN || g.dtype != OC_DTYPE_BF16 || g.self_match) return false;
    if (g.sy * g.sx > MAX_LATTICES) return false;
    if (g.C % 8 != 0) return false;
    if ((long long)g.B * g.T > 0x7FFFFFFFll) return false;
    return encode_fn() != nullptr;
}

void tc_cache_free(oc_ctx*) {}

oc_status launch_match_token_tc(oc_ctx* ctx, const Geo& g, const void* x, const float* inv_norm,
                                unsigned long long* keys, float* aux_sim, cudaStream_t s) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return OC_ERR_UNSUPPORTED;
    const TcPlan p = make_plan(g, ctx->sm_count);
    if (p.items > 0x7FFFFFFFll) return OC_ERR_UNSUPPORTED;

    TcParams P;
    memset(&P, 0, sizeof(P));
    const cuuint64_t dims[4] = {(cuuint64_t)g.C, (cuuint64_t)(g.W / g.sx), (cuuint64_t)(g.H / g.sy),
                                (cuuint64_t)g.B * g.T};
    const cuuint64_t strides[3] = {(cuuint64_t)g.sx * g.C * 2, (cuuint64_t)g.sy * g.W * g.C * 2,
                                   (cuuint64_t)g.H * g.W * g.C * 2};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const cuuint32_t boxA[4] = {(cuuint32_t)BK, (cuuint32_t)(1 << p.bwA_log2), (cuuint32_t)p.bhA, 1};
    const cuuint32_t boxQ[4] = {(cuuint32_t)BK, (cuuint32_t)(1 << p.bwQ_log2), (cuuint32_t)p.bhQ, 1};
    const int rep_member = g.oy * g.sx + g.ox;
    for (int m = 0; m <= g.sy * g.sx; ++m) {
        const bool quantum_map = m == g.sy * g.sx;
        const int member = quantum_map ? rep_member : m;
        if (!quantum_map && member == rep_member) continue;              // representatives are never candidates
        const int my = member / g.sx, mx = member - my * g.sx;
        void* base = (uint8_t*)x + ((size_t)my * g.W + mx) * g.C * 2;
        CUresult r = enc(quantum_map ? &P.mapQ : &P.mapsA[m], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides,
                         quantum_map ? boxQ : boxA, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return OC_ERR_UNSUPPORTED;     // the FMA matcher takes over
    }
    P.H = g.H; P.W = g.W; P.sy = g.sy; P.sx = g.sx; P.gy = g.gy; P.gx = g.gx;
    P.Hp = g.Hp; P.Wp = g.Wp; P.Hs = g.Hs; P.Ws = g.Ws;
    P.rep_member = rep_member; P.n_cand_lat = g.sy * g.sx - 1;
    P.kblocks = (g.C + BK - 1) / BK;
    P.bwA_log2 = p.bwA_log2; P.bhA = p.bhA; P.n_wtA = p.n_wtA; P.n_tilesA = p.n_tilesA; P.tpp = p.tpp; P.n_apairs = p.n_apairs;
    P.bwQ_log2 = p.bwQ_log2; P.bhQ = p.bhQ; P.n_wq = p.n_wq; P.n_quanta = p.n_quanta;
    P.pieces_per_row = p.pieces_per_row; P.total_items = (int)p.items;
    P.n_stages = p.n_stages; P.stage_bytes = p.stage_bytes;
    P.units_per_group = (int)g.units_per_group; P.reps_per_group = (int)g.reps_per_group;
    P.inv_norm = inv_norm; P.keys = keys; P.aux = aux_sim; P.status = ctx->d_status;

    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(match_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_TOTAL) != cudaSuccess)
            return OC_ERR_CUDA;
        attr_set = true;
    }
    // one CTA per SM, or one per piece when there are fewer pieces
    long long grid = p.items;
    if (grid > ctx->sm_count) grid = ctx->sm_count;
    if (grid < 1) grid = 1;
    LaunchScope scope(ctx, OC_K_MATCH_TC, s);
    match_tc_kernel<<<(unsigned)grid, TC_THREADS, SMEM_TOTAL, s>>>(P);
    return last_launch_status();
}

}  // namespace oc
