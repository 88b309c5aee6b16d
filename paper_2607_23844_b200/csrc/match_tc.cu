// Dense (Token Cache) matcher on the 5th-generation tensor cores.
//
// For every token group the candidates x representatives similarity matrix is a dense contraction
// over the channel axis, S = A * B^T with A = candidate rows, B = representative rows, both read IN
// PLACE from the channel-last feature tensor: each sub-lattice of the (sy, sx)-strided grid is one
// 4-D TMA tensor map {C, W/sx, H/sy, B*T}, so a box {64 channels, bw, bh, 1} lands in shared memory
// as a canonical K-major, 128-byte-swizzled tile.  No operand is gathered or copied beforehand.
//
// What bounds it.  Measured on B200 (in-kernel timestamps, timing-only builds with the copies or the
// epilogue's arithmetic left out, and micro-benchmarks of the copy ring, the MMA issue and the key
// arithmetic):
//   * the L2 -> shared-memory path delivers ~70-80 B/clk/SM to all SMs at once, some 500-800 cycles
//     after the copy is issued; an MMA of 128 x 256 x 16 takes ~140 cycles;
//   * shared memory serves the copies' writes AND the MMAs' operand reads: one tile of 128 rows against
//     256 columns reads 12 KB per MMA and is sent 8 KB, which is more than 128 B/clk -- a single CTA's
//     stage then takes ~700 cycles for 560 of MMA.  In a CTA pair each CTA reads and is sent half of the
//     representatives, and the tensor pipe is the bound again;
//   * the tensor pipe runs dry while the issuing warp is between two stages or two pieces unless that
//     warp is back within about one MMA's time: the look at the next stage's barrier and all commits
//     of a stage sit inside the block that issues its MMAs, and descriptors are kept by additions;
//   * a lone warp runs dependent integer arithmetic at full latency (~6 cycles an instruction) and pays
//     for every branch; a lone diverged LANE also has its operands moved into uniform registers before
//     every copy or MMA.  So the producer and the MMA issuer run their loops with the whole warp and
//     elect the lane that issues, and the epilogue does index arithmetic per group and per row, not
//     per piece, branch-free and ahead of time;
//   * the arg-max epilogue is bound by the ALU and FMA pipes (two warps per scheduler): per element
//     half a packed FMA, one integer multiply-add and half a three-input maximum.
//
// Tile.  One CTA multiplies ONE or TWO 128-row candidate tiles by the same N <= 256 representatives.
// Two tiles (M = 256 per CTA, 128 FLOP/B at N = 256) use all 512 TMEM columns as two accumulators;
// one tile - or two tiles whose pieces are at most 128 columns wide - leave half of TMEM free, so two
// sets of accumulators take turns and the epilogue of a piece runs under the MMAs of the next (what
// pays on short-K problems, where the arg-max epilogue is a third of the time).  Optionally two CTAs of a cluster form a pair (cta_group::2): each
// holds its own candidate tiles and fetches HALF of the representatives, and the tensor cores of
// both SMs read both halves: the same MMA work per SM for fewer fetched bytes.
//
// Work split.  The representatives of a group are cut into "quanta" of 32 lattice points (one 4 KB
// box per 64 channels).  A row of the problem is the candidate tiles of one CTA (or pair) against all
// representatives of its group; it is cut into P pieces of nearly equal width (<= 256 columns; in the
// single-CTA form in steps of half a quantum, so that 1024 columns split six ways as 176/176/160
// rather than 192/160/160: a piece that begins in mid-quantum fetches that quantum whole and starts
// its B descriptor 16 rows in), and the pieces are dealt out evenly, in contiguous runs, to one
// persistent CTA (pair) per SM (pair of SMs).
// The host picks the form, the tiles per CTA and P with a small cost model.
// Joint form (Token Cache on the frame pairs of Frame Cache, Section 3.2.3): the rows are not the
// regular (frame, patch, sub-lattice) enumeration but a list of {representative frame, candidate
// frame, sub-lattice} units that another kernel wrote; its length exists only on the device, so every
// walker reads it, takes its share of (unit, tile run, piece) triples and looks a unit up once.  The
// candidate tiles then come from one frame and the representatives from another -- a different fourth
// TMA coordinate for the two operands -- and nothing else changes.
//
// Warp specialised:
//   warp 0 (and, for one-tile plans, the last warp, taking turns with it stage by stage)
//               TMA producer: global -> smem ring (as many stages as fit), mbarrier complete_tx.  A
//               CTA's candidate tiles are one box, and so are its quanta of a piece, whenever they
//               stack into a rectangle of lattice rows: the whole warp then walks the loop and one
//               elected lane issues; otherwise one lane per box.  With "resident" candidate tiles
//               (plans whose rows have several pieces and few channels) all 64-channel steps of a row's
//               tiles sit in front of the ring and are fetched once per row.
//   warp 1      MMA issuer     (all lanes walk the loop so that addresses stay warp-uniform, one
//               elected lane issues): tcgen05.mma kind::f16 (bf16 x bf16 -> fp32 in TMEM), all MMAs
//               of a stage in one instruction block with the look at the next stage's barrier and
//               the stage's commits folded in; owns tcgen05.alloc / dealloc
//   warps 2..9  epilogue, two halves of four warps (one warp per TMEM lane quarter, thread r owns row
//               r of the candidate tiles).  With two accumulator sets the halves take alternate
//               pieces; with one set of two tiles one tile each; with one set of one tile half of
//               the columns each.  tcgen05.ld 32 columns at a time, scale by the
//               representative's inverse norm, and a running
//               maximum over integer keys: the scaled similarity, lifted into one binade (where a
//               float's bits are linear in its value), times 32, plus 31 - column (one three-input max
//               per three keys, no compare-and-select per element, no cross-thread reduction; the
//               lowest column wins among equal similarities whatever their sign);
//               then ONE 64-bit atomicMax per row merges the piece into the packed key array (largest
//               value, then lowest index: independent of arrival order, hence deterministic).
//               The lift rounds the reported cosine by at most 2.4e-7, and among representatives
//               whose similarities agree to that precision the lowest index wins.  The epilogue warps
//               never wait for one another from piece to piece: each half keeps the column scales of
//               the whole group in shared memory (rebuilt, behind a barrier over the half's four warps,
//               only when its pieces move to another group), and a row's own norms are fetched while
//               the piece before is reduced.
// Rows / columns of a box that fall outside the patch are masked in the epilogue (their scale is NaN
// and their key is zeroed), so ragged lattices need no padding.  Every mbarrier wait is bounded: on expiry the CTA
// records OC_ERR_TIMEOUT in the context's status word, lets its outstanding copies land, frees TMEM
// and exits.
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace oc {

static constexpr int BM = 128;           // rows per candidate tile (UMMA M)
static constexpr int QN = 32;            // representatives per quantum
static constexpr int MAXQ = 8;           // quanta per piece -> N <= 256
static constexpr int BK = 64;            // channels per stage: 128 bytes of bf16 = one swizzle row
static constexpr int A_BYTES = BM * BK * 2;
static constexpr int Q_BYTES = QN * BK * 2;
static constexpr int MAX_STAGES = 8;
static constexpr int MAX_AKB = 10;       // most 64-channel steps whose candidate tiles may stay resident
static constexpr int SMEM_LIMIT = 232448;         // 227 KB: the most dynamic shared memory a CTA may have
#ifndef OC_EPI_WARPS
#define OC_EPI_WARPS 8
#endif
static constexpr int EPI_WARPS = OC_EPI_WARPS;            // 8 or 16: two or four per TMEM lane quarter
static constexpr int EPI_PARTS = EPI_WARPS / 4;           // a piece's columns are cut into this many parts
#ifndef OC_PRODUCERS
#define OC_PRODUCERS 2
#endif
static constexpr int N_PRODUCERS = OC_PRODUCERS;          // copy-producer warps: warp 0 and, with two, the last warp
static constexpr int PRODUCER2_WARP = 2 + EPI_WARPS;
// The epilogue warps come in two halves (each with one warp per TMEM lane quarter).  With two accumulator
// sets the halves take alternate pieces (set = piece parity), each warp all columns of its rows; with one
// set of two tiles, one tile each; with one set of one tile, half of the columns each.  The first two
// give a warp twice the columns per piece it touches and half the pieces: its per-piece overhead halves.
enum { EPI_BY_COLUMNS = 0, EPI_BY_PIECE = 1, EPI_BY_TILE = 2 };
static constexpr int TC_THREADS = 64 + 32 * EPI_WARPS + 32 * (N_PRODUCERS - 1);   // producer, MMA, epilogue warps[, producer]
static constexpr int MAX_LATTICES = 9;
static constexpr uint32_t TMEM_COLS = 512;

// Everything but the tensor maps.
struct TcScalars {
    int H, W, sy, sx, gy, gx;
    int Hp, Wp, Hs, Ws;                  // patch size; lattice size per patch (same for every member)
    int rep_member;                      // oy*sx + ox
    int n_cand_lat;                      // sy*sx - 1
    int kblocks;
    int bwA_log2, bhA, n_wtA, n_tilesA;  // candidate box: (1 << bwA_log2) x bhA lattice points = 128 rows
    int tpp;                             // candidate tiles per piece: 2 (M = 256), or 1 for small problems
    int narrow;                          // tpp == 2 and no piece wider than 128 columns: the two tiles' accumulators
                                         // are 128 columns apart and take 256 columns, so two sets take turns
    int n_apairs;                        // tile rows per lattice member = ceil(n_tilesA / tpp)
    int bwQ_log2, bhQ, n_wq, n_quanta;   // quantum box:   (1 << bwQ_log2) x bhQ lattice points = 32 rows
    int pieces_per_row, total_items;     // a row = the candidate tiles of one piece against all representatives
    int q_unit, n_q_units;               // pieces are cut in units of q_unit quanta (2 for a CTA pair), or, when
    int half_units;                      // half_units is set, in units of half a quantum (16 columns)
    int a_merged, q_merged, q_lo;        // one box for a CTA's candidate tiles / for its quanta of a piece
    int items_base, items_rem;           // every walker takes items_base pieces, the first items_rem one more
    unsigned cum[5];                     // pieces per tile run, lattice, patch, patch row, frame
    float rcp_cum[5], rcp_ppr;           // their reciprocals, and 1 / pieces_per_row
    float rcp_n_wtA, rcp_n_wq;
    int my_rep, mx_rep;                  // rep_member / sx and the remainder
    int sx_magic;                        // ceil(65536 / sx): (m * sx_magic) >> 16 == m / sx for m < 256
    int u_step_q, u_step_r;              // n_q_units / pieces_per_row and the remainder
    int n_stages, stage_bytes;           // operand ring of this launch
    int n_prod;                          // copy-producer warps at work: 1, or 2 taking turns stage by stage
    unsigned key_mul;                    // 32, as a run-time value: keeps half of the key multiplies on the FMA pipe
    int epi_split;                       // how the two halves of the epilogue warps share the work (EPI_BY_*)
    int gt_off, gt_half_bytes, gt_quanta; // the group's column-scale tables (one per half of the epilogue warps):
                                         // byte offset in shared memory, size of one, quanta per group
    int a_res, a_region_bytes;           // candidate tiles resident: all 64-channel steps of a CTA's candidate tiles
                                         // sit in front of the ring (one slot per step) for all pieces of a row, and
                                         // the ring carries representatives only
    int units_per_group, reps_per_group;
    // Joint form (Token Cache on the frame pairs of Frame Cache, Section 3.2.3): the work is a list of
    // units {representative frame, candidate frame, candidate sub-lattice member} written by another
    // kernel, whose length is only known on the device; every walker derives its share from it.
    const int4* units;                   // null: the regular (frame, patch, member) enumeration
    const int* n_units_dev;
    unsigned n_walkers;
    float rcp_walkers;
    const float* inv_norm;
    unsigned long long* keys;
    float* aux;
    unsigned long long* span;            // nullable: {~first entry, last exit} of this launch, GPU-timer ns
    int* status;
};
struct TcParams {
    CUtensorMap mapsA[MAX_LATTICES];     // 128-row boxes, one map per sub-lattice member (my*sx + mx)
    CUtensorMap mapQ[2];                 // representative boxes: one quantum (32 rows), or when a piece's quanta
                                         // stack into one rectangle, q_lo quanta ([0]) and q_lo + 1 quanta ([1])
    TcScalars s;
};

// ---- the walk over this CTA's share of the piece list ----------------------------------------------
struct Piece {
    int bt, py, px, member;              // frame (of the representatives), patch, candidate sub-lattice member
    int bt_a;                            // frame of the candidates (differs from bt only in the joint form)
    int a_pair;                          // which run of candidate tiles (tpp per CTA) of the member's lattice
    int q0, nq;                          // quanta [q0, q0 + nq) of the group's representatives are fetched
    int c_off, ncol;                     // of which columns [c_off, c_off + ncol) are the piece (c_off is 0 or 16,
                                         // ncol a multiple of 16: pieces may begin and end in mid-quantum)
    int first, last;                     // the first / last piece this walker has of the piece's row (the same
                                         // candidate tiles serve all pieces of a row)
    long long g;
};
// floor(a / d) for a < 2^22 from the float reciprocal (one multiply and a fix-up; an integer division
// costs a lone warp several hundred cycles), by integer division otherwise.
__device__ __forceinline__ unsigned div_small(unsigned a, unsigned d, float rcp_d) {
    if (a >= (1u << 22)) return a / d;
    unsigned q = (unsigned)((float)a * rcp_d);
    const int r = (int)(a - q * d);
    if (r < 0) --q; else if ((unsigned)r >= d) ++q;
    return q;
}

// Pieces are numbered row-major over (frame, patch row, patch column, candidate lattice, tile run,
// piece of the row); a walker takes a contiguous range.  The first piece is decoded by division,
// the following ones by counting up.
template <bool JOINT>
struct Walk {
    int left;                            // pieces still to hand out
    int j, a_pair, k, px, py, bt;
    int u_cur, r_cur;                    // floor(j * n_q_units / pieces_per_row) and the remainder
    int bt_a, member_u;                  // joint form: the current unit's candidate frame and member
    int fresh;                           // nothing handed out yet
    long long g;
    __device__ __forceinline__ void load_unit(const TcScalars& P) {
        const int4 v = __ldg(P.units + g);
        bt = v.x; bt_a = v.y; member_u = v.z;
    }
    __device__ __forceinline__ Walk(const TcScalars& P, int c) {
        fresh = 1;
        if (JOINT) {
            // pieces are numbered (unit, tile run, piece of the row); the list length is read here
            const unsigned total = (unsigned)__ldg(P.n_units_dev) * P.cum[1];
            const unsigned base = div_small(total, P.n_walkers, P.rcp_walkers), rem = total - base * P.n_walkers;
            const unsigned i0 = (unsigned)c * base + ((unsigned)c < rem ? (unsigned)c : rem);
            left = (int)(base + ((unsigned)c < rem ? 1u : 0u));
            const unsigned q0 = div_small(i0, P.cum[0], P.rcp_cum[0]), q1 = div_small(i0, P.cum[1], P.rcp_cum[1]);
            j = (int)(i0 - q0 * P.cum[0]);
            a_pair = (int)(q0 - q1 * (unsigned)P.n_apairs);
            g = q1; k = 0; px = 0; py = 0; bt = 0; bt_a = 0; member_u = 0;
            if (left > 0) load_unit(P);
            const unsigned ju = (unsigned)j * (unsigned)P.n_q_units;
            u_cur = (int)div_small(ju, (unsigned)P.pieces_per_row, P.rcp_ppr);
            r_cur = (int)(ju - (unsigned)u_cur * (unsigned)P.pieces_per_row);
            return;
        }
        bt_a = 0; member_u = 0;
        const unsigned i0 = (unsigned)(c * P.items_base + (c < P.items_rem ? c : P.items_rem));
        left = P.items_base + (c < P.items_rem ? 1 : 0);
        const unsigned q0 = div_small(i0, P.cum[0], P.rcp_cum[0]), q1 = div_small(i0, P.cum[1], P.rcp_cum[1]),
                       q2 = div_small(i0, P.cum[2], P.rcp_cum[2]), q3 = div_small(i0, P.cum[3], P.rcp_cum[3]),
                       q4 = div_small(i0, P.cum[4], P.rcp_cum[4]);
        j = (int)(i0 - q0 * P.cum[0]);
        a_pair = (int)(q0 - q1 * (unsigned)P.n_apairs);
        k = (int)(q1 - q2 * (unsigned)P.n_cand_lat);
        g = q2;
        px = (int)(q2 - q3 * (unsigned)P.gx);
        py = (int)(q3 - q4 * (unsigned)P.gy);
        bt = (int)q4;
        const unsigned ju = (unsigned)j * (unsigned)P.n_q_units;
        u_cur = (int)div_small(ju, (unsigned)P.pieces_per_row, P.rcp_ppr);
        r_cur = (int)(ju - (unsigned)u_cur * (unsigned)P.pieces_per_row);
    }
    __device__ __forceinline__ bool next(const TcScalars& P, Piece& p) {
        if (left <= 0) return false;
        --left;
        int u_next = u_cur + P.u_step_q, r_next = r_cur + P.u_step_r;
        if (r_next >= P.pieces_per_row) { r_next -= P.pieces_per_row; ++u_next; }
        if (P.half_units) {                  // units of 16 columns: half a quantum
            p.q0 = u_cur >> 1;
            p.nq = ((u_next - 1) >> 1) - p.q0 + 1;
            p.c_off = (u_cur & 1) << 4;
            p.ncol = (u_next - u_cur) << 4;
        } else {
            p.q0 = u_cur * P.q_unit;
            p.nq = (u_next - u_cur) * P.q_unit;
            p.c_off = 0;
            p.ncol = p.nq * QN;
        }
        u_cur = u_next; r_cur = r_next;
        p.first = (j == 0) | fresh; fresh = 0;
        p.last = (j + 1 == P.pieces_per_row) | (left == 0);
        p.a_pair = a_pair; p.g = g; p.px = px; p.py = py; p.bt = bt;
        p.bt_a = JOINT ? bt_a : bt;
        p.member = JOINT ? member_u : (k < P.rep_member ? k : k + 1);
        if (++j == P.pieces_per_row) {
            j = 0; u_cur = 0; r_cur = 0;
            if (++a_pair == P.n_apairs) {
                a_pair = 0;
                if (JOINT) {
                    ++g;
                    if (left > 0) load_unit(P);
                } else if (++k == P.n_cand_lat) {
                    k = 0; ++g;
                    if (++px == P.gx) { px = 0; if (++py == P.gy) { py = 0; ++bt; } }
                }
            }
        }
        return true;
    }
};

// Maximum of 32 arg-max keys by a tree of three-input maxima: 16 instructions, four levels deep.
__device__ __forceinline__ uint32_t key_tree_max(const uint32_t (&k)[32]) {
    uint32_t a[11];
#pragma unroll
    for (int i = 0; i < 10; ++i) a[i] = __vimax3_u32(k[3 * i], k[3 * i + 1], k[3 * i + 2]);
    a[10] = max(k[30], k[31]);
    const uint32_t b0 = __vimax3_u32(a[0], a[1], a[2]), b1 = __vimax3_u32(a[3], a[4], a[5]), b2 = __vimax3_u32(a[6], a[7], a[8]);
    const uint32_t c0 = __vimax3_u32(b0, b1, b2);
    return __vimax3_u32(c0, a[9], a[10]);
}

// d = a * b + {c, c} on two packed fp32 lanes: one FMA-pipe instruction for two columns
__device__ __forceinline__ void fma_pair(float& d0, float& d1, uint32_t a0, uint32_t a1, float b0, float b1, float c) {
    unsigned long long a, b, cc, d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(a) : "r"(a0), "r"(a1));
    asm("mov.b64 %0, {%1, %2};" : "=l"(b) : "f"(b0), "f"(b1));
    asm("mov.b64 %0, {%1, %1};" : "=l"(cc) : "f"(c));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(cc));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d0), "=f"(d1) : "l"(d));
}


static constexpr int GT_MAX_QUANTA = 150;                               // largest group whose scale tables fit beside the ring
static constexpr int N_BARS = 2 * MAX_STAGES + 5 + MAX_AKB;             // full[], empty[], acc_full[2], acc_empty[2], drain, a_empty[]
static constexpr int TAIL_BYTES = N_BARS * 8 + 32;                      // barriers, TMEM slot, flags
static constexpr int TILE_BYTES = (SMEM_LIMIT - TAIL_BYTES) / 1024 * 1024;   // operand ring: everything else
static constexpr int SMEM_TOTAL = TILE_BYTES + TAIL_BYTES;

// PAIR: two CTAs of a cluster work on one piece with cta_group::2 instructions.  Each holds its own
// tpp candidate tiles (256 accumulator rows per MMA across the pair) and fetches HALF of the piece's
// representative quanta; the tensor cores of both SMs read both halves, so every fetched operand
// byte feeds twice the FLOPs.  The leader (cluster rank 0) issues all MMAs; both CTAs' copies report
// to the leader's stage barrier, and the leader's commits free the stage in both CTAs.
// MODE 0: the hot instance; 1: also writes the full similarity rows (parity runs); 2: the joint work list.
template <bool PAIR, int MODE>
__global__ void __launch_bounds__(TC_THREADS, 1)
match_tc_kernel(const __grid_constant__ TcParams KP) {
    constexpr bool AUX = MODE == 1, JOINT = MODE == 2;
    // The operand ring starts at the base of dynamic shared memory, which must be 1024-byte aligned
    // for the 128-byte swizzle (this kernel has no static shared memory in front of it; checked below).
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = smem_raw;
    uint64_t* bars = (uint64_t*)(smem + TILE_BYTES);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * MAX_STAGES;
    const uint32_t bar_acc_full = bar_empty + 8 * MAX_STAGES, bar_acc_empty = bar_acc_full + 16;   // two of each
    const uint32_t bar_drain = bar_acc_empty + 16;
    const uint32_t bar_a_empty = bar_drain + 8;                        // resident candidate slots, one per 64-channel step
    uint32_t* tmem_slot = (uint32_t*)(bars + N_BARS);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
    const uint32_t tiles_base = smem_u32(smem);
    const TcScalars& P = KP.s;
    if (P.span && threadIdx.x == 0) atomicMax(P.span, ~global_ns());
    // First touches of parameter space miss the constant cache (several hundred cycles each, and
    // one after the other when a lone warp meets them on its way to the first copy): every warp
    // reads one word per 64 bytes of the scalars now, as independent loads.
    {
        const int w0 = P.H, w1 = P.n_apairs, w2 = P.items_base, w3 = P.sx_magic, w4 = P.units_per_group;
        asm volatile("" :: "r"(w0), "r"(w1), "r"(w2), "r"(w3), "r"(w4));
    }

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
    const bool leader = rank == 0;
    const int walker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    if ((tiles_base & 1023u) != 0) {                                   // never expected; refuse rather than compute garbage
        if (threadIdx.x == 0) atomicCAS(KP.s.status, 0, OC_ERR_ALIGNMENT);   // (same outcome in both CTAs of a pair)
        return;
    }

    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_acc_full + 8 * b, 1);
            // one arrival per epilogue warp (of both CTAs) that reads the accumulator set
            mbar_init(bar_acc_empty + 8 * b, (PAIR ? 2 : 1) * (KP.s.epi_split == EPI_BY_PIECE ? EPI_WARPS / 2 : EPI_WARPS));
        }
        mbar_init(bar_drain, 1);
        for (int k = 0; k < MAX_AKB; ++k) mbar_init(bar_a_empty + 8 * k, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 0 && lane == 0) {
        tma_prefetch_map(&KP.mapQ[0]);
        tma_prefetch_map(&KP.mapQ[1]);
        for (int m = 0; m <= KP.s.n_cand_lat; ++m)
            if (m != KP.s.rep_member || JOINT) tma_prefetch_map(&KP.mapsA[m]);
    }
    if (warp == 1) {
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         :: "r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         :: "r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    // The producer warp initialised the barriers itself (its lane 0, above), so in the single-CTA form
    // it does not wait for the rest of the set-up (the TMEM allocation): it goes on to decode its
    // first piece and issue its first stage, and joins this barrier from inside its loop.  In a pair the other
    // CTA's barriers must exist first, so everybody meets here.
    const bool early_producer = !PAIR && warp == 0;
    __syncwarp();
    if (!early_producer) {
        tc_fence_before();
        __syncthreads();
        if (PAIR) cluster_sync_all();      // the other CTA's barriers exist before anything signals them
        tc_fence_after();
    }
    const int STAGES = P.n_stages, STAGE_BYTES = P.stage_bytes;
    const bool dbl = P.tpp == 1 || P.narrow;                  // two accumulator sets take turns
    const uint32_t tile_stride = P.narrow ? 128u : 256u;      // TMEM columns between the two tiles' accumulators

    // (the joint form's work list is written by a kernel earlier in the stream: wait for it)
    if (JOINT) pdl_wait();
    Walk<JOINT> walk(P, walker);                  // every role walks the same pieces
    Piece c;
    const int bwA = 1 << P.bwA_log2, bwQ = 1 << P.bwQ_log2;
    const int my_rep = P.my_rep, mx_rep = P.mx_rep;
    const uint32_t tmem_base = early_producer ? 0u : *tmem_slot;    // (the producer warp never touches TMEM)

    if (warp == PRODUCER2_WARP && P.n_prod < 2) {
        // (the second producer warp sits this launch out)
    } else if (warp == 0 || warp == PRODUCER2_WARP) {
        // ================================ TMA producer ==========================================
        // Two producer warps take turns, stage by stage (the producer's own work per stage -- a look at a
        // barrier, one or two copy instructions, an arrival, all of them slow to issue beside the epilogue
        // warps -- is longer than the MMAs of a short stage; two of them halve it).  Each walks all pieces
        // and all stages, and acts on every other stage.
        const uint32_t my_turn = warp == 0 ? 0u : 1u;
        uint32_t gstage = 0;                          // stages handed out so far, over all pieces
        // Every stage costs the issuing thread one look at the stage's "empty" barrier, its copies and one
        // arrive on the "full" barrier.  When a CTA's candidate tiles are one box and its quanta of a piece
        // are one box (the usual case: see a_merged / q_merged) lane 0 does all of that by itself, with no
        // warp-wide exchange per stage; otherwise one lane per box: the first tpp lanes fetch the candidate
        // tiles, the next lanes one quantum each (in a pair: this CTA's half of the piece's quanta).
        int stage = 0; uint32_t phase = 0;
        uint32_t a_phase = 0;                         // resident candidate slots: flips with every row loaded
        uint32_t armed = 0;                           // stages with a copy possibly still in flight
        bool ok = true;
        bool joined = !early_producer;                // whether this warp has met the set-up barrier yet
        const uint32_t ring_base = tiles_base + (uint32_t)P.a_region_bytes;       // (a_region_bytes is 0 unless a_res)
        const bool solo = P.a_merged && P.q_merged;
        const uint32_t issue = elect_one();
        const uint32_t a_step = P.a_res ? (uint32_t)(P.tpp * A_BYTES) : 0u;     // resident slot pitch
        const uint32_t q_off = (uint32_t)(P.a_res ? 0 : P.tpp * A_BYTES);       // quanta inside a ring stage
        int trp = -1;
        while (ok && walk.next(P, c)) {
            ++trp;
            const int nq_mine = PAIR ? (c.nq >> 1) : c.nq;             // quanta this CTA fetches
            const int nA = P.a_merged ? 1 : P.tpp, nQ = P.q_merged ? 1 : nq_mine;   // boxes per stage
            // resident candidate tiles are fetched with the first piece of a row only, each 64-channel step
            // into its own slot, and reported to the barrier of the ring stage that carries the same step
            const bool load_a = !P.a_res || c.first;
            // what the leader's barrier expects per stage: the copies of both CTAs
            const uint32_t bytes = (uint32_t)((PAIR ? 2 : 1) * ((load_a ? P.tpp * A_BYTES : 0) + nq_mine * Q_BYTES));
            if (solo) {
                // (tiles past the lattice are fetched as zeros and masked in the epilogue)
                const int ta = (PAIR ? 2 : 1) * P.tpp * c.a_pair + (int)rank * P.tpp;
                const int htA = (int)div_small((unsigned)ta, (unsigned)P.n_wtA, P.rcp_n_wtA), wtA = ta - htA * P.n_wtA;
                const int wA = c.px * P.Ws + wtA * bwA, hA = c.py * P.Hs + htA * P.bhA;
                const int qi = c.q0 + (int)rank * nq_mine;
                const int hq = (int)div_small((unsigned)qi, (unsigned)P.n_wq, P.rcp_n_wq), wq = qi - hq * P.n_wq;
                const int wQ = c.px * P.Ws + wq * bwQ, hQ = c.py * P.Hs + hq * P.bhQ;
                const CUtensorMap* mapA = &KP.mapsA[c.member];
                const CUtensorMap* mapQ = &KP.mapQ[nq_mine != P.q_lo ? 1 : 0];
                for (int kb = 0; kb < P.kblocks; ++kb, ++gstage) {
                    // (the whole warp runs this; the elected lane issues)
                    if (ok && (P.n_prod < 2 || (gstage & 1u) == my_turn)) {
                        const uint32_t full_local = bar_full + 8 * stage;
                        const uint32_t full = PAIR ? map_to_cta(full_local, 0) : full_local;
                        bool go = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag);
                        // the slot of this step is free once the MMAs of the previous row's last piece have read it
                        if (go && P.a_res && load_a) go = mbar_wait(bar_a_empty + 8 * kb, a_phase ^ 1u, abort_flag);
                        if (__all_sync(0xFFFFFFFFu, go)) {
                            // the copies first, the arrival that carries their byte count after them: the barrier
                            // cannot complete before that arrival, and the copies are on their way sooner
                            tma_load_4d_elected<PAIR>(ring_base + stage * STAGE_BYTES + q_off, mapQ, kb * BK, wQ, hQ, c.bt, full, issue);
                            if (load_a)
                                tma_load_4d_elected<PAIR>(P.a_res ? tiles_base + (uint32_t)kb * a_step : ring_base + stage * STAGE_BYTES,
                                                          mapA, kb * BK, wA, hA, c.bt_a, full, issue);
                            if (leader) mbar_arrive_expect_tx_elected(full_local, bytes, issue);
                        } else {
                            ok = false;
                        }
                    }
                    armed |= 1u << stage;
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    if (!joined) { __syncwarp(); __syncthreads(); joined = true; }   // first stage on its way: meet the others
                }
            } else {
                const CUtensorMap* map;
                int w, h;
                uint32_t dst_off;
                if (lane < nA) {
                    map = &KP.mapsA[c.member];
                    const int ta = (PAIR ? 2 : 1) * P.tpp * c.a_pair + (int)rank * P.tpp + lane;
                    const int htA = (int)div_small((unsigned)ta, (unsigned)P.n_wtA, P.rcp_n_wtA), wtA = ta - htA * P.n_wtA;
                    w = c.px * P.Ws + wtA * bwA; h = c.py * P.Hs + htA * P.bhA;
                    dst_off = (uint32_t)(lane * A_BYTES);
                } else {
                    map = &KP.mapQ[(P.q_merged && nq_mine != P.q_lo) ? 1 : 0];
                    const int qi = c.q0 + (int)rank * nq_mine + lane - nA;
                    const int hq = (int)div_small((unsigned)qi, (unsigned)P.n_wq, P.rcp_n_wq), wq = qi - hq * P.n_wq;
                    w = c.px * P.Ws + wq * bwQ; h = c.py * P.Hs + hq * P.bhQ;
                    dst_off = q_off + (uint32_t)((lane - nA) * Q_BYTES);
                }
                const bool active = lane < nA ? load_a : lane < nA + nQ;
                for (int kb = 0; kb < P.kblocks; ++kb, ++gstage) {
                    if (P.n_prod > 1 && (gstage & 1u) != my_turn) {             // the other producer's stage
                        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                        continue;
                    }
                    const uint32_t full_local = bar_full + 8 * stage;
                    const uint32_t full = PAIR ? map_to_cta(full_local, 0) : full_local;
                    bool go = true;
                    if (lane == 0) {
                        go = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag);
                        if (go && P.a_res && load_a) go = mbar_wait(bar_a_empty + 8 * kb, a_phase ^ 1u, abort_flag);
                        if (go && leader) mbar_arrive_expect_tx(full_local, bytes);
                    }
                    go = __shfl_sync(0xFFFFFFFFu, (int)go, 0) != 0;
                    if (!go) { ok = false; break; }
                    if (active) {
                        const uint32_t dst = (lane < nA && P.a_res) ? tiles_base + (uint32_t)kb * a_step + dst_off
                                                                    : ring_base + stage * STAGE_BYTES + dst_off;
                        tma_load_4d<PAIR>(dst, map, kb * BK, w, h, lane < nA ? c.bt_a : c.bt, full);
                    }
                    armed |= 1u << stage;
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    if (!joined) { __syncthreads(); joined = true; }   // first stage on its way: meet the others
                }
            }
            if (P.a_res && load_a) a_phase ^= 1u;
        }
        if (!joined) { __syncthreads(); joined = true; }
        if (!ok && lane == 0) {
            atomicCAS(P.status, 0, OC_ERR_TIMEOUT);
            *abort_flag = 1;
            // copies already issued still write this CTA's shared memory: give each a bounded
            // chance to land before the CTA retires (the parity armed last is phase or phase^1)
            if (leader) {
                for (int s = 0; s < STAGES; ++s) {
                    if (!(armed & (1u << s))) continue;
                    const uint32_t par = (s < stage) ? phase : (phase ^ 1u);
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar_full + 8 * s, par) && global_ns() - t0 < 20000000ull) {}
                }
            } else {                                   // its copies report to the leader: allow them a fixed time
                const unsigned long long t0 = global_ns();
                while (global_ns() - t0 < 1000000ull) {}
            }
        }
    } else if (warp == 1) {
        // ================================ MMA issuer ============================================
        if (leader) {
            constexpr uint32_t IDESC_BASE = (1u << 4) | (1u << 7) | (1u << 10) |      // D=f32, A=B=bf16, K-major both,
                                            ((uint32_t)((PAIR ? 2 * BM : BM) >> 4) << 24);   // M=128 (256 across a pair)
            const uint32_t issue = elect_one();        // all lanes walk the loop, this one issues
            int stage = 0; uint32_t phase = 0;
            // K-major, 128-byte swizzle (as make_smem_desc): the constant part of every operand descriptor,
            // and the parts of the address field (16-byte units) that the loop adds up
            const uint64_t desc_hi = make_smem_desc(0);
            const bool a_res = P.a_res != 0;
            const int kblocks = P.kblocks;
            const uint32_t res_lo = (tiles_base >> 4) & 0x3FFFu, ring_lo = ((tiles_base + (uint32_t)P.a_region_bytes) >> 4) & 0x3FFFu;
            const uint32_t stage16 = (uint32_t)STAGE_BYTES >> 4, a_tile16 = (uint32_t)A_BYTES >> 4;
            const uint32_t a_slot16 = (uint32_t)(P.tpp * A_BYTES) >> 4, q_off16 = a_res ? 0u : a_slot16;
            bool ok = true, peeked = false;
            uint32_t it = 0;
            // (the commit that hands the accumulators to the epilogue is part of the last stage's block; taking
            //  the walk to the next piece between two stages instead of between two pieces measured slower)
            while (ok && walk.next(P, c)) {
                // one candidate tile per CTA leaves half of TMEM free: two accumulators take turns, and the
                // epilogue of a piece runs under the MMAs of the next one
                const uint32_t buf = dbl ? (it & 1u) : 0u, acc_phase = dbl ? ((it >> 1) & 1u) : (it & 1u);
                ++it;
                if (!__all_sync(0xFFFFFFFFu, mbar_wait(bar_acc_empty + 8 * buf, acc_phase ^ 1u, abort_flag))) { ok = false; break; }
                const uint32_t d_tmem = tmem_base + buf * 256u;
                tc_fence_after();
                const uint32_t idesc = IDESC_BASE | ((uint32_t)(c.ncol >> 3) << 17);
                // an odd number of candidate tiles leaves the last run with an empty second tile (in a pair:
                // empty in both CTAs): its MMAs are not issued, and the epilogue skips it likewise
                const bool two_tiles = P.tpp == 2 && (PAIR ? 2 : 1) * P.tpp * c.a_pair + 1 < P.n_tilesA;
                // descriptors of the piece's operands: low words only (the high word is one constant), kept
                // up to date by additions -- between two stages the tensor pipe runs dry unless this warp is
                // back with the next MMA within about one MMA's time
                const uint32_t c_off16 = (uint32_t)c.c_off * 8u;        // (c_off rows of 128 bytes, in 16-byte units)
                const uint32_t free_a = (a_res && c.last) ? 1u : 0u;
                for (int kb = 0; kb < kblocks; ++kb) {
                    // (each lane looked for itself; the barrier's phase cannot go back, so a lane that saw it
                    //  full stays right, and the others wait here)
                    if (!peeked) {
                        if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) ok = false;
                        if (!__all_sync(0xFFFFFFFFu, ok)) { ok = false; break; }
                    }
                    const uint32_t s_lo = ring_lo + (uint32_t)stage * stage16;
                    const uint32_t a_lo = a_res ? res_lo + (uint32_t)kb * a_slot16 : s_lo;
                    // (a piece that begins in mid-quantum skips 16 rows = 2 KB of its first box: a whole number
                    //  of 8-row swizzle groups)
                    const uint32_t b_lo = s_lo + q_off16 + c_off16;
                    int nstage = stage + 1; uint32_t nphase = phase;
                    if (nstage == STAGES) { nstage = 0; nphase ^= 1u; }
                    // UMMA K = 16 is 32 bytes along the swizzled row: +2 in the descriptor's address field.
                    // The commits free the stage (in both CTAs of a pair) when the MMAs retire, and with the
                    // row's last piece the resident candidate slot of this step.
                    peeked = tc_mma_stage<PAIR>(d_tmem, desc_hi | a_lo, desc_hi | (a_lo + a_tile16), desc_hi | b_lo, idesc,
                                                (uint32_t)(kb != 0), issue, two_tiles, bar_full + 8 * nstage, nphase, tile_stride,
                                                bar_empty + 8 * stage, free_a ? bar_a_empty + 8 * kb : 0u,
                                                kb + 1 == kblocks ? bar_acc_full + 8 * buf : 0u) != 0;
                    stage = nstage; phase = nphase;
                }
            }
            if (!ok && lane == 0) { atomicCAS(P.status, 0, OC_ERR_TIMEOUT); *abort_flag = 1; }
            // all MMAs issued by this warp must retire before TMEM is released
            tc_commit<PAIR>(PAIR ? map_to_cta(bar_drain, 0) : bar_drain, issue);
            const unsigned long long t0 = global_ns();
            while (!mbar_try_wait(bar_drain, 0) && global_ns() - t0 < WAIT_LIMIT_NS) {}
        }
    } else {
        // ================================ epilogue ==============================================
        const int et = threadIdx.x - 64;                               // 0..255
        const int part = et >> 7;                                      // which part of the piece's columns
        const int lane_group = warp & 3;                               // TMEM lanes this warp may read
        const int row = lane_group * 32 + lane;                        // tile row owned by this thread
        bool ok = true;
        uint32_t it = 0;
        const uint32_t acc_empty = PAIR ? map_to_cta(bar_acc_empty, 0) : bar_acc_empty;   // the leader's
        // Per representative slot of the GROUP (quantum by quantum, 32 lattice points each): the
        // representative's inverse norm, NaN where the slot is no representative of this patch, and per
        // quantum a bit mask of those slots (their keys are zeroed).  Each half of the epilogue warps
        // keeps its own table and rebuilds it when its pieces move on to another group (a barrier over
        // the half's four warps on either side: rare); a piece then costs a warp no table work at all,
        // its columns are a window into the table.
        const int ew = et >> 5;                                        // this warp among the epilogue warps
        float* gt_scale = (float*)(smem + P.gt_off + part * P.gt_half_bytes);
        uint32_t* gt_mask = (uint32_t*)(gt_scale + P.gt_quanta * QN);  // [gt_quanta + 1]
        const int split = P.epi_split;
        const int t_begin = split == EPI_BY_TILE ? part : 0, t_end = split == EPI_BY_TILE ? part + 1 : P.tpp;
        const uint32_t key_mul = P.key_mul;
        const int rowh = row >> P.bwA_log2, roww = row & (bwA - 1);
        // What a warp needs of a piece, gathered ahead of time.  A lone warp runs dependent integer
        // arithmetic at its full latency and pays for every branch, and this is on the one path that
        // bounds the kernel, so: no branches (selects and a clamped address instead), one division per
        // lookup, and that only when the row changes (the pieces of a row share their candidate tiles).
        struct Rows {
            int tokA[2];                     // the rows (candidate tokens) this thread owns in the piece's tiles
            bool row_ok[2];
            float inv_a[2];                  // their inverse norms
            float lift[2];
            int my, mx;
        };
        // floor(a / d) for 0 <= a < 2^22 from the float reciprocal, without a branch
        auto div_fast = [](int a, int d, float rcp_d) {
            int q = (int)((float)a * rcp_d);
            const int r = a - q * d;
            q += (r >= d ? 1 : 0) - (r < 0 ? 1 : 0);
            return q;
        };
        const float quiet_nan = __int_as_float(0x7FC00000);
        const int tok_per_lattice_row = P.sy * P.W;
        // The group's table: warp w of the half fills quanta w, w + 4, ...  Every warp of the half comes
        // here at the same piece (they take the same pieces), also one that has given up: it must not
        // leave the others waiting at the barriers.
        int table_bt = -1, table_py = -1, table_px = -1;
        auto rebuild_table = [&](const Piece& pc) {
            asm volatile("bar.sync %0, 128;" :: "r"(1 + part) : "memory");     // the old table is no longer read
            const int tok0 = (pc.bt * P.H + pc.py * P.Hs * P.sy + my_rep) * P.W + pc.px * P.Ws * P.sx + mx_rep;
            for (int q = ew & 3; q < P.gt_quanta; q += 4) {
                const int hq = div_fast(q, P.n_wq, P.rcp_n_wq), wq = q - hq * P.n_wq;
                const int hs = hq * P.bhQ + (lane >> P.bwQ_log2), ws = wq * bwQ + (lane & (bwQ - 1));
                const bool valid = (hs < P.Hs) & (ws < P.Ws);
                const float v = __ldg(P.inv_norm + (valid ? tok0 + hs * tok_per_lattice_row + ws * P.sx : 0));
                gt_scale[q * QN + lane] = valid ? v : quiet_nan;
                const uint32_t masked = __ballot_sync(0xFFFFFFFFu, !valid);
                if (lane == 0) gt_mask[q] = masked;
            }
            if ((ew & 3) == 0 && lane == 0) gt_mask[P.gt_quanta] = 0xFFFFFFFFu;     // (read with the last quantum's word)
            asm volatile("bar.sync %0, 128;" :: "r"(1 + part) : "memory");
            table_bt = pc.bt; table_py = pc.py; table_px = pc.px;
        };
        auto gather_rows = [&](const Piece& pc, Rows& a) {
            a.my = (pc.member * P.sx_magic) >> 16; a.mx = pc.member - a.my * P.sx;
            const int tok0 = (pc.bt_a * P.H + pc.py * P.Hs * P.sy + a.my) * P.W + pc.px * P.Ws * P.sx + a.mx;
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const int ta = (PAIR ? 2 : 1) * P.tpp * pc.a_pair + (int)rank * P.tpp + t;
                const int htA = div_fast(ta, P.n_wtA, P.rcp_n_wtA), wtA = ta - htA * P.n_wtA;
                const int hsA = htA * P.bhA + rowh, wsA = wtA * bwA + roww;
                a.row_ok[t] = (t < P.tpp) & (hsA < P.Hs) & (wsA < P.Ws);
                a.tokA[t] = a.row_ok[t] ? tok0 + hsA * tok_per_lattice_row + wsA * P.sx : 0;
                a.inv_a[t] = __ldg(P.inv_norm + a.tokA[t]);
            }
        };
        // The keys below want every scaled similarity of a row inside ONE binade, where the bits of a
        // float are linear in its value: the FMA that applies the scale also adds a lift of 3 * 2^k,
        // with 2^k the power of two at or above 1.001 x the row's own norm.  |<a, b>| / |b| <= |a|, so
        // the lifted values lie in [2^(k+1), 2^(k+2)); the lift is taken off the one value reported.
        auto set_lifts = [&](Rows& a) {
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const float bound = 1.001f / a.inv_a[t];
                a.lift[t] = 3.0f * __uint_as_float((__float_as_uint(bound) + 0x007FFFFFu) & 0x7F800000u);
            }
        };
        // Only from here on does this kernel touch what the norm pre-pass (the kernel before it in the
        // stream) writes: its operand copies and MMAs may run while that kernel still does.
        pdl_wait();
        if (et == 0) pdl_launch_dependents();
        Piece nx;
        Rows cur, rows_ahead;
        // this warp's next piece: every piece, or (EPI_BY_PIECE) every other one
        uint32_t handed = 0;                                           // pieces the walk has handed out
        auto next_mine = [&](Piece& pc, uint32_t& index, bool& new_row) -> bool {
            new_row = false;
            for (;;) {
                if (!walk.next(P, pc)) return false;
                index = handed++;
                new_row |= pc.first != 0;
                if (split != EPI_BY_PIECE || (index & 1u) == (uint32_t)part) return true;
            }
        };
        uint32_t it_nx = 0;
        bool new_row = false;
        bool have = next_mine(c, it, new_row);
        if (have) { gather_rows(c, cur); set_lifts(cur); }
        while (have) {
            const uint32_t buf = dbl ? (it & 1u) : 0u, acc_phase = dbl ? ((it >> 1) & 1u) : (it & 1u);
            const bool have_nx = next_mine(nx, it_nx, new_row);
            if (have_nx && new_row) gather_rows(nx, rows_ahead);       // in flight until the end of this piece
            if ((c.bt != table_bt) | (c.py != table_py) | (c.px != table_px)) rebuild_table(c);
            const int my = cur.my, mx = cur.mx;
            const float lift0 = cur.lift[0], lift1 = cur.lift[1];
            // chunks of 32 columns: all of them, or the first half to warps 2..5 and the rest to warps 6..9
            // (a last half chunk reads 16 columns of nothing: they are masked)
            const int n_ch = (c.ncol + 31) >> 5;
            const int ch_begin = split == EPI_BY_COLUMNS ? (part * n_ch + EPI_PARTS - 1) / EPI_PARTS : 0;
            const int ch_end = split == EPI_BY_COLUMNS ? ((part + 1) * n_ch + EPI_PARTS - 1) / EPI_PARTS : n_ch;
            // the piece's columns in the group's table (a piece may begin in mid-quantum)
            const int col0 = c.q0 * QN + c.c_off;
            const float* col_scale1 = gt_scale + col0;
            const float4* col_scale4 = (const float4*)col_scale1;
            // whether any column of the piece is masked: a slot outside the patch, or the tail of a last,
            // partial chunk (one mask word per lane)
            const int w_first = col0 >> 5, w_last = (col0 + c.ncol - 1) >> 5;
            const bool piece_masked = (c.ncol & 31) != 0 ||
                                      __any_sync(0xFFFFFFFFu, w_first + lane <= w_last && gt_mask[w_first + lane] != 0u);

            // warp-uniform outcome: the TMEM loads below are warp-collective
            const bool ready = ok && __all_sync(0xFFFFFFFFu, mbar_wait(bar_acc_full + 8 * buf, acc_phase, abort_flag));
            if (ready) {
                tc_fence_after();
                uint32_t won_key0 = 0, won_key1 = 0;                   // per tile: the row's largest key and its chunk
                int won_ch0 = -1, won_ch1 = -1;
                bool released = false;
#pragma unroll 1
                for (int t = t_begin; t < t_end; ++t) {                // the piece's candidate tiles (of this warp)
                    if ((PAIR ? 2 : 1) * P.tpp * c.a_pair + (int)rank * P.tpp + t >= P.n_tilesA) continue;   // past the lattice
                    const bool row_ok = (t ? cur.row_ok[1] : cur.row_ok[0]);
                    float inv_a = 0.f;
                    float* aux_row = nullptr;
                    if (AUX && P.aux && row_ok) {
                        inv_a = (t ? cur.inv_a[1] : cur.inv_a[0]);
                        const int ta = (PAIR ? 2 : 1) * P.tpp * c.a_pair + (int)rank * P.tpp + t;
                        const int htA = (int)div_small((unsigned)ta, (unsigned)P.n_wtA, P.rcp_n_wtA), wtA = ta - htA * P.n_wtA;
                        const int u_local = ((htA * P.bhA + rowh) * P.sy + my) * P.Wp + (wtA * bwA + roww) * P.sx + mx;
                        aux_row = P.aux + ((long long)c.g * P.units_per_group + u_local) * P.reps_per_group;
                    }
                    // Running maximum over "keys".  A key is the lifted similarity's bit pattern times 32
                    // plus 31 - (column within the chunk): the multiply drops the sign and the four high
                    // exponent bits, which all lifted values of a row share, and keeps every mantissa bit, so
                    // unsigned order of keys is order of similarity and then lowest column first, and ONE
                    // three-input integer max per three keys carries the arg max along.  Nothing is lost
                    // beyond the rounding of the FMA at the lift's magnitude (2^-23 of at most 4 x the row's
                    // norm: 5e-7 in units of the cosine).  Per element that is half a packed FMA, one
                    // multiply-add (every other one with a run-time factor, so that the compiler's shift-add
                    // on the ALU pipe and the integer FMA pipe share them) and half a max.  The 32 keys of a
                    // chunk are reduced by a tree of depth 4 (a running maximum would be a chain of 16
                    // dependent instructions, and with two epilogue warps per scheduler nothing else hides
                    // that latency); bc = the chunk in which the row's maximum last rose.
                    uint32_t bm = 0;
                    int bc = -1;
                    const float row_lift = t ? lift1 : lift0;
                    const uint32_t t_row = tmem_base + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)t * tile_stride + buf * 256u;
                    uint32_t va[32];
// (the scales of a chunk are asked for before the wait for its accumulators: shared memory is busy with
//  the MMAs' operand reads, and the answers take a few hundred cycles)
#define OC_LOAD_SCALES(ch)                                                                                       \
    do {                                                                                                         \
        _Pragma("unroll") for (int q = 0; q < 8; ++q) sc4[q] = col_scale4[(ch) * 8 + q];                         \
    } while (0)
// The keys of a chunk (and, in the parity instance, its row of the full similarity matrix): everything
// that reads the loaded accumulators and the scales, so that both registers sets are free afterwards.
#define OC_KEYS(v, ch, MASKED)                                                                                   \
    do {                                                                                                         \
        _Pragma("unroll") for (int j = 0; j < 32; j += 4) {                                                      \
            const float4 s4 = sc4[j >> 2];                                                                       \
            float x0, x1, x2, x3;                                                                                \
            fma_pair(x0, x1, v[j], v[j + 1], s4.x, s4.y, row_lift);                                              \
            fma_pair(x2, x3, v[j + 2], v[j + 3], s4.z, s4.w, row_lift);                                          \
            kf[j] = __float_as_uint(x0) * 32u + (uint32_t)(31 - j);                                              \
            kf[j + 1] = __float_as_uint(x1) * key_mul + (uint32_t)(30 - j);                                      \
            kf[j + 2] = __float_as_uint(x2) * 32u + (uint32_t)(29 - j);                                          \
            kf[j + 3] = __float_as_uint(x3) * key_mul + (uint32_t)(28 - j);                                      \
        }                                                                                                        \
        if (MASKED) {                                                  /* (a literal: two copies of the loop) */ \
            const int gcol = col0 + (ch) * 32, left = c.ncol - (ch) * 32;                                        \
            uint32_t masked = gt_mask[gcol >> 5];                                                                \
            if (gcol & 16) masked = (masked >> 16) | (gt_mask[(gcol >> 5) + 1] << 16);                           \
            if (left < 32) masked |= 0xFFFFFFFFu << left;              /* columns of the next piece */          \
            _Pragma("unroll") for (int j = 0; j < 32; ++j)                                                       \
                if ((masked >> j) & 1u) kf[j] = 0u;                                                              \
        }                                                                                                        \
        if (AUX && aux_row) {                                                                                    \
            for (int j = 0; j < 32; ++j) {                                                                       \
                const float sc = col_scale1[(ch) * 32 + j];                                                      \
                if ((ch) * 32 + j < c.ncol && sc == sc) {                                                        \
                    const int gp_ = c.c_off + (ch) * 32 + j;                                                     \
                    const int qi = c.q0 + (gp_ >> 5), r = gp_ & 31;                                              \
                    const int hq = (int)div_small((unsigned)qi, (unsigned)P.n_wq, P.rcp_n_wq), wq = qi - hq * P.n_wq;                                           \
                    const int hs = hq * P.bhQ + (r >> P.bwQ_log2), ws = wq * bwQ + (r & (bwQ - 1));              \
                    aux_row[hs * P.Ws + ws] = clamp_unit(__uint_as_float(v[j]) * sc * inv_a);                    \
                }                                                                                                \
            }                                                                                                    \
        }                                                                                                        \
    } while (0)
                    // The accumulators are handed back as soon as this warp's LAST load of them has landed in
                    // registers, before that chunk is reduced: the MMAs of the piece after next wait for it.
                    const bool last_tile = t + 1 == t_end;
#define OC_RELEASE_ACCUMULATORS()                                                                                \
    do {                                                                                                         \
        tc_fence_before();                                                                                       \
        __syncwarp();                                                                                            \
        if (lane == 0) {                                                                                         \
            if (PAIR) mbar_arrive_cluster(acc_empty + 8 * buf); else mbar_arrive(bar_acc_empty + 8 * buf);       \
        }                                                                                                        \
        released = true;                                                                                         \
    } while (0)
                    float4 sc4[8];
                    uint32_t kf[32];
                    // One register buffer for the accumulators: the next chunk's load and its scales are asked for
                    // as soon as this chunk's keys are formed, and arrive under the maximum tree.  The loop exists
                    // twice (with the mask test inside it every key of a chunk has to sit in a register before the
                    // first maximum is taken, masked columns or not).  A later chunk wins only with a strictly
                    // larger similarity (the index bits set aside); a zeroed key never does: a lifted similarity
                    // lies strictly above the binade's lower end, so a key is > 31.
#define OC_CHUNK_LOOP(MASKED)                                                                                    \
                    for (int ch = ch_begin; ch < ch_end; ++ch) {                                                 \
                        tmem_ld_wait();                                                                          \
                        if (ch + 1 == ch_end && last_tile) OC_RELEASE_ACCUMULATORS();                            \
                        OC_KEYS(va, ch, MASKED);                                                                 \
                        if (ch + 1 < ch_end) { tmem_ld32(t_row + (uint32_t)((ch + 1) * 32), va); OC_LOAD_SCALES(ch + 1); } \
                        const uint32_t cm = key_tree_max(kf);                                                    \
                        if (cm > (bm | 31u)) { bm = cm; bc = ch; }                                               \
                    }
                    if (ch_begin < ch_end) { tmem_ld32(t_row + (uint32_t)(ch_begin * 32), va); OC_LOAD_SCALES(ch_begin); }
                    if (piece_masked) {
#pragma unroll 1
                        OC_CHUNK_LOOP(1)
                    } else {
#pragma unroll 1
                        OC_CHUNK_LOOP(0)
                    }
#undef OC_CHUNK_LOOP
#undef OC_LOAD_SCALES
#undef OC_KEYS
                    if (t) { won_key1 = bm; won_ch1 = row_ok ? bc : -1; } else { won_key0 = bm; won_ch0 = row_ok ? bc : -1; }
                }
                if (!released) OC_RELEASE_ACCUMULATORS();              // (no chunk of a last tile: nothing was loaded)
#undef OC_RELEASE_ACCUMULATORS
                // The rows' results go out only after the arrival: it releases what its thread wrote before
                // it, and would wait for these atomics to be performed.
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const uint32_t bm = t ? won_key1 : won_key0;
                    const int bc = t ? won_ch1 : won_ch0;
                    if (bc < 0) continue;
                    const float row_lift = t ? lift1 : lift0;
                    const int n0 = bc * 32 + 31 - (int)(bm & 31u);
                    // the winner's bits again: what the multiply dropped is what the lift's own bits have there
                    const float best = __uint_as_float((bm >> 5) | (__float_as_uint(row_lift) & 0xF8000000u)) - row_lift;   // (exact)
                    const int gp = c.c_off + n0;
                    const int qi = c.q0 + (gp >> 5), r = gp & 31;
                    const int hq = (int)div_small((unsigned)qi, (unsigned)P.n_wq, P.rcp_n_wq), wq = qi - hq * P.n_wq;
                    const int hs = hq * P.bhQ + (r >> P.bwQ_log2), ws = wq * bwQ + (r & (bwQ - 1));
                    const int y = (c.py * P.Hs + hs) * P.sy + my_rep, x = (c.px * P.Ws + ws) * P.sx + mx_rep;
                    const long long tokB = ((long long)c.bt * P.H + y) * P.W + x;
                    atomicMax(P.keys + (t ? cur.tokA[1] : cur.tokA[0]), pack_key(best, (uint32_t)tokB));
                }
            } else if (ok) {
                ok = false;
                atomicCAS(P.status, 0, OC_ERR_TIMEOUT);
                *abort_flag = 1;                                       // the other roles give up at their next wait
            }
            // (a warp that has given up still walks its remaining pieces, without waiting for anything: the
            //  other warps of its half may be at a table's barriers, which want all four of them)
            if (have_nx && new_row) { cur = rows_ahead; set_lifts(cur); }
            c = nx; have = have_nx;
            it = it_nx;
        }
        if (!ok) { atomicCAS(P.status, 0, OC_ERR_TIMEOUT); *abort_flag = 1; }
    }

    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();          // nobody signals a barrier of, or reads operands from, a retired CTA
    tc_fence_after();
    if (warp == 1) {
        if (PAIR)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"(TMEM_COLS) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
    if (P.span && threadIdx.x == 0) atomicMax(P.span + 1, global_ns());
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
    int pair, q_unit, n_q_units, half_units, a_merged, q_merged, q_lo, q_hi, q_rows;
    int pieces_per_row, qmax, n_stages, stage_bytes, narrow;
    int a_res, a_region_bytes;
    int gt_half_bytes;                   // one group table: a scale per representative slot and a mask word per quantum (+1)
    long long rows, items;
};
// quanta of 32 lattice points that cover one group's representatives
static int group_quanta(const Geo& g) {
    int lq = pow2_ceil_log2(g.Ws); if ((1 << lq) > QN) lq = pow2_ceil_log2(QN);
    const int bhQ = QN >> lq;
    return ((g.Ws + (1 << lq) - 1) >> lq) * ((g.Hs + bhQ - 1) / bhQ);
}

// A forced work split (oc_tc_plan_override): the tests run every form of the kernel this way.
struct TcForce { bool on; int pair, tiles, pieces, no_narrow, a_res /* -1: the planner's choice */; };

// walkers: CTAs that can run at once; pair_walkers: CTA pairs that can (0 = pairs not available)
static TcPlan make_plan(const Geo& g, int walkers, int pair_walkers, const TcForce& force) {
    TcPlan p;
    int la = pow2_ceil_log2(g.Ws); if ((1 << la) > BM) la = pow2_ceil_log2(BM);
    p.bwA_log2 = la; p.bhA = BM >> la;
    p.n_wtA = (g.Ws + (1 << la) - 1) >> la;
    p.n_tilesA = p.n_wtA * ((g.Hs + p.bhA - 1) / p.bhA);
    int lq = pow2_ceil_log2(g.Ws); if ((1 << lq) > QN) lq = pow2_ceil_log2(QN);
    p.bwQ_log2 = lq; p.bhQ = QN >> lq;
    p.n_wq = (g.Ws + (1 << lq) - 1) >> lq;
    p.n_quanta = p.n_wq * ((g.Hs + p.bhQ - 1) / p.bhQ);
    // two tables (one per half of the epilogue warps) at the end of the operand region: the ring gets the rest
    p.gt_half_bytes = (p.n_quanta * (QN * 4 + 4) + 4 + 15) / 16 * 16;
    const int ring_cap = TILE_BYTES - 2 * p.gt_half_bytes;
    // Form (single CTA or CTA pair), candidate tiles per CTA (1 or 2), pieces per row and whether the
    // candidate tiles stay resident, by estimated cycles of the busiest walker.  The shape of the estimate
    // follows the kernel; its constants were fitted (least squares on the logarithm, over 40 timed plans)
    // to sweeps of forced plans on four workloads (the SD3-shaped token cache and the three SVD UNet
    // levels); the estimate picks the fastest measured plan on each of them:
    //   * a 64-channel stage issues tpp*64*q tensor cycles (x0.9 as fitted) and cannot go faster than
    //     the hand-over of a ring slot (~490 cycles), than its copies arrive (~81 B/clk), nor than shared
    //     memory serves the copies' writes and the MMAs' operand reads together (~138 B/clk: one tile of
    //     256 columns reads 48 KB and is sent 32 KB per stage; a CTA pair halves the representatives' part
    //     of both, which is what makes the pair faster on wide pieces);
    //   * the epilogue costs ~340 cycles per 32 columns per tile.  With two accumulator sets (one tile, or
    //     two tiles and pieces of at most 128 columns) each half of its warps takes every other piece and
    //     runs under the MMAs of the next one: the piece takes the longest of its MMAs, half its epilogue,
    //     and half of (epilogue + MMAs) plus ~720 (a set is not reused before its epilogue is over);
    //     otherwise the epilogue follows the MMAs;
    //   * ~3400 cycles before a CTA's first MMA and after its last.
    const int kblocks = (g.C + BK - 1) / BK;
    // Single-CTA pieces are cut in units of HALF a quantum (16 columns) whenever that is valid: no piece
    // wider than 256 columns, none that would have to fetch more than MAXQ quanta (one that begins in
    // mid-quantum fetches its first quantum whole).  Returns the widest piece in half units, or 0.
    const int n_half = 2 * p.n_quanta;
    auto half_widest = [&](int P) -> int {
        if (P < 1 || P > p.n_quanta) return 0;
        const int h_max = (n_half + P - 1) / P;
        if (h_max > 2 * MAXQ) return 0;
        if (h_max == 2 * MAXQ && !(n_half % P == 0 && (h_max & 1) == 0)) return 0;   // 256 columns only from even starts
        return h_max;
    };
    double best_cost = 0; int best_P = 0, best_tpp = 2, best_pair = 0, best_ar = 0;
    for (int pair = 0; pair <= (pair_walkers > 0 ? 1 : 0); ++pair) {
        const int ncta = pair ? 2 : 1, q_unit = pair ? 2 : 1;
        const int n_units = (p.n_quanta + q_unit - 1) / q_unit, max_units = MAXQ / q_unit;
        const int nw = pair ? pair_walkers : walkers;
        for (int tpp = 1; tpp <= 2; ++tpp) {
            const long long rows = g.n_groups * (long long)(g.sy * g.sx - 1) *
                                   ((p.n_tilesA + tpp * ncta - 1) / (tpp * ncta));
            for (int P = (n_units + max_units - 1) / max_units; P <= n_units; ++P) {
                int q = ((n_units + P - 1) / P) * q_unit;             // quanta of the largest piece: for the MMAs ...
                int q_load = q;                                       // ... and fetched per stage
                const int hw = pair ? 0 : half_widest(P);
                if (hw) { q_load = (hw + 2) >> 1; if (q_load > MAXQ) q_load = MAXQ; }
                const double qe = hw ? hw * 0.5 : (double)q;          // width in quanta (may end in a half)
                if (hw) q = (hw + 1) >> 1;
                const long long per_walker = (rows * P + nw - 1) / nw;
                const double mma = tpp * 64.0 * qe * 0.897;
                // (two tiles whose pieces are at most 128 columns wide leave room for a second set of
                //  accumulators, like one tile does)
                const int cols = hw ? hw * 16 : q * 32, chunks = (cols + 31) / 32;
                const bool overlapped = tpp == 1 || cols <= 128;
                const double epi_all = 338.4 * (overlapped ? tpp * chunks : (tpp == 2 ? chunks : (chunks + 1) / 2));
                const double epi = overlapped ? 0.5 * epi_all : epi_all;   // per piece and warp
                for (int ar = 1; ar >= 0; --ar) {                           // (equal estimates: fewer bytes fetched wins)
                    const double a_kb = tpp * 16.0, q_kb = 4.0 * q_load / ncta;
                    if (ar && (kblocks > MAX_AKB || a_kb * kblocks + 3 * q_kb > ring_cap / 1024 || P == 1)) continue;
                    const double sent_kb = (ar ? 0.0 : a_kb) + q_kb, read_kb = tpp * (16.0 + 4.0 * qe / ncta);
                    const double feed = sent_kb * 1024.0 / 80.7, smem = (sent_kb + read_kb) * 7.42;
                    double piece;
                    if (overlapped) {
                        double stage = mma + 54.0; if (stage < 488.0) stage = 488.0; if (stage < feed) stage = feed; if (stage < smem) stage = smem;
                        const double loop = kblocks * stage + 530.0, reuse = 0.5 * (epi_all + loop) + 723.0;
                        piece = loop; if (piece < epi + 66.0) piece = epi + 66.0; if (piece < reuse) piece = reuse;
                    } else {
                        double stage = mma + 213.0; if (stage < 307.0) stage = 307.0; if (stage < feed) stage = feed; if (stage < smem) stage = smem;
                        piece = kblocks * stage + epi + 955.0;
                    }
                    if (pair) piece += 123.0;
                    const double cost = 3377.0 + per_walker * piece + (overlapped ? epi_all : 0.0);
                    if (best_P == 0 || cost < best_cost) { best_cost = cost; best_P = P; best_tpp = tpp; best_pair = pair; best_ar = ar; }
                }
            }
        }
    }
    // A forced split replaces the choice (ignored unless the shape admits it).
    if (force.on) {
        const int o_pair = force.pair, o_tpp = force.tiles, o_P = force.pieces;
        if ((o_pair == 0 || (o_pair == 1 && pair_walkers > 0)) && (o_tpp == 1 || o_tpp == 2)) {
            const int q_unit = o_pair ? 2 : 1;
            const int n_units = (p.n_quanta + q_unit - 1) / q_unit, max_units = MAXQ / q_unit;
            if (o_P >= (n_units + max_units - 1) / max_units && o_P <= n_units) { best_pair = o_pair; best_tpp = o_tpp; best_P = o_P; }
        }
    }
    p.pair = best_pair; p.tpp = best_tpp;
    p.half_units = (!p.pair && half_widest(best_P)) ? 1 : 0;
    p.q_unit = p.pair ? 2 : 1;
    p.n_q_units = p.half_units ? n_half : (p.n_quanta + p.q_unit - 1) / p.q_unit;
    const int ncta = p.pair ? 2 : 1;
    p.n_apairs = (p.n_tilesA + p.tpp * ncta - 1) / (p.tpp * ncta);
    p.rows = g.n_groups * (long long)(g.sy * g.sx - 1) * p.n_apairs;
    p.pieces_per_row = best_P;
    // fewest and most quanta any piece fetches (per CTA); and whether every CTA's run of quanta is a whole
    // number of lattice rows (lattices wider than one quantum: the run is then one rectangle of rows)
    int q_min = 1 << 30, q_max = 0;
    bool whole_rows = p.n_wq > 1 && p.bhQ == 1 && p.n_wq * QN <= 256;
    for (int j = 0; j < best_P; ++j) {
        const int u0 = (int)((long long)j * p.n_q_units / best_P), u1 = (int)((long long)(j + 1) * p.n_q_units / best_P);
        const int q0 = p.half_units ? (u0 >> 1) : u0 * p.q_unit;
        int nq = p.half_units ? ((u1 - 1) >> 1) - (u0 >> 1) + 1 : (u1 - u0) * p.q_unit / ncta;
        if (nq < q_min) q_min = nq;
        if (nq > q_max) q_max = nq;
        for (int r = 0; r < ncta; ++r)
            if ((q0 + r * nq) % p.n_wq != 0 || nq % p.n_wq != 0) whole_rows = false;
    }
    p.qmax = q_max * ncta;
    {   // widest piece in columns (a forced split may keep such plans on one accumulator set)
        const int hw = p.half_units ? half_widest(best_P) : 0;
        const int cols = hw ? hw * 16 : ((p.n_q_units + best_P - 1) / best_P) * p.q_unit * 32;
        p.narrow = (p.tpp == 2 && cols <= 128 && !(force.on && force.no_narrow)) ? 1 : 0;
    }
    // Candidate tiles resident (all 64-channel steps of a CTA's tiles in front of the ring, fetched once per
    // row instead of once per piece): possible when they leave room for at least three ring stages of
    // representatives.
    const int a_region = p.tpp * A_BYTES * kblocks;
    const bool a_res_ok = kblocks <= MAX_AKB && a_region + 3 * q_max * Q_BYTES <= ring_cap && best_P > 1;
    p.a_res = a_res_ok ? (force.on ? (force.a_res != 0) : (best_ar != 0)) : 0;
    p.a_region_bytes = p.a_res ? a_region : 0;
    p.stage_bytes = (p.a_res ? 0 : p.tpp * A_BYTES) + q_max * Q_BYTES;
    p.n_stages = (ring_cap - p.a_region_bytes) / p.stage_bytes;
    if (p.n_stages > MAX_STAGES) p.n_stages = MAX_STAGES;
    p.items = p.rows * p.pieces_per_row;
    // One copy instruction costs the producer ~100 cycles whatever the box size, so a CTA's candidate
    // tiles, and its quanta of a piece, travel as ONE box each whenever they stack into a rectangle
    // of lattice rows (always the case when the patch's lattice is at most one box wide).
    p.a_merged = (p.tpp == 1 || p.n_wtA == 1) ? 1 : 0;
    p.q_rows = whole_rows ? 1 : 0;            // ... or when every run of quanta is a rectangle of whole lattice rows
    p.q_merged = (p.n_wq == 1 || whole_rows) ? 1 : 0;
    p.q_lo = q_min;                           // merged boxes come in two heights: q_lo and q_hi quanta
    p.q_hi = q_max;
    return p;
}

bool tc_match_supported(const Geo& g) {
    if (g.kind != OC_KIND_TOKEN || g.dtype != OC_DTYPE_BF16 || g.self_match) return false;
    if (g.sy * g.sx > MAX_LATTICES) return false;
    if (g.C % 8 != 0) return false;
    if ((long long)g.B * g.T > 0x7FFFFFFFll) return false;
    if (group_quanta(g) > GT_MAX_QUANTA) return false;           // the group's scale tables would not fit beside the ring
    return encode_fn() != nullptr;
}

// Once per device (the context's device is current): opt in to the large dynamic shared memory and ask
// how many CTA pairs fit.  False if the attributes could not be set.
static bool tc_device_setup(oc_ctx* ctx, int* pair_walkers_out) {
    static PerDeviceOnce attr_once;
    static int max_pairs[PerDeviceOnce::MAX_DEV];
    const int dev = ctx->device;
    const int sm_count = ctx->sm_count;
    const bool attr_ok = attr_once.ensure(dev, [dev, sm_count] {
        const bool ok =
            cudaFuncSetAttribute(match_tc_kernel<false, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_TOTAL) == cudaSuccess &&
            cudaFuncSetAttribute(match_tc_kernel<true, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_TOTAL) == cudaSuccess &&
            cudaFuncSetAttribute(match_tc_kernel<false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_TOTAL) == cudaSuccess &&
            cudaFuncSetAttribute(match_tc_kernel<true, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_TOTAL) == cudaSuccess &&
            cudaFuncSetAttribute(match_tc_kernel<false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_TOTAL) == cudaSuccess &&
            cudaFuncSetAttribute(match_tc_kernel<true, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_TOTAL) == cudaSuccess;
        if (!ok) { cudaGetLastError(); return false; }
        if (dev >= 0 && dev < PerDeviceOnce::MAX_DEV) {
            cudaLaunchConfig_t q = {};
            cudaLaunchAttribute qa[1];
            qa[0].id = cudaLaunchAttributeClusterDimension;
            qa[0].val.clusterDim.x = 2; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
            q.gridDim = dim3(2 * (unsigned)(sm_count / 2)); q.blockDim = dim3(TC_THREADS);
            q.dynamicSmemBytes = SMEM_TOTAL; q.attrs = qa; q.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, match_tc_kernel<true, 0>, &q) != cudaSuccess) { cudaGetLastError(); n = 0; }
            if (n > sm_count / 2) n = sm_count / 2;
            max_pairs[dev] = n;
        }
        return true;
    });
    *pair_walkers_out = (attr_ok && dev >= 0 && dev < PerDeviceOnce::MAX_DEV) ? max_pairs[dev] : 0;
    return attr_ok;
}

oc_status tc_plan_describe(oc_ctx* ctx, const Geo& g, int32_t* out) {
    if (!tc_match_supported(g)) return OC_ERR_UNSUPPORTED;
    int pair_walkers = 0;
    if (!tc_device_setup(ctx, &pair_walkers)) return OC_ERR_CUDA;
    const TcForce force = {ctx->tc_plan_forced, ctx->tc_plan_pair, ctx->tc_plan_tiles, ctx->tc_plan_pieces, ctx->tc_plan_no_narrow,
                           ctx->tc_plan_a_res};
    const TcPlan p = make_plan(g, ctx->sm_count, pair_walkers, force);
    long long walkers = p.items;
    const int cap = p.pair ? pair_walkers : ctx->sm_count;
    if (walkers > cap) walkers = cap;
    const int widest = p.half_units ? ((2 * p.n_quanta + p.pieces_per_row - 1) / p.pieces_per_row) * 16
                                    : ((p.n_q_units + p.pieces_per_row - 1) / p.pieces_per_row) * p.q_unit * 32;
    const int v[12] = {p.pair, p.tpp, p.pieces_per_row, (p.tpp == 1 || p.narrow) ? 1 : 0, p.n_stages, p.stage_bytes, p.a_res,
                       (int)(p.items > 0x7FFFFFFFll ? 0x7FFFFFFF : p.items), (int)walkers, widest, (g.C + BK - 1) / BK, 0};
    for (int i = 0; i < 12; ++i) out[i] = v[i];
    return OC_OK;
}

static oc_status launch_tc(oc_ctx* ctx, const Geo& g, const void* x, const float* inv_norm, unsigned long long* keys,
                           float* aux_sim, const int4* units, const int* n_units_dev, long long max_units, cudaStream_t s);

oc_status launch_match_token_tc(oc_ctx* ctx, const Geo& g, const void* x, const float* inv_norm,
                                unsigned long long* keys, float* aux_sim, cudaStream_t s) {
    return launch_tc(ctx, g, x, inv_norm, keys, aux_sim, nullptr, nullptr, 0, s);
}

// Joint form: `units` (device) lists {representative frame, candidate frame, member} triples, `n_units_dev`
// (device) how many; max_units bounds the list (it sizes the launch).  g: one patch per frame.
oc_status launch_match_joint_tc(oc_ctx* ctx, const Geo& g, const void* x, const float* inv_norm,
                                unsigned long long* keys, const int4* units, const int* n_units_dev,
                                long long max_units, cudaStream_t s) {
    if (g.gy != 1 || g.gx != 1 || !units || !n_units_dev || max_units <= 0) return OC_ERR_UNSUPPORTED;
    return launch_tc(ctx, g, x, inv_norm, keys, nullptr, units, n_units_dev, max_units, s);
}

static oc_status launch_tc(oc_ctx* ctx, const Geo& g, const void* x, const float* inv_norm, unsigned long long* keys,
                           float* aux_sim, const int4* units, const int* n_units_dev, long long max_units, cudaStream_t s) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return OC_ERR_UNSUPPORTED;
    int pair_walkers = 0;
    if (!tc_device_setup(ctx, &pair_walkers)) return OC_ERR_CUDA;
    const TcForce force = {ctx->tc_plan_forced, ctx->tc_plan_pair, ctx->tc_plan_tiles, ctx->tc_plan_pieces, ctx->tc_plan_no_narrow,
                           ctx->tc_plan_a_res};
    const TcPlan p = make_plan(g, ctx->sm_count, pair_walkers, force);
    if (p.items > 0x7FFFFFFFll) return OC_ERR_UNSUPPORTED;

    TcParams KP;
    memset(&KP, 0, sizeof(KP));
    TcScalars& P = KP.s;
    const cuuint64_t dims[4] = {(cuuint64_t)g.C, (cuuint64_t)(g.W / g.sx), (cuuint64_t)(g.H / g.sy),
                                (cuuint64_t)g.B * g.T};
    const cuuint64_t strides[3] = {(cuuint64_t)g.sx * g.C * 2, (cuuint64_t)g.sy * g.W * g.C * 2,
                                   (cuuint64_t)g.H * g.W * g.C * 2};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const cuuint32_t boxA[4] = {(cuuint32_t)BK, (cuuint32_t)(1 << p.bwA_log2),
                                (cuuint32_t)(p.bhA * (p.a_merged ? p.tpp : 1)), 1};
    const int q_hi = p.q_hi;
    // (a run of whole lattice rows: the box is n_wq quanta wide and one lattice row per n_wq quanta high)
    const cuuint32_t q_box_w = (cuuint32_t)(p.q_rows ? p.n_wq * QN : (1 << p.bwQ_log2));
    const int q_per_h = p.q_rows ? p.n_wq : 1;
    const cuuint32_t boxQ[2][4] = {
        {(cuuint32_t)BK, q_box_w, (cuuint32_t)(p.bhQ * (p.q_merged ? p.q_lo / q_per_h : 1)), 1},
        {(cuuint32_t)BK, q_box_w, (cuuint32_t)(p.bhQ * (p.q_merged ? q_hi / q_per_h : 1)), 1}};
    const int rep_member = g.oy * g.sx + g.ox;
    const int n_members = g.sy * g.sx;
    for (int m = 0; m < n_members + 2; ++m) {
        const bool quantum_map = m >= n_members;
        const int member = quantum_map ? rep_member : m;
        if (!quantum_map && member == rep_member && !units) continue;    // representatives are candidates only across frames
        const int my = member / g.sx, mx = member - my * g.sx;
        void* base = (uint8_t*)x + ((size_t)my * g.W + mx) * g.C * 2;
        CUresult r = enc(quantum_map ? &KP.mapQ[m - n_members] : &KP.mapsA[m], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base,
                         dims, strides, quantum_map ? boxQ[m - n_members] : boxA, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return OC_ERR_UNSUPPORTED;     // the FMA matcher takes over
    }
    P.H = g.H; P.W = g.W; P.sy = g.sy; P.sx = g.sx; P.gy = g.gy; P.gx = g.gx;
    P.Hp = g.Hp; P.Wp = g.Wp; P.Hs = g.Hs; P.Ws = g.Ws;
    P.rep_member = rep_member; P.n_cand_lat = g.sy * g.sx - 1;
    P.kblocks = (g.C + BK - 1) / BK;
    P.bwA_log2 = p.bwA_log2; P.bhA = p.bhA; P.n_wtA = p.n_wtA; P.n_tilesA = p.n_tilesA; P.tpp = p.tpp; P.narrow = p.narrow; P.n_apairs = p.n_apairs;
    P.bwQ_log2 = p.bwQ_log2; P.bhQ = p.bhQ; P.n_wq = p.n_wq; P.n_quanta = p.n_quanta;
    P.pieces_per_row = p.pieces_per_row; P.total_items = (int)p.items;
    P.q_unit = p.q_unit; P.n_q_units = p.n_q_units; P.half_units = p.half_units;
    P.a_merged = p.a_merged; P.q_merged = p.q_merged; P.q_lo = p.q_lo;
    P.n_stages = p.n_stages; P.stage_bytes = p.stage_bytes;
    P.a_res = p.a_res; P.a_region_bytes = p.a_region_bytes;
    // two producers pay where a stage is short (one candidate tile per CTA); with two tiles the MMAs of a
    // stage cover one producer's work and the second warp only competes for issue slots
    P.n_prod = (N_PRODUCERS > 1 && p.tpp == 1) ? 2 : 1;
    P.key_mul = 32u;
    P.gt_half_bytes = p.gt_half_bytes; P.gt_off = TILE_BYTES - 2 * p.gt_half_bytes; P.gt_quanta = p.n_quanta;
    P.epi_split = (p.tpp == 1 || p.narrow) ? EPI_BY_PIECE : (p.tpp == 2 ? EPI_BY_TILE : EPI_BY_COLUMNS);
    P.units_per_group = (int)g.units_per_group; P.reps_per_group = (int)g.reps_per_group;
    P.inv_norm = inv_norm; P.keys = keys; P.aux = aux_sim; P.status = ctx->d_status;
    if (ctx->span_on) {
        P.span = ctx->d_span + 2 * (ctx->span_count & 255);
        ++ctx->span_count;
        if (cudaMemsetAsync(P.span, 0, 2 * sizeof(unsigned long long), s) != cudaSuccess) return OC_ERR_CUDA;
    }
    // one walker (CTA or CTA pair) per SM (pair of SMs), or one per piece when there are fewer pieces
    P.units = units; P.n_units_dev = n_units_dev;
    long long walkers = units ? max_units * (long long)p.pieces_per_row * p.n_apairs : p.items;
    const int cap = p.pair ? pair_walkers : ctx->sm_count;
    if (walkers > cap) walkers = cap;
    if (walkers < 1) walkers = 1;
    P.items_base = (int)(p.items / walkers); P.items_rem = (int)(p.items % walkers);
    P.n_walkers = (unsigned)walkers; P.rcp_walkers = 1.0f / (float)walkers;
    if (units && max_units * (long long)p.pieces_per_row * p.n_apairs > 0x7FFFFFFFll) return OC_ERR_UNSUPPORTED;
    P.cum[0] = (unsigned)p.pieces_per_row; P.cum[1] = P.cum[0] * (unsigned)p.n_apairs;
    P.cum[2] = P.cum[1] * (unsigned)P.n_cand_lat; P.cum[3] = P.cum[2] * (unsigned)g.gx; P.cum[4] = P.cum[3] * (unsigned)g.gy;
    P.u_step_q = p.n_q_units / p.pieces_per_row; P.u_step_r = p.n_q_units % p.pieces_per_row;
    for (int i = 0; i < 5; ++i) P.rcp_cum[i] = 1.0f / (float)P.cum[i];
    P.rcp_ppr = 1.0f / (float)p.pieces_per_row;
    P.rcp_n_wtA = 1.0f / (float)p.n_wtA; P.rcp_n_wq = 1.0f / (float)p.n_wq;
    P.my_rep = rep_member / g.sx; P.mx_rep = rep_member % g.sx;
    P.sx_magic = (65536 + g.sx - 1) / g.sx;
    LaunchScope scope(ctx, OC_K_MATCH_TC, s);
    if (p.pair) {
        PdlLaunch l(dim3(2 * (unsigned)walkers), dim3(TC_THREADS), SMEM_TOTAL, s, 2);
        const cudaError_t e = units ? cudaLaunchKernelEx(&l.cfg, match_tc_kernel<true, 2>, KP)
                            : aux_sim ? cudaLaunchKernelEx(&l.cfg, match_tc_kernel<true, 1>, KP)
                                      : cudaLaunchKernelEx(&l.cfg, match_tc_kernel<true, 0>, KP);
        if (e != cudaSuccess) { cudaGetLastError(); return OC_ERR_CUDA; }
        return OC_OK;
    }
    if (units) OC_LAUNCH((match_tc_kernel<false, 2>), (unsigned)walkers, TC_THREADS, SMEM_TOTAL, s, KP);
    else if (aux_sim) OC_LAUNCH((match_tc_kernel<false, 1>), (unsigned)walkers, TC_THREADS, SMEM_TOTAL, s, KP);
    else OC_LAUNCH((match_tc_kernel<false, 0>), (unsigned)walkers, TC_THREADS, SMEM_TOTAL, s, KP);
    return last_launch_status();
}

}  // namespace oc

