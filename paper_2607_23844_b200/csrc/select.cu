// select: threshold / keep-count selection, order-preserving compaction, match map.
//
// One CTA per group (a group is an independent selection problem).  Everything is decided in
// ascending unit order, so the result is deterministic and comparable bit for bit:
//   COUNT mode  - the candidates' best_sim are staged once in shared memory as order-preserving
//                 keys; a radix select finds the value at the cut (fast kernel: 12-bit digits of the
//                 key relative to the smallest candidate key, two passes for the narrow range one
//                 group's similarities span; general kernel: 4 x 8-bit digits of the raw key with
//                 warp-aggregated histogram updates); candidates above the cut are reused, candidates
//                 equal to it are admitted lowest index first;
//   both modes  - kept units are compacted with block-wide prefix sums (stable, ascending original
//                 index).
// Two kernels: select_fast_kernel (groups up to 40960 units, the usual case) reads every input once
// up front, gives each thread a contiguous run of units so that only two block-wide scans are needed,
// and writes all outputs in one coalesced pass at the end; select_general_kernel covers self-match
// and larger groups with a round-by-round loop.
#include "common.cuh"

namespace oc {

static constexpr int SEL_THREADS = 1024;
static constexpr int SEL_MAX_UNITS = 65536;
static constexpr int SEL_SMEM_KEYS = 40960;          // keys cached in shared memory up to this many units

// Per-CTA view of one group: unit index and candidate test with as few instructions as possible
// (one CTA serves a whole group, so the kernel is bound by instruction issue on a single SM):
// shifts and masks when the row width / lattice strides are powers of two, divisions otherwise.
template <bool JOINT = false>
struct GroupView {
    long long base;     // global index of local unit 0 (TOKEN: of the patch's first token)
    int unit_stride;    // FRAME: distance between consecutive frames of a patch position
    int row_pitch;      // TOKEN, BLOCK: frame width W
    int w_local;        // row width of the local unit grid (TOKEN, BLOCK: Wp; FRAME: 0)
    int w_shift;        // log2(w_local) if it is a power of two, else -1
    int lat_pow2;       // sy and sx are both powers of two
    int contig;         // local units are equally spaced in unit order (FRAME; patches as wide as the frame)
    long long base1;    // joint form: global index of the second frame's first token
    int frame_units;    // joint form: tokens per frame (0 otherwise)
    int rep_half;       // joint form: which of the two frames holds the representatives
    __device__ GroupView(const GroupMap& m, long long g) {
        base1 = 0; frame_units = 0; rep_half = 0;
        if (JOINT) {                                    // one or two whole frames, in time order
            const int2 fr = m.frames[g];
            const int f0 = (fr.y >= 0 && fr.y < fr.x) ? fr.y : fr.x, f1 = (fr.y >= 0 && fr.y < fr.x) ? fr.x : fr.y;
            frame_units = m.H * m.W;
            base = (long long)f0 * frame_units; base1 = (long long)f1 * frame_units;
            rep_half = fr.x == f0 ? 0 : 1;
            unit_stride = 1; row_pitch = m.W; w_local = m.W;
        } else if (m.kind != OC_KIND_FRAME) {                  // TOKEN: bt = frame; BLOCK: bt = batch element
            const int px = (int)(g % m.gx), py = (int)((g / m.gx) % m.gy);
            const long long bt = g / ((long long)m.gx * m.gy);
            base = (bt * m.H + (long long)py * m.Hp) * m.W + (long long)px * m.Wp;
            row_pitch = m.W;
            w_local = m.Wp;
            unit_stride = 1;
        } else {
            const long long np = (long long)m.gy * m.gx, b = g / np;
            base = b * m.units_per_group * np + (g - b * np);
            unit_stride = (int)np;
            row_pitch = 0;
            w_local = 0;
        }
        contig = m.kind == OC_KIND_FRAME || m.Wp == m.W;
        w_shift = (w_local > 0 && (w_local & (w_local - 1)) == 0) ? 31 - __clz(w_local) : -1;
        lat_pow2 = (m.sy & (m.sy - 1)) == 0 && (m.sx & (m.sx - 1)) == 0;
    }
    __device__ __forceinline__ void split(int u, int& ly, int& lx) const {
        if (w_shift >= 0) { ly = u >> w_shift; lx = u & (w_local - 1); }
        else { ly = u / w_local; lx = u - ly * w_local; }
    }
    __device__ __forceinline__ long long index(const GroupMap& m, int u) const {
        if (JOINT && u >= frame_units) return base1 + (u - frame_units);
        if (contig) return base + (long long)u * unit_stride;
        int ly, lx; split(u, ly, lx);
        return base + (long long)ly * row_pitch + lx;
    }
    __device__ __forceinline__ bool is_cand(const GroupMap& m, int u) const {
        if (JOINT) {                                    // every token of the partner frame is a candidate
            const int half = u >= frame_units ? 1 : 0;
            if (half != rep_half) return true;
            u -= half * frame_units;
        }
        if (m.kind == OC_KIND_FRAME) return (u & 1) != 0;
        if (m.self_match) return true;
        int ly, lx; split(u, ly, lx);
        if (lat_pow2) return !(((ly & (m.sy - 1)) == m.oy) && ((lx & (m.sx - 1)) == m.ox));
        return !((ly % m.sy) == m.oy && (lx % m.sx) == m.ox);
    }
};

// exclusive prefix of a per-thread 0/1 flag over the CTA (thread order) and the CTA total; `sums`
// is one of two alternating 33-int buffers, so consecutive calls need no trailing barrier.
__device__ __forceinline__ int block_scan(bool flag, int* sums, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned b = __ballot_sync(0xFFFFFFFFu, flag);
    const int within = __popc(b & ((1u << lane) - 1u));
    if (lane == 0) sums[warp] = __popc(b);
    __syncthreads();
    if (warp == 0) {
        const int v = sums[lane];
        int incl = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int n = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= d) incl += n;
        }
        sums[lane] = incl - v;
        if (lane == 31) sums[32] = incl;
    }
    __syncthreads();
    total = sums[32];
    return sums[warp] + within;
}

__global__ void __launch_bounds__(SEL_THREADS)
select_general_kernel(GroupMap gm, const float* __restrict__ best_sim, const int32_t* __restrict__ best_idx,
              int mode, float thr, int n_reuse, int y_stride, int keys_in_smem,
              int32_t* __restrict__ kept_idx, int32_t* __restrict__ kept_count,
              int32_t* __restrict__ match_map, int32_t* __restrict__ slot_of) {
    pdl_enter();
    extern __shared__ unsigned key_cache[];                    // [U] when keys_in_smem
    __shared__ unsigned reuse_bits[SEL_MAX_UNITS / 32];
    __shared__ int scan_sums[2][33];
    __shared__ unsigned hist[256];
    __shared__ unsigned sh_prefix, sh_remaining;
    __shared__ int sh_ncand;

    const int U = gm.units_per_group;
    const long long g = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_rounds = (U + SEL_THREADS - 1) / SEL_THREADS;
    const GroupView<> gv(gm, g);
    int scan_flip = 0;

    // ---- COUNT mode: value at the cut ----------------------------------------------------------
    unsigned cut_key = 0xFFFFFFFFu;  // candidates with key > cut_key are reused
    int need_eq = 0;                 // ... plus the first need_eq candidates with key == cut_key
    bool all_reused = false;
    if (mode == OC_SELECT_COUNT) {
        // stage keys (0 marks a non-candidate: every real key is > 0) and count the candidates
        if (tid == 0) sh_ncand = 0;
        __syncthreads();
        int local = 0;
        for (int u = tid; u < U; u += SEL_THREADS) {
            unsigned key = 0;
            if (gm_is_cand(gm, u)) { key = f32_to_ordered(best_sim[gv.index(gm, u)]); key = key ? key : 1u; ++local; }
            if (keys_in_smem) key_cache[u] = key;
        }
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) local += __shfl_xor_sync(0xFFFFFFFFu, local, d);
        if (lane == 0 && local) atomicAdd(&sh_ncand, local);
        __syncthreads();
        const int n_cand = sh_ncand;
        const int k = n_reuse < n_cand ? n_reuse : n_cand;
        if (k >= n_cand) {
            all_reused = true;
        } else if (k > 0) {
            if (tid == 0) { sh_prefix = 0; sh_remaining = (unsigned)k; }
            for (int pass = 0; pass < 4; ++pass) {
                const int shift = 24 - 8 * pass;
                if (tid < 256) hist[tid] = 0;
                __syncthreads();
                const unsigned prefix = sh_prefix;
                const unsigned himask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
                for (int r = 0; r < n_rounds; ++r) {
                    const int u = r * SEL_THREADS + tid;
                    unsigned key = 0;
                    if (u < U) {
                        if (keys_in_smem) key = key_cache[u];
                        else if (gm_is_cand(gm, u)) { key = f32_to_ordered(best_sim[gv.index(gm, u)]); key = key ? key : 1u; }
                    }
                    const bool take = key != 0 && (key & himask) == prefix;
                    // warp-aggregated update: one shared-memory atomic per distinct digit in the warp
                    const unsigned digit = take ? ((key >> shift) & 255u) : 256u;
                    const unsigned peers = __match_any_sync(0xFFFFFFFFu, digit);
                    if (take && lane == __ffs(peers) - 1) atomicAdd(&hist[digit], (unsigned)__popc(peers));
                }
                __syncthreads();
                if (warp == 0) {
                    // lane l owns bins 255-8l .. 248-8l (descending); find where the running count reaches rem
                    const unsigned rem = sh_remaining;
                    unsigned c[8], tot = 0;
#pragma unroll
                    for (int i = 0; i < 8; ++i) { c[i] = hist[255 - 8 * lane - i]; tot += c[i]; }
                    unsigned incl = tot;
#pragma unroll
                    for (int d = 1; d < 32; d <<= 1) {
                        const unsigned n = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                        if (lane >= d) incl += n;
                    }
                    const unsigned before = incl - tot;           // count in higher bins owned by lower lanes
                    const bool here = before < rem && rem <= incl;
                    if (here) {
                        unsigned acc = before;
                        int bin = 255 - 8 * lane;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            if (acc + c[i] >= rem) { bin = 255 - 8 * lane - i; break; }
                            acc += c[i];
                        }
                        sh_prefix = prefix | ((unsigned)bin << shift);
                        sh_remaining = rem - acc;                 // still to take inside that bin (>= 1)
                    }
                }
                __syncthreads();
            }
            cut_key = sh_prefix;
            need_eq = (int)sh_remaining;
        }
    }

    // ---- reuse flags, ascending unit order -----------------------------------------------------
    int eq_seen = 0;
    for (int r = 0; r < n_rounds; ++r) {
        const int u = r * SEL_THREADS + tid;
        bool reuse = false, eq = false;
        if (u < U && gm_is_cand(gm, u)) {
            if (mode == OC_SELECT_THRESHOLD) {
                const long long i = gv.index(gm, u);
                reuse = best_sim[i] >= thr;
                if (gm.self_match) reuse = reuse && (best_idx[i] < (int)i);
            } else if (all_reused) {
                reuse = true;
            } else {
                unsigned key;
                if (keys_in_smem) key = key_cache[u];
                else { key = f32_to_ordered(best_sim[gv.index(gm, u)]); key = key ? key : 1u; }
                reuse = key > cut_key;
                eq = key == cut_key;
            }
        }
        if (need_eq > 0) {                                         // uniform over the CTA
            int tot;
            const int rank = block_scan(eq, scan_sums[scan_flip], tot);
            scan_flip ^= 1;
            if (eq && eq_seen + rank < need_eq) reuse = true;
            eq_seen += tot;
        }
        const unsigned bits = __ballot_sync(0xFFFFFFFFu, reuse);
        if (lane == 0 && u < U) reuse_bits[u >> 5] = bits;
    }
    __syncthreads();

    // ---- compaction + maps ---------------------------------------------------------------------
    int kept_base = 0;
    for (int r = 0; r < n_rounds; ++r) {
        const int u = r * SEL_THREADS + tid;
        const bool valid = u < U;
        const bool reuse = valid && ((reuse_bits[u >> 5] >> (u & 31)) & 1u);
        const bool kept = valid && !reuse;
        int tot;
        const int rank = block_scan(kept, scan_sums[scan_flip], tot);
        scan_flip ^= 1;
        if (valid) {
            const long long i = gv.index(gm, u);
            if (kept) {
                const int pos = kept_base + rank;
                if (pos < y_stride) kept_idx[g * y_stride + pos] = (int32_t)i;
                slot_of[i] = (int32_t)(g * y_stride + pos);
                match_map[i] = (int32_t)i;
            } else {
                slot_of[i] = -1;
                int m = best_idx[i];
                if (gm.self_match) {
                    // follow the chain to a kept token; indices strictly decrease, so it ends
                    const int g0 = (int)(g * U);
                    for (int hop = 0; hop < U; ++hop) {
                        const int lu = m - g0;
                        if (lu < 0 || lu >= U || !((reuse_bits[lu >> 5] >> (lu & 31)) & 1u)) break;
                        m = best_idx[m];
                    }
                }
                match_map[i] = m;
            }
        }
        kept_base += tot;
    }
    for (int p = kept_base + tid; p < y_stride; p += SEL_THREADS) kept_idx[g * y_stride + p] = -1;
    if (tid == 0) kept_count[g] = kept_base;
}

// inclusive-to-exclusive block scan of one int per thread; returns this thread's exclusive prefix
__device__ __forceinline__ int block_scan_int(int v, int* sums /*[33]*/, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int n = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += n;
    }
    if (lane == 31) sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const int w = lane < (int)(blockDim.x >> 5) ? sums[lane] : 0;     // (CTAs of fewer than 32 warps)
        int wi = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int n = __shfl_up_sync(0xFFFFFFFFu, wi, d);
            if (lane >= d) wi += n;
        }
        sums[lane] = wi - w;
        if (lane == 31) sums[32] = wi;
    }
    __syncthreads();
    total = sums[32];
    return sums[warp] + incl - v;
}

template <bool JOINT>
__global__ void __launch_bounds__(1024)
select_fast_kernel(GroupMap gm, const float* __restrict__ best_sim, const int32_t* __restrict__ best_idx,
                   int mode, float thr, int n_reuse, int y_stride,
                   int32_t* __restrict__ kept_idx, int32_t* __restrict__ kept_count,
                   int32_t* __restrict__ match_map, int32_t* __restrict__ slot_of) {
    pdl_enter();
    extern __shared__ unsigned key_cache[];                    // [U] keys, later reused as kept positions
    __shared__ int scan_sums[2][33];
    __shared__ unsigned hist[4096];
    __shared__ unsigned sh_prefix, sh_remaining;
    __shared__ int sh_ncand;
    __shared__ unsigned sh_kmin, sh_kmax;

    const int NT = (int)blockDim.x;                             // 128..1024 threads, chosen by the host for the group size
    int U = gm.units_per_group;
    const long long g = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31;
    if (JOINT) {                                                // joint form: the slot decides the group's size and budget
        const int2 fr = gm.frames[g];
        if (fr.x < 0) {                                         // absorbed into its partner's group: keeps nothing
            for (int p = tid; p < y_stride; p += NT) kept_idx[g * y_stride + p] = -1;
            if (tid == 0) kept_count[g] = 0;
            return;
        }
        if (fr.y < 0) { U = gm.H * gm.W; n_reuse = gm.n_reuse_single; }
    }
    const int n_rounds = (U + NT - 1) / NT;
    const GroupView<JOINT> gv(gm, g);

    // ---- phase 0: every input is read once, coalesced, all loads issued before any is used --------
    // key 0 marks a non-candidate (every real key is >= 1)
    constexpr int PF = 8;                                       // rounds whose loads are kept in registers
    if (tid == 0) { sh_ncand = 0; sh_kmin = 0xFFFFFFFFu; sh_kmax = 0u; }
    __syncthreads();
    int local = 0;
    unsigned kmin = 0xFFFFFFFFu, kmax = 0u;
    int idx_pf[PF];                                             // best_idx of this thread's units (phase 3)
    for (int r0 = 0; r0 < n_rounds; r0 += PF) {
        float sim_pf[PF];
        long long gi[PF];
#pragma unroll
        for (int k = 0; k < PF; ++k) {
            if (r0 + k >= n_rounds) break;                          // (uniform: whole rounds that do not exist)
            const int u = (r0 + k) * NT + tid;
            gi[k] = u < U ? gv.index(gm, u) : -1;
        }
#pragma unroll
        for (int k = 0; k < PF; ++k) {
            if (r0 + k >= n_rounds) break;
            sim_pf[k] = gi[k] >= 0 ? best_sim[gi[k]] : 0.f;
            if (r0 == 0) idx_pf[k] = gi[k] >= 0 ? best_idx[gi[k]] : 0;
        }
#pragma unroll
        for (int k = 0; k < PF; ++k) {
            if (r0 + k >= n_rounds) break;
            const int u = (r0 + k) * NT + tid;
            if (u < U) {
                unsigned key = 0;
                if (gv.is_cand(gm, u)) {
                    key = f32_to_ordered(sim_pf[k]); key = key ? key : 1u; ++local;
                    kmin = min(kmin, key); kmax = max(kmax, key);
                }
                key_cache[u] = key;
            }
        }
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        local += __shfl_xor_sync(0xFFFFFFFFu, local, d);
        kmin = min(kmin, __shfl_xor_sync(0xFFFFFFFFu, kmin, d));
        kmax = max(kmax, __shfl_xor_sync(0xFFFFFFFFu, kmax, d));
    }
    if (lane == 0 && local) { atomicAdd(&sh_ncand, local); atomicMin(&sh_kmin, kmin); atomicMax(&sh_kmax, kmax); }
    __syncthreads();

    // ---- the cut: candidates with key > cut_key are reused, plus the first need_eq with key == cut_key
    unsigned cut_key = 0xFFFFFFFFu;
    int need_eq = 0;
    bool all_reused = false;
    if (mode == OC_SELECT_THRESHOLD) {
        // sim >= thr  <=>  key >= ordered(thr)  (-0.0 and +0.0 share one key); as "key > cut": cut = ordered(thr) - 1
        unsigned tk = f32_to_ordered(thr); tk = tk ? tk : 1u;
        cut_key = tk - 1u;
    } else {
        const int n_cand = sh_ncand;
        const int k = n_reuse < n_cand ? n_reuse : n_cand;
        if (k >= n_cand) {
            all_reused = true;
        } else if (k > 0) {
            // Radix select of the k-th largest key, 12 bits at a time, on keys taken relative to the
            // smallest candidate key: similarities of one group span a narrow range, so two passes
            // cover it where 8-bit digits of the raw key needed four (three cover any 32-bit span).
            if (tid == 0) { sh_prefix = 0; sh_remaining = (unsigned)k; }
            const unsigned base = sh_kmin;
            const unsigned span = sh_kmax - base;
            const int nbits = 32 - __clz(span);                    // 0 when all candidate keys are equal
            const int n_pass = (nbits + 11) / 12;
            for (int pass = 0; pass < n_pass; ++pass) {
                const int shift = 12 * (n_pass - 1 - pass);
                for (int i = tid; i < 4096; i += NT) hist[i] = 0;
                __syncthreads();
                const unsigned prefix = sh_prefix;                  // the digits fixed so far (high part of rel)
                for (int r = 0; r < n_rounds; ++r) {
                    const int u = r * NT + tid;
                    const unsigned key = u < U ? key_cache[u] : 0u;
                    if (key != 0) {
                        const unsigned rel = key - base;
                        // (a shift by 32 would be undefined: the first pass has no fixed digits)
                        if (pass == 0 || (rel >> (shift + 12)) == prefix) atomicAdd(&hist[(rel >> shift) & 4095u], 1u);
                    }
                }
                __syncthreads();
                // thread t owns bins 4095 - bpt*t downwards (bpt = 4096 / threads): where does the running
                // count reach rem?
                const unsigned rem = sh_remaining;
                const int bpt = 4096 / NT, top = 4095 - bpt * tid;
                unsigned tot = 0;
                for (int i = 0; i < bpt; ++i) tot += hist[top - i];
                int all;
                const unsigned before = (unsigned)block_scan_int((int)tot, scan_sums[pass & 1], all);
                if (before < rem && rem <= before + tot) {
                    unsigned acc = before;
                    int bin = top;
                    for (int i = 0; i < bpt; ++i) {
                        const unsigned ci = hist[top - i];
                        if (acc + ci >= rem) { bin = top - i; break; }
                        acc += ci;
                    }
                    sh_prefix = (prefix << 12) | (unsigned)bin;
                    sh_remaining = rem - acc;
                }
                __syncthreads();
            }
            // (with no pass at all every candidate has the key `base`: the cut is that key, k of them reused)
            cut_key = base + sh_prefix;
            need_eq = (int)sh_remaining;
        }
    }

    // ---- phase 2: each thread owns a contiguous run of units -------------------------------------
    const int run = n_rounds;                                   // units per thread
    const int u0 = tid * run, u1 = min(U, u0 + run);
    int eq_base = 0;
    if (need_eq > 0) {
        int n_eq = 0;
        for (int u = u0; u < u1; ++u) n_eq += key_cache[u] == cut_key ? 1 : 0;
        int tot;
        eq_base = block_scan_int(n_eq, scan_sums[0], tot);
    }
    unsigned long long reuse_mask = 0;                          // run <= 40 units
    int n_kept = 0;
    for (int u = u0; u < u1; ++u) {
        const unsigned key = key_cache[u];
        bool reuse = false;
        if (key != 0) {
            if (all_reused) reuse = true;
            else if (key > cut_key) reuse = true;
            else if (need_eq > 0 && key == cut_key) { reuse = eq_base < need_eq; ++eq_base; }
        }
        if (reuse) reuse_mask |= 1ull << (u - u0); else ++n_kept;
    }
    int kept_total;
    int pos = block_scan_int(n_kept, scan_sums[1], kept_total);
    __syncthreads();                                            // all reads of the keys are done
    for (int u = u0; u < u1; ++u)
        key_cache[u] = ((reuse_mask >> (u - u0)) & 1ull) ? 0xFFFFFFFFu : (unsigned)pos++;
    __syncthreads();

    // ---- phase 3: one coalesced pass writes every output ------------------------------------------
    auto emit = [&](int u, int m_pf, bool have_pf) {
        const long long i = gv.index(gm, u);
        const unsigned p = key_cache[u];
        if (p != 0xFFFFFFFFu) {
            if ((int)p < y_stride) kept_idx[g * y_stride + p] = (int32_t)i;
            slot_of[i] = (int32_t)(g * y_stride + p);
            match_map[i] = (int32_t)i;
        } else {
            slot_of[i] = -1;
            match_map[i] = have_pf ? m_pf : best_idx[i];            // registers of the first PF rounds, else reload
        }
    };
#pragma unroll
    for (int r = 0; r < PF; ++r) {
        const int u = r * NT + tid;
        if (r < n_rounds && u < U) emit(u, idx_pf[r], true);
    }
    for (int r = PF; r < n_rounds; ++r) {
        const int u = r * NT + tid;
        if (u < U) emit(u, 0, false);
    }
    for (int p = kept_total + tid; p < y_stride; p += NT) kept_idx[g * y_stride + p] = -1;
    if (tid == 0) kept_count[g] = kept_total;
}

// ------------------------------------------------------------------------------------------------
// Small groups (at most 64 units: the frames of a clip, the positions of a small patch): one WARP
// per group, two units per lane, everything in registers.  The count-mode rank of a candidate is
// counted directly -- how many candidates of the group precede it in (similarity descending, index
// ascending) order -- by passing every key round the warp; positions come from ballots.  No shared
// memory, no CTA barrier: the kernel costs a launch plus a few hundred cycles.
// ------------------------------------------------------------------------------------------------
static constexpr int SEL_SMALL_UNITS = 64;
static constexpr int SEL_SMALL_THREADS = 128;

__global__ void __launch_bounds__(SEL_SMALL_THREADS)
select_small_kernel(GroupMap gm, long long n_groups, const float* __restrict__ best_sim,
                    const int32_t* __restrict__ best_idx, int mode, float thr, int n_reuse, int y_stride,
                    int32_t* __restrict__ kept_idx, int32_t* __restrict__ kept_count,
                    int32_t* __restrict__ match_map, int32_t* __restrict__ slot_of) {
    pdl_enter();
    const long long g = (long long)blockIdx.x * (SEL_SMALL_THREADS / 32) + (threadIdx.x >> 5);
    if (g >= n_groups) return;                                 // whole warps leave together
    const int lane = threadIdx.x & 31;
    const int U = gm.units_per_group;
    const GroupView<> gv(gm, g);
    long long gi[2];
    unsigned key[2];
    int m_idx[2];
    bool valid[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int u = lane + 32 * h;
        valid[h] = u < U;
        gi[h] = valid[h] ? gv.index(gm, u) : 0;
        key[h] = 0; m_idx[h] = 0;
        if (valid[h] && gv.is_cand(gm, u)) {
            key[h] = f32_to_ordered(best_sim[gi[h]]); key[h] = key[h] ? key[h] : 1u;   // 0 marks a non-candidate
            m_idx[h] = best_idx[gi[h]];
        }
    }
    bool reuse[2] = {false, false};
    if (mode == OC_SELECT_THRESHOLD) {
        unsigned tk = f32_to_ordered(thr); tk = tk ? tk : 1u;      // sim >= thr  <=>  key >= ordered(thr)
#pragma unroll
        for (int h = 0; h < 2; ++h) reuse[h] = key[h] != 0 && key[h] >= tk;
    } else {
        const int n_cand = __popc(__ballot_sync(0xFFFFFFFFu, key[0] != 0)) + __popc(__ballot_sync(0xFFFFFFFFu, key[1] != 0));
        const int k = n_reuse < n_cand ? n_reuse : n_cand;
        int rank[2] = {0, 0};
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2) {
            if (32 * h2 >= U) break;                            // (uniform)
            for (int l = 0; l < 32; ++l) {
                const unsigned ko = __shfl_sync(0xFFFFFFFFu, key[h2], l);
                const int uo = l + 32 * h2;
#pragma unroll
                for (int h = 0; h < 2; ++h)
                    rank[h] += (ko != 0 && (ko > key[h] || (ko == key[h] && uo < lane + 32 * h))) ? 1 : 0;
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) reuse[h] = key[h] != 0 && rank[h] < k;
    }
    const unsigned lt = (1u << lane) - 1u;
    const unsigned k0 = __ballot_sync(0xFFFFFFFFu, valid[0] && !reuse[0]);
    const unsigned k1 = __ballot_sync(0xFFFFFFFFu, valid[1] && !reuse[1]);
    const int pos[2] = {__popc(k0 & lt), __popc(k0) + __popc(k1 & lt)};
    const int kept_total = __popc(k0) + __popc(k1);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        if (!valid[h]) continue;
        if (!reuse[h]) {
            if (pos[h] < y_stride) kept_idx[g * y_stride + pos[h]] = (int32_t)gi[h];
            slot_of[gi[h]] = (int32_t)(g * y_stride + pos[h]);
            match_map[gi[h]] = (int32_t)gi[h];
        } else {
            slot_of[gi[h]] = -1;
            match_map[gi[h]] = m_idx[h];
        }
    }
    for (int p = kept_total + lane; p < y_stride; p += 32) kept_idx[g * y_stride + p] = -1;
    if (lane == 0) kept_count[g] = kept_total;
}

oc_status launch_select(oc_ctx* ctx, const Geo& geo, const float* best_sim, const int32_t* best_idx,
                        int mode, float thr, int64_t n_reuse, int64_t y_stride, int32_t* kept_idx,
                        int32_t* kept_count, int32_t* match_map, int32_t* slot_of, cudaStream_t s) {
    if (geo.units_per_group > SEL_MAX_UNITS) return OC_ERR_UNSUPPORTED;
    if (geo.n_groups == 0) return OC_OK;
    GroupMap gm = make_group_map(geo);
    int nr = (int)(n_reuse > 0x7FFFFFFF ? 0x7FFFFFFF : n_reuse);
    static PerDeviceOnce attr_once;                 // (the context's device is current here)
    if (!attr_once.ensure(ctx->device, [] {
            const bool ok = cudaFuncSetAttribute(select_general_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 SEL_SMEM_KEYS * (int)sizeof(unsigned)) == cudaSuccess &&
                            cudaFuncSetAttribute(select_fast_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 SEL_SMEM_KEYS * (int)sizeof(unsigned)) == cudaSuccess;
            if (!ok) cudaGetLastError();
            return ok;
        }))
        return OC_ERR_CUDA;
    LaunchScope scope(ctx, OC_K_SELECT, s);
    if (!geo.self_match && geo.units_per_group <= SEL_SMALL_UNITS) {
        const int wpc = SEL_SMALL_THREADS / 32;
        OC_LAUNCH(select_small_kernel, (unsigned)((geo.n_groups + wpc - 1) / wpc), SEL_SMALL_THREADS, 0, s,
                  gm, (long long)geo.n_groups, best_sim, best_idx, mode, thr, nr, (int)y_stride, kept_idx, kept_count,
                  match_map, slot_of);
    } else if (!geo.self_match && geo.units_per_group <= SEL_SMEM_KEYS) {
        // A group wants every thread it can get (the kernel is latency-bound per thread); only when the
        // groups do not all fit on the device at once, and are small, do smaller CTAs pay (more groups in
        // flight).  A thread's run of units must fit its 64-bit reuse mask.
        int nt = SEL_THREADS, min_nt = 512;          // (measured: below 512 threads a group only gets slower)
        while (min_nt < SEL_THREADS && min_nt * 4 < geo.units_per_group) min_nt <<= 1;      // at most ~4 units per thread
        while (nt > min_nt && (long long)geo.n_groups * nt > 2048ll * ctx->sm_count) nt >>= 1;
        while (nt < SEL_THREADS && (geo.units_per_group + nt - 1) / nt > 40) nt <<= 1;
        OC_LAUNCH(select_fast_kernel<false>, (unsigned)geo.n_groups, nt, (size_t)geo.units_per_group * sizeof(unsigned), s,
                  gm, best_sim, best_idx, mode, thr, nr, (int)y_stride, kept_idx, kept_count, match_map, slot_of);
    } else {
        const int keys_in_smem = (mode == OC_SELECT_COUNT && geo.units_per_group <= SEL_SMEM_KEYS) ? 1 : 0;
        const size_t dyn = keys_in_smem ? (size_t)geo.units_per_group * sizeof(unsigned) : 0;
        OC_LAUNCH(select_general_kernel, (unsigned)geo.n_groups, SEL_THREADS, dyn, s, gm, best_sim, best_idx, mode, thr, nr,
                  (int)y_stride, keys_in_smem, kept_idx, kept_count, match_map, slot_of);
    }
    return last_launch_status();
}

// Joint form: one CTA per frame slot; pairs are groups of 2*H*W tokens, single frames of H*W.
oc_status launch_select_joint(oc_ctx* ctx, const Geo& geo, const int2* frames, const float* best_sim,
                              const int32_t* best_idx, int mode, float thr, int64_t n_reuse_pair,
                              int64_t n_reuse_single, int64_t y_stride, int32_t* kept_idx, int32_t* kept_count,
                              int32_t* match_map, int32_t* slot_of, cudaStream_t s) {
    const long long P = (long long)geo.H * geo.W, slots = (long long)geo.B * geo.T;
    if (geo.kind != OC_KIND_TOKEN || geo.self_match || geo.gy != 1 || geo.gx != 1) return OC_ERR_UNSUPPORTED;
    if (2 * P > SEL_SMEM_KEYS) return OC_ERR_UNSUPPORTED;
    if (slots == 0) return OC_OK;
    GroupMap gm = make_group_map(geo);
    gm.frames = frames;
    gm.units_per_group = (int)(2 * P);
    gm.n_reuse_single = (int)(n_reuse_single > 0x7FFFFFFF ? 0x7FFFFFFF : n_reuse_single);
    const int nr = (int)(n_reuse_pair > 0x7FFFFFFF ? 0x7FFFFFFF : n_reuse_pair);
    static PerDeviceOnce attr_once;
    if (!attr_once.ensure(ctx->device, [] {
            const bool ok = cudaFuncSetAttribute(select_fast_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 SEL_SMEM_KEYS * (int)sizeof(unsigned)) == cudaSuccess;
            if (!ok) cudaGetLastError();
            return ok;
        }))
        return OC_ERR_CUDA;
    LaunchScope scope(ctx, OC_K_SELECT, s);
    OC_LAUNCH(select_fast_kernel<true>, (unsigned)slots, SEL_THREADS, (size_t)(2 * P) * sizeof(unsigned), s,
              gm, best_sim, best_idx, mode, thr, nr, (int)y_stride, kept_idx, kept_count, match_map, slot_of);
    return last_launch_status();
}

}  // namespace oc
