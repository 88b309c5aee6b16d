// select: threshold / keep-count selection, order-preserving compaction, match map.
//
// One CTA per group (a group is an independent selection problem).  Everything is decided in
// ascending unit order, so the result is deterministic and comparable bit for bit:
//   COUNT mode  - 4 x 8-bit radix select over order-preserving keys of the candidates' best_sim
//                 finds the value at the cut; candidates above it are reused, candidates equal to it
//                 are admitted lowest index first;
//   both modes  - reuse flags live in a shared-memory bitmask; kept units are compacted with a
//                 warp-ballot prefix sum (stable, ascending original index).
#include "common.cuh"

namespace oc {

static constexpr int SEL_THREADS = 1024;
static constexpr int SEL_MAX_UNITS = 65536;

struct BlockScan {
    // exclusive prefix of a per-thread 0/1 flag over the CTA (thread order), plus the CTA total.
    __device__ static int run(bool flag, int* warp_sums /*[33]*/, int& total) {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        unsigned b = __ballot_sync(0xFFFFFFFFu, flag);
        int within = __popc(b & ((1u << lane) - 1u));
        if (lane == 0) warp_sums[warp] = __popc(b);
        __syncthreads();
        if (warp == 0) {
            int v = warp_sums[lane];
            int incl = v;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                int n = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                if (lane >= d) incl += n;
            }
            warp_sums[lane] = incl - v;
            if (lane == 31) warp_sums[32] = incl;
        }
        __syncthreads();
        int res = warp_sums[warp] + within;
        total = warp_sums[32];
        __syncthreads();          // warp_sums is reused by the next call
        return res;
    }
};

__global__ void __launch_bounds__(SEL_THREADS)
select_kernel(GroupMap gm, const float* __restrict__ best_sim, const int32_t* __restrict__ best_idx,
              int mode, float thr, int n_reuse, int y_stride, int32_t* __restrict__ kept_idx,
              int32_t* __restrict__ kept_count, int32_t* __restrict__ match_map,
              int32_t* __restrict__ slot_of) {
    __shared__ unsigned reuse_bits[SEL_MAX_UNITS / 32];
    __shared__ int warp_sums[33];
    __shared__ unsigned hist[256];
    __shared__ unsigned sh_prefix, sh_remaining;

    const int U = gm.units_per_group;
    const long long g = blockIdx.x;
    const int tid = threadIdx.x;
    const int n_rounds = (U + SEL_THREADS - 1) / SEL_THREADS;

    // ---- COUNT mode: value at the cut ----------------------------------------------------------
    unsigned cut_key = 0;       // candidates with key > cut_key are reused
    int need_eq = 0;            // ... plus the first need_eq candidates with key == cut_key
    bool all_reused = false;
    if (mode == OC_SELECT_COUNT) {
        // number of candidates in the group
        int local = 0;
        for (int u = tid; u < U; u += SEL_THREADS) local += gm_is_cand(gm, u) ? 1 : 0;
        // CTA sum through the scan helper (flag-wise), done on counts via shared atomics instead
        if (tid == 0) sh_remaining = 0;
        __syncthreads();
        if (local) atomicAdd(&sh_remaining, (unsigned)local);
        __syncthreads();
        const int n_cand = (int)sh_remaining;
        __syncthreads();
        const int k = n_reuse < n_cand ? n_reuse : n_cand;
        if (k >= n_cand) {
            all_reused = true;
        } else if (k > 0) {
            if (tid == 0) { sh_prefix = 0; sh_remaining = (unsigned)k; }
            __syncthreads();
            for (int pass = 0; pass < 4; ++pass) {
                const int shift = 24 - 8 * pass;
                if (tid < 256) hist[tid] = 0;
                __syncthreads();
                const unsigned prefix = sh_prefix;
                const unsigned himask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
                for (int u = tid; u < U; u += SEL_THREADS) {
                    if (!gm_is_cand(gm, u)) continue;
                    unsigned key = f32_to_ordered(best_sim[gm_unit_index(gm, g, u)]);
                    if ((key & himask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
                }
                __syncthreads();
                if (tid == 0) {
                    unsigned rem = sh_remaining;   // how many still to take among keys matching prefix
                    int d = 255;
                    for (; d > 0; --d) {
                        if (hist[d] >= rem) break;
                        rem -= hist[d];
                    }
                    sh_prefix = prefix | ((unsigned)d << shift);
                    sh_remaining = rem;            // taken from bin d (1 <= rem <= hist[d])
                }
                __syncthreads();
            }
            cut_key = sh_prefix;
            need_eq = (int)sh_remaining;
        }
        // k == 0: nothing reused (cut_key = 0xFFFFFFFF semantics handled below)
        if (k == 0) { cut_key = 0xFFFFFFFFu; need_eq = 0; }
    }

    // ---- reuse flags, ascending unit order -----------------------------------------------------
    int eq_seen = 0;
    for (int r = 0; r < n_rounds; ++r) {
        const int u = r * SEL_THREADS + tid;
        bool cand = false, reuse = false, eq = false;
        if (u < U) {
            cand = gm_is_cand(gm, u);
            if (cand) {
                const long long i = gm_unit_index(gm, g, u);
                const float s = best_sim[i];
                if (mode == OC_SELECT_THRESHOLD) {
                    reuse = s >= thr;
                    if (gm.self_match) reuse = reuse && (best_idx[i] < (int)i);
                } else if (all_reused) {
                    reuse = true;
                } else {
                    unsigned key = f32_to_ordered(s);
                    reuse = key > cut_key;
                    eq = key == cut_key;
                }
            }
        }
        if (mode == OC_SELECT_COUNT && !all_reused && need_eq > 0) {
            int tot;
            int rank = BlockScan::run(eq, warp_sums, tot);
            if (eq && eq_seen + rank < need_eq) reuse = true;
            eq_seen += tot;
        }
        unsigned bits = __ballot_sync(0xFFFFFFFFu, reuse);
        if ((tid & 31) == 0 && (u < U)) reuse_bits[u >> 5] = bits;
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
        int rank = BlockScan::run(kept, warp_sums, tot);
        if (valid) {
            const long long i = gm_unit_index(gm, g, u);
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

oc_status launch_select(oc_ctx* ctx, const Geo& geo, const float* best_sim, const int32_t* best_idx,
                        int mode, float thr, int64_t n_reuse, int64_t y_stride, int32_t* kept_idx,
                        int32_t* kept_count, int32_t* match_map, int32_t* slot_of, cudaStream_t s) {
    if (geo.units_per_group > SEL_MAX_UNITS) return OC_ERR_UNSUPPORTED;
    if (geo.n_groups == 0) return OC_OK;
    GroupMap gm = make_group_map(geo);
    int nr = (int)(n_reuse > 0x7FFFFFFF ? 0x7FFFFFFF : n_reuse);
    LaunchScope scope(ctx, OC_K_SELECT, s);
    select_kernel<<<(unsigned)geo.n_groups, SEL_THREADS, 0, s>>>(gm, best_sim, best_idx, mode, thr, nr,
                                                                  (int)y_stride, kept_idx, kept_count,
                                                                  match_map, slot_of);
    return last_launch_status();
}

}  // namespace oc
