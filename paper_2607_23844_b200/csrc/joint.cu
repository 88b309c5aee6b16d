// Token Cache on the frame pairs of Frame Cache (Section 3.2.3).  Token Cache reuses the feature map
// and the frame pairing of Frame Cache: a matched pair is treated as one token group of 2*H*W tokens
// (the paper's (B*r_f, 2HW, C) arrangement) with one representative per 2x2x2 cube, and a frame that
// found no partner is matched inside its own 2x2 neighbourhoods as usual.
//
// Nothing is reshaped here: a pair is two frame indices, and the matcher, the selection and the row
// movers address the two frames in place.
//   joint_groups_kernel   Frame Cache's result -> one slot per frame: {representative frame, partner}
//   joint_units_kernel    slots -> the tensor-core matcher's work list {rep frame, cand frame, member}
//   finalize_joint_kernel packed arg-max keys -> best_sim / best_idx (every token of an absorbed frame
//                         is a candidate)
// The matching itself is match_tc.cu's kernel walking the work list; the selection is select.cu's
// kernel with two-frame groups.
#include "common.cuh"

namespace oc {

// A reused candidate frame t claims its matched representative frame u; when both neighbours of u
// claim it, the more similar one wins (equal: the earlier frame) and the other stays on its own.
// One thread per frame; frames of different batch elements never interact.
__global__ void __launch_bounds__(256)
joint_groups_kernel(int B, int T, const float* __restrict__ frame_best_sim, const int32_t* __restrict__ frame_best_idx,
                    const int32_t* __restrict__ frame_slot_of, int2* __restrict__ frames) {
    pdl_enter();
    const int f = blockIdx.x * 256 + threadIdx.x;
    if (f >= B * T) return;
    const int b = f / T, t = f - b * T;
    auto claims = [&](int ft, int fu) {           // does candidate frame ft (in range) claim representative fu?
        return frame_slot_of[ft] < 0 && frame_best_idx[ft] == fu;
    };
    if ((t & 1) == 0) {                           // a representative frame: which neighbour, if any, joins it
        int win = -1;
        if (t >= 1 && claims(f - 1, f)) win = f - 1;
        if (t + 1 < T && claims(f + 1, f) && (win < 0 || frame_best_sim[f + 1] > frame_best_sim[win])) win = f + 1;
        frames[f] = make_int2(f, win);
    } else {                                      // a candidate frame: absorbed iff it wins its claim
        bool absorbed = false;
        if (frame_slot_of[f] < 0) {
            const int fu = frame_best_idx[f];     // f - 1 or f + 1 (adjacent representatives only)
            const int other = 2 * fu - f;         // the representative's other neighbour
            const bool other_in = other >= b * T && other < (b + 1) * T;
            if (fu >= b * T && fu < (b + 1) * T && (fu == f - 1 || fu == f + 1)) {
                absorbed = true;
                if (other_in && claims(other, fu)) {
                    const float mine = frame_best_sim[f], theirs = frame_best_sim[other];
                    absorbed = mine > theirs || (mine == theirs && f < other);
                }
            }
        }
        frames[f] = absorbed ? make_int2(-1, -1) : make_int2(f, -1);
    }
}

// Work list of the matcher, in slot order: for a group with representative frame u, the sy*sx - 1
// non-representative sub-lattices of u itself, then (pairs) all sy*sx sub-lattices of the partner.
// One CTA; a block scan over the slots gives every slot its place.
__global__ void __launch_bounds__(1024)
joint_units_kernel(int n_slots, const int2* __restrict__ frames, int n_members, int rep_member,
                   int4* __restrict__ units, int* __restrict__ n_units) {
    pdl_enter();
    __shared__ int warp_sums[32];
    __shared__ int carry;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) carry = 0;
    __syncthreads();
    for (int s0 = 0; s0 < n_slots; s0 += 1024) {
        const int slot = s0 + tid;
        int2 fr = make_int2(-1, -1);
        if (slot < n_slots) fr = frames[slot];
        const int mine = fr.x < 0 ? 0 : (n_members - 1) + (fr.y >= 0 ? n_members : 0);
        int incl = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int n = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= d) incl += n;
        }
        if (lane == 31) warp_sums[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int v = warp_sums[lane];
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int n = __shfl_up_sync(0xFFFFFFFFu, v, d);
                if (lane >= d) v += n;
            }
            warp_sums[lane] = v;                  // inclusive over warps
        }
        __syncthreads();
        int at = carry + (warp ? warp_sums[warp - 1] : 0) + incl - mine;
        if (fr.x >= 0) {
            for (int m = 0; m < n_members; ++m)
                if (m != rep_member) units[at++] = make_int4(fr.x, fr.x, m, 0);
            if (fr.y >= 0)
                for (int m = 0; m < n_members; ++m) units[at++] = make_int4(fr.x, fr.y, m, 0);
        }
        __syncthreads();
        if (tid == 0) carry += warp_sums[31];
        __syncthreads();
    }
    if (tid == 0) *n_units = carry;
}

__global__ void __launch_bounds__(256)
finalize_joint_kernel(int H, int W, int sy, int sx, int oy, int ox, long long n_tok, const int2* __restrict__ frames,
                      const float* __restrict__ inv_norm, const unsigned long long* __restrict__ keys,
                      float* __restrict__ best_sim, int32_t* __restrict__ best_idx) {
    pdl_enter();
    const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
    if (i >= n_tok) return;
    const int P = H * W;
    const int f = (int)(i / P), p = (int)(i - (long long)f * P);
    const int y = p / W, x = p - y * W;
    const bool absorbed = frames[f].x < 0;
    const bool rep = !absorbed && (y % sy) == oy && (x % sx) == ox;
    const unsigned long long key = keys[i];
    if (rep || key == 0ull) {
        best_sim[i] = -INFINITY; best_idx[i] = (int32_t)i;
        return;
    }
    const float v = ordered_to_f32((uint32_t)(key >> 32));
    best_sim[i] = clamp_unit(v * inv_norm[i]);
    best_idx[i] = (int32_t)(0xFFFFFFFFu - (uint32_t)(key & 0xFFFFFFFFull));
}

// workspace: keys, inverse norms (as the token matcher), then the work list and its length
static size_t joint_units_offset(const Geo& g) {
    const size_t n = (size_t)g.n_units;
    return n * sizeof(unsigned long long) + ((n * sizeof(float) + 255) / 256) * 256 + 256;
}
static long long joint_max_units(const Geo& g) {
    const long long slots = (long long)g.B * g.T, m = (long long)g.sy * g.sx;
    return slots * (m - 1) + ((slots + 1) / 2) * m;
}
size_t joint_workspace_bytes(const Geo& g) {
    return joint_units_offset(g) + (size_t)joint_max_units(g) * sizeof(int4) + 256;
}

oc_status launch_joint_groups(oc_ctx* ctx, int B, int T, const float* frame_best_sim, const int32_t* frame_best_idx,
                              const int32_t* frame_slot_of, int2* frames, cudaStream_t s) {
    (void)ctx;
    OC_LAUNCH(joint_groups_kernel, (unsigned)((B * T + 255) / 256), 256, 0, s, B, T, frame_best_sim, frame_best_idx,
              frame_slot_of, frames);
    return last_launch_status();
}

void launch_norms(oc_ctx* ctx, const Geo& g, const void* x, float* inv_norm, unsigned long long* keys, cudaStream_t s);

oc_status launch_match_joint(oc_ctx* ctx, const Geo& g, const void* x, const int2* frames, float* best_sim,
                             int32_t* best_idx, cudaStream_t s) {
    const long long n_tok = g.n_units;
    if (n_tok == 0) return OC_OK;
    if (!tc_match_supported(g) || g.gy != 1 || g.gx != 1) return OC_ERR_UNSUPPORTED;
    unsigned long long* keys = (unsigned long long*)ctx->workspace;
    float* inv_norm = (float*)((uint8_t*)ctx->workspace + (size_t)n_tok * sizeof(unsigned long long));
    int4* units = (int4*)((uint8_t*)ctx->workspace + joint_units_offset(g));
    int* n_units = (int*)((uint8_t*)units + (size_t)joint_max_units(g) * sizeof(int4));
    OC_LAUNCH(joint_units_kernel, 1, 1024, 0, s, g.B * g.T, frames, g.sy * g.sx, g.oy * g.sx + g.ox, units, n_units);
    if (last_launch_status() != OC_OK) return OC_ERR_CUDA;
    launch_norms(ctx, g, x, inv_norm, keys, s);
    oc_status st = launch_match_joint_tc(ctx, g, x, inv_norm, keys, units, n_units, joint_max_units(g), s);
    if (st != OC_OK) return st;
    {
        LaunchScope scope(ctx, OC_K_MATCH_FIN, s);
        OC_LAUNCH(finalize_joint_kernel, (unsigned)((n_tok + 255) / 256), 256, 0, s, g.H, g.W, g.sy, g.sx, g.oy, g.ox,
                  n_tok, frames, inv_norm, keys, best_sim, best_idx);
    }
    return last_launch_status();
}

}  // namespace oc
