/*
 * omnicache.h - C-ABI of the B200 (sm_100a) OmniCache hot path.
 *
 * The operator wrapped around one attention / FFN layer call by Token Cache, Frame Cache and Block
 * Cache (Sections 3.2.1-3.2.3), plus the Layered Cache store (Section 3.4):
 *
 *     match  ->  select  ->  gather  ->  [ the wrapped layer, outside this library ]  ->  restore
 *
 * Conventions
 *   - All data pointers are DEVICE pointers unless a name ends in `_host`.  The caller owns every
 *     feature / index / output buffer and the stream.  The library never allocates caller-visible
 *     memory, never frees caller memory and never synchronises the stream (exceptions are stated).
 *   - `stream` is a cudaStream_t passed as void*.  All work is stream-ordered.
 *   - Feature tensors are row-major [B][T][H][W][C], channel last (Section 3.2.2 writes spatial
 *     inputs as (B, T, H, W, C)); images have T = 1.  Base pointers are 16-byte aligned and
 *     C * element size is a multiple of 16 bytes.
 *   - A "unit" is a token (OC_KIND_TOKEN), a frame (OC_KIND_FRAME) or a 1x1xT temporal block
 *     (OC_KIND_BLOCK).  Unit indices are global and int32:
 *         token ((b*T + t)*H + y)*W + x,     frame b*T + t,     block b*H*W + y*W + x;
 *     with patch-local Frame Cache (gy*gx > 1) the unit is one patch of one frame,
 *         ((b*T + t)*gy + py)*gx + px.
 *   - Every call returns an oc_status.  On a host-detected error nothing is launched and no output
 *     is written.  Device-side conditions (an expired bounded wait) land in a status word read by
 *     oc_device_status().  No call aborts or throws.
 *   - A context is bound to one device and is not thread-safe; use one per host thread.
 */
#ifndef OMNICACHE_H_
#define OMNICACHE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int oc_status;
enum {
    OC_OK = 0,
    OC_ERR_INVALID_ARG = 1,  /* null pointer, non-positive size, inconsistent layout            */
    OC_ERR_ALIGNMENT = 2,    /* pointer or row size not a multiple of 16 bytes                  */
    OC_ERR_UNSUPPORTED = 3,  /* valid request outside what the kernels implement                */
    OC_ERR_WORKSPACE = 4,    /* context workspace smaller than oc_match_workspace_bytes()       */
    OC_ERR_CUDA = 5,         /* a CUDA runtime / driver call failed (no device, launch error)   */
    OC_ERR_TIMEOUT = 6,      /* a bounded device-side wait expired (see oc_device_status)       */
    OC_ERR_OOM = 7,          /* device allocation for library-owned storage failed              */
    OC_CACHE_MISS = 8        /* oc_layer_cache_get: nothing reusable for (layer, step)          */
};

enum { OC_KIND_TOKEN = 0, OC_KIND_FRAME = 1, OC_KIND_BLOCK = 2 };
enum { OC_DTYPE_F32 = 0, OC_DTYPE_BF16 = 1 };
enum { OC_SELECT_THRESHOLD = 0, OC_SELECT_COUNT = 1 };
enum { OC_RESTORE_FROM_CACHE = 0, OC_RESTORE_FROM_REPRESENTATIVE = 1 };
enum { OC_FRAME_MEAN_POS_COS = 0, OC_FRAME_FLAT_COS = 1 };

/* Which units are compared with which (Sections 3.2.1-3.2.3, 3.3).
 *   TOKEN: each frame is cut into gy x gx equal patches ("token groups", Section 3.3); inside a
 *          patch the tokens on the (oy, ox) + (sy, sx)-strided lattice are the representatives and
 *          every other token is a candidate, compared with all representatives of its patch.
 *          self_match = 1: every token is both (all pairs, self excluded); needs gy = gx = 1.
 *   FRAME: even frames are representatives, odd frames candidates, each compared with its two
 *          adjacent frames (alternating sets, Section 3.2.2).  sy..ox are ignored.  gy x gx > 1
 *          is the patch-local form of Section 3.3: each frame is cut into gy x gx equal patches,
 *          every patch position (b, py, px) is a matching and selection problem of its own over
 *          its T frame-patches (the paper's (B*k*k, T, (H/k)*(W/k)*C) arrangement, read in place),
 *          and the statistic runs over the patch's positions only.  gy = gx = 0 means 1.
 *   BLOCK: positions are cut into sy x sx neighbourhoods; the (oy, ox) member is the
 *          representative, the others are compared with it over the T*C block descriptor
 *          (Section 3.2.1).  gy x gx > 1 cuts the positions into patches of whole neighbourhoods
 *          (Section 3.3): matching is unchanged, the selection is taken per patch (b, py, px).
 * H must be a multiple of gy and W of gx; H/gy must be a multiple of sy and W/gx of sx (TOKEN, BLOCK). */
typedef struct oc_layout {
    int kind;        /* OC_KIND_*  */
    int dtype;       /* OC_DTYPE_* of the feature tensor */
    int B, T, H, W, C;
    int sy, sx;      /* representative lattice stride, >= 1, sy*sx >= 2 unless self_match */
    int oy, ox;      /* representative offset inside a neighbourhood, 0 <= oy < sy, 0 <= ox < sx */
    int gy, gx;      /* patches per frame (TOKEN, FRAME) */
    int self_match;  /* TOKEN only */
    int frame_stat;  /* FRAME only: OC_FRAME_* */
    float eps;       /* floor applied to each vector norm; cos = <a,b> / (max(|a|,eps) max(|b|,eps)) */
} oc_layout;

/* Rows of a strided tensor, used by gather / restore so that one pair of kernels moves tokens,
 * whole frames and 1x1xT blocks (the fused permutation/scatter of Appendix A).  The row of unit i
 * is n_seg segments of seg_bytes; segment s starts at byte
 *     (i / units_per_outer) * outer_pitch + (i % units_per_outer) * unit_pitch + s * seg_stride.
 * The dense side (gather output, restore input) is packed [row][segment][seg_bytes].
 * seg_bytes and all pitches are multiples of 16. */
typedef struct oc_rows {
    int64_t seg_bytes;
    int64_t n_seg;
    int64_t seg_stride;
    int64_t unit_pitch;
    int64_t units_per_outer;
    int64_t outer_pitch;
} oc_rows;

typedef struct oc_ctx oc_ctx;

/* ---------------------------------------------------------------------------------------------
 * Host-only helpers: no device is touched, usable without a GPU.
 * ------------------------------------------------------------------------------------------- */

/* Human-readable name of a status code (static storage). */
const char* oc_status_str(oc_status s);

/* Validates a layout against the rules above.  OC_OK, OC_ERR_INVALID_ARG, OC_ERR_ALIGNMENT
 * (C * element size not a multiple of 16) or OC_ERR_UNSUPPORTED (e.g. more than 2^31-1 units). */
oc_status oc_layout_check(const oc_layout* layout);

/* Group structure of a layout: a group is an independent selection problem (TOKEN: one patch of one
 * frame; FRAME: one patch position of one batch element, its units being T frame-patches that lie
 * gy*gx apart in unit order; BLOCK: one batch element).  Any output pointer may be null. */
oc_status oc_layout_counts(const oc_layout* layout, int64_t* n_groups, int64_t* units_per_group,
                           int64_t* reps_per_group);

/* Bytes of context workspace oc_match() needs for this layout (norms, packed arg-max keys,
 * partial sums). */
oc_status oc_match_workspace_bytes(const oc_layout* layout, size_t* bytes);

/* Row geometry of this layout's units inside a [B][T][H][W][channels] tensor of elem_bytes-sized
 * elements (the layer input, or a layer output with another channel count). */
oc_status oc_rows_from_layout(const oc_layout* layout, int channels, int elem_bytes, oc_rows* rows);

/* The Layered Cache reuse rule (Section 3.4; the (l, t, N) triples of Algorithm 1): an output stored
 * at stored_step serves step iff 0 <= step - stored_step < interval.  Returns 1 or 0. */
int oc_layer_cache_would_hit(int stored_step, int step, int interval);

/* Kernel ids for the launch counters / timers below. */
enum {
    OC_K_NORMS = 0,       /* row inverse norms + key reset (dense match pre-pass)     */
    OC_K_MATCH_TC = 1,    /* tcgen05 dense matcher                                    */
    OC_K_MATCH_SIMT = 2,  /* FFMA dense matcher (fp32 inputs, self-match, odd shapes) */
    OC_K_MATCH_FIN = 3,   /* key unpack -> best_sim / best_idx                        */
    OC_K_FRAME = 4,       /* Frame Cache streaming cosine                             */
    OC_K_FRAME_FIN = 5,
    OC_K_BLOCK = 6,       /* Block Cache streaming cosine                             */
    OC_K_BLOCK_FIN = 7,
    OC_K_SELECT = 8,
    OC_K_GATHER = 9,
    OC_K_RESTORE = 10,
    OC_K_COPY = 11,       /* layered-cache put / copying get                          */
    OC_K_LINEAR = 12,     /* projection with gather / scatter folded in               */
    OC_K_COUNT = 13
};
const char* oc_kernel_name(int kernel_id);

/* ---------------------------------------------------------------------------------------------
 * Context
 * ------------------------------------------------------------------------------------------- */

/* Creates a context on `device` with `workspace_bytes` of library-owned scratch (may be 0 if
 * oc_match is never called).  The context also owns the Layered Cache storage and a device status
 * word.  OC_ERR_CUDA if the device cannot be used, OC_ERR_OOM if the scratch cannot be allocated. */
oc_status oc_create(oc_ctx** out, int device, size_t workspace_bytes);

/* Frees everything the context owns.  Synchronises the device. */
oc_status oc_destroy(oc_ctx* ctx);

/* Synchronises the device, reads and clears the device status word: *code is OC_OK or the first
 * device-side condition recorded since the last call (OC_ERR_TIMEOUT). */
oc_status oc_device_status(oc_ctx* ctx, int* code);

/* Self-test of the device-side failure path.  Every wait inside the kernels is bounded; when one
 * runs out the kernel records OC_ERR_TIMEOUT in the status word and returns instead of hanging.
 * This call launches a one-warp kernel that waits, for at most limit_us microseconds
 * (1 .. 1000000), on a barrier that nothing completes, so that path can be observed on demand:
 * afterwards oc_device_status() reports OC_ERR_TIMEOUT once, and the context works as before. */
oc_status oc_selftest_bounded_wait(oc_ctx* ctx, unsigned int limit_us, void* stream);

/* Self-test of the once-per-device bookkeeping (host only: no CUDA call, no device needed).  Kernel
 * attributes such as the opt-in to large dynamic shared memory belong to a device, and one process may
 * use the library on several; the launchers therefore run their set-up once per DEVICE.  This call
 * drives a fresh instance of that bookkeeping: for round = 0 .. n_rounds-1 and dev = 0 .. n_devices-1
 * it asks for the set-up of `dev`, with a set-up routine that counts its runs per device and fails on
 * device fail_dev (-1: never).  runs[dev] receives how often the routine ran (1 for every device, also
 * the failing one: a failure is remembered, not retried), ok[dev] how often the request succeeded
 * (n_rounds, or 0 for fail_dev).  Both arrays are host memory of n_devices ints (1 .. 64 devices). */
oc_status oc_selftest_per_device_once(int n_devices, int n_rounds, int fail_dev, int* runs, int* ok);

/* Launch counters and optional per-kernel timers.  Counters always run.  oc_profile_enable takes
 * 0 (timers off), 1 (each kernel launch is bracketed by CUDA events on the caller's stream) or 2
 * (device-side spans of the tensor-core matcher, see oc_profile_span_read; no events).
 * oc_profile_read waits for the recorded events and returns the number of launches and their
 * summed device time since the last reset.  total_ms is 0 when the event timers were off. */
oc_status oc_profile_enable(oc_ctx* ctx, int on);
oc_status oc_profile_reset(oc_ctx* ctx);
oc_status oc_profile_read(oc_ctx* ctx, int kernel_id, int64_t* launches, double* total_ms);

/* Test hook: forces the work split of the tensor-core matcher for this context's later oc_match /
 * oc_match_joint calls instead of the planner's choice: a single CTA (pair = 0) or a CTA pair
 * (pair = 1) per piece, 1 or 2 candidate tiles per CTA, pieces_per_row pieces per row of the
 * problem; single_accumulator != 0 keeps narrow pieces on one accumulator set; candidates_resident
 * 1 / 0 turns on / off keeping a CTA's candidate tiles in shared memory for all pieces of a row
 * (only where they fit), -1 leaves that to the planner.  A split the shape does not admit is ignored
 * (the planner's choice runs).  on = 0 returns to the planner.  Results never depend on the split;
 * the parity tests use this to run every form of the kernel.  OC_ERR_INVALID_ARG for values outside
 * the ranges above.  The paper has no counterpart. */
oc_status oc_tc_plan_override(oc_ctx* ctx, int on, int pair, int tiles_per_cta, int pieces_per_row,
                              int single_accumulator, int candidates_resident);

/* Test hook: the work split oc_match would use for this (bf16, no self-match) OC_KIND_TOKEN layout on
 * this context, forced split included.  out receives 12 ints: pair, tiles per CTA, pieces per row,
 * two accumulator sets (0/1), ring stages, bytes per stage, candidate tiles resident (0/1), pieces in
 * total, walkers (CTAs or CTA pairs launched), widest piece in columns, 64-channel steps, reserved.
 * Host only.  OC_ERR_UNSUPPORTED when the layout does not take the tensor-core kernel. */
oc_status oc_tc_plan_describe(oc_ctx* ctx, const oc_layout* layout, int32_t* out);

/* Device-side span of the tensor-core matcher (kernel_id must be OC_K_MATCH_TC).  With
 * oc_profile_enable(ctx, 2) every launch of that kernel stamps the GPU's nanosecond timer when its
 * first CTA starts and when its last CTA ends (two atomics per CTA; no events are recorded in this
 * mode).  oc_profile_span_read synchronises the device and returns how many launches were stamped
 * since the last reset (at most the 256 most recent are kept) and the sum of their spans.  A span
 * leaves out what an event bracket adds around a kernel (launch latency, the event records
 * themselves): it is the time the kernel's CTAs occupy the device.  The paper has no counterpart;
 * this is a measurement aid. */
oc_status oc_profile_span_read(oc_ctx* ctx, int kernel_id, int64_t* launches, double* total_ms);

/* Event brackets inside a CUDA graph.  Launches made while the event timers are on (mode 1) AND the
 * caller's stream is being captured are bracketed by event-record nodes of the captured graph; those
 * brackets are taken again every time the graph runs and are not counted by oc_profile_read.
 * oc_profile_captured_read returns, for one kernel, how many such brackets exist (over all graphs
 * captured so far with this context) and the sum of their MOST RECENT recordings; call it after
 * synchronising a replay.  The events live until oc_destroy: graphs captured this way must not be
 * launched after the context is destroyed. */
oc_status oc_profile_captured_read(oc_ctx* ctx, int kernel_id, int64_t* launches, double* total_ms);

/* ---------------------------------------------------------------------------------------------
 * The hot path
 * ------------------------------------------------------------------------------------------- */

/* match (Background: candidates are paired with representatives by cosine similarity; Sections
 * 3.2.1-3.2.3).  For every candidate unit: the most similar representative it may be matched with.
 *   x         [B][T][H][W][C] features of layout->dtype (the wrapped layer's input)
 *   best_sim  [n_units] float: cosine of the best match; -inf for representatives
 *   best_idx  [n_units] int32: global unit index of that representative (ties: lowest index; the
 *             tensor-core matcher compares cosines rounded to within 2.4e-7, so values that agree to
 *             that precision count as tied);
 *             a representative's own index for representatives
 *   aux_sim   nullable.  TOKEN: [n_groups][units_per_group][reps_per_group] float, every candidate
 *             row's full similarity row (rows of representatives and the self-match diagonal are
 *             not written).  FRAME: [B][T-1][H*W] per-position cosines of frame t vs t-1.
 *   pair_sim  nullable, FRAME only: [B][T-1][gy*gx] statistic of every adjacent pair (t, t-1),
 *             per patch.
 * bf16 TOKEN layouts without self_match run on the tcgen05 tensor cores (fp32 accumulation) when the
 * lattice has at most 9 members, C is a multiple of 8 and a group has at most 4800 representative
 * slots (150 boxes of 32 lattice points; the SVD-XT frame has 2304, the SD3 image 1024);
 * everything else on fp32 FMA pipelines, with the same results up to the tolerances above.  Needs oc_match_workspace_bytes() of context workspace
 * (OC_ERR_WORKSPACE otherwise).  Calls on one context must not overlap on the device. */
oc_status oc_match(oc_ctx* ctx, const oc_layout* layout, const void* x, float* best_sim,
                   int32_t* best_idx, float* aux_sim, float* pair_sim, void* stream);

/* Frame Cache at several patch sizes from ONE pass over the tensor (Section 3.3: the patch-level pass
 * may be followed by coarser ones, with larger patches or with whole frames).  `layout` is an OC_KIND_FRAME layout whose (gy, gx) is the finest grid; `grids` (HOST
 * memory, [n_levels][2] ints) lists (gy_l, gx_l) per level, each dividing (gy, gx) -- (1, 1) is the
 * whole frame.  Level l's results are what oc_match() gives for the same layout with (gy_l, gx_l)
 * (equal up to fp32 summation order), stored one level after another:
 *   best_sim, best_idx  [sum_l B*T*gy_l*gx_l], unit indices local to their level
 *   pair_sim  nullable, [sum_l B*(T-1)*gy_l*gx_l]
 *   pos_sim   nullable, [B][T-1][H*W] per-position cosines (shared by all levels)
 * The streaming kernel runs once; only the small per-unit reduction runs per level.
 * 1 <= n_levels <= OC_MAX_FRAME_LEVELS.  Workspace: oc_match_workspace_bytes(layout).
 * Errors: as oc_match(); OC_ERR_INVALID_ARG for a grid that does not divide the layout's. */
#define OC_MAX_FRAME_LEVELS 8
oc_status oc_match_frame_levels(oc_ctx* ctx, const oc_layout* layout, const void* x, int n_levels,
                                const int32_t* grids, float* best_sim, int32_t* best_idx, float* pos_sim,
                                float* pair_sim, void* stream);

/* ---------------------------------------------------------------------------------------------
 * The wrapped layer's projection with the gather folded into its operand load and the restore into
 * its store (Appendix A's compaction and fused scatter taken one step further: the dense buffers on
 * both sides of the layer are never written):
 *     out[dst(r), :] = bf16( sum_k a[src(r), k] * w[n, k] ),     r = 0 .. n_rows-1
 *   a        [a_rows][K] bf16, row-major (e.g. the token rows of the feature tensor)
 *   a_idx    nullable, [n_rows] int32: src(r) = a_idx[r] (the kept_idx list); null: src(r) = r
 *   w        [N][K] bf16, row-major (the layout of a linear layer's weight)
 *   out      [out_rows][N] bf16; out_idx nullable, [n_rows]: dst(r) = out_idx[r]; null: dst(r) = r
 * A row whose src or dst is negative (or out of range) is skipped; rows of `out` that no r names keep
 * their contents, so with out = the cached activations and out_idx = kept_idx the call IS the restore.
 * bf16 x bf16 products, fp32 accumulation on the tcgen05 tensor cores, one rounding to bf16.
 * K % 8 == 0, N % 8 == 0, N >= 128; a, w, out 16-byte aligned.  Errors: OC_ERR_INVALID_ARG,
 * OC_ERR_ALIGNMENT, OC_ERR_UNSUPPORTED (shape limits), OC_ERR_CUDA.
 * ------------------------------------------------------------------------------------------- */
oc_status oc_linear_gather_scatter(oc_ctx* ctx, const void* a, int64_t a_rows, int64_t K, const int32_t* a_idx,
                                   int64_t n_rows, const void* w, int64_t N, void* out, int64_t out_rows,
                                   const int32_t* out_idx, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Token Cache on the frame pairs of Frame Cache (Section 3.2.3): it works on the feature map and the
 * frame pairing Frame Cache has just produced; matched pairs become token groups of 2*H*W tokens
 * with one representative per 2x2x2 cube, unmatched frames keep their 2x2 groups.
 * `layout` is the OC_KIND_TOKEN layout of the tensor (bf16, gy = gx = 1, no self_match, a layout
 * that oc_match runs on the tensor cores; OC_ERR_UNSUPPORTED otherwise).  `frames` is a device array of B*T slots {rep, partner} (int32
 * pairs, 8-byte aligned): slot f = {f, t} if frame f is the representative frame of the pair
 * (f, t), {f, -1} if frame f is a group of its own, {-1, -1} if frame f was absorbed into its
 * partner's group.
 *
 * oc_joint_groups: builds `frames` from a Frame Cache result on the same tensor (whole frames,
 *   gy = gx = 1): a candidate frame t with frame_slot_of[t] < 0 (reused) claims the representative
 *   frame_best_idx[t]; if both neighbours of a representative claim it, the one with the larger
 *   frame_best_sim wins (equal: the earlier frame) and the other stays on its own.
 * oc_match_joint: for every group, every candidate token against all representatives of the group
 *   (the lattice tokens of the representative frame); candidates are the other tokens of that frame
 *   and ALL tokens of the partner frame.  Outputs as oc_match (indexed by token).  One launch of
 *   the tensor-core matcher over a device-side work list; needs oc_joint_workspace_bytes().
 * oc_select_joint: as oc_select with one group per slot, a pair's units being the tokens of its two
 *   frames in time order; n_reuse_pair / n_reuse_single are the count-mode budgets of the two kinds
 *   of group; kept_idx is [B*T][y_stride] (absorbed slots keep nothing, kept_count 0), y_stride at
 *   most 2*H*W and at least what either kind of group can keep; 2*H*W at most 40960.
 * gather / restore then move token rows as for any Token Cache selection (n_slots = B*T*y_stride).
 * Errors: as oc_match / oc_select.
 * ------------------------------------------------------------------------------------------- */
oc_status oc_joint_workspace_bytes(const oc_layout* layout, size_t* bytes);
oc_status oc_joint_groups(oc_ctx* ctx, const oc_layout* layout, const float* frame_best_sim,
                          const int32_t* frame_best_idx, const int32_t* frame_slot_of, int32_t* frames,
                          void* stream);
oc_status oc_match_joint(oc_ctx* ctx, const oc_layout* layout, const void* x, const int32_t* frames,
                         float* best_sim, int32_t* best_idx, void* stream);
oc_status oc_select_joint(oc_ctx* ctx, const oc_layout* layout, const int32_t* frames, const float* best_sim,
                          const int32_t* best_idx, int mode, float thr, int64_t n_reuse_pair,
                          int64_t n_reuse_single, int64_t y_stride, int32_t* kept_idx, int32_t* kept_count,
                          int32_t* match_map, int32_t* slot_of, void* stream);

/* select (Sections 3.2.1-3.2.3: the r candidates most similar to their match are restored from the
 * cache, everything else goes through the layer).  Representatives are always kept.
 *   mode OC_SELECT_THRESHOLD: a candidate is reused iff best_sim >= thr (self_match: and its best
 *        match has a lower index; match_map then follows best_idx down to a kept token).
 *   mode OC_SELECT_COUNT: in every group the n_reuse_per_group candidates with the largest
 *        best_sim are reused (equal values: lower index first; clamped to the candidates present).
 *   y_group_stride  rows reserved per group in the dense buffer: at least the number of kept units
 *        (units_per_group always suffices; units_per_group - n_reuse in COUNT mode packs it tight)
 *   kept_idx   [n_groups][y_group_stride] int32: kept units in ascending original index, tail -1
 *   kept_count [n_groups] int32 (stays on the device: no host synchronisation)
 *   match_map  [n_units] int32: i for kept units, else the representative standing for i
 *   slot_of    [n_units] int32: row of unit i in the dense buffer (g*y_group_stride + rank), -1 if reused
 * OC_ERR_UNSUPPORTED for COUNT with self_match or more than 65536 units per group. */
oc_status oc_select(oc_ctx* ctx, const oc_layout* layout, const float* best_sim,
                    const int32_t* best_idx, int mode, float thr, int64_t n_reuse_per_group,
                    int64_t y_group_stride, int32_t* kept_idx, int32_t* kept_count,
                    int32_t* match_map, int32_t* slot_of, void* stream);

/* gather (Appendix A: compaction of the kept rows): y[slot] = row kept_idx[slot] of x for every slot
 * in [0, n_slots) with kept_idx[slot] >= 0; other slots of y are left untouched.  Bit copy. */
oc_status oc_gather(oc_ctx* ctx, const oc_rows* rows, const void* x, const int32_t* kept_idx,
                    int64_t n_slots, void* y, void* stream);

/* restore (Sections 3.2.1-3.2.3: a skipped position takes the activation cached for that same
 * position at the previous denoising step; rows are copied, never averaged).
 *   z      dense layer output, row slot_of[i] belongs to unit i
 *   cache  strided like out: the previous step's restored output (nullable in
 *          OC_RESTORE_FROM_REPRESENTATIVE mode)
 *   out    out[i] = z[slot_of[i]] if slot_of[i] >= 0; otherwise cache[i] (FROM_CACHE) or
 *          z[slot_of[match_map[i]]] (FROM_REPRESENTATIVE, for a first step without a cache).
 *          out may equal cache: then only computed rows are written. */
oc_status oc_restore(oc_ctx* ctx, const oc_rows* rows, const void* z, const void* cache,
                     int64_t n_units, const int32_t* slot_of, const int32_t* match_map, void* out,
                     int src_mode, void* stream);

/* Layered Cache (Section 3.4): keep a layer's output at a scheduled step and reuse it for the
 * following steps of the interval.
 *   put  copies `bytes` from src into library-owned storage for `layer` (allocated on the first
 *        put of that size: that put calls cudaMalloc) and records `step`.
 *   get  OC_OK iff an entry exists and 0 <= step - stored_step < interval, else OC_CACHE_MISS.
 *        On a hit: if dst != null the stored bytes are copied to dst (stream-ordered); if
 *        view != null *view receives the library-owned device pointer (zero copy, valid until the
 *        next put / clear for that layer); if bytes != null *bytes receives the entry size.
 *   clear frees all entries (synchronises the device). */
oc_status oc_layer_cache_put(oc_ctx* ctx, int layer, int step, const void* src, size_t bytes,
                             void* stream);
oc_status oc_layer_cache_get(oc_ctx* ctx, int layer, int step, int interval, void* dst,
                             const void** view, size_t* bytes, void* stream);
oc_status oc_layer_cache_clear(oc_ctx* ctx);

/* Frame Cache match for callers that must not allocate.  The paper has no counterpart for this
 * call; it exists for hosts where the calling code is not allowed to obtain device memory at all:
 * an inference server that hands its whole memory budget to one pool at start-up and treats any
 * later driver allocation as a fault, a plug-in running inside another framework's allocator, or
 * code that may already be inside a region where cudaMalloc is illegal or would stall every stream.
 * oc_match() needs a context, and a context owns cudaMalloc'd scratch; this variant needs neither.
 *
 * It computes exactly what oc_match() computes for an OC_KIND_FRAME layout (best_sim, best_idx and,
 * if pair_sim is not null, the [B][T-1][gy*gx] adjacent-pair statistic), with the same kernels, but keeps
 * its partial sums in a fixed array of OC_NOALLOC_SCRATCH_BYTES bytes that is part of the library
 * image: every GPU that loads the library holds that array until the process exits.
 *   - A layout whose scratch need (oc_match_workspace_bytes) exceeds OC_NOALLOC_SCRATCH_BYTES is
 *     refused with OC_ERR_WORKSPACE and nothing is launched.  Other kinds: OC_ERR_INVALID_ARG.
 *   - The call itself makes no cudaMalloc / cudaFree and uses no allocating library routine; the
 *     caller passes every input and output buffer.
 *   - The first call on each device looks up the array's device address (with that device current),
 *     reads the device's SM count and makes the driver load every kernel the call can launch, and
 *     remembers all that; make that first call before any stream capture begins.  (Later calls with
 *     a layout of another dtype or row length launch other instances of the same kernels; those
 *     were loaded by the first call.)
 *   - All calls on a device share the one array and it keeps whatever the previous call left.  No
 *     part of it needs to start at zero (each call writes every value it later reads), but two calls
 *     whose kernels overlap on the GPU - different streams, or one stream replayed concurrently -
 *     race on it.  Serialise them. */
#define OC_NOALLOC_SCRATCH_BYTES (1u << 20)
oc_status oc_match_frame_noalloc(int device, const oc_layout* layout, const void* x, float* best_sim,
                                 int32_t* best_idx, float* pair_sim, void* stream);

/* Layered Cache schedule proposal (Algorithm 1, Section 3.4).  Host-side; launches nothing and needs
 * no context.
 *   latency[i], quality_loss[i]  the profiled L and Q of candidate i (a layer-timestep pair), n of
 *                                them, host arrays; every latency must be > 0 and finite, every
 *                                quality loss finite
 *   target_speedup               s_r >= 1
 * Candidates are ranked by quality loss per unit of latency, cheapest first (equal scores: lower
 * index first); the result is the shortest prefix of that ranking whose latencies add up to at least
 * the budget (1 - 1/s_r) * sum(latency) -- the whole ranking if none does.  Double precision.
 *   chosen     host array of capacity n: receives the taken candidate indices in the order taken
 *              (each is to be cached with the caller's interval N, which does not influence the choice)
 *   n_chosen   receives how many were taken
 *   saved      nullable: receives the accumulated latency of the taken candidates
 * OC_ERR_INVALID_ARG on null pointers, n < 0, s_r < 1 or non-finite / non-positive inputs; nothing
 * is written then.  The refinement pass over the model graph (Algorithm 2) is not part of this
 * library. */
oc_status oc_schedule_propose(const double* latency, const double* quality_loss, int64_t n, double target_speedup,
                              int32_t* chosen, int64_t* n_chosen, double* saved);

/* One whole cache-wrapped layer call on HOST buffers, for callers that keep activations in host
 * memory: copies x_host (layer input) and cache_host (previous output, same shape) to library-owned
 * device staging, runs match -> select -> gather -> restore with the identity as the wrapped layer
 * (z = the gathered rows), copies the restored tensor to out_host and the per-group kept counts to
 * kept_count_host, and synchronises the stream before returning.  When cache_host / out_host are
 * pinned (page-locked, device-mapped, 16-byte aligned) the restore kernel reads and writes them in
 * place: of the cache only the rows of reused units cross the bus, and the output streams out while
 * they stream in; pageable buffers go through staging copies of the whole tensors.  x_host is always
 * copied whole (the matcher reads it several times).  Token Cache layouts of several frames are
 * processed in up to 8 chunks of whole frames, the copies of later chunks overlapping the work on
 * earlier ones (a second, library-owned stream carries those copies; the caller's stream orders the
 * call as a whole). */
oc_status oc_cache_step_host(oc_ctx* ctx, const oc_layout* layout, int mode, float thr,
                             int64_t n_reuse_per_group, const void* x_host, const void* cache_host,
                             void* out_host, int32_t* kept_count_host, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* OMNICACHE_H_ */
