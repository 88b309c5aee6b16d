/*
 * CPU oracle for the OmniCache match / select / gather / restore path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition of what the path computes,
 * written from the paper; it shares no code, header, table or constant with the CUDA library and
 * must never be linked into or called from the product path.  Only the test-suite, the smoke
 * check and the CPU-baseline leg of the benchmark use it.
 *
 * Conventions (the paper writes spatial-layer inputs as (B, T, H, W, C), Section 3.2.2):
 *   - features are row-major [B][T][H][W][C], channel last; a "token" is one C-vector;
 *   - dtype 0 = IEEE fp32, dtype 1 = bf16 stored as 16-bit patterns; every stored value is
 *     widened exactly to double and all arithmetic is double;
 *   - a unit is a token (kind 0), a frame (kind 1) or a 1x1xT block (kind 2); unit indices are
 *     global: token ((b*T+t)*H+y)*W+x, frame b*T+t, block b*H*W + y*W+x; with patch-local
 *     Frame Cache (Section 3.3, gy*gx > 1) the unit is one patch of one frame,
 *     ((b*T+t)*gy+py)*gx+px;
 *   - outputs that the library produces in fp32 are rounded to fp32 once, at the end.
 *
 * Every function has at least one pin in the CPU test-suite (brute force in NumPy, closed forms,
 * invariants); none is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int kind;        /* 0 token, 1 frame, 2 block */
    int dtype;       /* 0 fp32, 1 bf16 bits */
    int B, T, H, W, C;
    int sy, sx;      /* representative lattice stride (Section 3.2.1 / 3.2.3: local 2x2 groups) */
    int oy, ox;      /* which member of a group is the representative */
    int gy, gx;      /* patches per frame, Section 3.3 (token and frame kinds) */
    int self_match;  /* every token is candidate and representative (tiny all-pairs config) */
    int frame_stat;  /* 0 mean of same-position token cosines, 1 cosine of the flat H*W*C descriptor */
    double eps;      /* floor applied to each norm */
} ocr_layout;

int ocr_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void ocr_set_num_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* ---- stored value -> double ------------------------------------------------------------- */
static double load_elem(const void* x, int dtype, int64_t i) {
    if (dtype == 0) return (double)((const float*)x)[i];
    uint32_t bits = ((uint32_t)((const uint16_t*)x)[i]) << 16;   /* bf16 = top half of an fp32 */
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* ---- O1: cosine similarity of two length-n vectors ---------------------------------------
 * cos(a,b) = <a,b> / (max(|a|,eps) * max(|b|,eps)), clamped to [-1, 1].
 * (Background, "matches similar pairs by cosine similarity".)  a, b: element offsets into x. */
static double clamp1(double v) { return v > 1.0 ? 1.0 : (v < -1.0 ? -1.0 : v); }

double ocr_cosine(const void* x, int dtype, int64_t a_off, int64_t b_off, int64_t n, double eps) {
    double dot = 0.0, na = 0.0, nb = 0.0;
    for (int64_t c = 0; c < n; ++c) {
        double a = load_elem(x, dtype, a_off + c), b = load_elem(x, dtype, b_off + c);
        dot += a * b; na += a * a; nb += b * b;
    }
    na = sqrt(na); nb = sqrt(nb);
    if (na < eps) na = eps;
    if (nb < eps) nb = eps;
    return clamp1(dot / (na * nb));
}

/* ---- group structure -----------------------------------------------------------------------
 * token kind : a group is one patch of one frame, (b, t, py, px); units = (H/gy)*(W/gx) tokens,
 *              local index u = ly*(W/gx)+lx in row-major order of the patch.
 * frame kind : a group is one patch position of one batch element, (b, py, px) (Section 3.3's
 *              (B*k*k, T, .) arrangement; gy = gx = 1 is the whole frame); units = the T
 *              frame-patches at that position, local index u = t.
 * block kind : a group is one patch of one batch element, (b, py, px) (gy = gx = 1: all positions);
 *              units = the (H/gy)*(W/gx) spatial positions of the patch, row-major.  A block is
 *              always compared with the representative of its own sy x sx neighbourhood; the patch
 *              confines the selection ("the r most redundant" of the patch, Section 3.3). */
int64_t ocr_num_groups(const ocr_layout* L) {
    if (L->kind == 0) return (int64_t)L->B * L->T * L->gy * L->gx;
    return (int64_t)L->B * L->gy * L->gx;
}
int64_t ocr_units_per_group(const ocr_layout* L) {
    if (L->kind == 1) return L->T;
    return (int64_t)(L->H / L->gy) * (L->W / L->gx);
}
int64_t ocr_num_units(const ocr_layout* L) { return ocr_num_groups(L) * ocr_units_per_group(L); }

/* global unit index of local unit u of group g */
int64_t ocr_unit_index(const ocr_layout* L, int64_t g, int64_t u) {
    if (L->kind != 1) {                        /* token: bt = frame b*T+t; block: bt = batch element */
        int Hp = L->H / L->gy, Wp = L->W / L->gx;
        int64_t px = g % L->gx, py = (g / L->gx) % L->gy, bt = g / ((int64_t)L->gx * L->gy);
        int64_t ly = u / Wp, lx = u % Wp;
        return (bt * L->H + py * Hp + ly) * L->W + px * Wp + lx;
    }
    int64_t np = (int64_t)L->gy * L->gx, b = g / np, patch = g % np;
    return (b * L->T + u) * np + patch;
}

/* is local unit u a representative (always computed, never reused)? */
int ocr_is_rep(const ocr_layout* L, int64_t u) {
    if (L->kind == 1) return (u % 2) == 0;                 /* alternating frame sets, Section 3.2.2 */
    if (L->self_match) return 1;
    int Wl = L->W / L->gx;                     /* patches hold whole sy x sx neighbourhoods */
    int64_t ly = u / Wl, lx = u % Wl;
    return (ly % L->sy) == L->oy && (lx % L->sx) == L->ox;
}

static int is_cand(const ocr_layout* L, int64_t u) {
    if (L->kind == 0 && L->self_match) return 1;
    return !ocr_is_rep(L, u);
}

/* ---- O2: dense match (Token Cache) ---------------------------------------------------------
 * For each candidate token of a group, the cosine against every representative of the same group
 * (self-match: every other token); best = maximum, ties to the lowest token index; second = the
 * runner-up value (used only to classify near-ties).  Representatives get best_idx = own index,
 * best_sim = -inf.  If rows != NULL only those global token indices are evaluated.
 * full_sim (nullable): [group][local unit][representative rank] doubles; rows of representatives
 * and, in self-match, the diagonal are left untouched.
 * Outputs are indexed by global token index. */
int ocr_match_token(const ocr_layout* L, const void* x, const int32_t* rows, int64_t n_rows,
                    float* best_sim, int32_t* best_idx, float* second_sim, double* full_sim) {
    if (L->kind != 0) return 1;
    const int64_t G = ocr_num_groups(L), U = ocr_units_per_group(L), C = L->C;
    const int64_t n_tok = G * U;
    /* norms of every token */
    double* norm = (double*)malloc(sizeof(double) * (size_t)n_tok);
    if (!norm) return 2;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n_tok; ++i) {
        double s = 0.0;
        for (int64_t c = 0; c < C; ++c) { double v = load_elem(x, L->dtype, i * C + c); s += v * v; }
        s = sqrt(s);
        norm[i] = s < L->eps ? L->eps : s;
    }
    /* representative list of each group, ascending global index (= ascending local index) */
    int64_t n_rep = 0;
    for (int64_t u = 0; u < U; ++u) n_rep += ocr_is_rep(L, u);
    int64_t* rep_local = (int64_t*)malloc(sizeof(int64_t) * (size_t)(n_rep > 0 ? n_rep : 1));
    if (!rep_local) { free(norm); return 2; }
    { int64_t r = 0; for (int64_t u = 0; u < U; ++u) if (ocr_is_rep(L, u)) rep_local[r++] = u; }

    const int64_t n_work = rows ? n_rows : n_tok;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t w = 0; w < n_work; ++w) {
        int64_t g, u, i;
        if (rows) {
            /* invert the global index: find (g, u) by search over groups of the same frame */
            i = rows[w];
            int Hp = L->H / L->gy, Wp = L->W / L->gx;
            int64_t xx = i % L->W, yy = (i / L->W) % L->H, bt = i / ((int64_t)L->W * L->H);
            int64_t py = yy / Hp, px = xx / Wp;
            g = (bt * L->gy + py) * L->gx + px;
            u = (yy % Hp) * Wp + (xx % Wp);
        } else {
            g = w / U; u = w % U; i = ocr_unit_index(L, g, u);
        }
        if (!is_cand(L, u)) {
            best_sim[i] = -INFINITY; best_idx[i] = (int32_t)i;
            if (second_sim) second_sim[i] = -INFINITY;
            continue;
        }
        double best = -INFINITY, second = -INFINITY; int64_t arg = i;
        for (int64_t r = 0; r < n_rep; ++r) {
            int64_t j = ocr_unit_index(L, g, rep_local[r]);
            if (j == i) continue;                                  /* self-match excludes self */
            double dot = 0.0;
            for (int64_t c = 0; c < C; ++c)
                dot += load_elem(x, L->dtype, i * C + c) * load_elem(x, L->dtype, j * C + c);
            double s = clamp1(dot / (norm[i] * norm[j]));
            if (full_sim) full_sim[(g * U + u) * n_rep + r] = s;
            if (s > best) { second = best; best = s; arg = j; }
            else if (s > second) second = s;
        }
        best_sim[i] = (float)best; best_idx[i] = (int32_t)arg;
        if (second_sim) second_sim[i] = (float)second;
    }
    free(rep_local); free(norm);
    return 0;
}

/* ---- O3: Frame Cache match -----------------------------------------------------------------
 * Even frames are representatives, odd frames candidates (alternating sets, Section 3.2.2).  The
 * similarity of two frames is, by default, the mean over positions p of cos(x[t,p,:], x[u,p,:]);
 * with frame_stat = 1 it is the cosine of the two flattened H*W*C descriptors (the paper's literal
 * (B, T, H*W*C) reshape).  A candidate t is compared with its adjacent frames t-1 and t+1 only;
 * best = maximum, ties to the lower frame.
 * Patch-local form (Section 3.3): the frame is cut into gy x gx equal patches and everything above
 * is done per patch position, the descriptor being the patch's (H/gy)*(W/gx)*C elements; a unit is
 * one patch of one frame and best_idx names the matched patch of the adjacent frame.
 * pair_sim[b][t-1][patch], t = 1..T-1, is the statistic of (t, t-1) for every adjacent pair;
 * pos_sim (nullable) [b][t-1][p] the per-position cosines (p = y*W+x in the frame). */
static double patch_stat(const ocr_layout* L, const void* x, int64_t fa, int64_t fb, int64_t py, int64_t px) {
    const int64_t Hp = L->H / L->gy, Wp = L->W / L->gx, C = L->C, P = (int64_t)L->H * L->W;
    double acc = 0.0, dot = 0.0, na = 0.0, nb = 0.0;
    for (int64_t ly = 0; ly < Hp; ++ly)
        for (int64_t lx = 0; lx < Wp; ++lx) {
            int64_t p = (py * Hp + ly) * L->W + px * Wp + lx;
            int64_t ao = (fa * P + p) * C, bo = (fb * P + p) * C;
            if (L->frame_stat == 1) {
                for (int64_t c = 0; c < C; ++c) {
                    double a = load_elem(x, L->dtype, ao + c), b = load_elem(x, L->dtype, bo + c);
                    dot += a * b; na += a * a; nb += b * b;
                }
            } else {
                acc += ocr_cosine(x, L->dtype, ao, bo, C, L->eps);
            }
        }
    if (L->frame_stat == 1) {
        na = sqrt(na); nb = sqrt(nb);
        if (na < L->eps) na = L->eps;
        if (nb < L->eps) nb = L->eps;
        return clamp1(dot / (na * nb));
    }
    return acc / (double)(Hp * Wp);
}

int ocr_match_frame(const ocr_layout* L, const void* x, float* best_sim, int32_t* best_idx,
                    float* pair_sim, float* pos_sim) {
    if (L->kind != 1) return 1;
    if (L->gy <= 0 || L->gx <= 0 || L->H % L->gy || L->W % L->gx) return 1;
    const int64_t T = L->T, P = (int64_t)L->H * L->W, C = L->C;
    const int64_t np = (int64_t)L->gy * L->gx;
    const int64_t n_pairs = (int64_t)L->B * (T - 1);
    double* pair = (double*)malloc(sizeof(double) * (size_t)(n_pairs * np > 0 ? n_pairs * np : 1));
    if (!pair) return 2;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t q = 0; q < n_pairs; ++q) {
        int64_t b = q / (T - 1), t = q % (T - 1) + 1;
        int64_t fa = b * T + t, fb = fa - 1;
        for (int64_t patch = 0; patch < np; ++patch) {
            pair[q * np + patch] = patch_stat(L, x, fa, fb, patch / L->gx, patch % L->gx);
            if (pair_sim) pair_sim[q * np + patch] = (float)pair[q * np + patch];
        }
        if (pos_sim)
            for (int64_t p = 0; p < P; ++p)
                pos_sim[q * P + p] = (float)ocr_cosine(x, L->dtype, (fa * P + p) * C, (fb * P + p) * C, C, L->eps);
    }
    for (int64_t b = 0; b < L->B; ++b)
        for (int64_t t = 0; t < T; ++t)
            for (int64_t patch = 0; patch < np; ++patch) {
                int64_t i = (b * T + t) * np + patch;
                if (t % 2 == 0) { best_sim[i] = -INFINITY; best_idx[i] = (int32_t)i; continue; }
                double best = pair[(b * (T - 1) + (t - 1)) * np + patch]; int64_t arg = i - np;   /* (t, t-1) */
                if (t + 1 < T) {
                    double nxt = pair[(b * (T - 1) + t) * np + patch];                             /* (t+1, t) */
                    if (nxt > best) { best = nxt; arg = i + np; }
                }
                best_sim[i] = (float)best; best_idx[i] = (int32_t)arg;
            }
    free(pair);
    return 0;
}

/* ---- O4: Block Cache match -----------------------------------------------------------------
 * The descriptor of spatial position p is the concatenation over t of x[b,t,p,:] (length T*C,
 * Section 3.2.1's (B, H*W, T*C) reshape).  Positions are partitioned into sy x sx neighbourhoods;
 * the (oy, ox) member is the representative, every other member is compared with it. */
int ocr_match_block(const ocr_layout* L, const void* x, float* best_sim, int32_t* best_idx) {
    if (L->kind != 2) return 1;
    if (L->gy <= 0 || L->gx <= 0 || L->H % (L->gy * L->sy) || L->W % (L->gx * L->sx)) return 1;
    const int64_t T = L->T, H = L->H, W = L->W, C = L->C, P = H * W;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t i = 0; i < (int64_t)L->B * P; ++i) {
        int64_t b = i / P, p = i % P, y = p / W, xx = p % W;
        if ((y % L->sy) == L->oy && (xx % L->sx) == L->ox) {
            best_sim[i] = -INFINITY; best_idx[i] = (int32_t)i; continue;
        }
        int64_t ry = y - (y % L->sy) + L->oy, rx = xx - (xx % L->sx) + L->ox, rp = ry * W + rx;
        double dot = 0.0, na = 0.0, nb = 0.0;
        for (int64_t t = 0; t < T; ++t)
            for (int64_t c = 0; c < C; ++c) {
                double a = load_elem(x, L->dtype, ((b * T + t) * P + p) * C + c);
                double r = load_elem(x, L->dtype, ((b * T + t) * P + rp) * C + c);
                dot += a * r; na += a * a; nb += r * r;
            }
        na = sqrt(na); nb = sqrt(nb);
        if (na < L->eps) na = L->eps;
        if (nb < L->eps) nb = L->eps;
        best_sim[i] = (float)clamp1(dot / (na * nb));
        best_idx[i] = (int32_t)(b * P + rp);
    }
    return 0;
}

/* ---- O5: selection -------------------------------------------------------------------------
 * Representatives are always kept.  mode 0 (threshold): a candidate is reused iff its fp32
 * best_sim >= thr (self-match: and its best match has a lower index; match_map then follows
 * best_idx down to a kept token).  mode 1 (count): the n_reuse candidates of each group with the
 * largest best_sim are reused, equal values broken towards the lower index ("the r most redundant",
 * Sections 3.2.1-3.2.3).  Kept units are listed in ascending original index (order preserving, no
 * averaging).  kept_idx: [group][y_group_stride] global unit indices, unused tail = -1;
 * slot_of[i] = g*y_group_stride + position for kept i, -1 for reused i; match_map[i] = i if kept,
 * else the representative whose cache position/row stands for it. */
typedef struct { float sim; int64_t u; } ocr_rank;
static int rank_cmp(const void* pa, const void* pb) {
    const ocr_rank* a = (const ocr_rank*)pa; const ocr_rank* b = (const ocr_rank*)pb;
    if (a->sim > b->sim) return -1;
    if (a->sim < b->sim) return 1;
    return (a->u > b->u) - (a->u < b->u);
}

int ocr_select(const ocr_layout* L, const float* best_sim, const int32_t* best_idx, int mode,
               float thr, int64_t n_reuse, int64_t y_group_stride, int32_t* kept_idx,
               int32_t* kept_count, int32_t* match_map, int32_t* slot_of) {
    const int64_t G = ocr_num_groups(L), U = ocr_units_per_group(L);
    if (mode == 1 && L->kind == 0 && L->self_match) return 1;
    uint8_t* reuse = (uint8_t*)calloc((size_t)(G * U > 0 ? G * U : 1), 1);  /* by global unit index */
    ocr_rank* rk = (ocr_rank*)malloc(sizeof(ocr_rank) * (size_t)(U > 0 ? U : 1));
    if (!reuse || !rk) { free(reuse); free(rk); return 2; }
    for (int64_t g = 0; g < G; ++g) {
        if (mode == 0) {
            for (int64_t u = 0; u < U; ++u) {
                int64_t i = ocr_unit_index(L, g, u);
                if (!is_cand(L, u)) continue;
                int r = best_sim[i] >= thr;
                if (L->kind == 0 && L->self_match) r = r && (best_idx[i] < i);
                reuse[i] = (uint8_t)r;
            }
        } else {
            int64_t n = 0;
            for (int64_t u = 0; u < U; ++u)
                if (is_cand(L, u)) { rk[n].sim = best_sim[ocr_unit_index(L, g, u)]; rk[n].u = u; ++n; }
            qsort(rk, (size_t)n, sizeof(ocr_rank), rank_cmp);
            int64_t m = n_reuse < n ? n_reuse : n;
            for (int64_t k = 0; k < m; ++k) reuse[ocr_unit_index(L, g, rk[k].u)] = 1;
        }
        int64_t pos = 0;
        for (int64_t u = 0; u < U; ++u) {
            int64_t i = ocr_unit_index(L, g, u);
            if (reuse[i]) { slot_of[i] = -1; continue; }
            if (pos >= y_group_stride) { free(reuse); free(rk); return 3; }
            kept_idx[g * y_group_stride + pos] = (int32_t)i;
            slot_of[i] = (int32_t)(g * y_group_stride + pos);
            ++pos;
        }
        kept_count[g] = (int32_t)pos;
        for (int64_t s = pos; s < y_group_stride; ++s) kept_idx[g * y_group_stride + s] = -1;
    }
    for (int64_t g = 0; g < G; ++g)
        for (int64_t u = 0; u < U; ++u) {
            int64_t i = ocr_unit_index(L, g, u);
            int64_t m = i;
            while (reuse[m]) m = best_idx[m];          /* self-match chains strictly decrease */
            match_map[i] = (int32_t)m;
        }
    free(reuse); free(rk);
    return 0;
}

/* ---- O5b: Token Cache on the frame pairs of Frame Cache (Section 3.2.3) -----------------------
 * "Token Cache consumes the same feature map and frame-pair metadata used by Frame Cache ... For
 * frame pairs selected by Frame Cache, we reshape the paired features from (B, 2 r_f, H, W, C) to
 * (B r_f, 2HW, C).  Within each local 2x2x2 cube, Token Cache retains representative tokens ...
 * For unmatched frames, the same procedure is applied within local 2x2 spatial neighborhoods."
 *
 * Reading (the paper fixes neither the cube's representative nor what happens when two candidate
 * frames pick the same representative frame):
 *   - a candidate frame t that Frame Cache marked for reuse claims its matched representative
 *     frame u = frame_best_idx[t]; if both neighbours of u claim it, the one with the larger frame
 *     similarity wins (equal: the earlier frame), the other stays unmatched;
 *   - a pair (u, t) is ONE token group of 2HW tokens: the lattice tokens of frame u are its
 *     representatives (one per 2x2x2 cube: the cube's (oy, ox) member in the representative
 *     frame), the other 3HW/4 tokens of u and ALL HW tokens of t are candidates, each compared
 *     with all representatives of the group;
 *   - every other frame is a group of its own with the usual lattice (unmatched frames).
 * frames[f] = (u, t) for slot f: (f, partner) if f is the representative frame of a pair,
 * (f, -1) if f is a group of its own, (-1, -1) if f was absorbed into its partner's group.
 * Units of a pair are ordered by time: the earlier frame's tokens first. */
int ocr_joint_groups(int B, int T, const float* frame_best_sim, const int32_t* frame_best_idx,
                     const int32_t* frame_slot_of, int32_t* frames) {
    for (int64_t f = 0; f < (int64_t)B * T; ++f) { frames[2 * f] = (int32_t)f; frames[2 * f + 1] = -1; }
    for (int b = 0; b < B; ++b)
        for (int u = 0; u < T; u += 2) {                       /* representative frames */
            int64_t fu = (int64_t)b * T + u, win = -1;
            for (int d = -1; d <= 1; d += 2) {
                int t = u + d;
                if (t < 0 || t >= T) continue;
                int64_t ft = (int64_t)b * T + t;
                if (frame_slot_of[ft] >= 0 || frame_best_idx[ft] != fu) continue;   /* not reused / matched elsewhere */
                if (win < 0 || frame_best_sim[ft] > frame_best_sim[win]) win = ft;  /* equal: the earlier one stays */
            }
            if (win >= 0) { frames[2 * fu + 1] = (int32_t)win; frames[2 * win] = -1; frames[2 * win + 1] = -1; }
        }
    return 0;
}

/* is token i (frame f = i / HW) a representative of its joint group? */
static int joint_is_rep(const ocr_layout* L, const int32_t* frames, int64_t i) {
    int64_t P = (int64_t)L->H * L->W, f = i / P, p = i % P, y = p / L->W, xx = p % L->W;
    if (frames[2 * f] < 0) return 0;                            /* absorbed frame: all candidates */
    return (y % L->sy) == L->oy && (xx % L->sx) == L->ox;
}

int ocr_match_joint(const ocr_layout* L, const void* x, const int32_t* frames, float* best_sim,
                    int32_t* best_idx, float* second_sim) {
    if (L->kind != 0 || L->gy != 1 || L->gx != 1 || L->self_match) return 1;
    const int64_t P = (int64_t)L->H * L->W, F = (int64_t)L->B * L->T, C = L->C;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t slot = 0; slot < F; ++slot) {
        int64_t u = frames[2 * slot], t = frames[2 * slot + 1];
        if (u < 0) continue;
        for (int half = 0; half < 2; ++half) {
            int64_t f = half ? t : u;
            if (f < 0) continue;
            for (int64_t p = 0; p < P; ++p) {
                int64_t i = f * P + p;
                if (joint_is_rep(L, frames, i)) {
                    best_sim[i] = -INFINITY; best_idx[i] = (int32_t)i;
                    if (second_sim) second_sim[i] = -INFINITY;
                    continue;
                }
                double best = -INFINITY, second = -INFINITY; int64_t arg = i;
                for (int64_t r = 0; r < P; ++r) {             /* representatives: the lattice of frame u */
                    int64_t j = u * P + r;
                    if (!joint_is_rep(L, frames, j)) continue;
                    double s = ocr_cosine(x, L->dtype, i * C, j * C, C, L->eps);
                    if (s > best) { second = best; best = s; arg = j; }
                    else if (s > second) second = s;
                }
                best_sim[i] = (float)best; best_idx[i] = (int32_t)arg;
                if (second_sim) second_sim[i] = (float)second;
            }
        }
    }
    return 0;
}

/* Selection over the joint groups: as ocr_select, the group of slot f being the tokens of its one
 * or two frames in time order.  n_reuse_pair / n_reuse_single: count-mode budgets of a pair group
 * and of a single-frame group.  kept_idx: [B*T slots][y_group_stride]; absorbed slots keep nothing. */
int ocr_select_joint(const ocr_layout* L, const int32_t* frames, const float* best_sim,
                     const int32_t* best_idx, int mode, float thr, int64_t n_reuse_pair,
                     int64_t n_reuse_single, int64_t y_group_stride, int32_t* kept_idx,
                     int32_t* kept_count, int32_t* match_map, int32_t* slot_of) {
    if (L->kind != 0 || L->gy != 1 || L->gx != 1 || L->self_match) return 1;
    const int64_t P = (int64_t)L->H * L->W, F = (int64_t)L->B * L->T;
    uint8_t* reuse = (uint8_t*)calloc((size_t)(F * P > 0 ? F * P : 1), 1);
    ocr_rank* rk = (ocr_rank*)malloc(sizeof(ocr_rank) * (size_t)(2 * P > 0 ? 2 * P : 1));
    int64_t* unit = (int64_t*)malloc(sizeof(int64_t) * (size_t)(2 * P > 0 ? 2 * P : 1));
    if (!reuse || !rk || !unit) { free(reuse); free(rk); free(unit); return 2; }
    for (int64_t slot = 0; slot < F; ++slot) {
        int64_t u = frames[2 * slot], t = frames[2 * slot + 1];
        for (int64_t s = 0; s < y_group_stride; ++s) kept_idx[slot * y_group_stride + s] = -1;
        kept_count[slot] = 0;
        if (u < 0) continue;
        /* the group's tokens in time order */
        int64_t n = 0, f0 = (t >= 0 && t < u) ? t : u, f1 = (t >= 0 && t < u) ? u : t;
        for (int64_t p = 0; p < P; ++p) unit[n++] = f0 * P + p;
        if (f1 >= 0) for (int64_t p = 0; p < P; ++p) unit[n++] = f1 * P + p;
        if (mode == 0) {
            for (int64_t k = 0; k < n; ++k)
                if (!joint_is_rep(L, frames, unit[k])) reuse[unit[k]] = best_sim[unit[k]] >= thr;
        } else {
            int64_t m = 0;
            for (int64_t k = 0; k < n; ++k)
                if (!joint_is_rep(L, frames, unit[k])) { rk[m].sim = best_sim[unit[k]]; rk[m].u = k; ++m; }
            qsort(rk, (size_t)m, sizeof(ocr_rank), rank_cmp);
            int64_t want = t >= 0 ? n_reuse_pair : n_reuse_single;
            if (want > m) want = m;
            for (int64_t k = 0; k < want; ++k) reuse[unit[rk[k].u]] = 1;
        }
        int64_t pos = 0;
        for (int64_t k = 0; k < n; ++k) {
            int64_t i = unit[k];
            if (reuse[i]) { slot_of[i] = -1; match_map[i] = best_idx[i]; continue; }
            if (pos >= y_group_stride) { free(reuse); free(rk); free(unit); return 3; }
            kept_idx[slot * y_group_stride + pos] = (int32_t)i;
            slot_of[i] = (int32_t)(slot * y_group_stride + pos);
            match_map[i] = (int32_t)i;
            ++pos;
        }
        kept_count[slot] = (int32_t)pos;
    }
    free(reuse); free(rk); free(unit);
    return 0;
}

/* ---- rows of a strided tensor --------------------------------------------------------------
 * A unit's row is n_seg segments of seg_bytes; segment s of unit i starts at byte
 *   (i / units_per_outer) * outer_pitch + (i % units_per_outer) * unit_pitch + s * seg_stride.
 * Tokens and frames: one contiguous segment.  A 1x1xT block in a [B,T,H,W,C] tensor: T segments of
 * C elements, seg_stride = H*W*C elements, outer = batch element.  The dense side is packed
 * [row][segment][seg_bytes]. */
typedef struct {
    int64_t seg_bytes, n_seg, seg_stride, unit_pitch, units_per_outer, outer_pitch;
} ocr_rows;

static const uint8_t* row_seg_c(const ocr_rows* R, const void* base, int64_t i, int64_t s) {
    return (const uint8_t*)base + (i / R->units_per_outer) * R->outer_pitch
           + (i % R->units_per_outer) * R->unit_pitch + s * R->seg_stride;
}
static uint8_t* row_seg(const ocr_rows* R, void* base, int64_t i, int64_t s) {
    return (uint8_t*)base + (i / R->units_per_outer) * R->outer_pitch
           + (i % R->units_per_outer) * R->unit_pitch + s * R->seg_stride;
}

/* ---- O6: gather: y[slot] = x[kept_idx[slot]] for every slot whose index is >= 0 ------------- */
int ocr_gather(const ocr_rows* R, const void* x, const int32_t* kept_idx, int64_t n_slots, void* y) {
    const int64_t row_bytes = R->seg_bytes * R->n_seg;
    for (int64_t r = 0; r < n_slots; ++r) {
        if (kept_idx[r] < 0) continue;
        for (int64_t s = 0; s < R->n_seg; ++s)
            memcpy((uint8_t*)y + r * row_bytes + s * R->seg_bytes, row_seg_c(R, x, kept_idx[r], s),
                   (size_t)R->seg_bytes);
    }
    return 0;
}

/* ---- O7: restore ---------------------------------------------------------------------------
 * out[i] = z[slot_of[i]] for computed units; for skipped units, src_mode 0: out[i] = cache[i]
 * (the activation cached at the same position, Sections 3.2.1-3.2.3), src_mode 1:
 * out[i] = z[slot_of[match_map[i]]] (cold start: the matched representative's fresh row).
 * Every output row is a bit copy of exactly one source row.  out == cache: skipped rows untouched. */
int ocr_restore(const ocr_rows* R, const void* z, const void* cache, int64_t n_units,
                const int32_t* slot_of, const int32_t* match_map, void* out, int src_mode) {
    const int64_t row_bytes = R->seg_bytes * R->n_seg;
    for (int64_t i = 0; i < n_units; ++i) {
        int64_t slot = slot_of[i];
        if (slot < 0 && src_mode == 1) slot = slot_of[match_map[i]];
        for (int64_t s = 0; s < R->n_seg; ++s) {
            uint8_t* dst = row_seg(R, out, i, s);
            if (slot >= 0) memcpy(dst, (const uint8_t*)z + slot * row_bytes + s * R->seg_bytes, (size_t)R->seg_bytes);
            else if (out != cache) memcpy(dst, row_seg_c(R, cache, i, s), (size_t)R->seg_bytes);
        }
    }
    return 0;
}

/* ---- O8: Layered Cache reuse rule (Section 3.4, Algorithm 1's (l, t, N) triples) -------------
 * An output stored at step s0 is reused at step s iff 0 <= s - s0 < N. */
int ocr_layer_cache_hit(int stored_step, int step, int interval) {
    int d = step - stored_step;
    return d >= 0 && d < interval;
}
