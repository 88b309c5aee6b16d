// gather / restore / copy: the bandwidth-bound row movers (Appendix A's compaction of the kept rows
// and its permutation/scatter back into place, written gather-style so that every output row has
// one writer).
//
// All three are flat over 16-byte chunks: a thread moves UNROLL independent chunks (all loads issued
// before the first store), consecutive threads touch consecutive chunks, so a warp reads and writes
// whole 512-byte runs of a row.  Index arrays are read through the L1/L2 path once per chunk (they
// are tiny and hit); feature rows are streamed with no-allocate loads.
#include "common.cuh"

namespace oc {

static constexpr int MOVE_THREADS = 256;
static constexpr int MOVE_UNROLL = 4;

struct RowsDev {
    long long seg_bytes, seg_stride, unit_pitch, outer_pitch;
    unsigned n_seg, units_per_outer;   // units_per_outer == 0 : no outer split
    unsigned cps;                      // 16-byte chunks per segment
    unsigned cpr;                      // 16-byte chunks per row
};

static RowsDev make_rows_dev(const oc_rows& r) {
    RowsDev d;
    d.seg_bytes = r.seg_bytes; d.seg_stride = r.seg_stride; d.unit_pitch = r.unit_pitch;
    d.outer_pitch = r.outer_pitch;
    d.n_seg = (unsigned)r.n_seg;
    d.units_per_outer = (r.outer_pitch == 0 || r.units_per_outer > 0x7FFFFFFFll) ? 0u : (unsigned)r.units_per_outer;
    d.cps = (unsigned)(r.seg_bytes / 16);
    d.cpr = d.cps * d.n_seg;
    return d;
}

// byte offset of chunk `col` of unit `unit` inside the strided tensor
template <bool SEG>
__device__ __forceinline__ long long strided_offset(const RowsDev& R, unsigned unit, unsigned col) {
    if (!SEG) return (long long)unit * R.unit_pitch + (long long)col * 16;
    unsigned seg = col / R.cps, off = col - seg * R.cps;
    long long base;
    if (R.units_per_outer) {
        unsigned o = unit / R.units_per_outer, in = unit - o * R.units_per_outer;
        base = (long long)o * R.outer_pitch + (long long)in * R.unit_pitch;
    } else {
        base = (long long)unit * R.unit_pitch;
    }
    return base + (long long)seg * R.seg_stride + (long long)off * 16;
}

template <bool SEG>
__global__ void __launch_bounds__(MOVE_THREADS)
gather_kernel(const uint8_t* __restrict__ x, const int32_t* __restrict__ kept_idx,
              uint8_t* __restrict__ y, unsigned total_chunks, RowsDev R) {
    pdl_enter();
    const unsigned base = blockIdx.x * (MOVE_THREADS * MOVE_UNROLL) + threadIdx.x;
    uint4 v[MOVE_UNROLL];
    bool ok[MOVE_UNROLL];
#pragma unroll
    for (int k = 0; k < MOVE_UNROLL; ++k) {
        unsigned c = base + k * MOVE_THREADS;
        ok[k] = false;
        if (c < total_chunks) {
            unsigned slot = c / R.cpr, col = c - slot * R.cpr;
            int unit = __ldg(kept_idx + slot);
            if (unit >= 0) {
                ok[k] = true;
                v[k] = ld_nc_v4(x + strided_offset<SEG>(R, (unsigned)unit, col));
            }
        }
    }
#pragma unroll
    for (int k = 0; k < MOVE_UNROLL; ++k) {
        unsigned c = base + k * MOVE_THREADS;
        if (ok[k]) st_v4(y + (long long)c * 16, v[k]);
    }
}

// MODE 0: skipped rows from cache; 1: skipped rows from the representative's z row; 2: in place
// (skipped rows untouched).  slot_of / match_map / cache / out are this launch's slice of the units;
// slot_of_all is the whole array, which MODE 1 indexes with the (global) unit a match_map entry names.
template <bool SEG, int MODE>
__global__ void __launch_bounds__(MOVE_THREADS)
restore_kernel(const uint8_t* __restrict__ z, const uint8_t* __restrict__ cache,
               const int32_t* __restrict__ slot_of, const int32_t* __restrict__ match_map,
               const int32_t* __restrict__ slot_of_all,
               uint8_t* __restrict__ out, unsigned total_chunks, RowsDev R) {
    pdl_enter();
    const unsigned base = blockIdx.x * (MOVE_THREADS * MOVE_UNROLL) + threadIdx.x;
    uint4 v[MOVE_UNROLL];
    long long dst[MOVE_UNROLL];
#pragma unroll
    for (int k = 0; k < MOVE_UNROLL; ++k) {
        unsigned c = base + k * MOVE_THREADS;
        dst[k] = -1;
        if (c < total_chunks) {
            unsigned unit = c / R.cpr, col = c - unit * R.cpr;
            int slot = __ldg(slot_of + unit);
            if (MODE == 1 && slot < 0) slot = __ldg(slot_of_all + __ldg(match_map + unit));
            long long off = strided_offset<SEG>(R, unit, col);
            if (slot >= 0) {
                v[k] = ld_nc_v4(z + ((long long)slot * R.cpr + col) * 16);
                dst[k] = off;
            } else if (MODE == 0) {
                v[k] = ld_nc_v4(cache + off);
                dst[k] = off;
            }
        }
    }
#pragma unroll
    for (int k = 0; k < MOVE_UNROLL; ++k)
        if (dst[k] >= 0) st_v4(out + dst[k], v[k]);
}

__global__ void __launch_bounds__(MOVE_THREADS)
copy_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, unsigned long long n_chunks,
            unsigned long long tail_begin, unsigned tail_bytes) {
    pdl_enter();
    const unsigned long long base = (unsigned long long)blockIdx.x * (MOVE_THREADS * MOVE_UNROLL) + threadIdx.x;
    uint4 v[MOVE_UNROLL];
#pragma unroll
    for (int k = 0; k < MOVE_UNROLL; ++k) {
        unsigned long long c = base + (unsigned long long)k * MOVE_THREADS;
        if (c < n_chunks) v[k] = ld_nc_v4(src + c * 16);
    }
#pragma unroll
    for (int k = 0; k < MOVE_UNROLL; ++k) {
        unsigned long long c = base + (unsigned long long)k * MOVE_THREADS;
        if (c < n_chunks) st_v4(dst + c * 16, v[k]);
    }
    if (blockIdx.x == 0 && threadIdx.x < tail_bytes) dst[tail_begin + threadIdx.x] = src[tail_begin + threadIdx.x];
}

// Rows are processed in launches of fewer than 2^31 chunks so that chunk arithmetic stays 32-bit.
static constexpr unsigned long long MAX_CHUNKS_PER_LAUNCH = 1ull << 31;

oc_status launch_gather(oc_ctx* ctx, const oc_rows& rows, const void* x, const int32_t* kept_idx,
                        int64_t n_slots, void* y, cudaStream_t s) {
    if (n_slots == 0) return OC_OK;
    RowsDev R = make_rows_dev(rows);
    const bool seg = R.n_seg > 1 || R.units_per_outer != 0;
    int64_t slots_per_launch = (int64_t)(MAX_CHUNKS_PER_LAUNCH / R.cpr);
    if (slots_per_launch < 1) return OC_ERR_UNSUPPORTED;
    for (int64_t s0 = 0; s0 < n_slots; s0 += slots_per_launch) {
        int64_t ns = n_slots - s0 < slots_per_launch ? n_slots - s0 : slots_per_launch;
        unsigned total = (unsigned)(ns * R.cpr);
        unsigned blocks = (total + MOVE_THREADS * MOVE_UNROLL - 1) / (MOVE_THREADS * MOVE_UNROLL);
        uint8_t* yy = (uint8_t*)y + s0 * (int64_t)R.cpr * 16;
        LaunchScope scope(ctx, OC_K_GATHER, s);
        if (seg) OC_LAUNCH(gather_kernel<true>, blocks, MOVE_THREADS, 0, s, (const uint8_t*)x, kept_idx + s0, yy, total, R);
        else     OC_LAUNCH(gather_kernel<false>, blocks, MOVE_THREADS, 0, s, (const uint8_t*)x, kept_idx + s0, yy, total, R);
    }
    return last_launch_status();
}

template <bool SEG>
static void restore_dispatch(int mode, unsigned blocks, cudaStream_t s, const uint8_t* z, const uint8_t* cache,
                             const int32_t* slot_of, const int32_t* match_map, const int32_t* slot_of_all, uint8_t* out,
                             unsigned total, const RowsDev& R) {
    if (mode == 0) OC_LAUNCH((restore_kernel<SEG, 0>), blocks, MOVE_THREADS, 0, s, z, cache, slot_of, match_map, slot_of_all, out, total, R);
    else if (mode == 1) OC_LAUNCH((restore_kernel<SEG, 1>), blocks, MOVE_THREADS, 0, s, z, cache, slot_of, match_map, slot_of_all, out, total, R);
    else OC_LAUNCH((restore_kernel<SEG, 2>), blocks, MOVE_THREADS, 0, s, z, cache, slot_of, match_map, slot_of_all, out, total, R);
}

oc_status launch_restore(oc_ctx* ctx, const oc_rows& rows, const void* z, const void* cache,
                         int64_t n_units, const int32_t* slot_of, const int32_t* match_map, void* out,
                         int src_mode, cudaStream_t s) {
    if (n_units == 0) return OC_OK;
    RowsDev R = make_rows_dev(rows);
    const bool seg = R.n_seg > 1 || R.units_per_outer != 0;
    int mode = src_mode == OC_RESTORE_FROM_REPRESENTATIVE ? 1 : (out == cache ? 2 : 0);
    int64_t units_per_launch = (int64_t)(MAX_CHUNKS_PER_LAUNCH / R.cpr);
    if (units_per_launch < 1) return OC_ERR_UNSUPPORTED;
    if (n_units > units_per_launch && seg) return OC_ERR_UNSUPPORTED;   // segmented rows: one launch only
    for (int64_t u0 = 0; u0 < n_units; u0 += units_per_launch) {
        int64_t nu = n_units - u0 < units_per_launch ? n_units - u0 : units_per_launch;
        unsigned total = (unsigned)(nu * R.cpr);
        unsigned blocks = (total + MOVE_THREADS * MOVE_UNROLL - 1) / (MOVE_THREADS * MOVE_UNROLL);
        // contiguous rows: shifting the strided base by u0 rows keeps unit indices launch-local
        const uint8_t* cc = cache ? (const uint8_t*)cache + u0 * R.unit_pitch : nullptr;
        uint8_t* oo = (uint8_t*)out + u0 * R.unit_pitch;
        LaunchScope scope(ctx, OC_K_RESTORE, s);
        if (seg) restore_dispatch<true>(mode, blocks, s, (const uint8_t*)z, cc, slot_of + u0, match_map + u0, slot_of, oo, total, R);
        else     restore_dispatch<false>(mode, blocks, s, (const uint8_t*)z, cc, slot_of + u0, match_map + u0, slot_of, oo, total, R);
    }
    return last_launch_status();
}

oc_status launch_copy(oc_ctx* ctx, const void* src, void* dst, size_t bytes, cudaStream_t s) {
    if (bytes == 0) return OC_OK;
    const bool aligned = (((uintptr_t)src | (uintptr_t)dst) & 15u) == 0;
    unsigned long long n_chunks = aligned ? bytes / 16 : 0;
    unsigned long long tail_begin = n_chunks * 16;
    size_t tail = bytes - tail_begin;
    if (tail >= (size_t)MOVE_THREADS) return OC_ERR_ALIGNMENT;          // unaligned bulk is not supported
    unsigned long long per_block = MOVE_THREADS * MOVE_UNROLL;
    unsigned long long blocks = (n_chunks + per_block - 1) / per_block;
    if (blocks == 0) blocks = 1;
    if (blocks > 0x7FFFFFFFull) return OC_ERR_UNSUPPORTED;
    LaunchScope scope(ctx, OC_K_COPY, s);
    OC_LAUNCH(copy_kernel, (unsigned)blocks, MOVE_THREADS, 0, s, (const uint8_t*)src, (uint8_t*)dst, n_chunks, tail_begin, (unsigned)tail);
    return last_launch_status();
}

}  // namespace oc
