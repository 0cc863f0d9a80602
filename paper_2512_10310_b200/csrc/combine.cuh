// Split-reduction combine kernel: merges the per-split partial outputs of the step attention.
//
//   M = max_s lse_s,  w_s = e^{lse_s - M},  O = sum_s w_s O_s / sum_s w_s,  lse = M + log sum_s w_s
//
// One warp per packed query row: lane s holds lse_s (at most 32 splits), the maximum and the
// weight sum are warp-shuffle reductions, then each lane merges D/32 contiguous channels with
// vector loads.  The row is rounded once to the storage dtype and written to its place in the
// token-major [n, Hq, D] output.  HBM/L2-bound: S*(D+1) floats in, D elements out per row.
#pragma once

#include "common.cuh"

namespace evln {

struct CombineArgs {
    const float* o_part;     // [S, Hkv, R, D]
    const float* lse_part;   // [S, Hkv, R]
    void* out;               // [n, Hq, D]
    float* lse_out;          // [n, Hq] or null
    int Hkv, G, D;
    int rows;                // R = (total) new tokens * G
    int num_splits;          // contiguous: S for every row
    // batches: per-episode split counts are derived from the lengths
    int batch, unit_rows, chunk_tiles;
    int tail;                // batch of items sharing a cache prefix (own tokens tiled separately)
    FastDiv div_g;           // division by G, by the work-item size in KV tiles (chunk_tiles, at least 1):
    FastDiv div_chunk;       //   a row's warp decodes its place with multiplications (an integer division costs
                             //   as much as the rest of the merge)
    PackedMap map;           // where output token m goes (identity unless the call serves a packed sequence)
};

template <typename T, int D, bool PAGED, typename LensT>
__global__ void __launch_bounds__(128)
combine_kernel(const CombineArgs a, const __grid_constant__ LensT lens)
{
    constexpr int C = D / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t row = blockIdx.x * 4u + (uint32_t)warp;      // packed row within kv head (< 2^24, checked on the host)
    const int g = blockIdx.y;
    if (row >= (uint32_t)a.rows) return;
    const uint32_t row_tok = fast_div(row, a.div_g);            // its token among the call's new tokens ...
    const int row_head = (int)(row - row_tok * (uint32_t)a.G);  // ... and its query head within the group

    int S = a.num_splits;
    if (PAGED) {
        const int tok = (int)row_tok;
        int lo = 0, hi = a.batch;
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (lens.new_off[mid] <= tok) lo = mid; else hi = mid;
        }
        const int b = lo;
        const int n_b = lens.new_off[b + 1] - lens.new_off[b];
        const int local_row = (int)row - lens.new_off[b] * a.G;
        const int unit = local_row / kUnitRows;                  // (a power of two)
        const int nkv = a.tail ? tail_kv_tiles_fast(lens.cache_len[b], n_b, a.div_g, unit, kUnitRows)
                               : unit_kv_tiles_fast(lens.cache_len[b], n_b, a.div_g, unit, kUnitRows);
        S = (int)fast_div((uint32_t)(nkv + a.chunk_tiles - 1), a.div_chunk);
    }

    const long stride_s = (long)a.Hkv * a.rows;           // rows between consecutive splits
    const long prow0 = (long)g * a.rows + row;
    // (so far launch parameters only: a row's warp knows its place before the partials exist)
    asm volatile("griddepcontrol.wait;" ::: "memory");          // programmatic dependent launch: inputs ready
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    constexpr int kPre = 4;
    // (Letting every lane read all log-sum-exps of a row with few splits, so that the maximum and
    // the weights need no shuffles, was measured slower: 3.85 against 3.45 us at the 7B step.)
    float my_lse = (lane < S) ? a.lse_part[prow0 + lane * stride_s] : -INFINITY;
    // the first partial rows do not depend on the weights: their loads go out with the lse load
    float pre[kPre][C];
#pragma unroll
    for (int s = 0; s < kPre; ++s) {
        if (s < S) {
            const float* op = a.o_part + (prow0 + s * stride_s) * D + lane * C;
            if (C == 4) {
                float4 x = *reinterpret_cast<const float4*>(op);
                pre[s][0] = x.x; pre[s][1] = x.y; pre[s][2] = x.z; pre[s][3] = x.w;
            } else {
#pragma unroll
                for (int c = 0; c < C; ++c) pre[s][c] = op[c];
            }
        } else {
#pragma unroll
            for (int c = 0; c < C; ++c) pre[s][c] = 0.f;
        }
    }
    float M = my_lse;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
    float w = (my_lse == -INFINITY) ? 0.f : expf(my_lse - M);    // M = -inf only if all are
    float wsum = w;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) wsum += __shfl_xor_sync(0xffffffffu, wsum, off);

    float acc[C];
#pragma unroll
    for (int c = 0; c < C; ++c) acc[c] = 0.f;
#pragma unroll
    for (int s = 0; s < kPre; ++s) {
        const float ws = __shfl_sync(0xffffffffu, w, s);      // 0 for s >= S and for empty splits
#pragma unroll
        for (int c = 0; c < C; ++c) acc[c] = fmaf(ws, pre[s][c], acc[c]);
    }
    // the remaining splits four at a time: their loads are in flight together, the sums keep the
    // order of the splits
    constexpr int kBatch = 8;
    for (int s0 = kPre; s0 < S; s0 += kBatch) {
        float v[kBatch][C];
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
            const int s = s0 + k;
            if (s < S) {
                const float* op = a.o_part + (prow0 + s * stride_s) * D + lane * C;
                if (C == 4) {
                    float4 x = *reinterpret_cast<const float4*>(op);
                    v[k][0] = x.x; v[k][1] = x.y; v[k][2] = x.z; v[k][3] = x.w;
                } else {
#pragma unroll
                    for (int c = 0; c < C; ++c) v[k][c] = op[c];
                }
            } else {
#pragma unroll
                for (int c = 0; c < C; ++c) v[k][c] = 0.f;
            }
        }
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
            const float ws = (s0 + k < S) ? __shfl_sync(0xffffffffu, w, s0 + k) : 0.f;   // 0 for empty splits too
            if (ws != 0.f) {                                                            // uniform across the warp
#pragma unroll
                for (int c = 0; c < C; ++c) acc[c] = fmaf(ws, v[k][c], acc[c]);
            }
        }
    }
    const float inv = (wsum > 0.f) ? 1.f / wsum : 0.f;

    const long tok = packed_row(a.map, (long)row_tok);
    const int h = g * a.G + row_head;
    const int Hq = a.Hkv * a.G;
    T* dst = (T*)a.out + (tok * Hq + h) * D + lane * C;
#pragma unroll
    for (int c = 0; c < C; ++c) from_float(acc[c] * inv, dst[c]);
    if (a.lse_out && lane == 0) a.lse_out[tok * Hq + h] = (wsum > 0.f) ? M + logf(wsum) : -INFINITY;
}

}  // namespace evln
