// Re-indexing of an un-rotated cache (Sec. 3.2: the KV cache is stored before the rotation, the
// frame sampler picks the frames to keep, the kept tokens get contiguous position ids and RoPE is
// applied on the fly).
//
// store_append_kernel: the new frame's raw (un-rotated) K and V go to the store, head-major.
// gather_rope_kernel: the kept segments of the store are laid out back to back in a working cache;
// the token that lands in working slot p is rotated at position p (keys) or copied (values).  One
// CTA per destination token; angles in double precision as in the append kernel (or from the
// caller's position table).  HBM-bound: every
// kept element is read once and written once with 128-bit accesses.
#pragma once

#include "common.cuh"
#include "rope_append.cuh"

namespace evln {

constexpr int kMaxSegments = 256;

// Kept segments, passed by value: segment s = store slots [src[s], src[s] + dst_off[s+1] - dst_off[s])
// -> working slots [dst_off[s], dst_off[s+1]).
struct SegList {
    int src[kMaxSegments];
    int dst_off[kMaxSegments + 1];
};

struct GatherArgs {
    const void* k_src;      // store_append: k_new [n, Hkv, D] (token stride given); gather: store [Hkv, store_cap, D]
    const void* v_src;
    void* k_dst;            // store_append: store; gather: working cache [Hkv, work_cap, D]
    void* v_dst;
    long k_stride, v_stride;    // store_append only: token strides of k_new / v_new in elements
    int Hkv, D;
    int src_cap, dst_cap;
    int first_slot;         // store_append: first store slot written
    int num_tokens;         // destination tokens
    int num_segments;       // gather only
    double log2_theta;      // gather only
    const double2* table;   // gather only, optional: (cos, sin) per (position - table_first, j)
    int table_first;
};

template <typename T>
__global__ void __launch_bounds__(128)
store_append_kernel(const GatherArgs a)
{
    constexpr int V = VecTraits<T>::kVec;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int tok = blockIdx.x;
    const int per_row = a.D / V;
    const int items = 2 * a.Hkv * per_row;
    for (int it = threadIdx.x; it < items; it += blockDim.x) {
        const bool is_v = it >= a.Hkv * per_row;
        const int e = is_v ? it - a.Hkv * per_row : it;
        const int g = e / per_row, d0 = (e % per_row) * V;
        const T* src = (const T*)(is_v ? a.v_src : a.k_src) + (long)tok * (is_v ? a.v_stride : a.k_stride) + (long)g * a.D + d0;
        T* dst = (T*)(is_v ? a.v_dst : a.k_dst) + ((long)g * a.dst_cap + a.first_slot + tok) * a.D + d0;
        *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
    }
}

template <typename T>
__global__ void __launch_bounds__(128)
gather_rope_kernel(const GatherArgs a, const __grid_constant__ SegList segs)
{
    constexpr int V = VecTraits<T>::kVec;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __shared__ double s_cos[64];
    __shared__ double s_sin[64];

    const int pos = blockIdx.x;             // working slot = new position id
    const int D = a.D, half = D / 2;
    int lo = 0, hi = a.num_segments;        // largest s with dst_off[s] <= pos
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (segs.dst_off[mid] <= pos) lo = mid; else hi = mid;
    }
    const int src_slot = segs.src[lo] + (pos - segs.dst_off[lo]);

    if (threadIdx.x < half) {
        const int j = threadIdx.x;
        const double2 cs = a.table ? a.table[(long)(pos - a.table_first) * half + j] : rope_cos_sin(pos, j, D, a.log2_theta);
        s_cos[j] = cs.x;
        s_sin[j] = cs.y;
    }
    __syncthreads();

    const int vec_per_half = half / V;
    const int k_items = a.Hkv * vec_per_half;
    const int v_items = a.Hkv * (D / V);
    for (int it = threadIdx.x; it < k_items + v_items; it += blockDim.x) {
        if (it < k_items) {
            const int g = it / vec_per_half;
            const int j0 = (it % vec_per_half) * V;
            const T* src = (const T*)a.k_src + ((long)g * a.src_cap + src_slot) * D;
            T* dst = (T*)a.k_dst + ((long)g * a.dst_cap + pos) * D;
            uint4 lo_raw = *reinterpret_cast<const uint4*>(src + j0);
            uint4 hi_raw = *reinterpret_cast<const uint4*>(src + j0 + half);
            const T* xl = reinterpret_cast<const T*>(&lo_raw);
            const T* xh = reinterpret_cast<const T*>(&hi_raw);
            uint4 out_lo_raw, out_hi_raw;
            T* out_lo = reinterpret_cast<T*>(&out_lo_raw);
            T* out_hi = reinterpret_cast<T*>(&out_hi_raw);
#pragma unroll
            for (int v = 0; v < V; ++v) {
                // products and their difference in double, then one rounding to float and one to storage
                const double c = s_cos[j0 + v], s = s_sin[j0 + v];
                const double x0 = (double)to_float(xl[v]), x1 = (double)to_float(xh[v]);
                from_float((float)(x0 * c - x1 * s), out_lo[v]);
                from_float((float)(x1 * c + x0 * s), out_hi[v]);
            }
            *reinterpret_cast<uint4*>(dst + j0) = out_lo_raw;
            *reinterpret_cast<uint4*>(dst + j0 + half) = out_hi_raw;
        } else {
            const int e = it - k_items;
            const int g = e / (D / V);
            const int d0 = (e % (D / V)) * V;
            *reinterpret_cast<uint4*>((T*)a.v_dst + ((long)g * a.dst_cap + pos) * D + d0) =
                *reinterpret_cast<const uint4*>((const T*)a.v_src + ((long)g * a.src_cap + src_slot) * D + d0);
        }
    }
}

}  // namespace evln
