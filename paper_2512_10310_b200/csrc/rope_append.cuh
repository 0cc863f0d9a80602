// Fused RoPE-rotate-and-append kernel (Sec. 3.2: contiguous position ids, rotation,
// concatenation of the new frame with the reused cache).
//
// One CTA per new token.  Phase 1: D/2 threads get the token's cos/sin of phi_j = pos * theta^(-2j/D)
// in double precision (pos reaches tens of thousands; a float angle would be off by ~1e-3 rad)
// into shared memory for all heads: from the caller's position table when there is one (the
// table depends on the positions only, so a model makes it once per navigation step for all its
// layers: rope_table_kernel below), else formed on the spot.  Phase 2: every thread moves 16-byte
// vectors (a work item is a pair of vectors (j.., j + D/2..) of a query or key head, or one vector
// of a value head): rotated query halves to the kv-head-grouped q_rot scratch, rotated key halves
// and the unchanged values to the token's cache slot; the loads of a thread's first item are issued
// before the cos/sin are waited for.  HBM-bound by bytes (each element is read once and written
// once with 128-bit accesses); at the sizes of a step it is one chain of latencies, which is why
// nothing in it divides, and why a call of few tokens gets one thread per work item (all loads of
// a token in flight at once).  (Letting every thread read the table entries of its own vector
// instead of sharing them through shared memory was measured slower: 32 heads re-read the same 64
// entries.)
#pragma once

#include "common.cuh"

namespace evln {

struct RopeArgs {
    const void* q_new;
    const void* k_new;
    const void* v_new;
    void* q_rot;
    void* k_cache;      // contiguous: [Hkv, cap, D]; paged: pool [pages, Hkv, page, D]
    void* v_cache;
    const int* page_table;   // paged only: [batch, max_pages]
    long q_stride, k_stride, v_stride;   // token strides in elements
    int Hq, Hkv, D;
    int cache_len;      // contiguous only
    int num_new;        // contiguous: n; paged: total new tokens
    int cache_cap;      // contiguous only
    int batch, page_size, max_pages;     // paged only
    double log2_theta;
    const double2* table;   // optional: (cos, sin) per (position - table_first, j), [count][D/2]
    int table_first;
    int tail;               // batch mode without pages: K/V of new token m go to row m of k_cache / v_cache
                            // = buffers [Hkv, total new tokens, D] (the items' own tokens, not a shared cache)
    PackedMap map;          // where new token m sits in q_new / k_new / v_new (identity unless packed)
    // derived by the host (finish_rope_args): the threads decode their work with shifts and one
    // multiplication instead of integer divisions
    int G;                  // Hq / Hkv
    FastDiv div_g;
    int vph_shift;          // log2 of the 16-byte vectors per half head vector (D/2 / V)
    int page_shift;         // log2(page_size)
};

// cos/sin of pos * theta^(-2j/D): the one definition the append, gather and table kernels share
__device__ __forceinline__ double2 rope_cos_sin(long pos, int j, int D, double log2_theta)
{
    const double omega = exp2(-(2.0 * (double)j / (double)D) * log2_theta);
    double s, c;
    // sin/cos(pos * omega) through sincospi: its range reduction is exact and cheap, where a
    // plain sincos of an argument of thousands of radians takes the slow reduction path
    sincospi((double)pos * omega * 0.31830988618379067154, &s, &c);
    return make_double2(c, s);
}

// Position table: entry (p, j) = (cos, sin) of (first_pos + p) * theta^(-2j/D).
__global__ void __launch_bounds__(128)
rope_table_kernel(double2* table, int first_pos, int count, int D, double log2_theta)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int half = D / 2;
    const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long)count * half) return;
    const int p = (int)(i / half), j = (int)(i % half);
    table[i] = rope_cos_sin((long)first_pos + p, j, D, log2_theta);
}

// LensT is BatchLens for the paged kernel and NoLens (a stub) for the contiguous one.

// Block size: calls of few tokens (one wave of blocks) get one thread per work item, in whole warps,
// at most kRopeThreadsMax; batches of thousands of tokens are bound by throughput and take 256.
constexpr int kRopeThreadsMax = 384;
constexpr int kRopeThreads = 256;

template <typename T, bool PAGED, typename LensT>
__global__ void __launch_bounds__(kRopeThreadsMax)
rope_append_kernel(const RopeArgs a, const __grid_constant__ LensT lens)
{
    constexpr int V = VecTraits<T>::kVec;
    __shared__ double s_cos[128];
    __shared__ double s_sin[128];

    const int tok = blockIdx.x;           // index into the packed new tokens
    const int D = a.D, half = D / 2;
    const int G = a.G;

    int b = 0, i = tok, L = a.cache_len, n_b = a.num_new;
    if (PAGED) {
        int lo = 0, hi = a.batch;         // largest b with new_off[b] <= tok
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (lens.new_off[mid] <= tok) lo = mid; else hi = mid;
        }
        b = lo;
        i = tok - lens.new_off[b];
        L = lens.cache_len[b];
        n_b = lens.new_off[b + 1] - lens.new_off[b];
    }
    const long pos = (long)L + i;
    // (so far launch parameters only; what follows reads memory that earlier kernels may have written)
    asm volatile("griddepcontrol.wait;" ::: "memory");          // programmatic dependent launch: inputs ready
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const double2* trow = a.table ? a.table + (pos - a.table_first) * half : nullptr;

    if (threadIdx.x < half) {
        const int j = threadIdx.x;
        const double2 cs = trow ? trow[j] : rope_cos_sin(pos, j, D, a.log2_theta);
        s_cos[j] = cs.x;
        s_sin[j] = cs.y;
    }

    // destination of this token's K/V row for kv head g (element offset)
    long page_base = 0;     // paged: (page_id * Hkv) * page_size * D, slot within page
    int slot = 0;
    if (PAGED && !a.tail) {
        int pg = a.page_table[(long)b * a.max_pages + (int)(pos >> a.page_shift)];
        slot = (int)(pos & (a.page_size - 1));
        page_base = (long)pg * a.Hkv * a.page_size * D;
    }
    auto kv_row = [&](int g) -> long {
        if (PAGED && a.tail) return ((long)g * lens.new_off[a.batch] + tok) * D;
        if (PAGED) return page_base + ((long)g * a.page_size + slot) * D;
        return ((long)g * a.cache_cap + pos) * D;
    };

    const long src_tok = packed_row(a.map, tok);
    const T* q_tok = (const T*)a.q_new + src_tok * a.q_stride;
    const T* k_tok = (const T*)a.k_new + src_tok * a.k_stride;
    const T* v_tok = (const T*)a.v_new + src_tok * a.v_stride;

    const int vph = a.vph_shift, vpr = a.vph_shift + 1;       // vectors per half head vector / per head vector (log2)
    const int q_items = a.Hq << vph;
    const int k_items = a.Hkv << vph;
    const int v_items = a.Hkv << vpr;
    const int items = q_items + k_items + v_items;
    const long rows_per_head = PAGED ? (long)lens.new_off[a.batch] * G : (long)a.num_new * G;

    // a thread's work item `it`: a pair of 16-byte vectors (j0.., j0+half..) of a query or key head,
    // or one 16-byte vector of a value head
    auto load_item = [&](int it, uint4& r0, uint4& r1) {
        if (it < q_items + k_items) {
            const bool is_q = it < q_items;
            const int e = is_q ? it : it - q_items;
            const int h = e >> vph;
            const int j0 = (e & ((1 << vph) - 1)) * V;
            const T* src = (is_q ? q_tok : k_tok) + (long)h * D;
            r0 = *reinterpret_cast<const uint4*>(src + j0);
            r1 = *reinterpret_cast<const uint4*>(src + j0 + half);
        } else {
            const int e = it - q_items - k_items;
            const int g = e >> vpr;
            const int d0 = (e & ((1 << vpr) - 1)) * V;
            r0 = *reinterpret_cast<const uint4*>(v_tok + (long)g * D + d0);
        }
    };
    auto finish_item = [&](int it, const uint4& lo_raw, const uint4& hi_raw) {
        if (it < q_items + k_items) {
            const bool is_q = it < q_items;
            const int e = is_q ? it : it - q_items;
            const int h = e >> vph;
            const int j0 = (e & ((1 << vph) - 1)) * V;
            T* dst;
            if (is_q) {
                const int g = (int)fast_div((uint32_t)h, a.div_g);
                dst = (T*)a.q_rot + ((long)g * rows_per_head + (long)tok * G + (h - g * G)) * D;
            } else {
                dst = (T*)a.k_cache + kv_row(h);
            }
            const T* lo = reinterpret_cast<const T*>(&lo_raw);
            const T* hi = reinterpret_cast<const T*>(&hi_raw);
            uint4 out_lo_raw, out_hi_raw;
            T* out_lo = reinterpret_cast<T*>(&out_lo_raw);
            T* out_hi = reinterpret_cast<T*>(&out_hi_raw);
#pragma unroll
            for (int v = 0; v < V; ++v) {
                // products and the difference in double (a float product loses bits exactly where
                // x0*c and x1*s cancel), then one rounding to float and one to the storage dtype
                const double c = s_cos[j0 + v], s = s_sin[j0 + v];
                const double x0 = (double)to_float(lo[v]), x1 = (double)to_float(hi[v]);
                from_float((float)(x0 * c - x1 * s), out_lo[v]);
                from_float((float)(x1 * c + x0 * s), out_hi[v]);
            }
            *reinterpret_cast<uint4*>(dst + j0) = out_lo_raw;
            *reinterpret_cast<uint4*>(dst + j0 + half) = out_hi_raw;
        } else {
            const int e = it - q_items - k_items;
            const int g = e >> vpr;
            const int d0 = (e & ((1 << vpr) - 1)) * V;
            *reinterpret_cast<uint4*>((T*)a.v_cache + kv_row(g) + d0) = lo_raw;
        }
    };

    uint4 r0 = make_uint4(0u, 0u, 0u, 0u), r1 = r0;
    if ((int)threadIdx.x < items) load_item(threadIdx.x, r0, r1);     // in flight while the cos/sin arrive
    __syncthreads();
    if ((int)threadIdx.x < items) finish_item(threadIdx.x, r0, r1);
    for (int it = threadIdx.x + blockDim.x; it < items; it += blockDim.x) {
        load_item(it, r0, r1);
        finish_item(it, r0, r1);
    }

    if (PAGED && !a.tail && i == n_b - 1 && slot + 1 < a.page_size) {
        // the episode's last page is only partly filled: clear the value slots behind the last
        // token so that a tile load of the whole page never brings in stale bits
        const int tail = a.page_size - (slot + 1);
        const int vec_per_row = D / V;
        const int total = a.Hkv * tail * vec_per_row;
        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
        for (int it = threadIdx.x; it < total; it += blockDim.x) {
            const int g = it / (tail * vec_per_row);
            const int r = it % (tail * vec_per_row);
            const int s2 = slot + 1 + r / vec_per_row;
            const int d0 = (r % vec_per_row) * V;
            *reinterpret_cast<uint4*>((T*)a.v_cache + page_base + ((long)g * a.page_size + s2) * D + d0) = zero;
        }
    }
}

}  // namespace evln
