// fp32 SIMT step attention (no tensor cores).
//
// The fp32 configuration asks for 1e-5 agreement with the fp64 oracle, which tf32 tensor-core
// products cannot give, so this kernel evaluates the same split-KV causal attention with
// float FMAs.  One warp owns one packed query row (kv head g, row r = i*G + h%G): every lane
// scores one key of a 32-key chunk, the running maximum and sum of the online softmax are
// reduced across the warp with shuffles, and each lane accumulates D/32 output channels.
// It is also the on-device cross-check of the tensor-core kernel for bf16 inputs.
#pragma once

#include "common.cuh"

namespace evln {

struct SimtAttnArgs {
    const void* q_rot;     // [Hkv, R, D]
    const void* k_cache;   // [Hkv, cap, D]
    const void* v_cache;
    float* o_part;         // [S, Hkv, R, D]
    float* lse_part;       // [S, Hkv, R]
    int Hkv, G, D;
    int cache_len, num_new, cache_cap;
    int num_splits;
    float scale;
};

template <typename T, int D>
__global__ void __launch_bounds__(128)
attn_simt_kernel(const SimtAttnArgs a)
{
    constexpr int C = D / 32;                 // output channels per lane
    asm volatile("griddepcontrol.wait;" ::: "memory");          // programmatic dependent launch: inputs ready
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __shared__ float s_q[4][D];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int R = a.num_new * a.G;
    const int r = blockIdx.x * 4 + warp;
    const int g = blockIdx.y, split = blockIdx.z;
    const int T_total = a.cache_len + a.num_new;
    if (r >= R) return;

    const int i = r / a.G;
    const long t_lo = (long)split * T_total / a.num_splits;
    long t_hi = (long)(split + 1) * T_total / a.num_splits;
    const long bound = (long)a.cache_len + i + 1;          // keys 0 .. L+i are visible
    if (t_hi > bound) t_hi = bound;

    const T* q = (const T*)a.q_rot + ((long)g * R + r) * D;
    for (int d = lane; d < D; d += 32) s_q[warp][d] = to_float(q[d]);
    __syncwarp();

    const T* kbase = (const T*)a.k_cache + (long)g * a.cache_cap * D;
    const T* vbase = (const T*)a.v_cache + (long)g * a.cache_cap * D;

    float m = -INFINITY, l = 0.f;
    float o[C];
#pragma unroll
    for (int c = 0; c < C; ++c) o[c] = 0.f;

    for (long t0 = t_lo; t0 < t_hi; t0 += 32) {
        const long t = t0 + lane;
        float s = -INFINITY;
        if (t < t_hi) {
            const T* k = kbase + t * D;
            float acc = 0.f;
#pragma unroll 8
            for (int d = 0; d < D; ++d) acc = fmaf(s_q[warp][d], to_float(k[d]), acc);
            s = acc * a.scale;
        }
        float cmax = s;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, off));
        const float m_new = fmaxf(m, cmax);               // finite: the chunk holds >= 1 key
        const float alpha = expf(m - m_new);              // m = -inf on the first chunk -> 0
        const float p = (t < t_hi) ? expf(s - m_new) : 0.f;
        float psum = p;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, off);
        l = l * alpha + psum;
        m = m_new;
#pragma unroll
        for (int c = 0; c < C; ++c) o[c] *= alpha;
        const int cnt = (int)((t_hi - t0) < 32 ? (t_hi - t0) : 32);
        for (int j = 0; j < cnt; ++j) {
            const float pj = __shfl_sync(0xffffffffu, p, j);
            const T* v = vbase + (t0 + j) * D;
#pragma unroll
            for (int c = 0; c < C; ++c) o[c] = fmaf(pj, to_float(v[lane + 32 * c]), o[c]);
        }
    }

    const long prow = ((long)split * a.Hkv + g) * R + r;
    float* op = a.o_part + prow * D;
    const float inv = (l > 0.f) ? 1.f / l : 0.f;
#pragma unroll
    for (int c = 0; c < C; ++c) op[lane + 32 * c] = o[c] * inv;
    if (lane == 0) a.lse_part[prow] = (l > 0.f) ? m + logf(l) : -INFINITY;
}

}  // namespace evln
