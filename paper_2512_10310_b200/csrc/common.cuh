// Shared host/device declarations of libevln's kernels (internal; the public contract is
// include/evln.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace evln {

constexpr int kMaxBatch = 256;     // paged calls carry per-episode lengths as launch parameters
constexpr int kMaxSplits = 32;     // a warp merges one split per lane
constexpr int kTileM = 128;        // query rows per MMA tile
constexpr int kTileN = 128;        // keys per KV tile
constexpr int kUnitRows = 2 * kTileM;  // one CTA of the tensor-core kernel owns two query tiles

// Device status codes written by kernels whose bounded waits expire.
enum DeviceStatus : int {
    kDevOk = 0,
    kDevTimeoutProducer = 1,   // TMA producer waiting for a free K/V stage
    kDevTimeoutMmaQ = 2,       // MMA warp waiting for the Q tiles
    kDevTimeoutMmaKV = 3,      // MMA warp waiting for a K/V tile
    kDevTimeoutMmaP = 4,       // MMA warp waiting for the softmax warps' P tile
    kDevTimeoutSoftmaxS = 5,   // softmax warps waiting for S
    kDevTimeoutSoftmaxO = 6,   // softmax warps waiting for the final O
    kDevTimeoutSoftmaxX = 7,   // softmax warps of one lane quarter waiting for each other
    kDevTimeoutSelfTest = 8,   // the self-test's wait on a barrier nothing arrives on (EVLN_SELFTEST_STATUS_CODE)
};

// Per-episode lengths of a paged batch, passed by value.
struct BatchLens {
    int cache_len[kMaxBatch];
    int new_off[kMaxBatch + 1];
    int item_off[kMaxBatch + 1];   // first work item of the attention kernel per episode
};

template <typename T> struct VecTraits;
template <> struct VecTraits<__nv_bfloat16> { static constexpr int kVec = 8; };
template <> struct VecTraits<float> { static constexpr int kVec = 4; };

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_float(float x, float& y) { y = x; }
__device__ __forceinline__ void from_float(float x, __nv_bfloat16& y) { y = __float2bfloat16_rn(x); }

// Number of 128-key tiles the rows of unit u (rows [u*unit_rows, ...)) of an episode need.
__host__ __device__ inline int unit_kv_tiles(int L, int n, int G, int unit, int unit_rows)
{
    // 32-bit on purpose (rows per kv head are at most 2^24): a 64-bit division costs a CTA hundreds
    // of cycles before it has started anything
    unsigned last_row = (unsigned)(unit + 1) * (unsigned)unit_rows - 1u;
    unsigned last_tok = last_row / (unsigned)G;
    if (last_tok > (unsigned)(n - 1)) last_tok = (unsigned)(n - 1);
    return (int)(((unsigned)L + last_tok + 1u + (unsigned)kTileN - 1u) / (unsigned)kTileN);
}

__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Division of x < 2^31 by a constant d >= 1 as a multiplication: with l = ceil(log2 d) and
// mul = ceil(2^(31+l) / d) < 2^32, floor(x * mul / 2^(31+l)) = floor(x / d) exactly (the error
// x * (mul*d - 2^(31+l)) / (d * 2^(31+l)) stays below 2^-l <= 1/d).  An integer division costs a
// CTA a few hundred cycles of latency before it knows what to load.
struct FastDiv {
    uint32_t mul, shift;
};
inline FastDiv make_fast_div(uint32_t d)
{
    uint32_t l = 0;
    while ((1ull << l) < d) ++l;
    FastDiv f;
    f.shift = 31 + l;
    f.mul = (uint32_t)(((1ull << f.shift) + d - 1) / d);
    return f;
}
__host__ __device__ inline uint32_t fast_div(uint32_t x, FastDiv f)
{
    return (uint32_t)(((unsigned long long)x * f.mul) >> f.shift);
}
// unit_kv_tiles with the division by G prepared by the host
__host__ __device__ inline int unit_kv_tiles_fast(int L, int n, FastDiv div_g, int unit, int unit_rows)
{
    const uint32_t last_row = (uint32_t)(unit + 1) * (uint32_t)unit_rows - 1u;
    uint32_t last_tok = fast_div(last_row, div_g);
    if (last_tok > (uint32_t)(n - 1)) last_tok = (uint32_t)(n - 1);
    return (int)(((uint32_t)L + last_tok + 1u + (uint32_t)kTileN - 1u) / (uint32_t)kTileN);
}

// KV tiles of unit u of a SHARED-PREFIX batch item: the first L tokens of a cache that several items
// share (all of them visible to every row), then the item's own n new tokens from a separate buffer
// (causal).  The two parts are tiled separately: the own tokens start a new tile.
__host__ __device__ inline int tail_kv_tiles(int L, int n, int G, int unit, int unit_rows)
{
    unsigned last_row = (unsigned)(unit + 1) * (unsigned)unit_rows - 1u;
    unsigned last_tok = last_row / (unsigned)G;
    if (last_tok > (unsigned)(n - 1)) last_tok = (unsigned)(n - 1);
    return (int)(((unsigned)L + (unsigned)kTileN - 1u) / (unsigned)kTileN + (last_tok + (unsigned)kTileN) / (unsigned)kTileN);
}
__host__ __device__ inline int tail_kv_tiles_fast(int L, int n, FastDiv div_g, int unit, int unit_rows)
{
    const uint32_t last_row = (uint32_t)(unit + 1) * (uint32_t)unit_rows - 1u;
    uint32_t last_tok = fast_div(last_row, div_g);
    if (last_tok > (uint32_t)(n - 1)) last_tok = (uint32_t)(n - 1);
    return (int)(((uint32_t)L + (uint32_t)kTileN - 1u) / (uint32_t)kTileN + (last_tok + (uint32_t)kTileN) / (uint32_t)kTileN);
}

// Where token m of a dense run of tokens sits in a PACKED sequence I, v_1, a_1, ..., v_N, a_N
// (Sec. 3.3): `action` = 0 maps the run instruction + visual tokens, 1 the run of action tokens.
// F = 0 means "not packed": the identity.
struct PackedMap {
    int I, F, A, action;
};
__host__ __device__ inline long packed_row(const PackedMap& pm, long m)
{
    if (pm.F <= 0 && pm.A <= 0) return m;
    if (pm.action) return pm.I + (m / pm.A) * (long)(pm.F + pm.A) + pm.F + m % pm.A;
    if (m < pm.I || pm.F <= 0) return m;
    return pm.I + ((m - pm.I) / pm.F) * (long)(pm.F + pm.A) + (m - pm.I) % pm.F;
}

// Stub lengths for the kernels that serve one episode.
struct NoLens {
    int cache_len[1];
    int new_off[2];
    int item_off[2];
};

}  // namespace evln
