// Split-KV step attention on the 5th-generation tensor cores, one CTA pair per work item
// (bf16, head_dim 128).
//
// Sec. 3.2 leaves one attention per step: the n new (rotated) queries against all L+n cached
// keys.  With grouped-query attention the G query heads of a kv head share its K/V, so the
// G*n query rows of a kv head are packed row-major (row = token*G + head-in-group) and cut
// into 128-row tiles.  A UNIT is two consecutive tiles (256 rows); a work item is a unit and a
// contiguous range of 128-key KV tiles (a split).  A cluster of two CTAs owns a work item: CTA
// r of the pair holds query tile r, and both drive ONE tensor-core instruction stream
// (tcgen05.mma cta_group::2, M = 256) issued by the pair's CTA 0.  Each CTA stages only its
// half of every K tile (64 keys) and V tile (64 channels): the pair reads K/V once for 256
// query rows.  The item's normalised partial outputs + log-sum-exps go to the workspace that
// the combine kernel merges.
//
// Per CTA (640 threads, 1 CTA/SM, ~199 KB shared memory, all 512 TMEM columns):
//   warp 0      TMA producer: the CTA's Q tile once, then its K / V half tiles through two
//               5-deep rings of 16 KB stages (128B-swizzled); no multicast anywhere.  Bytes are
//               counted on barriers of CTA 0, where the MMA threads wait.
//   warp 1      (CTA 0) score issuer, one elected lane: S_j = Q K_j^T (SS) into score buffer
//               j % 2 as soon as the softmax has READ tile j-2 out of it.
//   warp 2      (CTA 0) product issuer: O += P_j V_j (A = P_j from tensor memory, buffer j % 2)
//               as soon as P_j is written.  Scores and products have buffers of their own, so
//               neither instruction stream waits for the other.
//   warps 4-19  softmax + epilogue, four warps per TMEM lane quarter (= per SM sub-partition), two
//               threads per query row and tile.  The warps of group 0 take the even KV tiles of the
//               item, those of group 1 the odd ones; within a group a thread owns 64 of the 128
//               score columns of its row: it pulls them into registers, gives the score buffer back
//               at once, and then works through its 64 exponentials while the other three warps
//               of the sub-partition are in other phases of their tiles.  (One warp needs ~2.5 K
//               cycles of mostly latency for its share of a tile, the tensor pipe ~1 K for the
//               tile's MMAs: four warps in flight per sub-partition are what hides the chain; a
//               tile's exponentials also keep the 4 SFU lanes of a sub-partition busy for ~1 K
//               cycles, so that unit must not idle either.)  The exponentials of a row are taken
//               against a reference that one thread of the row reads off the first 32 scores of
//               the first tile and passes to the other three through shared memory; they talk to
//               each other again only if a later score exceeds it by more than 2^64 (then O, the
//               row sums and the pending P tiles are rescaled by a power of two); the final
//               division by the row sum makes any reference exact.
//   warp 3      sets up barriers (with warp 2), then idles.
// TMEM columns: scores S_b at 128 b, b = 0..1; P_b (128 keys as 64 columns of packed bf16 pairs) at
// 256 + 64 b; O at 384.
//
// Every mbarrier wait is bounded: on expiry the CTA records a code in the device status word and
// raises a shared abort flag; all roles then leave their loops, TMEM is freed and the pair
// returns together (cluster barrier).
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "timeline_debug.cuh"

namespace evln {

constexpr int kTcThreads = 640;
constexpr int kParts = 4;                             // softmax threads per query row: tile parity x column half
constexpr int kTileBytes = kTileM * 128 * 2;          // Q tile: 128 rows x 128 channels x bf16
constexpr int kHalfBytes = kTileBytes / 2;            // 16 KB: a 64-channel half of Q; a K or V half tile
constexpr int kSmemBarBytes = 384;
constexpr int kSmemXchBytes = 128 * 4 + 2 * kParts * 128 * 4 + 128;

// Shared-memory plan of a CTA.  CTAS = 2: the CTA of a pair stages half tiles (16 KB) through two
// 5-deep rings.  CTAS = 1: a CTA on its own stages whole K / V tiles (32 KB: two 64-channel blocks
// of 128 keys) through a 3-deep K ring and a 2-deep V ring.
template <int CTAS>
struct SmemPlan {
    static constexpr int kKStages = CTAS == 2 ? 5 : 3;
    static constexpr int kVStages = CTAS == 2 ? 5 : 2;
    static constexpr int kStageBytes = CTAS == 2 ? kHalfBytes : kTileBytes;
    static constexpr int kQOff = 0;
    static constexpr int kKOff = kTileBytes;
    static constexpr int kVOff = kKOff + kKStages * kStageBytes;
    static constexpr int kBarOff = kVOff + kVStages * kStageBytes;
    static constexpr int kRefOff = kBarOff + kSmemBarBytes;          // float [128 rows]: published references
    static constexpr int kSumOff = kRefOff + 128 * 4;                // float [kParts][128 rows]: row-sum shares
    static constexpr int kCandOff = kSumOff + kParts * 128 * 4;      // float [kParts][128 rows]: reference requests
    static constexpr int kReqOff = kCandOff + kParts * 128 * 4;      // int [4] request flags, int [4][kParts] released tiles
    static constexpr int kBytes = kRefOff + kSmemXchBytes + 1024;    // + slack to align to 1024
    static_assert(kKStages * kStageBytes >= 16 * 32 * 144, "the epilogue stages its rows in the K ring");
    static_assert(kBytes <= 227 * 1024, "shared memory per CTA");
};
constexpr int kTcSmemBytes = SmemPlan<2>::kBytes;
constexpr int kSoloSmemBytes = SmemPlan<1>::kBytes;
constexpr long long kWaitLimitCycles = 2000000000LL;  // ~1 s at boost clocks
constexpr int kScoreBufs = 2;
// Registers per thread after the set-up.  setmaxnreg moves registers inside the pool the CTA got at
// launch (kTcThreads x the kernel's register count, kRegsLaunch): what the issue warpgroup gives up
// must cover what the softmax warpgroups take, or their request waits for ever.  The host checks
// the compiled register count against kRegsLaunch before the first launch.
constexpr int kRegsLaunch = 96, kRegsIssue = 32, kRegsSoftmax = 112;
static_assert((kRegsLaunch - kRegsIssue) * 128 >= (kRegsSoftmax - kRegsLaunch) * (kTcThreads - 128), "register pool of a CTA");
static_assert(kRegsLaunch * kTcThreads <= 65536, "register file of an SM");
constexpr uint32_t kColP = 256;
constexpr uint32_t kColO = 384;
#ifndef EVLN_REF_HEADROOM
#define EVLN_REF_HEADROOM 64.f
#endif
constexpr float kRefHeadroom = EVLN_REF_HEADROOM;     // a row's reference moves when a score exceeds it by 2^64

struct TcAttnArgs {
    float* o_part;            // [S, Hkv, rows, 128]
    float* lse_part;          // [S, Hkv, rows]
    const int* page_table;    // paged only
    int* status;              // device status word
    int Hkv, G;
    int rows;                 // packed rows per kv head over the whole call
    int cache_len, num_new;   // contiguous only
    int num_splits;           // contiguous only
    int units_per_head;       // contiguous only
    int batch, max_pages, chunk_tiles;   // paged only
    float scale_log2;         // softmax scale * log2(e)
    FastDiv div_g;            // division by G
    FastDiv div_s;            // contiguous only: division by num_splits
};

// --- descriptors --------------------------------------------------------------------------

// kind::f16 instruction descriptor: fp32 accumulate, bf16 A and B, M x N of the whole pair.
__device__ __forceinline__ constexpr uint32_t make_idesc(bool b_mn_major, int m, int n)
{
    return (1u << 4)                       // D format: f32
           | (1u << 7)                     // A format: bf16
           | (1u << 10)                    // B format: bf16
           | ((b_mn_major ? 1u : 0u) << 16)
           | ((uint32_t)(n >> 3) << 17)
           | ((uint32_t)(m >> 4) << 24);
}

// Shared-memory matrix descriptor, 128-byte swizzle, rows of 128 bytes, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t make_sdesc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;                // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                // SWIZZLE_128B
    return d;
}

__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, int code, int* status,
                                             volatile int* s_abort, long long limit_cycles = kWaitLimitCycles)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t spins = 0;
    while (!ptx::mbar_try_wait(bar, parity)) {
        if ((++spins & 0x3f) == 0) {
            if (*s_abort) return false;
            if (clock64() - t0 > limit_cycles) {
                *s_abort = 1;
                atomicCAS(status, 0, code);
                return false;
            }
        }
    }
    return true;
}

// One lane polls, the warp shares the outcome (fewer pollers on the barrier word).
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, int code, int* status,
                                          volatile int* s_abort, int lane)
{
    int r = 1;
    if (lane == 0) r = wait_bounded(bar, parity, code, status, s_abort) ? 1 : 0;
    return __shfl_sync(0xffffffffu, r, 0) != 0;
}

// --- softmax pieces on 32-column register blocks of a score row ------------------------------

__device__ __forceinline__ void mask32(uint32_t* s, int lim)
{
#pragma unroll
    for (int e = 0; e < 32; ++e)
        if (e > lim) s[e] = 0xff800000u;
}

__device__ __forceinline__ void rowmax32(const uint32_t* s, float& m0, float& m1, float& m2, float& m3)
{
#pragma unroll
    for (int e = 0; e < 32; e += 8) {
        m0 = ptx::max3(m0, __uint_as_float(s[e]), __uint_as_float(s[e + 1]));
        m1 = ptx::max3(m1, __uint_as_float(s[e + 2]), __uint_as_float(s[e + 3]));
        m2 = ptx::max3(m2, __uint_as_float(s[e + 4]), __uint_as_float(s[e + 5]));
        m3 = ptx::max3(m3, __uint_as_float(s[e + 6]), __uint_as_float(s[e + 7]));
    }
}

// 2^x for a pair of scores on the FMA pipe instead of the special-function unit: x = n + f with
// n = round(x) (magic-number addition), 2^f by a cubic fitted on [-0.5, 0.5] (relative error
// 1.0e-4, far below the 2^-9 of the bf16 rounding that follows), the exponent n added as an
// integer.  x is clamped at -126 (masked scores are -inf; 2^-126 counts as nothing).
__device__ __forceinline__ void poly_ex2_pair(uint64_t x2, float& p0, float& p1)
{
    float x0, x1;
    ptx::unpack2(x2, x0, x1);
    x0 = fmaxf(x0, -126.f);
    x1 = fmaxf(x1, -126.f);
    const uint64_t xc = ptx::pack2(x0, x1);
    const uint64_t magic = ptx::pack2(12582912.f, 12582912.f), nmagic = ptx::pack2(-12582912.f, -12582912.f);
    const uint64_t t = ptx::add2(xc, magic);
    const uint64_t nf = ptx::add2(t, nmagic);
    const uint64_t f = ptx::fma2(nf, ptx::pack2(-1.f, -1.f), xc);
    uint64_t q = ptx::fma2(f, ptx::pack2(0.055922035f, 0.055922035f), ptx::pack2(0.24264008f, 0.24264008f));
    q = ptx::fma2(q, f, ptx::pack2(0.69312102f, 0.69312102f));
    q = ptx::fma2(q, f, ptx::pack2(0.99992448f, 0.99992448f));
    float q0, q1, t0, t1;
    ptx::unpack2(q, q0, q1);
    ptx::unpack2(t, t0, t1);
    p0 = __uint_as_float(__float_as_uint(q0) + (__float_as_uint(t0) << 23));
    p1 = __uint_as_float(__float_as_uint(q1) + (__float_as_uint(t1) << 23));
}

// p = 2^(s*scale + negm) for 32 columns, accumulated into two packed sums, left as 16 packed
// bf16 pairs (= 16 columns of tensor memory).  A tile's 128x128 exponentials keep the 4 SFU lanes
// of a sub-partition busy for as long as the tile's MMAs keep the tensor pipe busy, so a quarter of
// them (one pair in eight scores) is computed on the FMA pipe, which has issue slots to spare;
// a larger share costs more issue slots than it frees SFU cycles (measured: 25 % is 2-3 % faster
// than none at every cache length, 50 % is slower).
__device__ __forceinline__ void exp32(const uint32_t* s, uint32_t (&packed)[16], uint64_t scale2,
                                      uint64_t negm2, uint64_t& sum2a, uint64_t& sum2b)
{
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
        const uint64_t xa = ptx::fma2(ptx::pack2(__uint_as_float(s[e]), __uint_as_float(s[e + 1])), scale2, negm2);
        const uint64_t xb = ptx::fma2(ptx::pack2(__uint_as_float(s[e + 2]), __uint_as_float(s[e + 3])), scale2, negm2);
        float x0, x1, p0, p1, p2, p3;
        ptx::unpack2(xa, x0, x1);
        p0 = ptx::ex2(x0); p1 = ptx::ex2(x1);
        if (((e >> 2) & 1) == 0) {
            poly_ex2_pair(xb, p2, p3);
        } else {
            float x2, x3;
            ptx::unpack2(xb, x2, x3);
            p2 = ptx::ex2(x2); p3 = ptx::ex2(x3);
        }
        sum2a = ptx::add2(sum2a, ptx::pack2(p0, p1));
        sum2b = ptx::add2(sum2b, ptx::pack2(p2, p3));
        packed[e >> 1] = ptx::pack_bf16x2(p0, p1);
        packed[(e >> 1) + 1] = ptx::pack_bf16x2(p2, p3);
    }
}

// The largest of a row's first 32 scores of a score buffer (columns 0 .. lim visible), scaled: what the
// publisher of the row's reference computes, for a thread that would rather read the scores itself
// than wait for the publication.  Kept out of line so that it does not disturb the tile loop's code.
__device__ __noinline__ float first_block_reference(uint32_t taddr, int lim, float scale_log2)
{
    uint32_t f[32];
    ptx::tmem_ld32(taddr, f);
    ptx::tmem_ld_wait();
    if (!__all_sync(0xffffffffu, lim >= 63)) mask32(f, lim);
    float x0 = -INFINITY, x1 = -INFINITY, x2 = -INFINITY, x3 = -INFINITY;
    rowmax32(f, x0, x1, x2, x3);
    return fmaxf(fmaxf(x0, x1), fmaxf(x2, x3)) * scale_log2;
}

// --- work decoding ------------------------------------------------------------------------

struct WorkItem {
    int b, g, unit, slot;     // episode, kv head, unit within the episode, partial slot
    int L, n;                 // episode lengths
    int row_base;             // first packed row of the episode within the kv head
    int j0, j1;               // KV tile range
};

// Contiguous cache: the grid is (CTAS * units, kv heads, splits), so a CTA reads its work item off
// its block index; the two divisions left (by G and by the split count) are multiplications by
// constants the host prepared.  Batches (paged cache, or episodes sharing a cache prefix): items are
// numbered episode by episode (kv head, unit, split inside), the host passes the first item of every
// episode and the CTA searches that table.
template <bool PAGED, bool TAIL, typename LensT, int CTAS>
__device__ __forceinline__ WorkItem decode_work(const TcAttnArgs& a, const LensT& lens)
{
    constexpr int UNIT_ROWS = CTAS * kTileM;
    WorkItem w;
    if (!PAGED && !TAIL) {
        w.b = 0;
        w.unit = CTAS == 2 ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
        w.g = (int)blockIdx.y;
        w.slot = (int)blockIdx.z;
        w.L = a.cache_len;
        w.n = a.num_new;
        w.row_base = 0;
        const uint32_t nkv = (uint32_t)unit_kv_tiles_fast(w.L, w.n, a.div_g, w.unit, UNIT_ROWS);
        w.j0 = (int)fast_div((uint32_t)w.slot * nkv, a.div_s);
        w.j1 = (int)fast_div((uint32_t)(w.slot + 1) * nkv, a.div_s);
    } else {
        const int item = (int)(blockIdx.x >> 1);
        int lo = 0, hi = a.batch;             // largest b with item_off[b] <= item
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (lens.item_off[mid] <= item) lo = mid; else hi = mid;
        }
        const int b = lo;
        w.b = b;
        w.L = lens.cache_len[b];
        w.n = lens.new_off[b + 1] - lens.new_off[b];
        w.row_base = lens.new_off[b] * a.G;
        w.g = w.unit = w.slot = 0;
        w.j0 = w.j1 = 0;
        const int per_head = (lens.item_off[b + 1] - lens.item_off[b]) / a.Hkv;
        int rem = item - lens.item_off[b];
        if (item >= lens.item_off[a.batch] || per_head <= 0) { w.b = -1; return w; }
        w.g = rem / per_head;
        rem -= w.g * per_head;
        const int units = ceil_div(w.n * a.G, UNIT_ROWS);
        for (int u = 0; u < units; ++u) {
            const int nkv = TAIL ? tail_kv_tiles_fast(w.L, w.n, a.div_g, u, UNIT_ROWS)
                                 : unit_kv_tiles_fast(w.L, w.n, a.div_g, u, UNIT_ROWS);
            const int S = ceil_div(nkv, a.chunk_tiles);
            if (rem < S) {
                w.unit = u;
                w.slot = rem;
                w.j0 = (int)((unsigned)rem * (unsigned)nkv / (unsigned)S);
                w.j1 = (int)((unsigned)(rem + 1) * (unsigned)nkv / (unsigned)S);
                break;
            }
            rem -= S;
        }
    }
    return w;
}

// --- the kernel ---------------------------------------------------------------------------
// CTAS = 2: launched with a cluster of 2 CTAs along x: query tile = cluster rank.
// CTAS = 1: no cluster; one query tile (all the rows of a kv head fit in it).

// TAIL: a batch of items that share the first L_b tokens of ONE contiguous cache (every row sees all
// of them) and bring their own n_b new tokens in a separate buffer (tm_kt / tm_vt, packed over the
// batch; causal among themselves): the action chunks of a packed sequence (Sec. 3.3), each after
// its own prefix of the visual tokens, none visible to another.
template <bool PAGED, bool TAIL, typename LensT, int CTAS>
__device__ __forceinline__ void attn_tc_body(const CUtensorMap& tm_q, const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                                             const CUtensorMap* tm_kt, const CUtensorMap* tm_vt,
                                             const TcAttnArgs& a, const LensT& lens)
{
    static_assert(CTAS == 2 || !(PAGED || TAIL), "the batch kernels run on CTA pairs");
    static_assert(!(PAGED && TAIL), "one cache layout at a time");
    using Plan = SmemPlan<CTAS>;
    constexpr int kKStages = Plan::kKStages, kVStages = Plan::kVStages, kStageBytes = Plan::kStageBytes;
    constexpr int kSmemQOff = Plan::kQOff, kSmemKOff = Plan::kKOff, kSmemVOff = Plan::kVOff;
    constexpr int kItemRows = CTAS * kTileM;           // query rows of a work item
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));

    // barriers: same offsets in both CTAs; "(CTA 0)" marks those of which only CTA 0's copy is used
    const uint32_t bar_base = smem_base + Plan::kBarOff;
    const uint32_t bar_q_full = bar_base;                        // (CTA 0) both CTAs' Q tiles landed
    const uint32_t bar_k_full = bar_q_full + 8;                  // (CTA 0) [kKStages]
    const uint32_t bar_v_full = bar_k_full + 8 * kKStages;       // (CTA 0) [kVStages]
    const uint32_t bar_s_free = bar_v_full + 8 * kVStages;       // (CTA 0) [kScoreBufs] scores read by both CTAs' softmax
    const uint32_t bar_p_full = bar_s_free + 8 * kScoreBufs;     // (CTA 0) [kScoreBufs] P written by both CTAs
    const uint32_t bar_k_empty = bar_p_full + 8 * kScoreBufs;    // [kKStages] stage consumed by the MMAs
    const uint32_t bar_v_empty = bar_k_empty + 8 * kKStages;     // [kVStages]
    const uint32_t bar_s_full = bar_v_empty + 8 * kVStages;      // [kScoreBufs] scores ready
    const uint32_t bar_pv_done = bar_s_full + 8 * kScoreBufs;    // [4] PV of tile j landed: barrier j % 4
    const uint32_t bar_o_full = bar_pv_done + 32;                // last PV landed
    const uint32_t bar_ref = bar_o_full + 8;                     // [4] the rows' references are published
    const uint32_t bar_xch = bar_ref + 32;                       // [4] the four warps of a lane quarter meet here (row sums)
    const uint32_t bar_rare = bar_xch + 32;                      // [4] ... and here when a row's reference has to move
    const uint32_t tmem_slot = bar_rare + 32;                    // uint32
    constexpr int kBarsCtas = 1 + kKStages + kVStages;                                 // arrival count CTAS
    constexpr int kBarsSoft = 2 * kScoreBufs;                                          // one per softmax warp of the tile
    constexpr int kBarsOne = kKStages + kVStages + kScoreBufs + 4 + 1 + 4;             // count 1
    constexpr int kNumBars = kBarsCtas + kBarsSoft + kBarsOne + 8;                     // + xch, rare: kParts
    static_assert(8 * kNumBars + 8 <= kSmemBarBytes, "barrier area");
    static_assert(kNumBars <= 64, "one thread of warps 2-3 per barrier");
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem_gen + (tmem_slot - smem_base));
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem_gen + (tmem_slot - smem_base) + 4);
    float* s_ref = reinterpret_cast<float*>(smem_gen + Plan::kRefOff);
    float* s_sum = reinterpret_cast<float*>(smem_gen + Plan::kSumOff);
    float* s_cand = reinterpret_cast<float*>(smem_gen + Plan::kCandOff);
    volatile int* s_req = reinterpret_cast<volatile int*>(smem_gen + Plan::kReqOff);        // [4]
    volatile int* s_rel = reinterpret_cast<volatile int*>(smem_gen + Plan::kReqOff) + 4;    // [4][kParts]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = CTAS == 2 ? ptx::cluster_ctarank() : 0u;   // 0: issues the MMAs, owns the "(CTA 0)" barriers
    if (threadIdx.x == 0) EVLN_STAMP(0);

    const WorkItem w = decode_work<PAGED, TAIL, LensT, CTAS>(a, lens);
    if ((PAGED || TAIL) && w.b < 0) return;                      // both CTAs of the pair decode the same item

    const int rows_valid = w.n * a.G;                            // packed rows of this episode
    const int row0 = w.unit * kItemRows + (int)rank * kTileM;    // first row of this CTA's tile (episode-local)
    const int ntiles = w.j1 - w.j0;
    const int nct = TAIL ? (w.L + kTileN - 1) / kTileN : 0;      // TAIL: tiles below nct come from the shared cache
    // Lane quarters (32 rows each) of the tile that hold rows of the episode.  A CTA on its own lets
    // the softmax warps of the others sit out; a pair keeps all of them (both CTAs count alike).
    int quarters = 4;
    if (CTAS == 1) {
        quarters = (rows_valid - row0 + 31) >> 5;
        quarters = quarters < 1 ? 1 : (quarters > 4 ? 4 : quarters);
    }

    // A split with no KV tiles (more splits than tiles): its partials are "empty".
    if (ntiles <= 0) {
        ptx::grid_dependency_wait();
        if (warp >= 4 && warp < 8) {
            const int r = row0 + ((warp & 3) << 5) + lane;
            if (r < rows_valid) {
                const long prow = ((long)w.slot * a.Hkv + w.g) * a.rows + w.row_base + r;
                float4* o = reinterpret_cast<float4*>(a.o_part + prow * 128);
                for (int c = 0; c < 32; ++c) o[c] = make_float4(0.f, 0.f, 0.f, 0.f);
                a.lse_part[prow] = -INFINITY;
            }
        }
        return;
    }

    // ---- setup: barriers, TMEM, then the pair synchronises once ----
    if (threadIdx.x == 0) {
        ptx::prefetch_tensormap(&tm_q);
        ptx::prefetch_tensormap(&tm_k);
        ptx::prefetch_tensormap(&tm_v);
        if (TAIL) {
            ptx::prefetch_tensormap(tm_kt);
            ptx::prefetch_tensormap(tm_vt);
        }
        if (!PAGED && !TAIL) {
            // this CTA's halves of the first K tiles and of the first V tile on their way into L2 while
            // the pair sets up (cached rows; a row the previous kernel is still writing stays coherent)
            const int pre = ntiles < 3 ? ntiles : 3;
            for (int jj = 0; jj < pre; ++jj) {
                const int key0 = (w.j0 + jj) * kTileN + (int)rank * 64;
                ptx::tma_prefetch_3d(&tm_k, 0, key0, w.g);
                ptx::tma_prefetch_3d(&tm_k, 64, key0, w.g);
            }
            ptx::tma_prefetch_3d(&tm_v, 64 * (int)rank, w.j0 * kTileN, w.g);
            if (CTAS == 1) ptx::tma_prefetch_3d(&tm_v, 64, w.j0 * kTileN, w.g);
        }
    }
    if (warp == 2 || warp == 3) {
        // one barrier per thread: arrival counts in the order of the barrier area
        const int i = (int)threadIdx.x - 64;
        if (i < kNumBars) {
            int count = 1;
            if (i < kBarsCtas) count = CTAS;                                   // q_full, k_full, v_full
            else if (i < kBarsCtas + kBarsSoft) count = CTAS * quarters * 2;   // s_free, p_full: the tile's softmax warps
            else if (i < kBarsCtas + kBarsSoft + kBarsOne) count = 1;          // k_empty .. ref
            else count = kParts;                                               // xch, rare
            ptx::mbar_init(bar_base + 8 * i, count);
            ptx::fence_barrier_init();
        }
        if (i < 4) s_req[i] = 0;
        if (i == 0) *s_abort = 0;
    }
    if (warp == 1) {
        if (CTAS == 2) {
            ptx::tmem_alloc_pair(tmem_slot, 512);
            ptx::tmem_relinquish_pair();
        } else {
            ptx::tmem_alloc(tmem_slot, 512);
            ptx::tmem_relinquish();
        }
    }
    ptx::fence_before_sync();
    __syncthreads();
    if (CTAS == 2) {
        // the other CTA's barriers exist before anything arrives on them (their initialisation was
        // released cluster-wide by fence.mbarrier_init; nothing else is shared yet)
        ptx::cluster_arrive_relaxed();
        ptx::cluster_wait();
    }
    ptx::fence_after_sync();
    const uint32_t tmem = *s_tmem;
    ptx::grid_launch_dependents();
    if (threadIdx.x == 0) EVLN_STAMP(1);

    auto on_cta0 = [&](uint32_t bar) -> uint32_t { return CTAS == 2 ? ptx::map_to_cta(bar, 0) : bar; };

    // ---- the TMA producer's tools (used by one thread of warp 0) ----
    bool ok_prod = true;
            auto expect = [&](uint32_t bar, uint32_t bytes) {
                if (CTAS == 2) ptx::mbar_expect_tx_cluster(bar, bytes); else ptx::mbar_expect_tx(bar, bytes);
            };
            auto tma3 = [&](uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
                if (CTAS == 2) ptx::tma_load_3d_pair(dst, map, bar, x, y, z); else ptx::tma_load_3d(dst, map, bar, x, y, z);
            };
            // K tile j.  Pair: this CTA's half, keys [128 j + 64 rank, +64), all channels (two 64-channel
            // blocks of 64 keys).  Alone: the whole tile (two 64-channel blocks of 128 keys).
            auto load_k = [&](int jj) {
                const int stage = jj % kKStages;
                if (jj >= kKStages)
                    ok_prod = wait_bounded(bar_k_empty + 8 * stage, ((jj / kKStages) & 1) ^ 1, kDevTimeoutProducer, a.status, s_abort);
                if (!ok_prod) return;
                const uint32_t dst = smem_base + kSmemKOff + stage * kStageBytes;
                const uint32_t bar = on_cta0(bar_k_full + 8 * stage);
                const int j = w.j0 + jj;
                expect(bar, kStageBytes);
                if (TAIL) {
                    // shared cache below tile nct (rows past L_b are other items' tokens: finite, masked),
                    // this item's own tokens after (rows past n_b: the next item's or zero fill, masked)
                    const bool own = j >= nct;
                    const int key0 = (own ? lens.new_off[w.b] + (j - nct) * kTileN : j * kTileN) + (int)rank * 64;
                    const CUtensorMap* map = own ? tm_kt : &tm_k;
                    tma3(dst, map, bar, 0, key0, w.g);
                    tma3(dst + kStageBytes / 2, map, bar, 64, key0, w.g);
                } else if (!PAGED) {
                    const int key0 = j * kTileN + (int)rank * 64;
                    tma3(dst, &tm_k, bar, 0, key0, w.g);
                    tma3(dst + kStageBytes / 2, &tm_k, bar, 64, key0, w.g);
                } else {
                    // a 64-token page is exactly this CTA's half; past the episode's last page the
                    // last page is read again (masked, but finite)
                    const int npages = (w.L + w.n + 63) >> 6;
                    int pi = 2 * j + (int)rank;
                    if (pi >= npages) pi = npages - 1;
                    const int pg = a.page_table[(long)w.b * a.max_pages + pi];
                    ptx::tma_load_4d_pair(dst, &tm_k, bar, 0, 0, w.g, pg);
                    ptx::tma_load_4d_pair(dst + 8192, &tm_k, bar, 64, 0, w.g, pg);
                }
            };
            // V tile j, all 128 keys.  Pair: channels [64 rank, +64).  Alone: both 64-channel blocks.
            auto load_v = [&](int jj) {
                const int stage = jj % kVStages;
                if (jj >= kVStages)
                    ok_prod = wait_bounded(bar_v_empty + 8 * stage, ((jj / kVStages) & 1) ^ 1, kDevTimeoutProducer, a.status, s_abort);
                if (!ok_prod) return;
                const uint32_t dst = smem_base + kSmemVOff + stage * kStageBytes;
                const uint32_t bar = on_cta0(bar_v_full + 8 * stage);
                const int j = w.j0 + jj;
                expect(bar, kStageBytes);
                if (TAIL) {
                    const bool own = j >= nct;
                    tma3(dst, own ? tm_vt : &tm_v, bar, 64 * (int)rank,
                         own ? lens.new_off[w.b] + (j - nct) * kTileN : j * kTileN, w.g);
                } else if (!PAGED) {
                    tma3(dst, &tm_v, bar, 64 * (int)rank, j * kTileN, w.g);
                    if (CTAS == 1) tma3(dst + kHalfBytes, &tm_v, bar, 64, j * kTileN, w.g);
                } else {
                    const int npages = (w.L + w.n + 63) >> 6;
                    const int p0 = 2 * j;
                    const int p1 = (p0 + 1 < npages) ? p0 + 1 : p0;
                    const int* pt = a.page_table + (long)w.b * a.max_pages;
                    ptx::tma_load_4d_pair(dst, &tm_v, bar, 64 * (int)rank, 0, w.g, pt[p0]);
                    ptx::tma_load_4d_pair(dst + 8192, &tm_v, bar, 64 * (int)rank, 0, w.g, pt[p1]);
                }
            };

    // The producer's first loads (Q, then the K tiles of the first scores) go out before the warps
    // change their register shares: that hand-over is a rendezvous of the whole warpgroup, and the
    // loads' latency is the longest item on the way to the first MMA.
    const int pre_k = ntiles < kScoreBufs ? ntiles : kScoreBufs;
    if (warp == 0 && lane == 0) {
        // everything this CTA reads or writes in global memory follows this thread's loads, so
        // one wait here orders the whole CTA after the kernels it depends on
        ptx::grid_dependency_wait();
            {
                const uint32_t q_full0 = on_cta0(bar_q_full);
                const uint32_t dst = smem_base + kSmemQOff;
                const int qrow = w.row_base + row0;
                expect(q_full0, kTileBytes);
                tma3(dst, &tm_q, q_full0, 0, qrow, w.g);
                tma3(dst + kHalfBytes, &tm_q, q_full0, 64, qrow, w.g);
            }
        for (int jj = 0; jj < pre_k; ++jj) load_k(jj);
    }
    __syncwarp();            // (the register hand-over below wants whole warps)

    // Registers go where the work is: the warpgroup of the producer and the issuers gives most of its
    // share back, the two softmax warpgroups (128 scores per thread in flight) take it.
    if (warp < 4) {
    ptx::setmaxnreg_dec<kRegsIssue>();
    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            // in the order the MMAs consume them: (K_0, K_1 are on their way,) then V_j, K_{j+2}
            for (int jj = 0; jj < ntiles && ok_prod; ++jj) {
                load_v(jj);
                if (ok_prod && jj + kScoreBufs < ntiles) load_k(jj + kScoreBufs);
            }
            if (!ok_prod || *s_abort) {
                // give this CTA's loads in flight time to land before the pair may leave
                const long long t0 = clock64();
                while (clock64() - t0 < 400000) { }
            }
        }
        __syncwarp();
    } else if (warp == 1 && rank == 0) {
        // ================= score issuer (CTA 0 of the pair): S_jj = Q K_jj^T =================
        const uint32_t idesc_s = make_idesc(false, CTAS * kTileM, kTileN);
        // descriptors differ only in their address field (units of 16 bytes): build them once
        const uint64_t qdesc0 = make_sdesc(smem_base + kSmemQOff, 16, 1024);
        const uint64_t kdesc0 = make_sdesc(smem_base + kSmemKOff, 16, 1024);            // K-major; 64 (pair) or 128 keys per CTA
        bool ok = warp_wait(bar_q_full, 0, kDevTimeoutMmaQ, a.status, s_abort, lane);
        for (int jj = 0; jj < ntiles && ok; ++jj) {
            // K_jj landed; the softmax has read tile jj - 2 out of this score buffer.  A wait costs
            // ~150 cycles even on a completed barrier, so two lanes take one each.
            {
                uint32_t bar = bar_k_full + 8 * (jj % kKStages), parity = (jj / kKStages) & 1;
                int code = kDevTimeoutMmaKV;
                if (lane == 1) { bar = bar_s_free + 8 * (jj & 1); parity = ((jj >> 1) - 1) & 1; code = kDevTimeoutMmaP; }
                bool mine = true;
                if (lane == 0 || (lane == 1 && jj >= kScoreBufs)) mine = wait_bounded(bar, parity, code, a.status, s_abort);
                if (lane < 2 && jj < 9) EVLN_STAMP(20 + 9 * lane + jj);
                ok = __all_sync(0xffffffffu, mine);
            }
            if (!ok) break;
            ptx::fence_after_sync();
            if (ptx::elect_one()) {
                const int stage = jj % kKStages;
                const uint64_t kd = kdesc0 + (uint64_t)((stage * kStageBytes) >> 4);
                const uint32_t d = tmem + (uint32_t)(jj & 1) * 128;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t qoff = (uint64_t)(((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4);
                    const uint64_t koff = (uint64_t)(((ks >> 2) * (kStageBytes / 2) + (ks & 3) * 32) >> 4);
                    if (CTAS == 2) ptx::mma_ss_pair(d, qdesc0 + qoff, kd + koff, idesc_s, ks > 0);
                    else ptx::mma_ss(d, qdesc0 + qoff, kd + koff, idesc_s, ks > 0);
                }
                if (CTAS == 2) {
                    ptx::mma_commit_pair(bar_s_full + 8 * (jj & 1), (uint16_t)3);
                    ptx::mma_commit_pair(bar_k_empty + 8 * stage, (uint16_t)3);
                } else {
                    ptx::mma_commit(bar_s_full + 8 * (jj & 1));
                    ptx::mma_commit(bar_k_empty + 8 * stage);
                }
            }
            if (lane == 0 && jj < 9) EVLN_STAMP(38 + jj);
            __syncwarp();
        }
    } else if (warp == 2 && rank == 0) {
        // ================= product issuer (CTA 0 of the pair): O (+)= P_jj V_jj =================
        const uint32_t idesc_pv = make_idesc(true, CTAS * kTileM, 128);
        const uint64_t vdesc0 = make_sdesc(smem_base + kSmemVOff, kHalfBytes, 1024);    // MN-major; 64-channel blocks 16 KB apart
        bool ok = true;
        for (int jj = 0; jj < ntiles && ok; ++jj) {
            {
                uint32_t bar = bar_v_full + 8 * (jj % kVStages), parity = (jj / kVStages) & 1;
                int code = kDevTimeoutMmaKV;
                if (lane == 1) { bar = bar_p_full + 8 * (jj & 1); parity = (jj >> 1) & 1; code = kDevTimeoutMmaP; }
                bool mine = true;
                if (lane < 2) mine = wait_bounded(bar, parity, code, a.status, s_abort);
                ok = __all_sync(0xffffffffu, mine);
            }
            if (!ok) break;
            if (lane == 0 && jj < 9) EVLN_STAMP(47 + jj);
            ptx::fence_after_sync();
            if (ptx::elect_one()) {
                const int stage = jj % kVStages;
                const uint64_t vd = vdesc0 + (uint64_t)((stage * kStageBytes) >> 4);
                const uint32_t p = tmem + kColP + (uint32_t)(jj & 1) * 64;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    if (CTAS == 2) ptx::mma_ts_pair(tmem + kColO, p + ks * 8, vd + (uint64_t)((ks * 2048) >> 4), idesc_pv, jj > 0 || ks > 0);
                    else ptx::mma_ts(tmem + kColO, p + ks * 8, vd + (uint64_t)((ks * 2048) >> 4), idesc_pv, jj > 0 || ks > 0);
                }
                if (CTAS == 2) {
                    ptx::mma_commit_pair(bar_pv_done + 8 * (jj & 3), (uint16_t)3);
                    ptx::mma_commit_pair(bar_v_empty + 8 * stage, (uint16_t)3);
                    if (jj == ntiles - 1) ptx::mma_commit_pair(bar_o_full, (uint16_t)3);
                } else {
                    ptx::mma_commit(bar_pv_done + 8 * (jj & 3));
                    ptx::mma_commit(bar_v_empty + 8 * stage);
                    if (jj == ntiles - 1) ptx::mma_commit(bar_o_full);
                }
            }
            __syncwarp();
        }
    }
    } else {
    ptx::setmaxnreg_inc<kRegsSoftmax>();
    if ((warp & 3) < quarters) {
        // ================= softmax + epilogue =================
        const int quarter = warp & 3;                      // TMEM lane quarter of this warp
        const int part = (warp - 4) >> 2;                  // its 32 channels of O (epilogue, rescales)
        const int grp = part >> 1;                         // its KV tiles: grp, grp + 2, ...
        const int half = part & 1;                         // its score columns: [64 half, +64), two blocks of 32
        const int r_tile = (quarter << 5) + lane;          // row within the tile = TMEM lane
        const int r_local = row0 + r_tile;                 // packed row within the episode
        const bool row_valid = r_local < rows_valid;
        // last visible key index; a padding row (beyond the episode's rows: its Q is zero fill or
        // another episode's) is never stored, so it takes everything unmasked rather than making its
        // warp mask every tile
        // (TAIL: `bound` is the row's last visible token among the item's OWN tokens)
        const int bound = row_valid ? (TAIL ? 0 : w.L) + (int)fast_div((uint32_t)r_local, a.div_g) : 0x3fffffff;
        const uint32_t t_lane = tmem + ((uint32_t)(quarter << 5) << 16);
        const uint32_t t_s = t_lane + (uint32_t)grp * 128 + (uint32_t)half * 64;          // its half of the group's score buffer
        const uint32_t t_p = t_lane + kColP + (uint32_t)grp * 64 + (uint32_t)half * 32;   // ... and of its P buffer
        const uint32_t t_o = t_lane + kColO + (uint32_t)part * 32;
        const uint32_t s_free0 = on_cta0(bar_s_free + 8 * grp);
        const uint32_t p_full0 = on_cta0(bar_p_full + 8 * grp);

        float m_ref = -INFINITY;      // reference maximum (log2 domain) the exponentials use
        float l = 0.f;                // this thread's share of the running sum of exponentials
        bool ok = true;
        const uint64_t scale2 = ptx::pack2(a.scale_log2, a.scale_log2);
        // Meeting of the four warps of this lane quarter (one phase of their barrier each): what any of
        // them wrote to shared memory before its arrival is visible to the others after the wait.
        auto meet = [&](uint32_t bar, int k) -> bool {
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar + 8 * quarter);
            return warp_wait(bar + 8 * quarter, k & 1, kDevTimeoutSoftmaxX, a.status, s_abort, lane);
        };
        // A wait that gives way when a warp of this lane quarter has asked for a new reference:
        // 0 = the barrier completed, 1 = a request is pending, 2 = gave up (bounded wait expired).
        // (Every lane probes once first: a barrier that is already complete costs one instruction.  The
        // exponentials keep the sub-partition's queue to the SFU, the shared-memory and the barrier units
        // full, so every dependent instruction on that path is worth ~100 cycles here.)
        auto wait_or_request = [&](uint32_t bar, uint32_t parity, int code) -> int {
            if (__all_sync(0xffffffffu, ptx::mbar_try_wait(bar, parity))) return 0;
            int r = 0;
            if (lane == 0) {
                if (s_req[quarter]) {
                    r = 1;
                } else if (!ptx::mbar_try_wait(bar, parity)) {
                    const long long t0 = clock64();
                    uint32_t spins = 0;
                    while (!ptx::mbar_try_wait(bar, parity)) {
                        if (s_req[quarter]) { r = 1; break; }
                        if ((++spins & 0x3f) == 0) {
                            if (*s_abort) { r = 2; break; }
                            if (clock64() - t0 > kWaitLimitCycles) {
                                *s_abort = 1;
                                atomicCAS(a.status, 0, code);
                                r = 2;
                                break;
                            }
                        }
                    }
                }
            }
            return __shfl_sync(0xffffffffu, r, 0);
        };

        // The exponentials of a row are taken against a reference m_ref that is fixed once (below) and
        // then left alone: the division by the row sum at the end makes any reference exact, and
        // floating point keeps the relative precision as long as nothing overflows, i.e. as long as
        // no score exceeds the reference by more than 2^kRefHeadroom.  So the four threads of a row
        // do not talk to each other while they work.  A thread that does meet such a score asks for a
        // new reference: all warps of the quarter come here at their next tile boundary (or out of a
        // wait), with `released` = the first tile it has not handed to the tensor core yet (it has
        // handed over all its tiles below, and written nothing of that one).  Nothing of a tile is
        // consumed before it is handed over and the products are issued in tile order, so the smallest
        // `released` bounds what the accumulator holds; all then move their own state to the new
        // reference (a power-of-two factor, exact): running sum, their channels of O, and their P
        // tile if it is written but not yet consumed.
        int nrare = 0;                // meetings on bar_rare so far
        bool sum_published = false;   // this thread's share of the row sum is out for the final exchange
        auto move_reference = [&](int released, bool mine, float want) -> bool {
            s_cand[part * 128 + r_tile] = mine ? want : m_ref;
            if (lane == 0) s_rel[quarter * kParts + part] = released;
            __syncwarp();
            if (lane == 0) s_req[quarter] = 1;
            if (!meet(bar_rare, nrare++)) return false;
            int r_min = released;
            float m_new = m_ref;
#pragma unroll
            for (int c = 0; c < kParts; ++c) {
                r_min = min(r_min, s_rel[quarter * kParts + c]);
                m_new = fmaxf(m_new, s_cand[c * 128 + r_tile]);
            }
            if (part == 0 && lane == 0) s_req[quarter] = 0;
            // whole powers of two only, so that what is already rounded stays exact
            float alpha = 1.f;
            if (m_new > m_ref) {
                if (m_ref == -INFINITY) {
                    alpha = 0.f;
                } else {
                    const float steps = ceilf(m_new - m_ref);
                    m_new = m_ref + steps;
                    alpha = ptx::ex2(-steps);
                }
            }
            const bool any_change = __any_sync(0xffffffffu, alpha != 1.f);
            if (any_change) {
                if (r_min > 0) {
                    // PV(r_min - 1) must have landed.  Every tile below r_min is handed over, tile r_min
                    // is not, and the products are issued in order: PV(r_min + 3) cannot have been
                    // issued, so barrier (r_min - 1) % 4 has seen (r_min - 1) / 4 phases or one more.
                    if (!warp_wait(bar_pv_done + 8 * ((r_min - 1) & 3), ((r_min - 1) >> 2) & 1, kDevTimeoutSoftmaxO, a.status,
                                   s_abort, lane))
                        return false;
                    ptx::fence_after_sync();
                    uint32_t regs[32];              // this thread's 32 of the row's 128 channels
                    ptx::tmem_ld32(t_o, regs);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e) regs[e] = __float_as_uint(__uint_as_float(regs[e]) * alpha);
                    ptx::tmem_st32(t_o, regs);
                }
                // written, not consumed: this warp's tiles in [r_min, released) (at most one: its half of the P buffer)
                for (int t = r_min; t < released; ++t) {
                    if ((t & 1) != grp) continue;
#pragma unroll
                    for (int blk = 0; blk < 2; ++blk) {
                        uint32_t pk[16];
                        ptx::tmem_ld16(t_p + blk * 16, pk);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const float lo = __uint_as_float(pk[e] << 16) * alpha;
                            const float hi = __uint_as_float(pk[e] & 0xffff0000u) * alpha;
                            pk[e] = ptx::pack_bf16x2(lo, hi);
                        }
                        ptx::tmem_st16(t_p + blk * 16, pk);
                    }
                }
                l *= alpha;
                ptx::tmem_st_wait();
                ptx::fence_before_sync();
            }
            m_ref = m_new;
            if (sum_published) s_sum[part * 128 + r_tile] = l;    // (ordered by the meeting below)
            return meet(bar_rare, nrare++);
        };

        // The row's reference: the largest of its first 32 scores of the item's first tile (-inf: the
        // row sees no key of this split, since the visible keys of a row are a prefix).  The
        // thread that owns those columns reads it off and publishes it; nobody can ask for a new
        // reference before, so the other threads of the row simply wait for it.
        if (part == 1 && ntiles > 0) {
            // The other half of the first tile's group does not wait for the publisher: it reads the
            // same 32 scores itself (the buffer is not given back before all of the group's warps
            // have arrived) and gets the same maximum, ~1 K cycles before the published one could
            // reach it: the first product starts that much earlier.
            ok = warp_wait(bar_s_full, 0, kDevTimeoutSoftmaxS, a.status, s_abort, lane);
            if (ok) {
                ptx::fence_after_sync();
                int lim0 = bound - w.j0 * kTileN;
                if (TAIL) lim0 = w.j0 < nct ? w.L - 1 - w.j0 * kTileN : bound - (w.j0 - nct) * kTileN;
                m_ref = first_block_reference(t_lane, lim0, a.scale_log2);
            }
        } else if (part != 0) {
            ok = warp_wait(bar_ref + 8 * quarter, 0, kDevTimeoutSoftmaxX, a.status, s_abort, lane);
            if (ok) m_ref = s_ref[r_tile];
        }

        for (int jj = grp; jj < ntiles && ok; jj += 2) {
            const uint32_t use = (uint32_t)(jj >> 1);           // how often this group's buffers were used before
            while (ok) {
                const int r = (jj == 0 && part == 0)
                                  ? (warp_wait(bar_s_full, 0, kDevTimeoutSoftmaxS, a.status, s_abort, lane) ? 0 : 2)
                                  : wait_or_request(bar_s_full + 8 * grp, use & 1, kDevTimeoutSoftmaxS);
                if (r == 0) break;
                ok = (r == 1) && move_reference(jj, false, 0.f);
            }
            if (!ok) break;
            ptx::fence_after_sync();
            if (quarter == 0 && half == 0 && lane == 0 && jj < 9) EVLN_STAMP(2 + jj);

            // this thread's 64 scores of the row into registers; the score buffer goes back to the tensor core
            uint32_t s[64];
#pragma unroll
            for (int blk = 0; blk < 2; ++blk) ptx::tmem_ld32(t_s + blk * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[blk * 32]));
            ptx::tmem_ld_wait();
            if (quarter == 0 && half == 0 && lane == 0 && jj == 4) EVLN_STAMP(56);
            ptx::fence_before_sync();
            if (ptx::elect_one()) {
                if (CTAS == 2) ptx::mbar_arrive_cluster(s_free0); else ptx::mbar_arrive(s_free0);
            }

            // columns 0..lim of this thread's 64 are visible
            int lim = bound - (w.j0 + jj) * kTileN - half * 64;
            if (TAIL) {
                const int j = w.j0 + jj;
                lim = (j < nct ? w.L - 1 - j * kTileN : bound - (j - nct) * kTileN) - half * 64;
            }
            if (!__all_sync(0xffffffffu, lim >= 63)) {
#pragma unroll
                for (int blk = 0; blk < 2; ++blk) mask32(&s[blk * 32], lim - blk * 32);   // -inf: masked keys (and stale slots) drop out
            }
            float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
            rowmax32(&s[0], mx0, mx1, mx2, mx3);
            if (jj == 0 && part == 0) {
                m_ref = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * a.scale_log2;   // scale > 0
                s_ref[r_tile] = m_ref;
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bar_ref + 8 * quarter);
            }
            rowmax32(&s[32], mx0, mx1, mx2, mx3);
            const float tmax = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * a.scale_log2;
            bool over = tmax > m_ref + kRefHeadroom;
            while (ok && __any_sync(0xffffffffu, over)) {
                ok = move_reference(jj, over, tmax);
                over = tmax > m_ref + kRefHeadroom;
            }
            if (!ok) break;
            if (quarter == 0 && half == 0 && lane == 0 && jj == 4) EVLN_STAMP(57);

            // P = 2^(s*scale_log2 - m_ref) (packed FMA), row sum (packed add), bf16 P.  The P buffer is
            // free once the product of tile jj - 2 has landed: this thread handed that tile over only a
            // moment ago, so it asks after the first block of exponentials, not before.
            const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
            const uint64_t negm2 = ptx::pack2(neg_m, neg_m);
            uint64_t sum2a = ptx::pack2(0.f, 0.f), sum2b = sum2a;
            {
                uint32_t pk[16];
                exp32(&s[0], pk, scale2, negm2, sum2a, sum2b);
                while (ok && jj >= 2) {
                    const int r = wait_or_request(bar_pv_done + 8 * ((jj - 2) & 3), ((jj - 2) >> 2) & 1, kDevTimeoutSoftmaxO);
                    if (r == 0) break;
                    // (the meeting moves what is written and handed over; this block is still in
                    // registers, so it follows by the same power of two)
                    const float m_old = m_ref;
                    ok = (r == 1) && move_reference(jj, false, 0.f);
                    if (ok && m_ref != m_old) {
                        const float alpha = (m_old == -INFINITY) ? 0.f : ptx::ex2(m_old - m_ref);
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const float lo = __uint_as_float(pk[e] << 16) * alpha;
                            const float hi = __uint_as_float(pk[e] & 0xffff0000u) * alpha;
                            pk[e] = ptx::pack_bf16x2(lo, hi);
                        }
                        float a0, a1, b0, b1;
                        ptx::unpack2(sum2a, a0, a1);
                        ptx::unpack2(sum2b, b0, b1);
                        sum2a = ptx::pack2(a0 * alpha, a1 * alpha);
                        sum2b = ptx::pack2(b0 * alpha, b1 * alpha);
                    }
                }
                if (!ok) break;
                ptx::fence_after_sync();
                if (quarter == 0 && half == 0 && lane == 0 && jj == 4) EVLN_STAMP(58);
                ptx::tmem_st16(t_p, pk);
            }
            {
                // (the reference may have moved while waiting)
                const float neg_m2 = (m_ref == -INFINITY) ? 0.f : -m_ref;
                const uint64_t negm2b = ptx::pack2(neg_m2, neg_m2);
                uint32_t pk[16];
                exp32(&s[32], pk, scale2, negm2b, sum2a, sum2b);
                ptx::tmem_st16(t_p + 16, pk);
            }
            {
                float a0, a1, b0, b1;
                ptx::unpack2(sum2a, a0, a1);
                ptx::unpack2(sum2b, b0, b1);
                l += (a0 + a1) + (b0 + b1);
            }
            if (quarter == 0 && half == 0 && lane == 0 && jj == 4) EVLN_STAMP(59);
            ptx::tmem_st_wait();
            ptx::fence_before_sync();
            if (quarter == 0 && half == 0 && lane == 0 && jj == 4) EVLN_STAMP(63);
            if (ptx::elect_one()) {
                if (CTAS == 2) ptx::mbar_arrive_cluster(p_full0); else ptx::mbar_arrive(p_full0);
            }
            if (quarter == 0 && half == 0 && lane == 0 && jj < 9) EVLN_STAMP(11 + jj);
        }

        // All tiles handed over.  The row sum is the sum of the row's four threads (same reference in
        // all): they exchange it while the last product is still running.  A slower warp of the
        // quarter may still ask for a new reference until it arrives here too; a warp that serves such
        // a request after publishing its share publishes the rescaled share again (inside move_reference).
        if (ok) {
            s_sum[part * 128 + r_tile] = l;
            sum_published = true;
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar_xch + 8 * quarter);
        }
        while (ok) {
            const int r = wait_or_request(bar_xch + 8 * quarter, 0, kDevTimeoutSoftmaxX);
            if (r == 0) break;
            ok = (r == 1) && move_reference(ntiles, false, 0.f);
        }
        // nobody of the quarter can ask any more; the last product
        if (ok) ok = warp_wait(bar_o_full, 0, kDevTimeoutSoftmaxO, a.status, s_abort, lane);
        if (ok) {
            ptx::fence_after_sync();
            if (warp == 4 && lane == 0) EVLN_STAMP(60);
            l = (s_sum[r_tile] + s_sum[128 + r_tile]) + (s_sum[256 + r_tile] + s_sum[384 + r_tile]);
            // Epilogue: O/l goes out through shared memory so that global stores are whole
            // 128-byte lines.  The K ring is dead (its last consumer has completed); each warp
            // stages its 32 rows x 32 channels there, rows 144 bytes apart.
            const float inv = (l > 0.f) ? 1.f / l : 0.f;
            const int wrow0 = quarter << 5;
            uint8_t* stage = smem_gen + kSmemKOff + (warp - 4) * (32 * 144);
            const int first_row = row0 + wrow0;                              // episode-local
            const int rows_here = rows_valid - first_row;                    // may be <= 0 or > 32
            const long prow0 = ((long)w.slot * a.Hkv + w.g) * a.rows + w.row_base + first_row;
            {
                float* gbase = a.o_part + prow0 * 128 + part * 32;
                uint32_t regs[32];
                ptx::tmem_ld32(t_o, regs);
                ptx::tmem_ld_wait();
                float4* srow = reinterpret_cast<float4*>(stage + lane * 144);
#pragma unroll
                for (int e = 0; e < 32; e += 4)
                    srow[e >> 2] = make_float4(__uint_as_float(regs[e]) * inv, __uint_as_float(regs[e + 1]) * inv,
                                               __uint_as_float(regs[e + 2]) * inv, __uint_as_float(regs[e + 3]) * inv);
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = i * 4 + (lane >> 3);
                    if (r < rows_here) {
                        const float4 v = *reinterpret_cast<const float4*>(stage + r * 144 + (lane & 7) * 16);
                        *reinterpret_cast<float4*>(gbase + (long)r * 128 + (lane & 7) * 4) = v;
                    }
                }
            }
            if (row_valid && part == 0)
                a.lse_part[prow0 + lane] = (l > 0.f) ? (m_ref + log2f(l)) * 0.6931471805599453f : -INFINITY;
            if (warp == 4 && lane == 0) EVLN_STAMP(61);
        }
    }
    }

    // ---- teardown: nobody leaves while the other CTA may still touch this CTA's memory ----
    ptx::fence_before_sync();
    __syncthreads();
    if (CTAS == 2) {
        // every cross-CTA signal and tensor-memory access of the item is behind the last commit both
        // CTAs waited for; this meeting only keeps either CTA from freeing the pair's tensor memory early
        ptx::cluster_arrive_relaxed();
        ptx::cluster_wait();
    }
    if (warp == 1) {
        ptx::fence_after_sync();
        if (CTAS == 2) ptx::tmem_dealloc_pair(tmem, 512); else ptx::tmem_dealloc(tmem, 512);
        if (lane == 0) EVLN_STAMP(62);
    }
}

// One CTA pair per work item (256 query rows): any number of rows, contiguous or paged cache.
template <bool PAGED, typename LensT>
__global__ void __launch_bounds__(kTcThreads, 1)
attn_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const TcAttnArgs a,
                 const __grid_constant__ LensT lens)
{
    attn_tc_body<PAGED, false, LensT, 2>(tm_q, tm_k, tm_v, nullptr, nullptr, a, lens);
}

// CTA pairs over a batch of items that share a prefix of one contiguous cache and bring their own
// new tokens in a separate buffer (the action chunks of a packed sequence, Sec. 3.3).
__global__ void __launch_bounds__(kTcThreads, 1)
attn_tail_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_kt,
                 const __grid_constant__ CUtensorMap tm_vt, const TcAttnArgs a,
                 const __grid_constant__ BatchLens lens)
{
    attn_tc_body<false, true, BatchLens, 2>(tm_q, tm_k, tm_v, &tm_kt, &tm_vt, a, lens);
}

// One CTA per work item, for steps whose rows per kv head fit one 128-row tile (the few action
// tokens that follow a frame, Sec. 3.1): the KV range is cut into as many splits as there are SMs,
// and each CTA streams whole K/V tiles, so the step runs at the rate HBM delivers the cache.
__global__ void __launch_bounds__(kTcThreads, 1)
attn_solo_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const TcAttnArgs a)
{
    attn_tc_body<false, false, NoLens, 1>(tm_q, tm_k, tm_v, nullptr, nullptr, a, NoLens{});
}

}  // namespace evln
