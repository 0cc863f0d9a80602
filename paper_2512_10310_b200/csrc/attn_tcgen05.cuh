// Split-KV step attention on the 5th-generation tensor cores (bf16, head_dim 128).
//
// Sec. 3.2 leaves one attention per step: the n new (rotated) queries against all L+n cached
// keys.  With grouped-query attention the G query heads of a kv head share its K/V, so the
// G*n query rows of a kv head are packed row-major (row = token*G + head-in-group) and cut
// into 128-row MMA tiles.  One CTA owns a UNIT of two such tiles and one contiguous range of
// 128-key KV tiles (a split); it writes normalised partial outputs + log-sum-exps that the
// combine kernel merges.
//
// CTA anatomy (384 threads, 1 CTA/SM, ~225 KB shared memory, all 512 TMEM columns):
//   warp 0      TMA producer: Q tiles once, then K_j, V_j tiles through a 5-deep ring of
//               32 KB stages (128B-swizzled, two 64-channel halves per tile); no multicast.
//   warp 1      MMA issuer (one lane): S = Q K^T  (SS, both K-major) into TMEM,
//               O += P V (A = P from TMEM, B = V MN-major).  The two query tiles ping-pong:
//               while the softmax warps work on tile A's scores the tensor pipe runs tile B.
//   warps 4-7   softmax of tile A, warps 8-11 softmax of tile B: one thread per query row
//               (TMEM lane), so row max / row sum need no cross-thread traffic; P is written
//               back over S as packed bf16; O is rescaled in TMEM only when the row maximum
//               grew by more than 2^8 (the final division by the row sum makes that exact).
//   warps 2-3   idle (register donors).
// TMEM columns: S_A [0,128) (P_A aliases [0,64)), S_B [128,256), O_A [256,384), O_B [384,512).
//
// Every mbarrier wait is bounded: on expiry the CTA records a code in the device status
// word, raises a shared abort flag, drains its own TMA loads, frees TMEM and returns.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace evln {

#ifdef EVLN_TIMELINE
#define EVLN_STAMP(slot) do { if (a.timeline && (slot) < 64) a.timeline[(long)blockIdx.x * 64 + (slot)] = clock64(); } while (0)
#else
#define EVLN_STAMP(slot) do { } while (0)
#endif

constexpr int kTcThreads = 384;
constexpr int kStages = 5;
constexpr int kTileBytes = kTileN * 128 * 2;          // 128 rows x 128 channels x bf16
constexpr int kHalfBytes = kTileBytes / 2;            // one 64-channel half: 128 rows x 128 B
constexpr int kSmemQOff = 0;
constexpr int kSmemKVOff = 2 * kTileBytes;
constexpr int kSmemBarOff = kSmemKVOff + kStages * kTileBytes;
constexpr int kSmemBarBytes = 256;
constexpr int kTcSmemBytes = kSmemBarOff + kSmemBarBytes + 1024;   // + slack to align to 1024
constexpr long long kWaitLimitCycles = 2000000000LL;  // ~1 s at boost clocks

constexpr uint32_t kColS = 0, kColO = 256;            // + 128 * tile

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
#ifdef EVLN_TIMELINE
    long long* timeline;      // debug builds only: 32 clock stamps per CTA
#endif
};

// --- descriptors --------------------------------------------------------------------------

// kind::f16 instruction descriptor: fp32 accumulate, bf16 A and B, M = 128, N = 128.
__device__ __forceinline__ constexpr uint32_t make_idesc(bool b_mn_major)
{
    return (1u << 4)                       // D format: f32
           | (1u << 7)                     // A format: bf16
           | (1u << 10)                    // B format: bf16
           | ((b_mn_major ? 1u : 0u) << 16)
           | ((uint32_t)(kTileN >> 3) << 17)
           | ((uint32_t)(kTileM >> 4) << 24);
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
                                             volatile int* s_abort)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t spins = 0;
    while (!ptx::mbar_try_wait(bar, parity)) {
        if ((++spins & 0x3f) == 0) {
            if (*s_abort) return false;
            if (clock64() - t0 > kWaitLimitCycles) {
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

// --- softmax pieces on one 32-column register block of a score row ---------------------------

__device__ __forceinline__ void mask32(uint32_t (&s)[32], int lim)
{
#pragma unroll
    for (int e = 0; e < 32; ++e)
        if (e > lim) s[e] = 0xff800000u;
}

__device__ __forceinline__ void rowmax32(const uint32_t (&s)[32], float& m0, float& m1, float& m2, float& m3)
{
#pragma unroll
    for (int e = 0; e < 32; e += 8) {
        m0 = ptx::max3(m0, __uint_as_float(s[e]), __uint_as_float(s[e + 1]));
        m1 = ptx::max3(m1, __uint_as_float(s[e + 2]), __uint_as_float(s[e + 3]));
        m2 = ptx::max3(m2, __uint_as_float(s[e + 4]), __uint_as_float(s[e + 5]));
        m3 = ptx::max3(m3, __uint_as_float(s[e + 6]), __uint_as_float(s[e + 7]));
    }
}

// p = 2^(s*scale + negm) for 32 columns, accumulated into two packed sums, written to TMEM as
// 16 columns of packed bf16 pairs
__device__ __forceinline__ void exp32_store(const uint32_t (&s)[32], uint32_t taddr, uint64_t scale2,
                                            uint64_t negm2, uint64_t& sum2a, uint64_t& sum2b)
{
    uint32_t packed[16];
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
        const uint64_t xa = ptx::fma2(ptx::pack2(__uint_as_float(s[e]), __uint_as_float(s[e + 1])), scale2, negm2);
        const uint64_t xb = ptx::fma2(ptx::pack2(__uint_as_float(s[e + 2]), __uint_as_float(s[e + 3])), scale2, negm2);
        float x0, x1, x2, x3;
        ptx::unpack2(xa, x0, x1);
        ptx::unpack2(xb, x2, x3);
        const float p0 = ptx::ex2(x0), p1 = ptx::ex2(x1), p2 = ptx::ex2(x2), p3 = ptx::ex2(x3);
        sum2a = ptx::add2(sum2a, ptx::pack2(p0, p1));
        sum2b = ptx::add2(sum2b, ptx::pack2(p2, p3));
        packed[e >> 1] = ptx::pack_bf16x2(p0, p1);
        packed[(e >> 1) + 1] = ptx::pack_bf16x2(p2, p3);
    }
    ptx::tmem_st16(taddr, packed);
}

// --- work decoding ------------------------------------------------------------------------

struct WorkItem {
    int b, g, unit, slot;     // episode, kv head, unit within the episode, partial slot
    int L, n;                 // episode lengths
    int row_base;             // first packed row of the episode within the kv head
    int j0, j1;               // KV tile range
};

template <bool PAGED, typename LensT>
__device__ __forceinline__ WorkItem decode_work(const TcAttnArgs& a, const LensT& lens, int bid)
{
    WorkItem w;
    if (!PAGED) {
        w.b = 0;
        w.unit = bid % a.units_per_head;
        w.g = (bid / a.units_per_head) % a.Hkv;
        w.slot = bid / (a.units_per_head * a.Hkv);
        w.L = a.cache_len;
        w.n = a.num_new;
        w.row_base = 0;
        const int nkv = unit_kv_tiles(w.L, w.n, a.G, w.unit, kUnitRows);
        w.j0 = (int)((long)w.slot * nkv / a.num_splits);
        w.j1 = (int)((long)(w.slot + 1) * nkv / a.num_splits);
    } else {
        int rem = bid;
        int b = 0;
        for (; b < a.batch; ++b) {
            const int n_b = lens.new_off[b + 1] - lens.new_off[b];
            const int units = ceil_div(n_b * a.G, kUnitRows);
            int per_head = 0;
            for (int u = 0; u < units; ++u)
                per_head += ceil_div(unit_kv_tiles(lens.cache_len[b], n_b, a.G, u, kUnitRows), a.chunk_tiles);
            if (rem < per_head * a.Hkv) {
                w.b = b;
                w.L = lens.cache_len[b];
                w.n = n_b;
                w.row_base = lens.new_off[b] * a.G;
                w.g = rem / per_head;
                rem -= w.g * per_head;
                for (int u = 0; u < units; ++u) {
                    const int nkv = unit_kv_tiles(w.L, n_b, a.G, u, kUnitRows);
                    const int S = ceil_div(nkv, a.chunk_tiles);
                    if (rem < S) {
                        w.unit = u;
                        w.slot = rem;
                        w.j0 = (int)((long)rem * nkv / S);
                        w.j1 = (int)((long)(rem + 1) * nkv / S);
                        break;
                    }
                    rem -= S;
                }
                break;
            }
            rem -= per_head * a.Hkv;
        }
        if (b == a.batch) { w.b = -1; w.j0 = w.j1 = 0; w.g = w.unit = w.slot = 0; w.L = w.n = w.row_base = 0; }
    }
    return w;
}

// --- the kernel ---------------------------------------------------------------------------

template <bool PAGED, typename LensT>
__global__ void __launch_bounds__(kTcThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const TcAttnArgs a,
               const __grid_constant__ LensT lens)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));

    const uint32_t bar_base = smem_base + kSmemBarOff;
    const uint32_t bar_q_full = bar_base;                    // [2]
    const uint32_t bar_kv_full = bar_base + 16;              // [kStages]
    const uint32_t bar_kv_empty = bar_kv_full + 8 * kStages; // [kStages]
    const uint32_t bar_s_full = bar_kv_empty + 8 * kStages;  // [2]
    const uint32_t bar_p_full = bar_s_full + 16;             // [2]
    const uint32_t bar_o_full = bar_p_full + 16;             // [2]
    const uint32_t tmem_slot = bar_o_full + 16;              // uint32
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem_gen + kSmemBarOff + (tmem_slot - bar_base) + 8);
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem_gen + kSmemBarOff + (tmem_slot - bar_base));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) EVLN_STAMP(0);

    const WorkItem w = decode_work<PAGED, LensT>(a, lens, blockIdx.x);
    if (PAGED && w.b < 0) return;

    const int rows_valid = w.n * a.G;                 // packed rows of this episode
    const int row0 = w.unit * kUnitRows;              // first row of the unit (episode-local)
    const bool tile_b_active = row0 + kTileM < rows_valid;
    const int ntiles = w.j1 - w.j0;
    const int nq = tile_b_active ? 2 : 1;

    // A split with no KV tiles (more splits than tiles): its partials are "empty".
    if (ntiles <= 0) {
        ptx::grid_dependency_wait();
        if (warp >= 4 && warp < 4 + 4 * nq) {
            const int x = (warp - 4) >> 2;
            const int r = row0 + x * kTileM + ((warp & 3) << 5) + lane;
            if (r < rows_valid) {
                const long prow = ((long)w.slot * a.Hkv + w.g) * a.rows + w.row_base + r;
                float4* o = reinterpret_cast<float4*>(a.o_part + prow * 128);
                for (int c = 0; c < 32; ++c) o[c] = make_float4(0.f, 0.f, 0.f, 0.f);
                a.lse_part[prow] = -INFINITY;
            }
        }
        return;
    }

    // ---- setup: barriers, TMEM; the producer starts loading before the CTA-wide sync ----
    // K/V ring entry k (K_j0, V_j0, K_j0+1, V_j0+1, ...): one tile of 32 KB into stage k % kStages
    auto issue_kv = [&](int k) {
        const int stage = k % kStages;
        const int j = w.j0 + (k >> 1);
        const CUtensorMap* map = (k & 1) ? &tm_v : &tm_k;
        const uint32_t dst = smem_base + kSmemKVOff + stage * kTileBytes;
        const uint32_t bar = bar_kv_full + 8 * stage;
        ptx::mbar_expect_tx(bar, kTileBytes);
        if (!PAGED) {
            ptx::tma_load_3d(dst, map, bar, 0, j * kTileN, w.g);
            ptx::tma_load_3d(dst + kHalfBytes, map, bar, 64, j * kTileN, w.g);
        } else {
            // two 64-token pages per tile; a tile that ends in the episode's last page
            // re-reads that page for its second half (masked, but finite)
            const int npages = (w.L + w.n + 63) >> 6;
            const int p0 = 2 * j;
            const int p1 = (p0 + 1 < npages) ? p0 + 1 : p0;
            const int* pt = a.page_table + (long)w.b * a.max_pages;
            const int pg0 = pt[p0], pg1 = pt[p1];
            ptx::tma_load_4d(dst, map, bar, 0, 0, w.g, pg0);
            ptx::tma_load_4d(dst + 8192, map, bar, 0, 0, w.g, pg1);
            ptx::tma_load_4d(dst + kHalfBytes, map, bar, 64, 0, w.g, pg0);
            ptx::tma_load_4d(dst + kHalfBytes + 8192, map, bar, 64, 0, w.g, pg1);
        }
    };
    const int kv_total = 2 * ntiles;
    const int kv_early = kv_total < kStages ? kv_total : kStages;   // entries that need no free-stage wait

    if (threadIdx.x == 32) {
        ptx::prefetch_tensormap(&tm_q);
        ptx::prefetch_tensormap(&tm_k);
        ptx::prefetch_tensormap(&tm_v);
    }
    if (threadIdx.x == 0) {
        ptx::mbar_init(bar_q_full, 1);
        ptx::mbar_init(bar_q_full + 8, 1);
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(bar_kv_full + 8 * s, 1);
            ptx::mbar_init(bar_kv_empty + 8 * s, 1);
        }
        for (int x = 0; x < 2; ++x) {
            ptx::mbar_init(bar_s_full + 8 * x, 1);
            ptx::mbar_init(bar_p_full + 8 * x, 128);
            ptx::mbar_init(bar_o_full + 8 * x, 1);
        }
        *s_abort = 0;
        ptx::fence_barrier_init();
        // everything this CTA reads or writes in global memory follows this thread's loads, so one
        // wait here orders the whole CTA after the kernels it depends on
        ptx::grid_dependency_wait();
        // first loads go out now: they only need the barriers this thread has just initialised
        const int qrow = w.row_base + row0;
        for (int x = 0; x < nq; ++x) {
            const uint32_t dst = smem_base + kSmemQOff + x * kTileBytes;
            ptx::mbar_expect_tx(bar_q_full + 8 * x, kTileBytes);
            ptx::tma_load_3d(dst, &tm_q, bar_q_full + 8 * x, 0, qrow + x * kTileM, w.g);
            ptx::tma_load_3d(dst + kHalfBytes, &tm_q, bar_q_full + 8 * x, 64, qrow + x * kTileM, w.g);
            if (x == 0) issue_kv(0);
        }
        for (int k = 1; k < kv_early; ++k) issue_kv(k);
    }
    if (warp == 1) {
        ptx::tmem_alloc(tmem_slot, 512);
        ptx::tmem_relinquish();
    }
    ptx::fence_before_sync();
    __syncthreads();
    ptx::fence_after_sync();
    const uint32_t tmem = *s_tmem;
    ptx::grid_launch_dependents();
    if (threadIdx.x == 0) EVLN_STAMP(1);

    // register budget: the producer / MMA warpgroup gives registers to the softmax warpgroups,
    // which hold a whole 128-column score row per thread
    if (warp < 4) ptx::setmaxnreg_dec<80>();

    if (warp == 0) {
        // ================= TMA producer (remaining ring entries) =================
        if (lane == 0) {
            bool ok = true;
            int issued = kv_early;
            for (int k = kv_early; k < kv_total; ++k) {
                const int stage = k % kStages;
                const uint32_t parity = ((k / kStages) & 1) ^ 1;
                ok = wait_bounded(bar_kv_empty + 8 * stage, parity, kDevTimeoutProducer, a.status, s_abort);
                if (!ok) break;
                issue_kv(k);
                ++issued;
            }
            if (!ok || *s_abort) {
                // drain: every load this thread issued must have landed before the CTA may exit
                for (int k = (issued > kStages ? issued - kStages : 0); k < issued; ++k) {
                    const int stage = k % kStages;
                    const uint32_t parity = (k / kStages) & 1;
                    const long long t0 = clock64();
                    while (!ptx::mbar_try_wait(bar_kv_full + 8 * stage, parity))
                        if (clock64() - t0 > kWaitLimitCycles) break;
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ================= MMA issuer =================
        const uint32_t idesc_s = make_idesc(false);
        const uint32_t idesc_pv = make_idesc(true);
        bool ok = true;
        uint32_t p_parity = 0;       // both tiles' P barriers advance in lockstep per iteration

        // every wait is taken by the whole warp and its outcome made uniform
        auto wait_u = [&](uint32_t bar, uint32_t parity, int code) -> bool {
            return warp_wait(bar, parity, code, a.status, s_abort, lane);
        };
        auto wait_kv = [&](int kk) -> bool {
            return wait_u(bar_kv_full + 8 * (kk % kStages), (kk / kStages) & 1, kDevTimeoutMmaKV);
        };
        // descriptors differ only in their address field (units of 16 bytes): build them once
        const uint64_t qdesc0 = make_sdesc(smem_base + kSmemQOff, 16, 1024);
        const uint64_t kdesc0 = make_sdesc(smem_base + kSmemKVOff, 16, 1024);            // K-major
        const uint64_t vdesc0 = make_sdesc(smem_base + kSmemKVOff, kHalfBytes, 1024);    // MN-major
        auto issue_s = [&](int x, int kk) {      // S_x = Q_x K^T, K in ring entry kk
            if (lane == 0) {
                const uint64_t qd = qdesc0 + (uint64_t)((x * kTileBytes) >> 4);
                const uint64_t kd = kdesc0 + (uint64_t)(((kk % kStages) * kTileBytes) >> 4);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t off = (uint64_t)(((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4);
                    ptx::mma_ss(tmem + kColS + x * 128, qd + off, kd + off, idesc_s, ks > 0);
                }
                ptx::mma_commit(bar_s_full + 8 * x);
            }
        };
        auto issue_pv = [&](int x, int kk, bool accumulate) {   // O_x (+)= P_x V, V in ring entry kk
            if (lane == 0) {
                const uint64_t vd = vdesc0 + (uint64_t)(((kk % kStages) * kTileBytes) >> 4);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    ptx::mma_ts(tmem + kColO + x * 128, tmem + kColS + x * 128 + ks * 8,
                                vd + (uint64_t)((ks * 2048) >> 4), idesc_pv, accumulate || ks > 0);
                }
            }
        };
        auto release = [&](int kk) {
            if (lane == 0) ptx::mma_commit(bar_kv_empty + 8 * (kk % kStages));
        };

        ok = wait_u(bar_q_full, 0, kDevTimeoutMmaQ);
        if (ok && nq == 2) ok = wait_u(bar_q_full + 8, 0, kDevTimeoutMmaQ);
        if (ok) ok = wait_kv(0);
        if (ok) {
            ptx::fence_after_sync();
            issue_s(0, 0);
            if (nq == 2) issue_s(1, 0);
            release(0);
            __syncwarp();
        }
        for (int it = 0; it < ntiles && ok; ++it) {
            const int kv = 2 * it + 1;           // ring entry of V_it
            const int kn = 2 * it + 2;           // ring entry of K_{it+1}
            const bool more = it + 1 < ntiles;
            ok = wait_kv(kv);
            if (ok && more) ok = wait_kv(kn);
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                if (x < nq && ok) {
                    ok = wait_u(bar_p_full + 8 * x, p_parity, kDevTimeoutMmaP);
                    if (ok) {
                        if (lane == 0 && it < 6) EVLN_STAMP(32 + 4 * it + 2 * x);
                        ptx::fence_after_sync();
                        issue_pv(x, kv, it > 0);
                        if (more) {
                            issue_s(x, kn);
                        } else if (lane == 0) {
                            ptx::mma_commit(bar_o_full + 8 * x);
                        }
                        if (x == nq - 1) {
                            release(kv);
                            if (more) release(kn);
                        }
                        if (lane == 0 && it < 6) EVLN_STAMP(33 + 4 * it + 2 * x);
                        __syncwarp();
                    }
                }
            }
            p_parity ^= 1;
        }
    } else if (warp >= 4 && warp < 4 + 4 * nq) {
        // ================= softmax + epilogue =================
        ptx::setmaxnreg_inc<208>();
        const int x = (warp - 4) >> 2;                     // which query tile
        const int quarter = warp & 3;                      // TMEM lane quarter of this warp
        const int r_tile = (quarter << 5) + lane;          // row within the tile = TMEM lane
        const int r_local = row0 + x * kTileM + r_tile;    // packed row within the episode
        const bool row_valid = r_local < rows_valid;
        const int bound = row_valid ? w.L + r_local / a.G : -1;   // last visible key index
        const uint32_t t_lane = tmem + ((uint32_t)(quarter << 5) << 16);
        const uint32_t t_s = t_lane + kColS + x * 128;
        const uint32_t t_o = t_lane + kColO + x * 128;

        float m_ref = -INFINITY;      // reference maximum (log2 domain) the exponentials use
        float l = 0.f;                // running sum of exponentials
        bool ok = true;
        const uint64_t scale2 = ptx::pack2(a.scale_log2, a.scale_log2);

        for (int it = 0; it < ntiles; ++it) {
            ok = warp_wait(bar_s_full + 8 * x, it & 1, kDevTimeoutSoftmaxS, a.status, s_abort, lane);
            if (!ok) break;
            ptx::fence_after_sync();
            if (warp == 4 && lane == 0) EVLN_STAMP(2 + 2 * it);

            const int j = w.j0 + it;
            const int lim = bound - j * kTileN;            // columns 0..lim are visible
            const bool no_mask = __all_sync(0xffffffffu, lim >= kTileN - 1);

            // the whole score row of this thread: 128 columns in registers, one wait
            uint32_t sA[32], sB[32], sC[32], sD[32];
            ptx::tmem_ld32(t_s, sA);
            ptx::tmem_ld32(t_s + 32, sB);
            ptx::tmem_ld32(t_s + 64, sC);
            ptx::tmem_ld32(t_s + 96, sD);
            ptx::tmem_ld_wait();
            if (warp == 4 && lane == 0 && it < 6) EVLN_STAMP(14 + 2 * it);
            if (!no_mask) {        // -inf: masked keys (and stale slots) drop out
                mask32(sA, lim);
                mask32(sB, lim - 32);
                mask32(sC, lim - 64);
                mask32(sD, lim - 96);
            }

            // row maximum (3-input max, four independent chains)
            float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
            rowmax32(sA, mx0, mx1, mx2, mx3);
            rowmax32(sB, mx0, mx1, mx2, mx3);
            rowmax32(sC, mx0, mx1, mx2, mx3);
            rowmax32(sD, mx0, mx1, mx2, mx3);
            const float tmax = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * a.scale_log2;   // scale > 0

            // move the reference maximum only when it would otherwise lose range
            float alpha = 1.f;
            const bool grow = tmax > m_ref + 8.f;           // also true for the first finite tile
            if (grow) {
                alpha = (m_ref == -INFINITY) ? 0.f : ptx::ex2(m_ref - tmax);
                m_ref = tmax;
                l *= alpha;
            }
            if (it > 0 && __any_sync(0xffffffffu, grow)) {
                // O_x holds PV sums up to tile it-1 (complete: the S commit follows them)
                uint32_t regs[32];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    ptx::tmem_ld32(t_o + c * 32, regs);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e) regs[e] = __float_as_uint(__uint_as_float(regs[e]) * alpha);
                    ptx::tmem_st32(t_o + c * 32, regs);
                }
            }

            if (warp == 4 && lane == 0 && it < 6) EVLN_STAMP(15 + 2 * it);
            // P = 2^(s*scale_log2 - m_ref) (packed FMA), row sum (packed add), bf16 P over the S columns
            const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
            const uint64_t negm2 = ptx::pack2(neg_m, neg_m);
            uint64_t sum2a = ptx::pack2(0.f, 0.f), sum2b = sum2a;
            exp32_store(sA, t_s, scale2, negm2, sum2a, sum2b);
            exp32_store(sB, t_s + 16, scale2, negm2, sum2a, sum2b);
            exp32_store(sC, t_s + 32, scale2, negm2, sum2a, sum2b);
            exp32_store(sD, t_s + 48, scale2, negm2, sum2a, sum2b);
            {
                float a0, a1, b0, b1;
                ptx::unpack2(sum2a, a0, a1);
                ptx::unpack2(sum2b, b0, b1);
                l += (a0 + a1) + (b0 + b1);
            }
            ptx::tmem_st_wait();
            ptx::fence_before_sync();
            ptx::mbar_arrive(bar_p_full + 8 * x);
            if (warp == 4 && lane == 0) EVLN_STAMP(3 + 2 * it);
        }

        if (ok) {
            ok = warp_wait(bar_o_full + 8 * x, 0, kDevTimeoutSoftmaxO, a.status, s_abort, lane);
        }
        if (ok) {
            ptx::fence_after_sync();
            if (warp == 4 && lane == 0) EVLN_STAMP(28);
            // Epilogue: O/l goes out through shared memory so that global stores are whole
            // 128-byte lines.  This tile's Q buffer is dead (its last S MMA has completed); each
            // warp stages its own 32 rows there, 32 channels at a time, rows 144 bytes apart.
            const float inv = (l > 0.f) ? 1.f / l : 0.f;
            const int wrow0 = quarter << 5;
            uint8_t* stage = smem_gen + kSmemQOff + x * kTileBytes + wrow0 * 144;
            const int first_row = row0 + x * kTileM + wrow0;                 // episode-local
            const int rows_here = rows_valid - first_row;                    // may be <= 0 or > 32
            const long prow0 = ((long)w.slot * a.Hkv + w.g) * a.rows + w.row_base + first_row;
            float* gbase = a.o_part + prow0 * 128;
            uint32_t regs[32];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                ptx::tmem_ld32(t_o + c * 32, regs);
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
                        *reinterpret_cast<float4*>(gbase + (long)r * 128 + c * 32 + (lane & 7) * 4) = v;
                    }
                }
                __syncwarp();
            }
            if (row_valid)
                a.lse_part[prow0 + lane] = (l > 0.f) ? (m_ref + log2f(l)) * 0.6931471805599453f : -INFINITY;
            if (warp == 4 && lane == 0) EVLN_STAMP(29);
        }
    }

    // ---- teardown ----
    ptx::fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::fence_after_sync();
        ptx::tmem_dealloc(tmem, 512);
        if (lane == 0) EVLN_STAMP(30);
    }
}

}  // namespace evln
