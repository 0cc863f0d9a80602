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
#define EVLN_STAMP(slot) do { if (a.timeline && (slot) < 32) a.timeline[(long)blockIdx.x * 32 + (slot)] = clock64(); } while (0)
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

    // ---- setup: barriers, TMEM ----
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
        ptx::prefetch_tensormap(&tm_q);
        ptx::prefetch_tensormap(&tm_k);
        ptx::prefetch_tensormap(&tm_v);
    }
    if (warp == 1) {
        ptx::tmem_alloc(tmem_slot, 512);
        ptx::tmem_relinquish();
    }
    ptx::fence_before_sync();
    __syncthreads();
    ptx::fence_after_sync();
    const uint32_t tmem = *s_tmem;
    if (threadIdx.x == 0) EVLN_STAMP(1);

    if (warp == 0) {
        // ================= TMA producer =================
        bool ok = true;
        int issued = 0;
        if (lane == 0) {
            const int qrow = w.row_base + row0;
            for (int x = 0; x < nq; ++x) {
                const uint32_t dst = smem_base + kSmemQOff + x * kTileBytes;
                ptx::mbar_expect_tx(bar_q_full + 8 * x, kTileBytes);
                ptx::tma_load_3d(dst, &tm_q, bar_q_full + 8 * x, 0, qrow + x * kTileM, w.g);
                ptx::tma_load_3d(dst + kHalfBytes, &tm_q, bar_q_full + 8 * x, 64, qrow + x * kTileM, w.g);
            }
            const int total = 2 * ntiles;          // K_j0, V_j0, K_j0+1, V_j0+1, ...
            for (int k = 0; k < total && ok; ++k) {
                const int stage = k % kStages;
                const uint32_t parity = ((k / kStages) & 1) ^ 1;
                ok = wait_bounded(bar_kv_empty + 8 * stage, parity, kDevTimeoutProducer, a.status, s_abort);
                if (!ok) break;
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
                ++issued;
            }
            if (!ok) {
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
            const bool r = wait_bounded(bar, parity, code, a.status, s_abort);
            return __all_sync(0xffffffffu, r);
        };
        auto wait_kv = [&](int kk) -> bool {
            return wait_u(bar_kv_full + 8 * (kk % kStages), (kk / kStages) & 1, kDevTimeoutMmaKV);
        };
        auto issue_s = [&](int x, int kk) {      // S_x = Q_x K^T, K in ring entry kk
            if (lane == 0) {
                const uint32_t qa = smem_base + kSmemQOff + x * kTileBytes;
                const uint32_t kb = smem_base + kSmemKVOff + (kk % kStages) * kTileBytes;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t off = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
                    ptx::mma_ss(tmem + kColS + x * 128, make_sdesc(qa + off, 16, 1024),
                                make_sdesc(kb + off, 16, 1024), idesc_s, ks > 0);
                }
                ptx::mma_commit(bar_s_full + 8 * x);
            }
        };
        auto issue_pv = [&](int x, int kk, bool accumulate) {   // O_x (+)= P_x V, V in ring entry kk
            if (lane == 0) {
                const uint32_t vb = smem_base + kSmemKVOff + (kk % kStages) * kTileBytes;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    ptx::mma_ts(tmem + kColO + x * 128, tmem + kColS + x * 128 + ks * 8,
                                make_sdesc(vb + ks * 2048, kHalfBytes, 1024), idesc_pv,
                                accumulate || ks > 0);
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
                        __syncwarp();
                    }
                }
            }
            p_parity ^= 1;
        }
    } else if (warp >= 4 && warp < 4 + 4 * nq) {
        // ================= softmax + epilogue =================
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
        uint32_t regs[32];

        for (int it = 0; it < ntiles; ++it) {
            ok = wait_bounded(bar_s_full + 8 * x, it & 1, kDevTimeoutSoftmaxS, a.status, s_abort);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            ptx::fence_after_sync();
            if (warp == 4 && lane == 0) EVLN_STAMP(2 + 2 * it);

            const int j = w.j0 + it;
            const int lim = bound - j * kTileN;            // columns 0..lim are visible
            const bool no_mask = __all_sync(0xffffffffu, lim >= kTileN - 1);

            // pass 1: row maximum of the visible scores
            float tmax = -INFINITY;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                ptx::tmem_ld32(t_s + c * 32, regs);
                ptx::tmem_ld_wait();
                if (no_mask) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) tmax = fmaxf(tmax, __uint_as_float(regs[e]));
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (c * 32 + e <= lim) tmax = fmaxf(tmax, __uint_as_float(regs[e]));
                }
            }
            tmax *= a.scale_log2;                           // scale > 0: max commutes with it

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
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    ptx::tmem_ld32(t_o + c * 32, regs);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e) regs[e] = __float_as_uint(__uint_as_float(regs[e]) * alpha);
                    ptx::tmem_st32(t_o + c * 32, regs);
                }
            }

            // pass 2: P = 2^(s*scale_log2 - m_ref), row sum, bf16 P over the S columns
            const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
            float lsum = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                ptx::tmem_ld32(t_s + c * 32, regs);
                ptx::tmem_ld_wait();
                uint32_t packed[16];
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    float p0 = ptx::ex2(fmaf(__uint_as_float(regs[e]), a.scale_log2, neg_m));
                    float p1 = ptx::ex2(fmaf(__uint_as_float(regs[e + 1]), a.scale_log2, neg_m));
                    if (!no_mask) {
                        if (c * 32 + e > lim) p0 = 0.f;
                        if (c * 32 + e + 1 > lim) p1 = 0.f;
                    }
                    lsum += p0 + p1;
                    packed[e >> 1] = ptx::pack_bf16x2(p0, p1);
                }
                ptx::tmem_st16(t_s + c * 16, packed);
            }
            l += lsum;
            ptx::tmem_st_wait();
            ptx::fence_before_sync();
            ptx::mbar_arrive(bar_p_full + 8 * x);
            if (warp == 4 && lane == 0) EVLN_STAMP(3 + 2 * it);
        }

        if (ok) {
            ok = wait_bounded(bar_o_full + 8 * x, 0, kDevTimeoutSoftmaxO, a.status, s_abort);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            ptx::fence_after_sync();
            if (warp == 4 && lane == 0) EVLN_STAMP(28);
            const float inv = (l > 0.f) ? 1.f / l : 0.f;
            const long prow = ((long)w.slot * a.Hkv + w.g) * a.rows + w.row_base + r_local;
            float4* dst = reinterpret_cast<float4*>(a.o_part + prow * 128);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                ptx::tmem_ld32(t_o + c * 32, regs);
                ptx::tmem_ld_wait();
                if (row_valid) {
#pragma unroll
                    for (int e = 0; e < 32; e += 4)
                        dst[c * 8 + (e >> 2)] = make_float4(__uint_as_float(regs[e]) * inv,
                                                            __uint_as_float(regs[e + 1]) * inv,
                                                            __uint_as_float(regs[e + 2]) * inv,
                                                            __uint_as_float(regs[e + 3]) * inv);
                }
            }
            if (row_valid)
                a.lse_part[prow] = (l > 0.f) ? (m_ref + log2f(l)) * 0.6931471805599453f : -INFINITY;
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
