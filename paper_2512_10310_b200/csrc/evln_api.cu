// C-ABI entry points of libevln (contract: include/evln.h).  Host-side validation, the split
// schedule, tensor-map encoding and kernel launches; no allocation in the per-step calls.
#include "../../include/evln.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "attn_simt.cuh"
#include "attn_pair.cuh"
#include "combine.cuh"
#include "gather_rope.cuh"
#include "common.cuh"
#include "rope_append.cuh"

using namespace evln;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct evlnContext {
    int device;
    int num_sms;
    int last_cuda_error;
    int* d_status;
    EncodeTiledFn encode;
};

#ifdef EVLN_TIMELINE
// debug builds only (see timeline_debug.cuh): where the attention kernel leaves its clock stamps
extern "C" int evlnDebugSetTimeline(void* p)
{
    long long* v = (long long*)p;
    return (int)cudaMemcpyToSymbol(evln::g_timeline_dev, &v, sizeof(v));
}
#endif

namespace {

// Every kernel is launched with programmatic stream serialisation: its prologue may overlap the
// tail of the previous kernel in the stream; each kernel waits (griddepcontrol.wait) before it
// touches global memory.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                       Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// The attention kernel runs as clusters of two CTAs (one CTA pair per work item).
template <typename... KArgs, typename... Args>
cudaError_t launch_pair_pdl(void (*kernel)(KArgs...), dim3 grid, size_t smem, cudaStream_t st, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;                 // x: two CTAs per work item
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// The attention kernels move registers between their warpgroups (setmaxnreg) inside the pool a CTA
// gets at launch; a request the pool cannot serve would wait for ever.  The plan in attn_pair.cuh is
// made for kRegsLaunch registers per thread: refuse to run a build that came out differently.
bool attention_register_pool_ok()
{
    cudaFuncAttributes fa;
    const void* kernels[4] = {(const void*)attn_pair_kernel<false, NoLens>, (const void*)attn_pair_kernel<true, BatchLens>,
                              (const void*)attn_solo_kernel, (const void*)attn_tail_kernel};
    for (const void* k : kernels) {
        if (cudaFuncGetAttributes(&fa, k) != cudaSuccess) return false;
        if (fa.numRegs != kRegsLaunch) return false;
    }
    return true;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int elem_bytes(int dtype) { return dtype == EVLN_BF16 ? 2 : 4; }

evlnStatus_t cuda_fail(evlnHandle_t h, cudaError_t e)
{
    h->last_cuda_error = (int)e;
    return EVLN_CUDA_ERROR;
}

// The handle's device must be current when work is launched: the kernels' attributes and the
// tensor maps belong to that device's context.
bool device_is_current(evlnHandle_t h)
{
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == h->device;
}

// An optional position table must cover the positions [first, first + count) of the call.
bool rope_table_covers(const void* table, int table_first, int table_count, long first, long count)
{
    if (!table) return true;
    if (!aligned16(table) || table_first < 0 || table_count < 0) return false;
    return (long)table_first <= first && first + count <= (long)table_first + table_count;
}

evlnStatus_t check_step_params(evlnHandle_t h, const evlnStepParams* p)
{
    if (!h || !p) return EVLN_INVALID_VALUE;
    if (p->struct_size != sizeof(evlnStepParams)) return EVLN_INVALID_VALUE;
    if (p->dtype != EVLN_BF16 && p->dtype != EVLN_F32) return EVLN_INVALID_VALUE;
    if (p->num_q_heads <= 0 || p->num_kv_heads <= 0 || p->num_q_heads % p->num_kv_heads != 0)
        return EVLN_INVALID_VALUE;
    if (p->cache_len < 0 || p->num_new < 0 || p->cache_capacity < 0) return EVLN_INVALID_VALUE;
    if (!(p->rope_theta > 0.0) || !(p->softmax_scale >= 0.f)) return EVLN_INVALID_VALUE;
    if (p->num_splits < 0 || p->num_splits > kMaxSplits) return EVLN_INVALID_VALUE;
    if (p->kernel != EVLN_KERNEL_AUTO && p->kernel != EVLN_KERNEL_SIMT) return EVLN_INVALID_VALUE;
    if (p->head_dim != 64 && p->head_dim != 128) return EVLN_NOT_SUPPORTED;
    if ((long)p->cache_len + p->num_new > (long)p->cache_capacity) return EVLN_CACHE_FULL;
    if ((long)p->num_new * p->num_q_heads / p->num_kv_heads > (1 << 24)) return EVLN_NOT_SUPPORTED;
    if (!rope_table_covers(p->rope_table, p->rope_table_first_pos, p->rope_table_count, p->cache_len, p->num_new))
        return EVLN_INVALID_VALUE;
    return EVLN_OK;
}

inline bool use_tensor_kernel(const evlnStepParams* p)
{
    return p->kernel == EVLN_KERNEL_AUTO && p->dtype == EVLN_BF16 && p->head_dim == 128;
}

// Cost model of the split-KV schedule of the tensor-core kernel: work items (unit x split) run
// in waves of one CTA pair per two SMs, each walks ceil(nkv / S) KV tiles plus a fixed
// prologue/epilogue; every extra split adds combine traffic.
int choose_splits_tc(int units_total, int nkv_max, int nkv_min, int num_sms)
{
    int best = 1;
    double best_cost = 1e30;
    const int pairs = num_sms / 2 > 0 ? num_sms / 2 : 1;
    const int smax = nkv_min < kMaxSplits ? (nkv_min < 1 ? 1 : nkv_min) : kMaxSplits;
    for (int s = 1; s <= smax; ++s) {
        const double waves = ceil((double)units_total * s / pairs);
        // per work item: set-up, first-tile latency, partial write-out and teardown cost about as
        // much as 7 KV tiles (measured); every split adds about half a tile of combine work
        const double cost = waves * (ceil((double)nkv_max / s) + 7.0) + 0.5 * s;
        if (cost < best_cost - 1e-9) { best_cost = cost; best = s; }
    }
    return best;
}

// A step whose rows per kv head fit one 128-row tile (a few new tokens: the action tokens after a
// frame) runs one CTA per (kv head, split) instead of CTA pairs.
inline bool use_solo_kernel(const evlnStepParams* p)
{
    return use_tensor_kernel(p) && (long)p->num_new * (p->num_q_heads / p->num_kv_heads) <= kTileM;
}

// Split schedule of the one-CTA-per-item kernel: the step is bound by streaming K/V once, so the
// KV range is spread over all SMs; an item's fixed cost is about 3 tiles of streaming, and a split
// adds a partial row set of R rows to merge.
int choose_splits_solo(int Hkv, int R, int nkv, int num_sms)
{
    int best = 1;
    double best_cost = 1e30;
    const int smax = nkv < kMaxSplits ? (nkv < 1 ? 1 : nkv) : kMaxSplits;
    for (int s = 1; s <= smax; ++s) {
        const double waves = ceil((double)Hkv * s / num_sms);
        const double cost = waves * (ceil((double)nkv / s) + 3.0) + 0.5 * s * R / 256.0;
        if (cost < best_cost - 1e-9) { best_cost = cost; best = s; }
    }
    return best;
}

int resolve_splits(evlnHandle_t h, const evlnStepParams* p)
{
    if (p->num_new == 0) return 1;
    if (p->num_splits > 0) return p->num_splits;
    const int G = p->num_q_heads / p->num_kv_heads;
    const int R = p->num_new * G;
    const int T = p->cache_len + p->num_new;
    if (use_solo_kernel(p))
        return choose_splits_solo(p->num_kv_heads, R, ceil_div(T, kTileN), h->num_sms);
    if (use_tensor_kernel(p)) {
        const int units = ceil_div(R, kUnitRows);
        const int nkv_max = unit_kv_tiles(p->cache_len, p->num_new, G, units - 1, kUnitRows);
        const int nkv_min = unit_kv_tiles(p->cache_len, p->num_new, G, 0, kUnitRows);
        return choose_splits_tc(units * p->num_kv_heads, nkv_max, nkv_min, h->num_sms);
    }
    const int blocks = ceil_div(R, 4) * p->num_kv_heads;
    int s = ceil_div(2 * h->num_sms, blocks);
    const int cap = ceil_div(T, 64);
    if (s > cap) s = cap;
    if (s > kMaxSplits) s = kMaxSplits;
    if (s < 1) s = 1;
    return s;
}

size_t partial_bytes(int splits, int Hkv, long rows, int D)
{
    return round_up((size_t)splits * Hkv * rows * (D + 1) * sizeof(float), 256);
}

bool encode_map(evlnHandle_t h, CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims,
                const cuuint64_t* strides_bytes, const cuuint32_t* box)
{
    cuuint32_t ones[5] = {1, 1, 1, 1, 1};
    CUresult r = h->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base),
                           dims, strides_bytes, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

evlnStatus_t check_paged_params(evlnHandle_t h, const evlnPagedParams* p, const int* lens, const int* offs)
{
    if (!h || !p || !lens || !offs) return EVLN_INVALID_VALUE;
    if (p->struct_size != sizeof(evlnPagedParams)) return EVLN_INVALID_VALUE;
    if (p->num_q_heads <= 0 || p->num_kv_heads <= 0 || p->num_q_heads % p->num_kv_heads != 0)
        return EVLN_INVALID_VALUE;
    if (p->batch < 1 || p->num_pages < 1 || p->max_pages_per_seq < 1 || p->kv_chunk_tiles < 0)
        return EVLN_INVALID_VALUE;
    if (!(p->rope_theta > 0.0) || !(p->softmax_scale >= 0.f)) return EVLN_INVALID_VALUE;
    if (p->dtype != EVLN_BF16 || p->head_dim != 128 || p->page_size != 64 || p->batch > kMaxBatch)
        return EVLN_NOT_SUPPORTED;
    if (offs[0] != 0) return EVLN_INVALID_VALUE;
    for (int b = 0; b < p->batch; ++b) {
        if (lens[b] < 0 || offs[b + 1] < offs[b]) return EVLN_INVALID_VALUE;
        const long tokens = (long)lens[b] + (offs[b + 1] - offs[b]);
        if ((tokens + p->page_size - 1) / p->page_size > p->max_pages_per_seq) return EVLN_CACHE_FULL;
        if (!rope_table_covers(p->rope_table, p->rope_table_first_pos, p->rope_table_count, lens[b], offs[b + 1] - offs[b]))
            return EVLN_INVALID_VALUE;
    }
    if ((long)offs[p->batch] * p->num_q_heads / p->num_kv_heads > (1 << 24)) return EVLN_NOT_SUPPORTED;
    return EVLN_OK;
}

// KV tiles of unit u of a batch item: paged episode, or item sharing a cache prefix (tail).
inline int batch_kv_tiles(bool tail, int L, int n, int G, int u)
{
    return tail ? tail_kv_tiles(L, n, G, u, kUnitRows) : unit_kv_tiles(L, n, G, u, kUnitRows);
}

// Work-item size (KV tiles) and the largest split count of a batch.
void batch_schedule(int num_sms, int G, int Hkv, int batch, const int* lens, const int* offs, bool tail,
                    int kv_chunk_tiles, int* chunk_tiles, int* max_splits, long* items)
{
    long total = 0;
    int nkv_max = 1;
    for (int b = 0; b < batch; ++b) {
        const int n = offs[b + 1] - offs[b];
        const int units = ceil_div(n * G, kUnitRows);
        for (int u = 0; u < units; ++u) {
            const int nkv = batch_kv_tiles(tail, lens[b], n, G, u);
            total += nkv;
            if (nkv > nkv_max) nkv_max = nkv;
        }
    }
    total *= Hkv;
    int chunk = kv_chunk_tiles;
    if (chunk <= 0) {
        const long pairs = num_sms / 2 > 0 ? num_sms / 2 : 1;
        chunk = (int)((total + pairs * 4 - 1) / (pairs * 4));
        if (chunk < 8) chunk = 8;
    }
    if (chunk < ceil_div(nkv_max, kMaxSplits)) chunk = ceil_div(nkv_max, kMaxSplits);
    long cnt = 0;
    for (int b = 0; b < batch; ++b) {
        const int n = offs[b + 1] - offs[b];
        const int units = ceil_div(n * G, kUnitRows);
        for (int u = 0; u < units; ++u) cnt += ceil_div(batch_kv_tiles(tail, lens[b], n, G, u), chunk);
    }
    *chunk_tiles = chunk;
    *max_splits = ceil_div(nkv_max, chunk);
    *items = cnt * Hkv;
}

void paged_schedule(evlnHandle_t h, const evlnPagedParams* p, const int* lens, const int* offs,
                    int* chunk_tiles, int* max_splits, long* items)
{
    batch_schedule(h->num_sms, p->num_q_heads / p->num_kv_heads, p->num_kv_heads, p->batch, lens, offs, false,
                   p->kv_chunk_tiles, chunk_tiles, max_splits, items);
}

// chunk_tiles > 0: also the first attention work item of every episode (items are numbered
// episode by episode: kv head, unit, split)
void fill_batch_lens(BatchLens* bl, int G, int Hkv, int batch, const int* lens, const int* offs, int chunk_tiles, bool tail)
{
    memset(bl, 0, sizeof(*bl));
    for (int b = 0; b < batch; ++b) bl->cache_len[b] = lens[b];
    for (int b = 0; b <= batch; ++b) bl->new_off[b] = offs[b];
    for (int b = batch + 1; b <= kMaxBatch; ++b) bl->new_off[b] = offs[batch];
    if (chunk_tiles > 0) {
        int items = 0;
        for (int b = 0; b < batch; ++b) {
            bl->item_off[b] = items;
            const int n = offs[b + 1] - offs[b];
            const int units = ceil_div(n * G, kUnitRows);
            int per_head = 0;
            for (int u = 0; u < units; ++u) per_head += ceil_div(batch_kv_tiles(tail, lens[b], n, G, u), chunk_tiles);
            items += per_head * Hkv;
        }
        for (int b = batch; b <= kMaxBatch; ++b) bl->item_off[b] = items;
    }
}

void fill_lens(BatchLens* bl, const evlnPagedParams* p, const int* lens, const int* offs, int chunk_tiles = 0)
{
    fill_batch_lens(bl, p->num_q_heads / p->num_kv_heads, p->num_kv_heads, p->batch, lens, offs, chunk_tiles, false);
}

template <typename T>
evlnStatus_t launch_combine(evlnHandle_t h, const CombineArgs& args, int D, bool paged, const BatchLens* bl,
                            cudaStream_t st)
{
    CombineArgs a = args;
    a.div_g = make_fast_div((uint32_t)a.G);
    a.div_chunk = make_fast_div((uint32_t)(a.chunk_tiles > 0 ? a.chunk_tiles : 1));
    dim3 grid(ceil_div(a.rows, 4), a.Hkv);
    if (paged) {
        if (D == 128) launch_pdl(combine_kernel<T, 128, true, BatchLens>, dim3(grid), dim3(128), 0, st, a, *bl);
        else return EVLN_NOT_SUPPORTED;
    } else {
        NoLens nl = {};
        if (D == 128) launch_pdl(combine_kernel<T, 128, false, NoLens>, dim3(grid), dim3(128), 0, st, a, nl);
        else launch_pdl(combine_kernel<T, 64, false, NoLens>, dim3(grid), dim3(128), 0, st, a, nl);
    }
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? EVLN_OK : cuda_fail(h, e);
}

// The fields of RopeArgs that follow from the others (vec: elements per 16-byte vector).
void finish_rope_args(RopeArgs* a, int vec)
{
    a->G = a->Hq / a->Hkv;
    a->div_g = make_fast_div((uint32_t)a->G);
    a->vph_shift = 0;
    while ((1 << a->vph_shift) < a->D / 2 / vec) ++a->vph_shift;
    a->page_shift = 0;
    while ((1 << a->page_shift) < a->page_size) ++a->page_shift;
}

// The append kernel for `tokens` tokens.  Few enough to be one wave of two blocks per SM: one thread
// per work item (in whole warps, at most kRopeThreadsMax).  Else 256 threads.
template <typename T, bool PAGED, typename LensT>
void launch_rope_append(evlnHandle_t h, const RopeArgs& a, int tokens, cudaStream_t st, const LensT& lens)
{
    const bool few = tokens <= 2 * h->num_sms;
    int t = kRopeThreads;
    if (few) {
        const int items = ((a.Hq + a.Hkv) << a.vph_shift) + (a.Hkv << (a.vph_shift + 1));
        t = (items + 31) / 32 * 32;
        if (t > kRopeThreadsMax) t = kRopeThreadsMax;
        if (t < 64) t = 64;
    }
    launch_pdl(rope_append_kernel<T, PAGED, LensT>, dim3(tokens), dim3(t), 0, st, a, lens);
}

evlnStatus_t noalloc_status_word(int** word);     // defined with the allocation-free variant below

}  // namespace

extern "C" {

const char* evlnGetErrorString(evlnStatus_t s)
{
    switch (s) {
        case EVLN_OK: return "EVLN_OK";
        case EVLN_INVALID_VALUE: return "EVLN_INVALID_VALUE";
        case EVLN_NOT_SUPPORTED: return "EVLN_NOT_SUPPORTED";
        case EVLN_CACHE_FULL: return "EVLN_CACHE_FULL";
        case EVLN_WORKSPACE_TOO_SMALL: return "EVLN_WORKSPACE_TOO_SMALL";
        case EVLN_CUDA_ERROR: return "EVLN_CUDA_ERROR";
        case EVLN_DEVICE_TIMEOUT: return "EVLN_DEVICE_TIMEOUT";
    }
    return "EVLN_UNKNOWN_STATUS";
}

evlnStatus_t evlnCreate(evlnHandle_t* handle, int device)
{
    if (!handle) return EVLN_INVALID_VALUE;
    *handle = nullptr;
    evlnContext* h = new (std::nothrow) evlnContext();
    if (!h) return EVLN_CUDA_ERROR;
    h->device = device;
    h->last_cuda_error = 0;
    h->d_status = nullptr;
    h->encode = nullptr;
    int prev_device = -1;
    cudaError_t e = cudaGetDevice(&prev_device);
    if (e == cudaSuccess) e = cudaSetDevice(device);
    // whatever happens below, the caller's current device is put back
    struct Restore {
        int dev;
        ~Restore() { if (dev >= 0) cudaSetDevice(dev); }
    } restore{prev_device};
    cudaDeviceProp prop;
    if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, device);
    if (e != cudaSuccess) { delete h; return EVLN_CUDA_ERROR; }
    if (prop.major != 10) { delete h; return EVLN_NOT_SUPPORTED; }
    h->num_sms = prop.multiProcessorCount;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) { delete h; return EVLN_CUDA_ERROR; }
    h->encode = reinterpret_cast<EncodeTiledFn>(fn);
    e = cudaMalloc(&h->d_status, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(h->d_status, 0, sizeof(int));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(attn_pair_kernel<false, NoLens>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kTcSmemBytes);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(attn_pair_kernel<true, BatchLens>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kTcSmemBytes);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(attn_solo_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSoloSmemBytes);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(attn_tail_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemBytes);
    if (e == cudaSuccess && !attention_register_pool_ok()) {
        cudaFree(h->d_status);
        delete h;
        return EVLN_NOT_SUPPORTED;
    }
    if (e != cudaSuccess) {
        if (h->d_status) cudaFree(h->d_status);
        delete h;
        return EVLN_CUDA_ERROR;
    }
    *handle = h;
    return EVLN_OK;
}

evlnStatus_t evlnDestroy(evlnHandle_t h)
{
    if (!h) return EVLN_INVALID_VALUE;
    if (h->d_status) cudaFree(h->d_status);
    delete h;
    return EVLN_OK;
}

int evlnGetLastCudaError(evlnHandle_t h) { return h ? h->last_cuda_error : 0; }

evlnStatus_t evlnGetDeviceStatus(evlnHandle_t h, void* stream, int* device_status)
{
    if (!device_status) return EVLN_INVALID_VALUE;
    int* word = nullptr;
    if (h) {
        if (!device_is_current(h)) return EVLN_INVALID_VALUE;
        word = h->d_status;
    } else {
        // the allocation-free call's status word on the current device (part of the library image)
        evlnStatus_t s = noalloc_status_word(&word);
        if (s != EVLN_OK) return s;
    }
    cudaStream_t st = (cudaStream_t)stream;
    int v = 0;
    cudaError_t e = cudaMemcpyAsync(&v, word, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e == cudaSuccess && v != 0) e = cudaMemsetAsync(word, 0, sizeof(int), st);
    if (e != cudaSuccess) return h ? cuda_fail(h, e) : EVLN_CUDA_ERROR;
    *device_status = v;
    return v == 0 ? EVLN_OK : EVLN_DEVICE_TIMEOUT;
}

// A bounded wait on a barrier nobody arrives on: it must run out and leave its code in the status word.
__global__ void selftest_wait_kernel(int* status, long long limit_cycles)
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int s_abort;
    const uint32_t b = ptx::smem_u32(&bar);
    if (threadIdx.x == 0) {
        s_abort = 0;
        ptx::mbar_init(b, 1);
        ptx::fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) wait_bounded(b, 0, EVLN_SELFTEST_STATUS_CODE, status, &s_abort, limit_cycles);
    __syncthreads();
}

evlnStatus_t evlnSelfTestBoundedWait(evlnHandle_t h, long long limit_cycles, void* stream)
{
    if (!h || limit_cycles < 1000 || limit_cycles > 1000000000LL) return EVLN_INVALID_VALUE;
    if (!device_is_current(h)) return EVLN_INVALID_VALUE;
    selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(h->d_status, limit_cycles);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? EVLN_OK : cuda_fail(h, e);
}

size_t evlnRopeTableBytes(int head_dim, int count)
{
    if ((head_dim != 64 && head_dim != 128) || count < 0) return 0;
    return (size_t)count * (head_dim / 2) * sizeof(double2);
}

evlnStatus_t evlnRopeTable(evlnHandle_t h, int head_dim, double rope_theta, int first_pos, int count, void* table,
                           void* stream)
{
    if (!h || first_pos < 0 || count < 0 || !(rope_theta > 0.0)) return EVLN_INVALID_VALUE;
    if (head_dim != 64 && head_dim != 128) return EVLN_NOT_SUPPORTED;
    if (count == 0) return EVLN_OK;
    if (!table || !aligned16(table)) return EVLN_INVALID_VALUE;
    if (!device_is_current(h)) return EVLN_INVALID_VALUE;
    const long total = (long)count * (head_dim / 2);
    launch_pdl(rope_table_kernel, dim3((unsigned)((total + 127) / 128)), dim3(128), 0, (cudaStream_t)stream,
               (double2*)table, first_pos, count, head_dim, log2(rope_theta));
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? EVLN_OK : cuda_fail(h, e);
}

evlnStatus_t evlnStepNumSplits(evlnHandle_t h, const evlnStepParams* p, int* num_splits)
{
    evlnStatus_t s = check_step_params(h, p);
    if (s != EVLN_OK) return s;
    if (!num_splits) return EVLN_INVALID_VALUE;
    *num_splits = resolve_splits(h, p);
    return EVLN_OK;
}

evlnStatus_t evlnStepWorkspaceSize(evlnHandle_t h, const evlnStepParams* p, size_t* bytes)
{
    evlnStatus_t s = check_step_params(h, p);
    if (s != EVLN_OK) return s;
    if (!bytes) return EVLN_INVALID_VALUE;
    const long rows = (long)p->num_new * (p->num_q_heads / p->num_kv_heads);
    *bytes = partial_bytes(resolve_splits(h, p), p->num_kv_heads, rows, p->head_dim);
    return EVLN_OK;
}

evlnStatus_t evlnStepQRotSize(evlnHandle_t h, const evlnStepParams* p, size_t* bytes)
{
    evlnStatus_t s = check_step_params(h, p);
    if (s != EVLN_OK) return s;
    if (!bytes) return EVLN_INVALID_VALUE;
    *bytes = round_up((size_t)p->num_new * p->num_q_heads * p->head_dim * elem_bytes(p->dtype), 256);
    return EVLN_OK;
}

static evlnStatus_t rope_append_impl(evlnHandle_t h, const evlnStepParams* p, const void* q_new, const void* k_new,
                                     const void* v_new, long q_stride_tok, long k_stride_tok, long v_stride_tok,
                                     void* q_rot, void* k_cache, void* v_cache, void* stream, const PackedMap& map)
{
    evlnStatus_t s = check_step_params(h, p);
    if (s != EVLN_OK) return s;
    if (p->num_new == 0) return EVLN_OK;
    if (!q_new || !k_new || !v_new || !q_rot || !k_cache || !v_cache) return EVLN_INVALID_VALUE;
    if (!aligned16(q_new) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(q_rot) ||
        !aligned16(k_cache) || !aligned16(v_cache))
        return EVLN_INVALID_VALUE;
    if (!device_is_current(h)) return EVLN_INVALID_VALUE;
    const int vec = 16 / elem_bytes(p->dtype);
    if (q_stride_tok < (long)p->num_q_heads * p->head_dim || k_stride_tok < (long)p->num_kv_heads * p->head_dim ||
        v_stride_tok < (long)p->num_kv_heads * p->head_dim)
        return EVLN_INVALID_VALUE;
    if (q_stride_tok % vec || k_stride_tok % vec || v_stride_tok % vec) return EVLN_INVALID_VALUE;

    RopeArgs a = {};
    a.q_new = q_new; a.k_new = k_new; a.v_new = v_new;
    a.q_rot = q_rot; a.k_cache = k_cache; a.v_cache = v_cache;
    a.page_table = nullptr;
    a.q_stride = q_stride_tok; a.k_stride = k_stride_tok; a.v_stride = v_stride_tok;
    a.Hq = p->num_q_heads; a.Hkv = p->num_kv_heads; a.D = p->head_dim;
    a.cache_len = p->cache_len; a.num_new = p->num_new; a.cache_cap = p->cache_capacity;
    a.log2_theta = log2(p->rope_theta);
    a.table = (const double2*)p->rope_table;
    a.table_first = p->rope_table_first_pos;
    a.map = map;
    finish_rope_args(&a, p->dtype == EVLN_BF16 ? 8 : 4);
    NoLens nl = {};
    cudaStream_t st = (cudaStream_t)stream;
    if (p->dtype == EVLN_BF16)
        launch_rope_append<__nv_bfloat16, false, NoLens>(h, a, p->num_new, st, nl);
    else
        launch_rope_append<float, false, NoLens>(h, a, p->num_new, st, nl);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? EVLN_OK : cuda_fail(h, e);
}

evlnStatus_t evlnRopeAppend(evlnHandle_t h, const evlnStepParams* p, const void* q_new, const void* k_new,
                            const void* v_new, long q_stride_tok, long k_stride_tok, long v_stride_tok,
                            void* q_rot, void* k_cache, void* v_cache, void* stream)
{
    return rope_append_impl(h, p, q_new, k_new, v_new, q_stride_tok, k_stride_tok, v_stride_tok, q_rot, k_cache,
                            v_cache, stream, PackedMap{0, 0, 0, 0});
}

evlnStatus_t evlnStepAttention(evlnHandle_t h, const evlnStepParams* p, const void* q_rot, const void* k_cache,
                               const void* v_cache, void* workspace, size_t workspace_bytes, void* stream)
{
    evlnStatus_t s = check_step_params(h, p);
    if (s != EVLN_OK) return s;
    if (p->num_new == 0) return EVLN_OK;
    if (!q_rot || !k_cache || !v_cache || !workspace) return EVLN_INVALID_VALUE;
    if (!aligned16(q_rot) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(workspace))
        return EVLN_INVALID_VALUE;
    if (!device_is_current(h)) return EVLN_INVALID_VALUE;
    const int G = p->num_q_heads / p->num_kv_heads;
    const int R = p->num_new * G;
    const int D = p->head_dim;
    const int S = resolve_splits(h, p);
    if (workspace_bytes < partial_bytes(S, p->num_kv_heads, R, D)) return EVLN_WORKSPACE_TOO_SMALL;
    float* o_part = (float*)workspace;
    float* lse_part = o_part + (size_t)S * p->num_kv_heads * R * D;
    const float scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)D);
    cudaStream_t st = (cudaStream_t)stream;

    if (use_tensor_kernel(p)) {
        const int T = p->cache_len + p->num_new;
        CUtensorMap tm_q, tm_k, tm_v;
        {
            cuuint64_t dims[3] = {128, (cuuint64_t)R, (cuuint64_t)p->num_kv_heads};
            cuuint64_t strides[2] = {256, (cuuint64_t)R * 256};
            cuuint32_t box[3] = {64, 128, 1};
            if (!encode_map(h, &tm_q, q_rot, 3, dims, strides, box)) return EVLN_INVALID_VALUE;
        }
        {
            // rows past L+n read as zeros, so stale slots never reach the tensor core
            cuuint64_t dims[3] = {128, (cuuint64_t)T, (cuuint64_t)p->num_kv_heads};
            cuuint64_t strides[2] = {256, (cuuint64_t)p->cache_capacity * 256};
            // per CTA of a pair: half a K tile is 64 keys x all channels (two boxes), half a V tile
            // is 128 keys x 64 channels (one box)
            // (a CTA on its own takes whole tiles: two 128-key boxes each)
            cuuint32_t box_k[3] = {64, 64, 1};
            cuuint32_t box_v[3] = {64, 128, 1};
            if (!encode_map(h, &tm_k, k_cache, 3, dims, strides, use_solo_kernel(p) ? box_v : box_k)) return EVLN_INVALID_VALUE;
            if (!encode_map(h, &tm_v, v_cache, 3, dims, strides, box_v)) return EVLN_INVALID_VALUE;
        }
        TcAttnArgs a = {};
        a.o_part = o_part; a.lse_part = lse_part; a.page_table = nullptr; a.status = h->d_status;
        a.Hkv = p->num_kv_heads; a.G = G; a.rows = R;
        a.cache_len = p->cache_len; a.num_new = p->num_new; a.num_splits = S;
        a.units_per_head = use_solo_kernel(p) ? 1 : ceil_div(R, kUnitRows);
        a.scale_log2 = scale * 1.4426950408889634f;
        a.div_g = make_fast_div((uint32_t)G);
        a.div_s = make_fast_div((uint32_t)S);
        NoLens nl = {};
        // one work item per (unit, kv head, split): the kernels read it off the block index
        if (a.units_per_head > 32767 || p->num_kv_heads > 65535) return EVLN_NOT_SUPPORTED;
        if (use_solo_kernel(p))
            launch_pdl(attn_solo_kernel, dim3(1, p->num_kv_heads, S), dim3(kTcThreads), kSoloSmemBytes, st, tm_q, tm_k, tm_v, a);
        else
            launch_pair_pdl(attn_pair_kernel<false, NoLens>, dim3(2 * a.units_per_head, p->num_kv_heads, S), kTcSmemBytes, st,
                            tm_q, tm_k, tm_v, a, nl);
    } else {
        SimtAttnArgs a = {};
        a.q_rot = q_rot; a.k_cache = k_cache; a.v_cache = v_cache;
        a.o_part = o_part; a.lse_part = lse_part;
        a.Hkv = p->num_kv_heads; a.G = G; a.D = D;
        a.cache_len = p->cache_len; a.num_new = p->num_new; a.cache_cap = p->cache_capacity;
        a.num_splits = S; a.scale = scale;
        dim3 grid(ceil_div(R, 4), p->num_kv_heads, S);
        if (p->dtype == EVLN_BF16) {
            if (D == 128) launch_pdl(attn_simt_kernel<__nv_bfloat16, 128>, dim3(grid), dim3(128), 0, st, a);
            else launch_pdl(attn_simt_kernel<__nv_bfloat16, 64>, dim3(grid), dim3(128), 0, st, a);
        } else {
            if (D == 128) launch_pdl(attn_simt_kernel<float, 128>, dim3(grid), dim3(128), 0, st, a);
            else launch_pdl(attn_simt_kernel<float, 64>, dim3(grid), dim3(128), 0, st, a);
        }
    }
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? EVLN_OK : cuda_fail(h, e);
}


static evlnStatus_t step_combine_impl(evlnHandle_t h, const evlnStepParams* p, const void* workspace, void* out,
                                      float* lse_out, void* stream, const PackedMap& map)
{
    evlnStatus_t s = check_step_params(h, p);
    if (s != EVLN_OK) return s;
    if (p->num_new == 0) return EVLN_OK;
    if (!workspace || !out || !aligned16(workspace) || !aligned16(out)) return EVLN_INVALID_VALUE;
    if (!device_is_current(h)) return EVLN_INVALID_VALUE;
    const int G = p->num_q_heads / p->num_kv_heads;
    const int R = p->num_new * G;
    const int S = resolve_splits(h, p);
    CombineArgs a = {};
    a.o_part = (const float*)workspace;
    a.lse_part = a.o_part + (size_t)S * p->num_kv_heads * R * p->head_dim;
    a.out = out; a.lse_out = lse_out;
    a.Hkv = p->num_kv_heads; a.G = G; a.D = p->head_dim; a.rows = R; a.num_splits = S;
    a.map = map;
    cudaStream_t st = (cudaStream_t)stream;
    if (p->dtype == EVLN_BF16) return launch_combine<__nv_bfloat16>(h, a, p->head_dim, false, nullptr, st);
    return launch_combine<float>(h, a, p->head_dim, false, nullptr, st);
}

evlnStatus_t evlnStepCombine(evlnHandle_t h, const evlnStepParams* p, const void* workspace, void* out,
                             float* lse_out, void* stream)
{
    return step_combine_impl(h, p, workspace, out, lse_out, stream, PackedMap{0, 0, 0, 0});
}

evlnStatus_t evlnStep(evlnHandle_t h, const evlnStepParams* p, const void* q_new, const void* k_new,
                      const void* v_new, long q_stride_tok, long k_stride_tok, long v_stride_tok, void* q_rot,
                      void* k_cache, void* v_cache, void* workspace, size_t workspace_bytes, void* out,
                      float* lse_out, void* stream)
{
    evlnStatus_t s = check_step_params(h, p);
    if (s != EVLN_OK) return s;
    if (p->num_new == 0) return EVLN_OK;
    // every argument is checked before the first launch, so a rejected call has done nothing
    if (!workspace || !out || !aligned16(workspace) || !aligned16(out)) return EVLN_INVALID_VALUE;
    const long rows = (long)p->num_new * (p->num_q_heads / p->num_kv_heads);
    if (workspace_bytes < partial_bytes(resolve_splits(h, p), p->num_kv_heads, rows, p->head_dim))
        return EVLN_WORKSPACE_TOO_SMALL;
    s = evlnRopeAppend(h, p, q_new, k_new, v_new, q_stride_tok, k_stride_tok, v_stride_tok, q_rot, k_cache, v_cache,
                       stream);
    if (s != EVLN_OK) return s;
    s = evlnStepAttention(h, p, q_rot, k_cache, v_cache, workspace, workspace_bytes, stream);
    if (s != EVLN_OK) return s;
    return evlnStepCombine(h, p, workspace, out, lse_out, stream);
}

// ---- paged -------------------------------------------------------------------------------

evlnStatus_t evlnPagedWorkspaceSize(evlnHandle_t h, const evlnPagedParams* p, const int* h_cache_lens,
                                    const int* h_new_offsets, size_t* bytes)
{
    evlnStatus_t s = check_paged_params(h, p, h_cache_lens, h_new_offsets);
    if (s != EVLN_OK) return s;
    if (!bytes) return EVLN_INVALID_VALUE;
    int chunk, smax;
    long items;
    paged_schedule(h, p, h_cache_lens, h_new_offsets, &chunk, &smax, &items);
    const long rows = (long)h_new_offsets[p->batch] * (p->num_q_heads / p->num_kv_heads);
    *bytes = partial_bytes(smax, p->num_kv_heads, rows, p->head_dim);
    return EVLN_OK;
}

evlnStatus_t evlnPagedRopeAppend(evlnHandle_t h, const evlnPagedParams* p, const void* q_new, const void* k_new,
                                 const void* v_new, const int* h_cache_lens, const int* h_new_offsets,
                                 const int* d_page_table, void* q_rot, void* k_pool, void* v_pool, void* stream)
{
    evlnStatus_t s = check_paged_params(h, p, h_cache_lens, h_new_offsets);
    if (s != EVLN_OK) return s;
    const int total = h_new_offsets[p->batch];
    if (total == 0) return EVLN_OK;
    if (!q_new || !k_new || !v_new || !d_page_table || !q_rot || !k_pool || !v_pool) return EVLN_INVALID_VALUE;
    if (!aligned16(q_new) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(q_rot) ||
        !aligned16(k_pool) || !aligned16(v_pool))
        return EVLN_INVALID_VALUE;
    if (!device_is_current(h)) return EVLN_INVALID_VALUE;
    RopeArgs a = {};
    a.q_new = q_new; a.k_new = k_new; a.v_new = v_new;
    a.q_rot = q_rot; a.k_cache = k_pool; a.v_cache = v_pool; a.page_table = d_page_table;
    a.q_stride = (long)p->num_q_heads * p->head_dim;
    a.k_stride = a.v_stride = (long)p->num_kv_heads * p->head_dim;
    a.Hq = p->num_q_heads; a.Hkv = p->num_kv_heads; a.D = p->head_dim;
    a.num_new = total; a.batch = p->batch; a.page_size = p->page_size; a.max_pages = p->max_pages_per_seq;
    a.log2_theta = log2(p->rope_theta);
    a.table = (const double2*)p->rope_table;
    a.table_first = p->rope_table_first_pos;
    finish_rope_args(&a, 8);
    BatchLens bl;
    fill_lens(&bl, p, h_cache_lens, h_new_offsets);
    launch_rope_append<__nv_bfloat16, true, BatchLens>(h, a, total, (cudaStream_t)stream, bl);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? EVLN_OK : cuda_fail(h, e);
}

evlnStatus_t evlnPagedStepAttention(evlnHandle_t h, const evlnPagedParams* p, const void* q_rot,
                                    const void* k_pool, const void* v_pool, const int* h_cache_lens,
                                    const int* h_new_offsets, const int* d_page_table, void* workspace,
                                    size_t workspace_bytes, void* stream)
{
    evlnStatus_t s = check_paged_params(h, p, h_cache_lens, h_new_offsets);
    if (s != EVLN_OK) return s;
    const int total = h_new_offsets[p->batch];
    if (total == 0) return EVLN_OK;
    if (!q_rot || !k_pool || !v_pool || !d_page_table || !workspace) return EVLN_INVALID_VALUE;
    if (!aligned16(q_rot) || !aligned16(k_pool) || !aligned16(v_pool) || !aligned16(workspace))
        return EVLN_INVALID_VALUE;
    if (!device_is_current(h)) return EVLN_INVALID_VALUE;
    const int G = p->num_q_heads / p->num_kv_heads;
    const long rows = (long)total * G;
    int chunk, smax;
    long items;
    paged_schedule(h, p, h_cache_lens, h_new_offsets, &chunk, &smax, &items);
    if (workspace_bytes < partial_bytes(smax, p->num_kv_heads, rows, 128)) return EVLN_WORKSPACE_TOO_SMALL;
    if (items <= 0 || items > 0x3fffffffL) return EVLN_NOT_SUPPORTED;

    CUtensorMap tm_q, tm_k, tm_v;
    {
        cuuint64_t dims[3] = {128, (cuuint64_t)rows, (cuuint64_t)p->num_kv_heads};
        cuuint64_t strides[2] = {256, (cuuint64_t)rows * 256};
        cuuint32_t box[3] = {64, 128, 1};
        if (!encode_map(h, &tm_q, q_rot, 3, dims, strides, box)) return EVLN_INVALID_VALUE;
    }
    {
        cuuint64_t dims[4] = {128, 64, (cuuint64_t)p->num_kv_heads, (cuuint64_t)p->num_pages};
        cuuint64_t strides[3] = {256, 64 * 256, (cuuint64_t)p->num_kv_heads * 64 * 256};
        cuuint32_t box[4] = {64, 64, 1, 1};
        if (!encode_map(h, &tm_k, k_pool, 4, dims, strides, box)) return EVLN_INVALID_VALUE;
        if (!encode_map(h, &tm_v, v_pool, 4, dims, strides, box)) return EVLN_INVALID_VALUE;
    }
    const float scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf(128.f);
    TcAttnArgs a = {};
    a.o_part = (float*)workspace;
    a.lse_part = a.o_part + (size_t)smax * p->num_kv_heads * rows * 128;
    a.page_table = d_page_table; a.status = h->d_status;
    a.Hkv = p->num_kv_heads; a.G = G; a.rows = (int)rows;
    a.batch = p->batch; a.max_pages = p->max_pages_per_seq; a.chunk_tiles = chunk;
    a.scale_log2 = scale * 1.4426950408889634f;
    a.div_g = make_fast_div((uint32_t)G);
    a.div_s = make_fast_div(1u);
    BatchLens bl;
    fill_lens(&bl, p, h_cache_lens, h_new_offsets, chunk);
    if (bl.item_off[p->batch] != (int)items) return EVLN_INVALID_VALUE;
    launch_pair_pdl(attn_pair_kernel<true, BatchLens>, dim3(2 * (int)items), kTcSmemBytes, (cudaStream_t)stream, tm_q, tm_k,
                    tm_v, a, bl);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? EVLN_OK : cuda_fail(h, e);
}

evlnStatus_t evlnPagedStepCombine(evlnHandle_t h, const evlnPagedParams* p, const void* workspace,
                                  const int* h_cache_lens, const int* h_new_offsets, void* out, float* lse_out,
                                  void* stream)
{
    evlnStatus_t s = check_paged_params(h, p, h_cache_lens, h_new_offsets);
    if (s != EVLN_OK) return s;
    const int total = h_new_offsets[p->batch];
    if (total == 0) return EVLN_OK;
    if (!workspace || !out || !aligned16(workspace) || !aligned16(out)) return EVLN_INVALID_VALUE;
    if (!device_is_current(h)) return EVLN_INVALID_VALUE;
    const int G = p->num_q_heads / p->num_kv_heads;
    const long rows = (long)total * G;
    int chunk, smax;
    long items;
    paged_schedule(h, p, h_cache_lens, h_new_offsets, &chunk, &smax, &items);
    CombineArgs a = {};
    a.o_part = (const float*)workspace;
    a.lse_part = a.o_part + (size_t)smax * p->num_kv_heads * rows * 128;
    a.out = out; a.lse_out = lse_out;
    a.Hkv = p->num_kv_heads; a.G = G; a.D = 128; a.rows = (int)rows; a.num_splits = smax;
    a.batch = p->batch; a.unit_rows = kUnitRows; a.chunk_tiles = chunk;
    BatchLens bl;
    fill_lens(&bl, p, h_cache_lens, h_new_offsets);
    return launch_combine<__nv_bfloat16>(h, a, 128, true, &bl, (cudaStream_t)stream);
}

evlnStatus_t evlnPagedCheckTable(const evlnPagedParams* p, const int* h_cache_lens, const int* h_new_offsets,
                                 const int* h_page_table, int* h_bad_episode, int* h_bad_index)
{
    if (!p || !h_cache_lens || !h_new_offsets || !h_page_table) return EVLN_INVALID_VALUE;
    if (p->struct_size != sizeof(evlnPagedParams)) return EVLN_INVALID_VALUE;
    if (p->batch < 1 || p->num_pages < 1 || p->max_pages_per_seq < 1 || p->page_size < 1) return EVLN_INVALID_VALUE;
    if (h_new_offsets[0] != 0) return EVLN_INVALID_VALUE;
    std::vector<unsigned char> used((size_t)p->num_pages, 0);
    for (int b = 0; b < p->batch; ++b) {
        if (h_cache_lens[b] < 0 || h_new_offsets[b + 1] < h_new_offsets[b]) return EVLN_INVALID_VALUE;
        const long tokens = (long)h_cache_lens[b] + (h_new_offsets[b + 1] - h_new_offsets[b]);
        const long need = (tokens + p->page_size - 1) / p->page_size;
        if (need > p->max_pages_per_seq) return EVLN_CACHE_FULL;
        for (long i = 0; i < need; ++i) {
            const int pg = h_page_table[(long)b * p->max_pages_per_seq + i];
            if (pg < 0 || pg >= p->num_pages || used[pg]) {
                if (h_bad_episode) *h_bad_episode = b;
                if (h_bad_index) *h_bad_index = (int)i;
                return EVLN_INVALID_VALUE;
            }
            used[pg] = 1;
        }
    }
    return EVLN_OK;
}

}  // extern "C"

// ---- packed sequence under the action-isolating mask (Sec. 3.3) -----------------------------

namespace {
struct PackedPlan {
    int n_vis, n_act;            // instruction + visual tokens; action tokens
    evlnStepParams vis;          // the visual run as one step on an empty cache
    int lens[kMaxBatch];         // per action chunk: visible prefix of the cache
    int offs[kMaxBatch + 1];     // per action chunk: first own token
    int chunk, smax;             // KV tiles per work item of the action batch, its largest split count
    long items;
    size_t off_qv, off_qa, off_tk, off_tv, off_part, bytes;   // workspace layout
};

evlnStatus_t plan_packed(evlnHandle_t h, const evlnPackedParams* p, PackedPlan* pl)
{
    if (!h || !p) return EVLN_INVALID_VALUE;
    if (p->struct_size != sizeof(evlnPackedParams)) return EVLN_INVALID_VALUE;
    if (p->num_q_heads <= 0 || p->num_kv_heads <= 0 || p->num_q_heads % p->num_kv_heads != 0) return EVLN_INVALID_VALUE;
    if (p->instr_len < 0 || p->frame_tokens < 0 || p->action_tokens < 0 || p->num_frames < 0 || p->kv_chunk_tiles < 0)
        return EVLN_INVALID_VALUE;
    if (!(p->rope_theta > 0.0) || !(p->softmax_scale >= 0.f)) return EVLN_INVALID_VALUE;
    if (p->dtype != EVLN_BF16 || p->head_dim != 128 || p->num_frames > kMaxBatch) return EVLN_NOT_SUPPORTED;
    const long n_vis = (long)p->instr_len + (long)p->num_frames * p->frame_tokens;
    const long n_act = (long)p->num_frames * p->action_tokens;
    const int G = p->num_q_heads / p->num_kv_heads;
    if ((n_vis + n_act) * G > (1 << 24)) return EVLN_NOT_SUPPORTED;
    if (n_vis > (long)p->cache_capacity) return EVLN_CACHE_FULL;
    pl->n_vis = (int)n_vis;
    pl->n_act = (int)n_act;
    evlnStepParams& sp = pl->vis;
    memset(&sp, 0, sizeof(sp));
    sp.struct_size = sizeof(sp);
    sp.dtype = EVLN_BF16;
    sp.num_q_heads = p->num_q_heads; sp.num_kv_heads = p->num_kv_heads; sp.head_dim = 128;
    sp.cache_len = 0; sp.num_new = (int)n_vis; sp.cache_capacity = p->cache_capacity;
    sp.num_splits = 0; sp.kernel = EVLN_KERNEL_AUTO;
    sp.softmax_scale = p->softmax_scale; sp.rope_theta = p->rope_theta;
    for (int t = 0; t < p->num_frames; ++t) {
        pl->lens[t] = p->instr_len + (t + 1) * p->frame_tokens;      // chunk t sees the instruction and v_1 .. v_{t+1}
        pl->offs[t] = t * p->action_tokens;
    }
    pl->offs[p->num_frames] = (int)n_act;
    pl->chunk = pl->smax = 1;
    pl->items = 0;
    if (n_act > 0)
        batch_schedule(h->num_sms, G, p->num_kv_heads, p->num_frames, pl->lens, pl->offs, true, p->kv_chunk_tiles,
                       &pl->chunk, &pl->smax, &pl->items);
    size_t part_v = 0;
    if (n_vis > 0) {
        evlnStatus_t s = check_step_params(h, &sp);
        if (s != EVLN_OK) return s;
        part_v = partial_bytes(resolve_splits(h, &sp), p->num_kv_heads, n_vis * G, 128);
    }
    const size_t part_a = n_act > 0 ? partial_bytes(pl->smax, p->num_kv_heads, n_act * G, 128) : 0;
    size_t off = 0;
    pl->off_qv = off; off += round_up((size_t)n_vis * p->num_q_heads * 128 * 2, 256);
    pl->off_qa = off; off += round_up((size_t)n_act * p->num_q_heads * 128 * 2, 256);
    pl->off_tk = off; off += round_up((size_t)n_act * p->num_kv_heads * 128 * 2, 256);
    pl->off_tv = off; off += round_up((size_t)n_act * p->num_kv_heads * 128 * 2, 256);
    pl->off_part = off; off += part_v > part_a ? part_v : part_a;
    pl->bytes = off > 256 ? off : 256;
    return EVLN_OK;
}
}  // namespace

extern "C" evlnStatus_t evlnPackedWorkspaceSize(evlnHandle_t h, const evlnPackedParams* p, size_t* bytes)
{
    PackedPlan pl;
    evlnStatus_t s = plan_packed(h, p, &pl);
    if (s != EVLN_OK) return s;
    if (!bytes) return EVLN_INVALID_VALUE;
    *bytes = pl.bytes;
    return EVLN_OK;
}

extern "C" evlnStatus_t evlnPackedForward(evlnHandle_t h, const evlnPackedParams* p, const void* q, const void* k,
                                          const void* v, long q_stride_tok, long k_stride_tok, long v_stride_tok,
                                          void* k_cache, void* v_cache, void* workspace, size_t workspace_bytes,
                                          void* out, float* lse_out, void* stream)
{
    PackedPlan pl;
    evlnStatus_t s = plan_packed(h, p, &pl);
    if (s != EVLN_OK) return s;
    if (pl.n_vis + pl.n_act == 0) return EVLN_OK;
    if (!q || !k || !v || !k_cache || !v_cache || !workspace || !out) return EVLN_INVALID_VALUE;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(k_cache) || !aligned16(v_cache) ||
        !aligned16(workspace) || !aligned16(out))
        return EVLN_INVALID_VALUE;
    if (q_stride_tok < (long)p->num_q_heads * 128 || k_stride_tok < (long)p->num_kv_heads * 128 ||
        v_stride_tok < (long)p->num_kv_heads * 128 || q_stride_tok % 8 || k_stride_tok % 8 || v_stride_tok % 8)
        return EVLN_INVALID_VALUE;
    if (workspace_bytes < pl.bytes) return EVLN_WORKSPACE_TOO_SMALL;
    if (!device_is_current(h)) return EVLN_INVALID_VALUE;
    char* ws = (char*)workspace;
    cudaStream_t st = (cudaStream_t)stream;
    const int G = p->num_q_heads / p->num_kv_heads;
    const PackedMap map_v{p->instr_len, p->frame_tokens, p->action_tokens, 0};
    const PackedMap map_a{p->instr_len, p->frame_tokens, p->action_tokens, 1};

    // the instruction and the visual tokens: ONE causal step on an empty cache; its query tiles never
    // load a KV tile past their own last token, and no action token is among the keys at all
    if (pl.n_vis > 0) {
        s = rope_append_impl(h, &pl.vis, q, k, v, q_stride_tok, k_stride_tok, v_stride_tok, ws + pl.off_qv, k_cache, v_cache,
                             stream, map_v);
        if (s != EVLN_OK) return s;
        const size_t part_v = partial_bytes(resolve_splits(h, &pl.vis), p->num_kv_heads, (long)pl.n_vis * G, 128);
        s = evlnStepAttention(h, &pl.vis, ws + pl.off_qv, k_cache, v_cache, ws + pl.off_part, part_v, stream);
        if (s != EVLN_OK) return s;
        s = step_combine_impl(h, &pl.vis, ws + pl.off_part, out, lse_out, stream, map_v);
        if (s != EVLN_OK) return s;
    }
    if (pl.n_act == 0) return EVLN_OK;

    // all action chunks in one batch: chunk t sees the first lens[t] tokens of the cache just written
    // and its own tokens, which live in a buffer of their own (nobody else's keys)
    BatchLens bl;
    fill_batch_lens(&bl, G, p->num_kv_heads, p->num_frames, pl.lens, pl.offs, pl.chunk, true);
    if (bl.item_off[p->num_frames] != (int)pl.items || pl.items <= 0 || pl.items > 0x3fffffffL) return EVLN_NOT_SUPPORTED;
    {
        RopeArgs a = {};
        a.q_new = q; a.k_new = k; a.v_new = v;
        a.q_rot = ws + pl.off_qa; a.k_cache = ws + pl.off_tk; a.v_cache = ws + pl.off_tv; a.page_table = nullptr;
        a.q_stride = q_stride_tok; a.k_stride = k_stride_tok; a.v_stride = v_stride_tok;
        a.Hq = p->num_q_heads; a.Hkv = p->num_kv_heads; a.D = 128;
        a.num_new = pl.n_act; a.batch = p->num_frames; a.page_size = 1; a.max_pages = 0;
        a.log2_theta = log2(p->rope_theta);
        a.tail = 1;
        a.map = map_a;
        finish_rope_args(&a, 8);
        launch_rope_append<__nv_bfloat16, true, BatchLens>(h, a, pl.n_act, st, bl);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(h, e);
    }
    const long rows = (long)pl.n_act * G;
    {
        CUtensorMap tm_q, tm_k, tm_v, tm_kt, tm_vt;
        cuuint32_t box_q[3] = {64, 128, 1}, box_k[3] = {64, 64, 1}, box_v[3] = {64, 128, 1};
        {
            cuuint64_t dims[3] = {128, (cuuint64_t)rows, (cuuint64_t)p->num_kv_heads};
            cuuint64_t strides[2] = {256, (cuuint64_t)rows * 256};
            if (!encode_map(h, &tm_q, ws + pl.off_qa, 3, dims, strides, box_q)) return EVLN_INVALID_VALUE;
        }
        {
            cuuint64_t dims[3] = {128, (cuuint64_t)pl.n_vis, (cuuint64_t)p->num_kv_heads};
            cuuint64_t strides[2] = {256, (cuuint64_t)p->cache_capacity * 256};
            if (!encode_map(h, &tm_k, k_cache, 3, dims, strides, box_k)) return EVLN_INVALID_VALUE;
            if (!encode_map(h, &tm_v, v_cache, 3, dims, strides, box_v)) return EVLN_INVALID_VALUE;
        }
        {
            cuuint64_t dims[3] = {128, (cuuint64_t)pl.n_act, (cuuint64_t)p->num_kv_heads};
            cuuint64_t strides[2] = {256, (cuuint64_t)pl.n_act * 256};
            if (!encode_map(h, &tm_kt, ws + pl.off_tk, 3, dims, strides, box_k)) return EVLN_INVALID_VALUE;
            if (!encode_map(h, &tm_vt, ws + pl.off_tv, 3, dims, strides, box_v)) return EVLN_INVALID_VALUE;
        }
        const float scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf(128.f);
        TcAttnArgs a = {};
        a.o_part = (float*)(ws + pl.off_part);
        a.lse_part = a.o_part + (size_t)pl.smax * p->num_kv_heads * rows * 128;
        a.page_table = nullptr; a.status = h->d_status;
        a.Hkv = p->num_kv_heads; a.G = G; a.rows = (int)rows;
        a.batch = p->num_frames; a.max_pages = 0; a.chunk_tiles = pl.chunk;
        a.scale_log2 = scale * 1.4426950408889634f;
        a.div_g = make_fast_div((uint32_t)G);
        a.div_s = make_fast_div(1u);
        launch_pair_pdl(attn_tail_kernel, dim3(2 * (int)pl.items), kTcSmemBytes, st, tm_q, tm_k, tm_v, tm_kt, tm_vt, a, bl);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(h, e);
    }
    CombineArgs c = {};
    c.o_part = (const float*)(ws + pl.off_part);
    c.lse_part = c.o_part + (size_t)pl.smax * p->num_kv_heads * rows * 128;
    c.out = out; c.lse_out = lse_out;
    c.Hkv = p->num_kv_heads; c.G = G; c.D = 128; c.rows = (int)rows; c.num_splits = pl.smax;
    c.batch = p->num_frames; c.unit_rows = kUnitRows; c.chunk_tiles = pl.chunk;
    c.tail = 1;
    c.map = map_a;
    return launch_combine<__nv_bfloat16>(h, c, 128, true, &bl, st);
}

// ---- un-rotated store + frame sampler ------------------------------------------------------

namespace {
evlnStatus_t check_gather_params(evlnHandle_t h, const evlnGatherParams* p)
{
    if (!h || !p) return EVLN_INVALID_VALUE;
    if (p->struct_size != sizeof(evlnGatherParams)) return EVLN_INVALID_VALUE;
    if (p->dtype != EVLN_BF16 && p->dtype != EVLN_F32) return EVLN_INVALID_VALUE;
    if (p->num_kv_heads <= 0 || p->store_capacity < 0 || p->work_capacity < 0) return EVLN_INVALID_VALUE;
    if (!(p->rope_theta > 0.0)) return EVLN_INVALID_VALUE;
    if (p->head_dim != 64 && p->head_dim != 128) return EVLN_NOT_SUPPORTED;
    if (!device_is_current(h)) return EVLN_INVALID_VALUE;
    return EVLN_OK;
}
}  // namespace

extern "C" int evlnSampleFrames(int sampler, int num_frames, int budget, int stride, int* h_indices)
{
    if (num_frames < 0 || budget < 0 || !h_indices) return -1;
    if (num_frames == 0 || budget == 0) return 0;
    if (sampler == EVLN_SAMPLE_UNIFORM) {
        if (num_frames <= budget) {
            for (int i = 0; i < num_frames; ++i) h_indices[i] = i;
            return num_frames;
        }
        if (budget == 1) { h_indices[0] = num_frames - 1; return 1; }
        for (int k = 0; k < budget; ++k)      // round(k (N-1) / (B-1)), halves up
            h_indices[k] = (int)((2L * k * (num_frames - 1) + (budget - 1)) / (2L * (budget - 1)));
        return budget;
    }
    if (sampler == EVLN_SAMPLE_SLIDING) {
        if (stride < 1) return -1;
        int count = 0;
        for (int f = num_frames - 1; f >= 0 && count < budget; f -= stride) ++count;
        for (int k = 0; k < count; ++k) h_indices[k] = num_frames - 1 - (count - 1 - k) * stride;
        return count;
    }
    return -1;
}

extern "C" evlnStatus_t evlnStoreAppend(evlnHandle_t h, const evlnGatherParams* p, const void* k_new,
                                        const void* v_new, long k_stride_tok, long v_stride_tok, int store_len,
                                        int num_new, void* k_store, void* v_store, void* stream)
{
    evlnStatus_t s = check_gather_params(h, p);
    if (s != EVLN_OK) return s;
    if (store_len < 0 || num_new < 0) return EVLN_INVALID_VALUE;
    if ((long)store_len + num_new > (long)p->store_capacity) return EVLN_CACHE_FULL;
    if (num_new == 0) return EVLN_OK;
    if (!k_new || !v_new || !k_store || !v_store) return EVLN_INVALID_VALUE;
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_store) || !aligned16(v_store)) return EVLN_INVALID_VALUE;
    const int vec = 16 / elem_bytes(p->dtype);
    const long row = (long)p->num_kv_heads * p->head_dim;
    if (k_stride_tok < row || v_stride_tok < row || k_stride_tok % vec || v_stride_tok % vec) return EVLN_INVALID_VALUE;
    GatherArgs a = {};
    a.k_src = k_new; a.v_src = v_new; a.k_dst = k_store; a.v_dst = v_store;
    a.k_stride = k_stride_tok; a.v_stride = v_stride_tok;
    a.Hkv = p->num_kv_heads; a.D = p->head_dim;
    a.dst_cap = p->store_capacity; a.first_slot = store_len; a.num_tokens = num_new;
    cudaStream_t st = (cudaStream_t)stream;
    if (p->dtype == EVLN_BF16) launch_pdl(store_append_kernel<__nv_bfloat16>, dim3(num_new), dim3(128), 0, st, a);
    else launch_pdl(store_append_kernel<float>, dim3(num_new), dim3(128), 0, st, a);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? EVLN_OK : cuda_fail(h, e);
}

extern "C" evlnStatus_t evlnGatherRope(evlnHandle_t h, const evlnGatherParams* p, int num_segments,
                                       const int* h_seg_src, const int* h_seg_len, const void* k_store,
                                       const void* v_store, void* k_work, void* v_work, int* h_total, void* stream)
{
    evlnStatus_t s = check_gather_params(h, p);
    if (s != EVLN_OK) return s;
    if (num_segments < 0 || (num_segments > 0 && (!h_seg_src || !h_seg_len))) return EVLN_INVALID_VALUE;
    if (num_segments > kMaxSegments) return EVLN_NOT_SUPPORTED;
    SegList segs;
    memset(&segs, 0, sizeof(segs));
    long total = 0;
    for (int i = 0; i < num_segments; ++i) {
        if (h_seg_src[i] < 0 || h_seg_len[i] < 0 || (long)h_seg_src[i] + h_seg_len[i] > (long)p->store_capacity)
            return EVLN_INVALID_VALUE;
        segs.src[i] = h_seg_src[i];
        segs.dst_off[i] = (int)total;
        total += h_seg_len[i];
        if (total > (long)p->work_capacity) return EVLN_CACHE_FULL;
    }
    for (int i = num_segments; i <= kMaxSegments; ++i) segs.dst_off[i] = (int)total;
    if (h_total) *h_total = (int)total;
    if (total == 0) return EVLN_OK;
    if (!rope_table_covers(p->rope_table, p->rope_table_first_pos, p->rope_table_count, 0, total)) return EVLN_INVALID_VALUE;
    if (!k_store || !v_store || !k_work || !v_work) return EVLN_INVALID_VALUE;
    if (!aligned16(k_store) || !aligned16(v_store) || !aligned16(k_work) || !aligned16(v_work)) return EVLN_INVALID_VALUE;
    GatherArgs a = {};
    a.k_src = k_store; a.v_src = v_store; a.k_dst = k_work; a.v_dst = v_work;
    a.Hkv = p->num_kv_heads; a.D = p->head_dim;
    a.src_cap = p->store_capacity; a.dst_cap = p->work_capacity;
    a.num_tokens = (int)total; a.num_segments = num_segments;
    a.log2_theta = log2(p->rope_theta);
    a.table = (const double2*)p->rope_table;
    a.table_first = p->rope_table_first_pos;
    cudaStream_t st = (cudaStream_t)stream;
    if (p->dtype == EVLN_BF16) launch_pdl(gather_rope_kernel<__nv_bfloat16>, dim3((int)total), dim3(128), 0, st, a, segs);
    else launch_pdl(gather_rope_kernel<float>, dim3((int)total), dim3(128), 0, st, a, segs);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? EVLN_OK : cuda_fail(h, e);
}

// ---- host-resident store: strided DMA between the pinned host store and the device store ----

namespace {
evlnStatus_t store_copy(evlnHandle_t h, const evlnGatherParams* p, const void* k_src, const void* v_src, int src_cap,
                        int src_slot, int len, void* k_dst, void* v_dst, int dst_cap, int dst_slot, cudaStream_t st,
                        cudaMemcpyKind kind)
{
    evlnStatus_t s = check_gather_params(h, p);
    if (s != EVLN_OK) return s;
    if (src_slot < 0 || dst_slot < 0 || len < 0 || src_cap < 0 || dst_cap < 0) return EVLN_INVALID_VALUE;
    if ((long)src_slot + len > (long)src_cap) return EVLN_INVALID_VALUE;
    if ((long)dst_slot + len > (long)dst_cap) return EVLN_CACHE_FULL;
    if (len == 0) return EVLN_OK;
    if (!k_src || !v_src || !k_dst || !v_dst) return EVLN_INVALID_VALUE;
    const size_t row = (size_t)p->head_dim * elem_bytes(p->dtype);       // one token of one head
    const size_t width = row * len;
    cudaError_t e = cudaMemcpy2DAsync((char*)k_dst + row * dst_slot, row * dst_cap, (const char*)k_src + row * src_slot,
                                      row * src_cap, width, p->num_kv_heads, kind, st);
    if (e == cudaSuccess)
        e = cudaMemcpy2DAsync((char*)v_dst + row * dst_slot, row * dst_cap, (const char*)v_src + row * src_slot,
                              row * src_cap, width, p->num_kv_heads, kind, st);
    return e == cudaSuccess ? EVLN_OK : cuda_fail(h, e);
}
}  // namespace

extern "C" evlnStatus_t evlnStoreOffload(evlnHandle_t h, const evlnGatherParams* p, const void* k_store,
                                         const void* v_store, int src_slot, int len, void* h_k_store, void* h_v_store,
                                         int host_capacity, int dst_slot, void* stream)
{
    if (!p) return EVLN_INVALID_VALUE;
    return store_copy(h, p, k_store, v_store, p->store_capacity, src_slot, len, h_k_store, h_v_store, host_capacity,
                      dst_slot, (cudaStream_t)stream, cudaMemcpyDeviceToHost);
}

extern "C" evlnStatus_t evlnStoreFetch(evlnHandle_t h, const evlnGatherParams* p, const void* h_k_store,
                                       const void* h_v_store, int host_capacity, int src_slot, int len, void* k_store,
                                       void* v_store, int dst_slot, void* stream)
{
    if (!p) return EVLN_INVALID_VALUE;
    return store_copy(h, p, h_k_store, h_v_store, host_capacity, src_slot, len, k_store, v_store, p->store_capacity,
                      dst_slot, (cudaStream_t)stream, cudaMemcpyHostToDevice);
}

// ---- allocation-free variant --------------------------------------------------------------

// Scratch for the split partials of evlnStepAttentionNoAlloc, part of the library image: every
// device that loads the library holds these bytes until the process exits.  In host code the
// names below are only stand-ins for the device objects; their device addresses come from
// cudaGetSymbolAddress (once per device) and are what the kernels receive.
static __device__ __align__(256) unsigned char g_noalloc_scratch[EVLN_NOALLOC_SCRATCH_BYTES];
static __device__ __align__(256) int g_noalloc_status;

namespace {
constexpr int kMaxDevices = 64;
struct NoAllocDevice {
    bool ready;
    evlnContext ctx;          // plain struct used as the handle of the regular entry points
    void* scratch;
};
NoAllocDevice g_noalloc_dev[kMaxDevices];
std::mutex g_noalloc_mutex;       // host threads may race for the first call on a device

// First call on a device: resolve device addresses and properties.  Allocates nothing.
evlnStatus_t noalloc_setup(int device, NoAllocDevice** out)
{
    if (device < 0 || device >= kMaxDevices) return EVLN_NOT_SUPPORTED;
    NoAllocDevice* d = &g_noalloc_dev[device];
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!d->ready) {
        cudaDeviceProp prop;
        cudaError_t e = cudaGetDeviceProperties(&prop, device);
        if (e != cudaSuccess) return EVLN_CUDA_ERROR;
        if (prop.major != 10) return EVLN_NOT_SUPPORTED;
        void* scratch = nullptr;
        void* status = nullptr;
        e = cudaGetSymbolAddress(&scratch, g_noalloc_scratch);
        if (e != cudaSuccess || !scratch) return EVLN_CUDA_ERROR;
        e = cudaGetSymbolAddress(&status, g_noalloc_status);
        if (e != cudaSuccess || !status) return EVLN_CUDA_ERROR;
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) return EVLN_CUDA_ERROR;
        e = cudaFuncSetAttribute(attn_pair_kernel<false, NoLens>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kTcSmemBytes);
        if (e != cudaSuccess) return EVLN_CUDA_ERROR;
        e = cudaFuncSetAttribute(attn_solo_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSoloSmemBytes);
        if (e != cudaSuccess) return EVLN_CUDA_ERROR;
        if (!attention_register_pool_ok()) return EVLN_NOT_SUPPORTED;
        d->ctx.device = device;
        d->ctx.num_sms = prop.multiProcessorCount;
        d->ctx.last_cuda_error = 0;
        d->ctx.d_status = static_cast<int*>(status);
        d->ctx.encode = reinterpret_cast<EncodeTiledFn>(fn);
        d->scratch = scratch;
        d->ready = true;
    }
    *out = d;
    return EVLN_OK;
}
// Device address of the allocation-free call's status word on the current device.
evlnStatus_t noalloc_status_word(int** word)
{
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return EVLN_CUDA_ERROR;
    NoAllocDevice* d = nullptr;
    evlnStatus_t s = noalloc_setup(device, &d);
    if (s != EVLN_OK) return s;
    *word = d->ctx.d_status;
    return EVLN_OK;
}
}  // namespace

extern "C" evlnStatus_t evlnStepAttentionNoAlloc(const evlnStepParams* p, const void* q_rot, const void* k_cache,
                                                 const void* v_cache, void* out, float* lse_out, void* stream)
{
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return EVLN_CUDA_ERROR;
    NoAllocDevice* d = nullptr;
    evlnStatus_t s = noalloc_setup(device, &d);
    if (s != EVLN_OK) return s;
    evlnHandle_t h = &d->ctx;
    size_t need = 0;
    s = evlnStepWorkspaceSize(h, p, &need);
    if (s != EVLN_OK) return s;
    if (need > (size_t)EVLN_NOALLOC_SCRATCH_BYTES) return EVLN_WORKSPACE_TOO_SMALL;
    if (p->num_new == 0) return EVLN_OK;
    if (!out) return EVLN_INVALID_VALUE;
    s = evlnStepAttention(h, p, q_rot, k_cache, v_cache, d->scratch, (size_t)EVLN_NOALLOC_SCRATCH_BYTES, stream);
    if (s != EVLN_OK) return s;
    return evlnStepCombine(h, p, d->scratch, out, lse_out, stream);
}
