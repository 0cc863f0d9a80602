/*
 * libevln: step attention for KV-cache reuse with contiguous RoPE on NVIDIA B200 (sm_100a).
 *
 * One navigation step of the paper's inference scheme (Sec. 3.2, "KV Cache Reuse with
 * Contiguous RoPE") processes only the newly observed frame: its n tokens receive the
 * position ids L .. L+n-1 that continue the cached sequence of length L, their queries and
 * keys are rotated by RoPE at those positions, the rotated keys and the values are appended
 * to the reused cache, and the n new queries attend causally to all L+n cached tokens
 * (grouped-query attention).  Per transformer layer this is three calls:
 *
 *     evlnRopeAppend  ->  evlnStepAttention  ->  evlnStepCombine      (or evlnStep: all three)
 *
 * plus evlnPaged* variants for a batch of episodes whose caches live in a page pool, and
 * evlnStoreAppend / evlnSampleFrames / evlnGatherRope for the paper's un-rotated store that a
 * frame sampler re-indexes every step (declared at the end of this file).
 *
 * Conventions
 *  - Every data pointer is DEVICE memory owned by the caller unless its name starts with
 *    h_ (host memory, read during the call).  The library never allocates or frees in
 *    these calls and keeps no reference to caller memory after a call returns.
 *  - All device base pointers must be 16-byte aligned, token strides multiples of 8
 *    elements (bf16) / 4 elements (f32); otherwise EVLN_INVALID_VALUE.
 *  - Calls validate on the host, then enqueue kernels on `stream` (a cudaStream_t passed as
 *    void*; NULL = default stream) and return without synchronising.  Argument errors
 *    launch nothing.  EVLN_CUDA_ERROR wraps a failed launch; evlnGetLastCudaError gives
 *    the cudaError_t value.
 *  - The library does not advance L: the caller passes the pre-step cache length to all
 *    three calls of a step and adds n afterwards.
 *  - For fixed parameters the split schedule is fixed, so results are bitwise reproducible, with
 *    one exception in the tensor-core kernel: when a score exceeds the maximum of its row's first
 *    KV tile by more than a factor 2^64, the row's softmax reference moves, and where it moves to
 *    depends on which of the row's threads noticed first; results then agree to rounding only.
 *  - One handle per host thread.  There is no CPU fallback.
 *
 * Layouts (D = head_dim, G = num_q_heads / num_kv_heads, query head h uses kv head h / G)
 *    q_new          [n, Hq, D]   token stride given in elements, head stride D
 *    k_new, v_new   [n, Hkv, D]  same
 *    k_cache,v_cache[Hkv, cache_capacity, D]            (contiguous cache, one layer)
 *    k_pool, v_pool [num_pages, Hkv, page_size, D]      (paged cache, one layer)
 *    q_rot          [Hkv, n*G, D] row r = i*G + (h % G) (scratch written by RopeAppend)
 *    out            [n, Hq, D]   contiguous, same dtype as the inputs
 *    lse_out        [n, Hq]      float, natural-log sum-exp of the scaled logits (optional)
 */
#ifndef EVLN_H_
#define EVLN_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    EVLN_OK = 0,
    EVLN_INVALID_VALUE = 1,      /* null / misaligned pointer, bad shape, bad struct_size      */
    EVLN_NOT_SUPPORTED = 2,      /* shape or dtype outside what the kernels implement          */
    EVLN_CACHE_FULL = 3,         /* cache_len + num_new > cache_capacity (or page table short) */
    EVLN_WORKSPACE_TOO_SMALL = 4,
    EVLN_CUDA_ERROR = 5,
    EVLN_DEVICE_TIMEOUT = 6      /* a bounded wait inside a kernel expired (see DeviceStatus)  */
} evlnStatus_t;

typedef enum { EVLN_BF16 = 0, EVLN_F32 = 1 } evlnDType_t;

/* Attention kernel choice.  AUTO: tensor-core kernel (tcgen05 MMA, TMEM accumulators, TMA
 * tiles) for bf16 with head_dim 128; the fp32 SIMT kernel otherwise.  SIMT forces the
 * SIMT kernel (any dtype), which exists for the fp32 precision target and as an
 * independent on-device cross-check.                                                        */
typedef enum { EVLN_KERNEL_AUTO = 0, EVLN_KERNEL_SIMT = 1 } evlnKernel_t;

typedef struct evlnContext* evlnHandle_t;

/* One layer, one episode, contiguous cache. */
typedef struct {
    size_t struct_size;      /* sizeof(evlnStepParams)                                       */
    int dtype;               /* evlnDType_t of q/k/v, cache, q_rot and out                   */
    int num_q_heads;         /* Hq                                                           */
    int num_kv_heads;        /* Hkv, divides Hq                                              */
    int head_dim;            /* D: 64 or 128                                                 */
    int cache_len;           /* L >= 0: tokens already cached (0 = instruction prefill)      */
    int num_new;             /* n >= 0: new tokens, rotated at positions L .. L+n-1          */
    int cache_capacity;      /* token slots per kv head in k_cache / v_cache                 */
    int num_splits;          /* KV splits; 0 = library heuristic                             */
    int kernel;              /* evlnKernel_t                                                 */
    float softmax_scale;     /* 0 -> 1/sqrt(D)                                               */
    double rope_theta;       /* RoPE base, > 0                                               */
    /* Optional position table written by evlnRopeTable (NULL: the kernels form the angles
     * themselves, once per call).  It must cover positions L .. L+n-1, i.e.
     * rope_table_first_pos <= L and L+n <= rope_table_first_pos + rope_table_count, and must
     * have been made for this head_dim and rope_theta.  Results are bit-identical either way. */
    const void* rope_table;
    int rope_table_first_pos;
    int rope_table_count;
} evlnStepParams;

/* A batch of episodes on a page pool (one layer).  Episode b has h_cache_lens[b] cached
 * tokens and its new tokens are rows h_new_offsets[b] .. h_new_offsets[b+1]-1 of the packed
 * q_new/k_new/v_new/out.  Row p of its page table lists pool pages in sequence order and
 * must already cover cache_len + num_new tokens (the caller hands out pages).              */
typedef struct {
    size_t struct_size;      /* sizeof(evlnPagedParams)                                      */
    int dtype;               /* EVLN_BF16 only                                               */
    int num_q_heads, num_kv_heads, head_dim;      /* head_dim 128                            */
    int batch;               /* number of episodes, 1 .. 256                                 */
    int page_size;           /* tokens per page: 64                                          */
    int num_pages;           /* pages in the pool                                            */
    int max_pages_per_seq;   /* row length of d_page_table                                   */
    int kv_chunk_tiles;      /* max 128-key tiles per work item; 0 = library heuristic       */
    float softmax_scale;     /* 0 -> 1/sqrt(D)                                               */
    double rope_theta;
    /* Optional position table written by evlnRopeTable (NULL: the append kernel forms the angles
     * itself).  It must cover the positions of every episode's new tokens, cache_len[b] ..
     * cache_len[b] + n_b - 1: a serving host makes one table for positions 0 .. its longest
     * context once, since the entries depend on head_dim and rope_theta only.  Results are
     * bit-identical either way.                                                                */
    const void* rope_table;
    int rope_table_first_pos;
    int rope_table_count;
} evlnPagedParams;

/* ---- handle, errors ------------------------------------------------------------------- */

/* Creates a handle bound to CUDA device `device` (allocates a 4-byte device status word and
 * resolves the driver's tensor-map encoder); the caller's current device is left as it was.
 * Every call that launches work must be made with that device current, otherwise it returns
 * EVLN_INVALID_VALUE and launches nothing.  Sec. 3.2 has no counterpart: plumbing.          */
evlnStatus_t evlnCreate(evlnHandle_t* handle, int device);
evlnStatus_t evlnDestroy(evlnHandle_t handle);
const char* evlnGetErrorString(evlnStatus_t status);
/* cudaError_t value of the most recent EVLN_CUDA_ERROR on this handle (0 if none). */
int evlnGetLastCudaError(evlnHandle_t handle);
/* Synchronises `stream`, reads and clears the device status word.  *device_status = 0 when no
 * kernel gave up on a bounded wait; otherwise a code identifying the wait that expired and
 * the function returns EVLN_DEVICE_TIMEOUT (the outputs of that step are then invalid).
 * handle == NULL addresses the status word of the allocation-free call
 * (evlnStepAttentionNoAlloc) on the CURRENT device; it allocates nothing either.             */
evlnStatus_t evlnGetDeviceStatus(evlnHandle_t handle, void* stream, int* device_status);

/* Self-test of the fault containment (Sec. 3.2 has no counterpart: plumbing).  Launches one
 * small kernel whose only act is a bounded wait on a barrier that nothing ever arrives on, with
 * a limit of `limit_cycles` SM clocks (1000 .. 10^9): the wait must run out, the kernel must
 * record EVLN_SELFTEST_STATUS_CODE in the handle's status word and return normally, so that the
 * next evlnGetDeviceStatus reports EVLN_DEVICE_TIMEOUT with that code and the context stays
 * usable.  No fault, trap or unbounded loop is involved.                                     */
#define EVLN_SELFTEST_STATUS_CODE 8
evlnStatus_t evlnSelfTestBoundedWait(evlnHandle_t handle, long long limit_cycles, void* stream);

/* ---- contiguous cache ------------------------------------------------------------------- */

/* Number of KV splits the attention/combine pair will use for these parameters.            */
evlnStatus_t evlnStepNumSplits(evlnHandle_t handle, const evlnStepParams* params, int* num_splits);
/* Bytes of `workspace` needed by evlnStepAttention / evlnStepCombine:
 * num_splits * Hkv * n*G * (D + 1) floats (per-split outputs and log-sum-exps), rounded up. */
evlnStatus_t evlnStepWorkspaceSize(evlnHandle_t handle, const evlnStepParams* params, size_t* bytes);
/* Bytes of the q_rot scratch: n * Hq * D elements, rounded up to 256. */
evlnStatus_t evlnStepQRotSize(evlnHandle_t handle, const evlnStepParams* params, size_t* bytes);

/* RoPE position table (Sec. 3.2: one set of contiguous position ids per navigation step, shared
 * by all layers).  Entry (p, j), p = 0 .. count-1, j = 0 .. head_dim/2-1, holds the pair
 * (cos, sin) of (first_pos + p) * rope_theta^(-2j/head_dim) as two doubles: exactly the values
 * evlnRopeAppend / evlnGatherRope would form themselves in every call.  The angles depend on the
 * position only, so a model computes the table once per step and passes it to the calls of all
 * its layers (evlnStepParams.rope_table, evlnGatherParams.rope_table).
 * evlnRopeTableBytes = count * (head_dim/2) * 16; `table` must be 16-byte aligned device memory. */
size_t evlnRopeTableBytes(int head_dim, int count);
evlnStatus_t evlnRopeTable(evlnHandle_t handle, int head_dim, double rope_theta, int first_pos,
                           int count, void* table, void* stream);

/* Step 1 (Sec. 3.2: contiguous position ids, RoPE, concatenation with the cache).
 * Rotates the new queries at positions L+i into q_rot (grouped by kv head), rotates the new
 * keys and stores them, with the values copied bit-exactly, into cache slots L .. L+n-1.
 * Angles, sines/cosines and the rotation products are formed in double precision and then
 * rounded to the storage dtype.  Slots outside L .. L+n-1 are not touched.
 * Errors: EVLN_CACHE_FULL if L+n > cache_capacity; n = 0 returns EVLN_OK and launches nothing. */
evlnStatus_t evlnRopeAppend(evlnHandle_t handle, const evlnStepParams* params,
                            const void* q_new, const void* k_new, const void* v_new,
                            long q_stride_tok, long k_stride_tok, long v_stride_tok,
                            void* q_rot, void* k_cache, void* v_cache, void* stream);

/* Step 2 (Sec. 3.2: prefill of the current frame only, against the reused cache).
 * Causal attention of the n rotated queries over cache slots 0 .. L+n-1 (query i sees slots
 * 0 .. L+i), split over the keys; writes per-split normalised outputs and log-sum-exps into
 * `workspace`.  Must run after evlnRopeAppend of the same step on the same stream.
 * bf16 with head_dim 128 runs on the tensor cores: CTA pairs over 256-row units of the packed
 * query rows, or, when all n * G rows of a kv head fit one 128-row tile (the few action tokens
 * decoded after a frame, Sec. 3.1), one CTA per (kv head, KV split) with the KV range spread
 * over all SMs.                                                                              */
evlnStatus_t evlnStepAttention(evlnHandle_t handle, const evlnStepParams* params,
                               const void* q_rot, const void* k_cache, const void* v_cache,
                               void* workspace, size_t workspace_bytes, void* stream);

/* Step 3: merges the splits, O = sum_s e^{lse_s-M} O_s / sum_s e^{lse_s-M}, M = max_s lse_s,
 * rounds once to the storage dtype and scatters rows back to [n, Hq, D].  lse_out may be NULL. */
evlnStatus_t evlnStepCombine(evlnHandle_t handle, const evlnStepParams* params,
                             const void* workspace, void* out, float* lse_out, void* stream);

/* The whole step in one call (Sec. 3.2): evlnRopeAppend, evlnStepAttention and evlnStepCombine
 * with the same arguments, enqueued back to back on `stream`; same results bit for bit.
 * All arguments are validated before the first launch; errors as for the three calls.          */
evlnStatus_t evlnStep(evlnHandle_t handle, const evlnStepParams* params,
                      const void* q_new, const void* k_new, const void* v_new,
                      long q_stride_tok, long k_stride_tok, long v_stride_tok,
                      void* q_rot, void* k_cache, void* v_cache,
                      void* workspace, size_t workspace_bytes, void* out, float* lse_out, void* stream);

/* ---- paged cache, batch of episodes ----------------------------------------------------- */

/* The three calls take the episode lengths from HOST arrays (h_cache_lens [batch],
 * h_new_offsets [batch+1]); they travel to the kernels as launch parameters, so no copy is
 * enqueued.  d_page_table is DEVICE memory, int [batch, max_pages_per_seq].                 */
evlnStatus_t evlnPagedWorkspaceSize(evlnHandle_t handle, const evlnPagedParams* params,
                                    const int* h_cache_lens, const int* h_new_offsets,
                                    size_t* bytes);
/* As evlnRopeAppend, slot of token L_b+i = page_table[b][(L_b+i)/page] * page + (L_b+i)%page.
 * Additionally zero-fills the value slots after the last appended token up to the end of
 * its page, so that a partly filled page never exposes stale bits to the attention kernel. */
evlnStatus_t evlnPagedRopeAppend(evlnHandle_t handle, const evlnPagedParams* params,
                                 const void* q_new, const void* k_new, const void* v_new,
                                 const int* h_cache_lens, const int* h_new_offsets,
                                 const int* d_page_table, void* q_rot, void* k_pool, void* v_pool,
                                 void* stream);
evlnStatus_t evlnPagedStepAttention(evlnHandle_t handle, const evlnPagedParams* params,
                                    const void* q_rot, const void* k_pool, const void* v_pool,
                                    const int* h_cache_lens, const int* h_new_offsets,
                                    const int* d_page_table, void* workspace,
                                    size_t workspace_bytes, void* stream);
evlnStatus_t evlnPagedStepCombine(evlnHandle_t handle, const evlnPagedParams* params,
                                  const void* workspace, const int* h_cache_lens,
                                  const int* h_new_offsets, void* out, float* lse_out,
                                  void* stream);
/* Host-side check of a page table BEFORE it is copied to the device (no GPU work; plumbing).
 * h_page_table is the host copy, int [batch, max_pages_per_seq].  For every episode the first
 * ceil((L_b + n_b) / page_size) entries must be pool pages in [0, num_pages) and no page may be
 * listed twice, by one episode or by two: the append kernel writes through this table, so a bad
 * entry would corrupt another episode's cache or write outside the pool.  Returns EVLN_OK,
 * EVLN_INVALID_VALUE (bad entry; *h_bad_episode / *h_bad_index, if not NULL, say where) or the
 * usual parameter errors.                                                                    */
evlnStatus_t evlnPagedCheckTable(const evlnPagedParams* params, const int* h_cache_lens,
                                 const int* h_new_offsets, const int* h_page_table,
                                 int* h_bad_episode, int* h_bad_index);

/* ---- packed sequence under the action-isolating mask (Sec. 3.3, packed training via action
 *      isolation; forward pass only) -----------------------------------------------------------
 *
 * A packed sequence is  I, v_1, a_1, v_2, a_2, ..., v_N, a_N : instr_len instruction tokens, then
 * N frames of frame_tokens visual tokens, each followed by its chunk of action_tokens action
 * tokens.  Under the mask of Sec. 3.3 a visual (or instruction) token attends causally to the
 * instruction and the visual tokens up to itself, never to an action token; an action token of
 * chunk t attends to the instruction, to v_1 .. v_t and to its own chunk up to itself, never to
 * another chunk.  Position ids (the paper does not print them): the instruction and the visual
 * tokens are numbered contiguously as if no action token were there, chunk t continues after v_t.
 *
 * evlnPackedForward runs the whole sequence in one call and six launches, whatever N is: the
 * instruction and visual rows as ONE causal step on an empty cache (a query tile never loads a
 * KV tile beyond its own last token, and action tokens are not among its keys at all), then all
 * N action chunks as ONE batch whose items share prefixes of the cache just written and keep
 * their own rotated keys / values in a separate buffer.  No mask operand exists: the blocks the
 * mask removes are never loaded.
 *   q [T, Hq, D], k, v [T, Hkv, D]: the packed sequence, T = instr_len + N (frame_tokens +
 *       action_tokens), token strides in elements (multiples of 8);
 *   k_cache, v_cache [Hkv, cache_capacity, D]: receive the rotated keys and the values of the
 *       instruction + visual tokens at slots 0 .. instr_len + N frame_tokens - 1 (the cache an
 *       inference run over the same frames would hold); EVLN_CACHE_FULL if they do not fit;
 *   workspace: evlnPackedWorkspaceSize bytes (rotated queries, the chunks' keys/values, split partials);
 *   out [T, Hq, D], lse_out [T, Hq] or NULL: rows in the order of the packed sequence.
 * bf16, head_dim 128, at most 256 frames; otherwise EVLN_NOT_SUPPORTED.                         */
typedef struct {
    size_t struct_size;      /* sizeof(evlnPackedParams)                                     */
    int dtype;               /* EVLN_BF16                                                    */
    int num_q_heads, num_kv_heads, head_dim;
    int instr_len;           /* |I|                                                          */
    int frame_tokens;        /* |v|                                                          */
    int action_tokens;       /* |a|                                                          */
    int num_frames;          /* N                                                            */
    int cache_capacity;      /* token slots per kv head in k_cache / v_cache                 */
    int kv_chunk_tiles;      /* max 128-key tiles per work item of the action batch; 0 = heuristic */
    float softmax_scale;     /* 0 -> 1/sqrt(D)                                               */
    double rope_theta;
} evlnPackedParams;

evlnStatus_t evlnPackedWorkspaceSize(evlnHandle_t handle, const evlnPackedParams* params, size_t* bytes);
evlnStatus_t evlnPackedForward(evlnHandle_t handle, const evlnPackedParams* params,
                               const void* q, const void* k, const void* v,
                               long q_stride_tok, long k_stride_tok, long v_stride_tok,
                               void* k_cache, void* v_cache, void* workspace, size_t workspace_bytes,
                               void* out, float* lse_out, void* stream);

/* ---- allocation-free variant ------------------------------------------------------------ */

/* Largest split workspace the allocation-free call can serve (bytes of its built-in scratch). */
#define EVLN_NOALLOC_SCRATCH_BYTES (32u << 20)

/* Attention + combine of one step for callers that cannot allocate device memory.  (The paper
 * has no counterpart for this call; it exists for deployment.)
 *
 * Who needs it: a host process that has handed all device memory to its own arena at start-up
 * (an inference server, a robot's control process with a fixed memory budget), or code that
 * runs where cudaMalloc is unwelcome because it synchronises the whole device and may fail
 * late.  Such a caller can neither create a handle (evlnCreate allocates its status word) nor
 * size and allocate the split workspace.  This call needs neither: it takes no handle, and the
 * per-split partial results go to a scratch array that is part of the library image itself
 * (EVLN_NOALLOC_SCRATCH_BYTES of device memory, held by every GPU that loads the library until
 * the process exits).  The caller passes only inputs and outputs:
 *   q_rot, k_cache, v_cache: the rotated queries and the cache exactly as evlnRopeAppend leaves
 *   them (that call allocates nothing either, but wants a handle made while allocating was
 *   still allowed, e.g. at start-up; the workspace size, in contrast, changes with L);
 *   out [n, Hq, D], lse_out [n, Hq] or NULL: as for evlnStepCombine.
 * It calls no cudaMalloc/cudaFree and no allocating library routine.
 *
 * Set-up: the first call on each device (with that device current) looks up the scratch
 * array's device address and the device's properties once; make that first call outside any
 * stream capture.  Later calls on that device only validate and launch.  Host threads may race
 * for the first call: the set-up runs once per device under a lock.
 * Status: a kernel of this call that gives up on a bounded wait records it in a status word
 * that is part of the library image as well; evlnGetDeviceStatus(NULL, stream, &code) reads and
 * clears it for the current device.
 * Limits and errors: parameters whose split workspace (evlnStepWorkspaceSize) exceeds
 * EVLN_NOALLOC_SCRATCH_BYTES are rejected with EVLN_WORKSPACE_TOO_SMALL and nothing is
 * launched; other errors as for evlnStepAttention / evlnStepCombine.
 * Sharing: every call on a device uses the same scratch array, which keeps the previous
 * call's contents (each call overwrites every partial it later reads, so nothing needs
 * clearing).  Two such calls that overlap on the GPU (different streams, or different host
 * threads) race on it: serialise them.                                                        */
evlnStatus_t evlnStepAttentionNoAlloc(const evlnStepParams* params, const void* q_rot,
                                      const void* k_cache, const void* v_cache, void* out,
                                      float* lse_out, void* stream);

/* ---- un-rotated store + frame sampler (Sec. 3.2: the cache is kept un-rotated; kept tokens are
 *      re-rotated at contiguous ids; uniform and sliding-window frame samplers) -----------
 *
 * The episode's raw keys and values (as projected, NOT rotated) live in a store
 * [Hkv, store_capacity, D] per layer.  Every step the caller
 *   1. appends the new frame's raw K/V to the store                    (evlnStoreAppend),
 *   2. lets a sampler choose the history frames to keep                (evlnSampleFrames, host),
 *   3. lays the kept segments out back to back in a working cache [Hkv, work_capacity, D],
 *      the token landing in slot p rotated at position p               (evlnGatherRope),
 *   4. runs the usual step on that working cache with cache_len = kept tokens:
 *      evlnRopeAppend (new frame at the next contiguous positions) -> evlnStepAttention ->
 *      evlnStepCombine.
 */
typedef struct {
    size_t struct_size;      /* sizeof(evlnGatherParams)                                     */
    int dtype;               /* evlnDType_t of store and working cache                       */
    int num_kv_heads;        /* Hkv                                                          */
    int head_dim;            /* D: 64 or 128                                                 */
    int store_capacity;      /* token slots per kv head in k_store / v_store                 */
    int work_capacity;       /* token slots per kv head in k_work / v_work                   */
    double rope_theta;
    /* optional evlnRopeTable table covering the positions 0 .. (tokens laid out)-1 (NULL: none) */
    const void* rope_table;
    int rope_table_first_pos;
    int rope_table_count;
} evlnGatherParams;

typedef enum { EVLN_SAMPLE_UNIFORM = 0, EVLN_SAMPLE_SLIDING = 1 } evlnSampler_t;

/* Host helper, no GPU work.  Chooses at most `budget` of the history frames 0 .. num_frames-1
 * and writes their indices in ascending order to h_indices (room for `budget` ints).
 *   UNIFORM: all frames if num_frames <= budget, else frame round(k (num_frames-1)/(budget-1)),
 *            k = 0 .. budget-1 (first and last frame always kept; `stride` ignored).
 *   SLIDING: frames num_frames-1, num_frames-1-stride, ... (the most recent ones, `stride`
 *            apart, stride >= 1), at most `budget` of them.
 * Returns the number of indices written, or -1 for bad arguments.                            */
int evlnSampleFrames(int sampler, int num_frames, int budget, int stride, int* h_indices);

/* Raw (un-rotated) k_new / v_new [n, Hkv, D] (token strides in elements) -> store slots
 * store_len .. store_len+n-1.  EVLN_CACHE_FULL if they do not fit.                           */
evlnStatus_t evlnStoreAppend(evlnHandle_t handle, const evlnGatherParams* params, const void* k_new,
                             const void* v_new, long k_stride_tok, long v_stride_tok, int store_len,
                             int num_new, void* k_store, void* v_store, void* stream);

/* Kept segments s = 0 .. num_segments-1 (at most 256): store slots
 * [h_seg_src[s], h_seg_src[s] + h_seg_len[s]) go to the working cache back to back, in the
 * order given; the key landing in working slot p is rotated by RoPE at position p, the value
 * is copied bit-exactly.  *h_total (optional) receives the number of tokens laid out.
 * Slots of the working cache beyond that are not touched.  EVLN_INVALID_VALUE for a segment
 * outside the store, EVLN_CACHE_FULL if the working cache is too small.                      */
evlnStatus_t evlnGatherRope(evlnHandle_t handle, const evlnGatherParams* params, int num_segments,
                            const int* h_seg_src, const int* h_seg_len, const void* k_store,
                            const void* v_store, void* k_work, void* v_work, int* h_total,
                            void* stream);

/* ---- host-resident store (Sec. 3.2, memory management: the cache lives in host memory and only
 *      the segments the sampler keeps come back to the GPU) -----------------------------------
 *
 * The full raw store of an episode may live in PINNED host memory, [Hkv, host_capacity, D],
 * while the device store only has room for the segments in use.  evlnStoreOffload copies token
 * slots of the device store to the host store, evlnStoreFetch copies token slots of the host
 * store into the device store; each is one strided DMA per tensor (all kv heads at once),
 * enqueued on `stream`, no kernel.  Which frames are resident, and where, is the caller's
 * bookkeeping (paper_2512_10310_b200/residency.py has one).  h_k_store / h_v_store must be
 * page-locked for the copies to be asynchronous.                                               */
evlnStatus_t evlnStoreOffload(evlnHandle_t handle, const evlnGatherParams* params, const void* k_store,
                              const void* v_store, int src_slot, int len, void* h_k_store, void* h_v_store,
                              int host_capacity, int dst_slot, void* stream);
evlnStatus_t evlnStoreFetch(evlnHandle_t handle, const evlnGatherParams* params, const void* h_k_store,
                            const void* h_v_store, int host_capacity, int src_slot, int len, void* k_store,
                            void* v_store, int dst_slot, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* EVLN_H_ */
