/*
 * rlkv.h -- C ABI of librlkv: decode attention over a head-mixed KV cache on one B200 (sm_100a).
 *
 * The operation (paper: Section 3.3, last paragraph; Section 4.3 "Inference Efficiency";
 * Appendix B "Local Attention Implementation"):
 *   every KV head of every layer is either FULL -- it keeps the keys/values of all tokens -- or
 *   COMPRESSED -- it keeps only the first `sink` tokens and the most recent `window` tokens in a
 *   constant-size circular buffer.  A decode step appends one token per layer and then runs
 *   ordinary scaled-dot-product attention, softmax(q.K^T / sqrt(head_dim)).V, of each query head
 *   over whatever its KV head retains.  Query head j reads KV head j / (q_heads / kv_heads).
 *
 * Conventions
 *   - Every function returns 0 (RLKV_OK) or a negative RLKV_E* code; nothing throws, exits or
 *     prints.  A call that returns RLKV_EINVAL, RLKV_EFULL, RLKV_EEMPTY, RLKV_ENOMEM or
 *     RLKV_ESCRATCH has changed nothing: these are found before anything is enqueued.  RLKV_ECUDA
 *     means a CUDA call failed part-way (normally the context is lost with it): lengths and cache
 *     contents are then unspecified and the cache should be destroyed.
 *   - "device" pointers are CUDA device memory on the GPU that was current at rlkv_cache_create;
 *     "host" pointers are ordinary host memory.  The caller owns every buffer it passes in.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  All GPU work is
 *     enqueued on it asynchronously; the library never synchronises on the hot path.  Calls on one
 *     cache must be ordered (one stream, or ordered by events): they share scratch memory.
 *   - bf16 = IEEE bfloat16 bit patterns, 2 bytes; all tensors are contiguous, row-major, and must
 *     be 16-byte aligned.
 *   - Lock-step batch: all `batch` sequences have the same length.  Each layer has its own length
 *     counter (append then attend, layer by layer).  The token appended in a step is visible to
 *     that step's attention (it is the newest token of the window).
 *   - Physical slot of token t in a compressed head: t if t < sink, else
 *     sink + ((t - sink) mod window).  While length <= sink + window nothing has been evicted.
 *   - Limits: head_dim in {64, 128}; 1 <= q_heads / kv_heads <= 8; kv_heads <= 128; sink >= 0;
 *     window >= 1.
 */
#ifndef RLKV_H
#define RLKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct rlkv_cache rlkv_cache; /* opaque, library-owned host object */

enum {
    RLKV_OK = 0,
    RLKV_EINVAL = -1, /* null/misaligned pointer, index out of range, unsupported shape */
    RLKV_EFULL = -2,  /* append/prefill would exceed max_len (any layer, uniform rule) */
    RLKV_EEMPTY = -3, /* decode on a layer that holds no token */
    RLKV_ENOMEM = -4, /* host or device allocation failed, or device_buf too small */
    RLKV_ECUDA = -5,  /* a CUDA call failed; rlkv_strerror(RLKV_ECUDA) carries the CUDA text */
    RLKV_EKERNEL = -6, /* a kernel gave up on a bounded wait (see rlkv_kernel_status) */
    RLKV_ESCRATCH = -7 /* rlkv_decode_attention_static_scratch: the static scratch array is too small */
};

/* Bytes of device memory a cache of this shape needs (pools, index tables, split scratch and the
 * staging area of rlkv_step_host).  head_is_full: host, [layers*kv_heads], 1 = full, 0 =
 * compressed.  A compressed head costs (sink+window) rows (rounded up to the 64-row tile) however
 * long the sequence grows -- the constant-size pool of Section 4.3. */
int rlkv_cache_size(int layers, int kv_heads, int q_heads, int head_dim, int batch, int max_len,
                    const uint8_t* head_is_full, int sink, int window, size_t* bytes_out);

/* Two-class cache layout (the two KV pools of Section 4.3).  device_buf == NULL: the library
 * cudaMallocs the memory and frees it in rlkv_cache_destroy.  Otherwise the caller provides
 * device_buf (1024-byte aligned, >= rlkv_cache_size bytes) and keeps it alive until destroy.
 * The pools are zero-filled, head_is_full is copied, all lengths start at 0.  Synchronous. */
int rlkv_cache_create(rlkv_cache** out, int layers, int kv_heads, int q_heads, int head_dim,
                      int batch, int max_len, const uint8_t* head_is_full, int sink, int window,
                      void* device_buf, size_t device_buf_bytes);
int rlkv_cache_destroy(rlkv_cache* cache);

/* The lock-step cache held in 8 bits: every K and V element of both head classes is stored as an
 * E4M3 code with one scale per (layer, KV head) for K and one for V (format, rounding and scales as
 * documented at rlkv_paged_create_fp8 below; k_scale, v_scale: HOST float [layers][kv_heads]).
 * head_dim must be 128.  The handle is a thin layer over the paged 8-bit cache with one request slot
 * per batch row and enough pages for every row to reach max_len, so no call finds the free list
 * empty.  On such a handle rlkv_append, rlkv_prefill, rlkv_decode_attention, rlkv_step,
 * rlkv_step_host (copies and kernels all on the caller's stream), rlkv_cache_reset (host bookkeeping
 * only: later work must go to the stream of the earlier), rlkv_set_step_mode, rlkv_set_output_bf16,
 * rlkv_length, rlkv_step_bytes (a K row and a V row of codes: 2 * head_dim bytes per token),
 * rlkv_kernel_status, rlkv_launch_count and rlkv_debug_export_head (the codes, one per 16-bit element;
 * rows that hold no token read as zero) work as documented; rlkv_set_decode_config, the overlapped
 * per-layer calls, rlkv_decode_attention_static_scratch, rlkv_decode_mixed_attention and
 * rlkv_debug_trace return RLKV_EINVAL. */
int rlkv_cache_size_fp8(int layers, int kv_heads, int q_heads, int head_dim, int batch, int max_len,
                        const uint8_t* head_is_full, int sink, int window, size_t* bytes_out);
int rlkv_cache_create_fp8(rlkv_cache** out, int layers, int kv_heads, int q_heads, int head_dim,
                          int batch, int max_len, const uint8_t* head_is_full, int sink, int window,
                          const float* k_scale, const float* v_scale, void* device_buf,
                          size_t device_buf_bytes);

/* All lengths back to 0 and the pools re-zeroed (asynchronous on `stream`). */
int rlkv_cache_reset(rlkv_cache* cache, void* stream);

/* Fused append (Section 4.3: circular buffer; Appendix B: the first sink tokens and the most
 * recent local tokens are kept).  k, v: device bf16 [batch][kv_heads][head_dim] -- all KV heads; the caller does
 * not need to know their classes.  Token t = length(layer) goes to row t of a full head and to
 * slot(t) of a compressed head; then length(layer) = t + 1.  Copies are bit-exact.
 * RLKV_EFULL if length(layer) == max_len. */
int rlkv_append(rlkv_cache* cache, int layer, const void* k, const void* v, void* stream);

/* Bulk append of n_tokens >= 1 tokens, defined as exactly n_tokens successive rlkv_append calls
 * (the resulting cache bytes are identical).  k, v: device bf16 [n_tokens][batch][kv_heads][head_dim].
 * RLKV_EFULL if length(layer) + n_tokens > max_len. */
int rlkv_prefill(rlkv_cache* cache, int layer, const void* k, const void* v, int n_tokens,
                 void* stream);

/* Split-KV decode attention over the heterogeneous heads of one layer, one launch for both head
 * classes (Section 3.3, last paragraph: a compressed head runs the same full attention, only over
 * the rows its smaller cache retains; Section 4.3 names a fused kernel for heterogeneous heads as
 * what would close the gap to the cost model).
 * q: device bf16 [batch][q_heads][head_dim]; out: device fp32 [batch][q_heads][head_dim].
 * Scores, softmax and accumulation are fp32.  RLKV_EEMPTY if length(layer) == 0. */
int rlkv_decode_attention(rlkv_cache* cache, int layer, const void* q, void* out, void* stream);

/* The per-layer calls for a model forward that wants them to overlap with the kernels around them.
 * (An integration call: the paper runs attention once per layer inside the model forward, Section 4.3
 * and Appendix B, and says nothing about how launches are ordered.)  A forward pass cannot use
 * rlkv_step: layer l + 1's q, k, v exist only after layer l's output has gone through its projections.
 * These two calls compute exactly what rlkv_append / rlkv_decode_attention compute, but are launched
 * with programmatic stream serialization, so they may START while the kernel before them on `stream`
 * is still running, and they let the kernel after them start early in turn:
 *   - the append executes griddepcontrol.wait before it reads k and v;
 *   - the attention launch sets up, and fetches K/V tiles that hold only older tokens (as many as its
 *     tile ring holds), before it waits; the query rows, the newest token's rows, the compressed
 *     heads' rings, the split-KV scratch and `out` are touched only after the wait.
 * So q, k and v may be written by the kernel directly before the call.  Requirements on the caller:
 * every kernel on `stream` that is itself launched with programmatic stream serialization must execute
 * griddepcontrol.wait (cudaGridDependencySynchronize) before it completes -- the usual way to use the
 * attribute -- so that a kernel's completion implies the completion of everything before it; a kernel
 * after the attention call that is launched that way must wait before it reads `out`.  After an
 * ordinary launch the calls behave like their ordinary counterparts.  Arguments, layouts, results and
 * error codes are those of rlkv_append and rlkv_decode_attention. */
int rlkv_append_overlapped(rlkv_cache* cache, int layer, const void* k, const void* v, void* stream);
int rlkv_decode_attention_overlapped(rlkv_cache* cache, int layer, const void* q, void* out,
                                     void* stream);
/* Both of them in ONE launch: the layer's step.  The attention launch appends the token itself --
 * the CTA that reads the tile a head's new token belongs to copies the caller's K and V rows there
 * first (bit for bit, after its wait), so no second kernel sits between the producer of k, v, q and
 * the attention.  Result and cache state are those of rlkv_append followed by
 * rlkv_decode_attention; the launch overlaps with its neighbours as described above.  k, v: device
 * bf16 [batch][kv_heads][head_dim]; q, out as for rlkv_decode_attention.  RLKV_EFULL if the layer is
 * at max_len. */
int rlkv_layer_step_overlapped(rlkv_cache* cache, int layer, const void* k, const void* v,
                               const void* q, void* out, void* stream);

/* rlkv_decode_attention for callers that must not allocate device memory.  (The paper has no
 * counterpart: this entry point exists for the integration, not for the method.)
 *
 * Who needs it: a host that has handed all device memory to its own pool before this library is
 * called -- a serving engine that sizes its KV pool to whatever cudaMalloc still grants at
 * start-up, a plugin running under a framework whose allocator owns the device, code running
 * where cudaMalloc is forbidden because it would synchronise the device in the middle of a step.
 * Such a host can give rlkv_cache_create a slice of its pool for the K/V rows, but may not want
 * the kernel's split-KV work area (tickets and partial results, rewritten by every launch) to
 * live there.  This call computes exactly what rlkv_decode_attention computes, with the same
 * kernel, and keeps that work area in an array that is part of the library image instead:
 * rlkv_static_scratch_bytes() bytes (4 MiB) of device memory on every GPU that loads librlkv,
 * held until the process exits.  The call itself allocates and frees nothing.
 *
 * - A launch that needs more than the array holds (batch * kv_heads tickets plus partial records
 *   of about (q_heads / kv_heads) * (head_dim + 2) floats each; rlkv_debug_schedule tells how many
 *   records a launch of a given shape may write) is refused with RLKV_ESCRATCH and nothing is
 *   launched.
 * - The first call on a device looks up the array's device address (one runtime query, kept for
 *   the life of the process; a driver that loads modules lazily gives the array its memory at that
 *   moment); make that first call at start-up, before starting any stream capture.  Two host
 *   threads may make their first calls on one device at the same time: both look the address up,
 *   get the same answer, and the slot that keeps it is written atomically.
 * - Every cache and every call on a device share the one array, which still holds the previous
 *   call's contents: each call clears the tickets and work-claim counters on `stream` before its launch.  Two such calls
 *   that overlap on the GPU (different streams, no ordering between them) race on the array and
 *   give wrong results; order them, or use rlkv_decode_attention for one of them.
 * Arguments, layouts and the other error codes are those of rlkv_decode_attention. */
int rlkv_decode_attention_static_scratch(rlkv_cache* cache, int layer, const void* q, void* out,
                                         void* stream);
size_t rlkv_static_scratch_bytes(void);

/* Mixed attention with gating adapters, the decode step of sample generation while the gates are
 * trained (Section 3.1, Eq. 1; Appendix B names custom decode kernels for it):
 *   out = alpha[h] * out_full_attn + (1 - alpha[h]) * out_local_attn        for q head j, h = j / G
 * where out_full_attn is attention over all length(layer) tokens of KV head h and out_local_attn
 * attention over its first `sink` tokens and its `window` most recent ones (the token appended last
 * included) -- what the head would see if it were compressed.  While length <= sink + window the two
 * branches are equal.  alpha = 1 gives rlkv_decode_attention's result for a full head, alpha = 0 the
 * result of a compressed head with the same history.
 * Every head of the layer must be a full head (the full branch needs every token): RLKV_EINVAL
 * otherwise.  q: device bf16 [batch][q_heads][head_dim]; alpha: DEVICE fp32 [kv_heads], the gates of
 * this layer, read when the kernel runs and used as they are (the paper keeps them in [0, 1]; the
 * library does not check); out: device fp32 [batch][q_heads][head_dim] (bf16 after
 * rlkv_set_output_bf16).  One launch and one pass: every K/V row is read once -- the softmax state
 * over the sink and window rows is the local branch and, merged with the state over the rows between
 * them, the full branch; whichever CTA delivers the last piece of a head merges them and writes
 * alpha * full + (1 - alpha) * local once.  K and V rows are assumed finite.
 * RLKV_EEMPTY if length(layer) == 0. */
int rlkv_decode_mixed_attention(rlkv_cache* cache, int layer, const void* q, const float* alpha,
                                void* out, void* stream);

/* Output element type of rlkv_decode_attention and its variants, rlkv_decode_mixed_attention,
 * rlkv_step and rlkv_step_host from now on: on != 0 stores results as bf16 (the fp32 result rounded
 * to nearest even when it is stored; `out` buffers then hold bf16 elements of the same shape, half
 * the bytes), on == 0 (the default) as fp32.  The arithmetic does not change. */
int rlkv_set_output_bf16(rlkv_cache* cache, int on);

/* One whole decode step: for every layer, append then attend.  Device buffers:
 * k, v bf16 [layers][batch][kv_heads][head_dim]; q bf16 [layers][batch][q_heads][head_dim];
 * out fp32 [layers][batch][q_heads][head_dim].  The results are those of the per-layer calls in
 * order (up to floating-point summation order: the step cuts the work differently).  Because all
 * inputs are there before the first launch, the step is issued as one append launch for all layers
 * and ONE attention launch over the K/V rows of every layer (the units of all layers form one flat
 * tile space, so a step of many small layers costs what its bytes cost, not a launch per layer);
 * where the layers hold different numbers of tokens, or the shape has more than 128 layers or 4096
 * (layer, KV head) pairs, it is one attention launch per layer, overlapped on the device (programmatic
 * dependent launch).  Every buffer must be complete when the call is made and stay untouched until
 * the work on `stream` has finished.  RLKV_EFULL (nothing done) if any layer is at max_len. */
int rlkv_step(rlkv_cache* cache, const void* k, const void* v, const void* q, void* out,
              void* stream);
/* How rlkv_step issues the attention of a step from now on: 0 (the default) lets the library choose as
 * described above, 1 forces one launch per layer, 2 one launch for the whole step (RLKV_EINVAL if
 * the shape does not allow it; a step whose layers differ in length still falls back to one launch
 * per layer).  Results do not depend on it beyond floating-point summation order. */
int rlkv_set_step_mode(rlkv_cache* cache, int mode);

/* The same step with HOST buffers of the same shapes (pinned memory makes the copies
 * asynchronous).  Inputs are copied host->device and results device->host inside the call, on two
 * streams of the library's own that run beside the kernels on `stream`: this call's inputs come in
 * while the kernels of the call before still run (the device staging area exists twice), and the
 * results of the first layers go out while the last layers are still computed.  The call returns
 * once the work is enqueued; work enqueued on `stream` afterwards waits for the results to have
 * arrived, so synchronising `stream` is enough before reading out_host.  The host input buffers
 * must stay untouched until then. */
int rlkv_step_host(rlkv_cache* cache, const void* k_host, const void* v_host, const void* q_host,
                   void* out_host, void* stream);

/* ---- the paged, ragged cache: the serving layout --------------------------------------------------
 * Section 4.3 of the paper serves requests of different lengths with continuous batching: the full
 * heads live in a paged pool, the compressed heads in a fixed-size pool with one constant-size
 * buffer per request, and the memory the compressed heads no longer need admits more requests.
 * rlkv_paged is that layout: max_seqs REQUEST SLOTS, each with its own length (per layer); the
 * full heads of all slots share n_pages PAGES of 64 tokens, handed out from one free list as
 * sequences grow and taken back when a slot is closed (page p of a sequence is page p of every full
 * head of every layer, as in the usual block table); every slot owns a sink + window ring per
 * compressed head.  What is computed per sequence is exactly what the lock-step cache computes for a
 * batch row (same slot rule, same attention); the calls name the request slots they act on, so a
 * decode step can serve any subset of the open slots, each at its own length.
 * Limits: max_seq_len <= 65536 tokens; at most min(max_seqs, 512) sequences per call; the other
 * shape limits of rlkv_cache_create.  Device memory: rlkv_paged_size bytes, library- or caller-owned
 * as for rlkv_cache_create.  Errors leave the cache unchanged. */
typedef struct rlkv_paged rlkv_paged;
int rlkv_paged_size(int layers, int kv_heads, int q_heads, int head_dim, int max_seqs, int n_pages,
                    int max_seq_len, const uint8_t* head_is_full, int sink, int window,
                    size_t* bytes_out);
int rlkv_paged_create(rlkv_paged** out, int layers, int kv_heads, int q_heads, int head_dim,
                      int max_seqs, int n_pages, int max_seq_len, const uint8_t* head_is_full,
                      int sink, int window, void* device_buf, size_t device_buf_bytes);
int rlkv_paged_destroy(rlkv_paged* cache);
/* The paged cache held in 8 bits.  (The paper names KV-cache quantisation as the direction to
 * combine head-level compression with and fixes no format; this is the format taken.)  Every K and
 * V element -- of the full heads' pages and of the compressed heads' rings -- is stored as an OCP E4M3 code (1 sign, 4 exponent bits
 * with bias 7, 3 mantissa bits, largest finite value 448, no infinities):
 *     code = E4M3(x * (1 / scale))   round to nearest even, magnitudes above 448 saturate;
 *     attention then runs on value(code) * scale
 * with one scale per (layer, KV head) for K and one for V: k_scale, v_scale, HOST float
 * [layers][kv_heads], positive and finite, copied (a scale of max|x| / 448 uses the whole range;
 * 1 is fine for activations of order one).  The cache then costs half the bytes per token, to store
 * and to read.  head_dim must be 128.  Every other call works as on a cache from rlkv_paged_create;
 * rlkv_paged_debug_export_head returns the codes, one per 16-bit element. */
int rlkv_paged_size_fp8(int layers, int kv_heads, int q_heads, int head_dim, int max_seqs, int n_pages,
                        int max_seq_len, const uint8_t* head_is_full, int sink, int window,
                        size_t* bytes_out);
int rlkv_paged_create_fp8(rlkv_paged** out, int layers, int kv_heads, int q_heads, int head_dim,
                          int max_seqs, int n_pages, int max_seq_len, const uint8_t* head_is_full,
                          int sink, int window, const float* k_scale, const float* v_scale,
                          void* device_buf, size_t device_buf_bytes);
/* Takes a free request slot (length 0 in every layer): RLKV_EFULL if all max_seqs are open. */
int rlkv_paged_seq_open(rlkv_paged* cache, int* slot_out);
/* Closes a slot: its pages go back to the free list.  The caller makes sure no work that uses the
 * slot is still in flight (host bookkeeping only, nothing is enqueued). */
int rlkv_paged_seq_close(rlkv_paged* cache, int slot);
/* One token for each of n sequences of one layer.  slots: HOST int[n], open slots, none twice;
 * k, v: device bf16 [n][kv_heads][head_dim], entry i for slots[i].  A sequence whose token opens a
 * page takes one from the free list.  RLKV_EFULL (nothing appended for any sequence) if a sequence
 * is at max_seq_len or the free list cannot serve every new page. */
int rlkv_paged_append(rlkv_paged* cache, int layer, const int* slots, int n, const void* k,
                      const void* v, void* stream);
/* n_tokens tokens for one sequence, exactly n_tokens single appends.  k, v: device bf16
 * [n_tokens][kv_heads][head_dim]. */
int rlkv_paged_prefill(rlkv_paged* cache, int layer, int slot, const void* k, const void* v,
                       int n_tokens, void* stream);
/* Decode attention for n sequences of one layer, each over its own length, one launch for both
 * head classes and all lengths.  q: device bf16 [n][q_heads][head_dim]; out: device fp32
 * [n][q_heads][head_dim]; entry i belongs to slots[i] (HOST int[n]).  RLKV_EEMPTY if a listed
 * sequence holds no token in this layer. */
int rlkv_paged_decode_attention(rlkv_paged* cache, int layer, const int* slots, int n,
                                const void* q, void* out, void* stream);
/* One whole decode step for n sequences: one token appended to every layer of each, then every
 * layer's attention.  k, v: device bf16 [layers][n][kv_heads][head_dim]; q: device bf16
 * [layers][n][q_heads][head_dim]; out: device fp32 [layers][n][q_heads][head_dim]; entry i of the
 * second dimension belongs to slots[i] (HOST int[n]).  Results are those of rlkv_paged_append and
 * rlkv_paged_decode_attention layer by layer (up to floating-point summation order).  As in rlkv_step
 * all inputs are there before the first launch, so the step is one append launch for all layers and
 * one attention launch over the K/V rows of every layer (or the layers' attention launches, overlapped
 * on the device: see rlkv_paged_set_step_mode); the buffers must be complete at the call
 * and stay untouched until the work on `stream` has finished.  Every listed sequence must have the
 * same length in all layers (RLKV_EINVAL otherwise); RLKV_EFULL as for rlkv_paged_append. */
int rlkv_paged_step(rlkv_paged* cache, const int* slots, int n, const void* k, const void* v,
                    const void* q, void* out, void* stream);
/* As rlkv_set_step_mode, for rlkv_paged_step: 0 (the default) one attention launch over the K/V rows
 * of every layer where the step's split-KV records fit the scratch (else one launch per layer), 1
 * always one launch per layer, 2 as 0 (RLKV_EINVAL if the shape has more than 128 layers or 4096
 * (layer, KV head) pairs). */
int rlkv_paged_set_step_mode(rlkv_paged* cache, int mode);
/* As rlkv_set_output_bf16, for rlkv_paged_decode_attention and rlkv_paged_step. */
int rlkv_paged_set_output_bf16(rlkv_paged* cache, int on);
int rlkv_paged_length(const rlkv_paged* cache, int layer, int slot, int* len_out);
/* Pages on the free list and pages in total. */
int rlkv_paged_pages(const rlkv_paged* cache, int* free_out, int* total_out);
/* Bytes of K and V rows the next rlkv_paged_decode_attention on these slots must read. */
int rlkv_paged_step_bytes(const rlkv_paged* cache, int layer, const int* slots, int n,
                          uint64_t* kv_bytes_out);
/* One head of one sequence copied to the host (synchronises the device).  A full head: its
 * length(layer, slot) rows in token order, gathered page by page (k_host, v_host hold up to
 * max_seq_len rows); a compressed head: its sink + window physical rows, as
 * rlkv_debug_export_head. */
int rlkv_paged_debug_export_head(rlkv_paged* cache, int layer, int slot, int kv_head, void* k_host,
                                 void* v_host, int* rows_out, int32_t* token_of_slot_host);
int rlkv_paged_kernel_status(rlkv_paged* cache, int* status_out);
/* The split bookkeeping of a paged decode launch, host arithmetic only (no GPU): n sequences of
 * lens[i] tokens (host int[n]) over n_full full and n_comp compressed heads, cap = sink + window,
 * cut for `ctas` CTAs into work items of at least item_tiles tiles.  For every unit (sequence i,
 * head slot f: index i * n_full + f; then the compressed units, i * n_comp + c after all full ones)
 * delivered_out counts the partial records the kernel's walk over the work items delivers,
 * expected_out the number its tickets wait for, complete_out the segments that hold the whole unit
 * and write its result directly (host int[n * (n_full + n_comp)] each).  A unit is served
 * correctly iff complete == 1 and delivered == 0, or complete == 0 and delivered == expected >= 1.
 * RLKV_EKERNEL if two segments of a unit would share a partial record. */
int rlkv_debug_paged_schedule(const int* lens, int n, int n_full, int n_comp, int cap, int ctas,
                              int item_tiles, int* n_items_out, int* delivered_out,
                              int* expected_out, int* complete_out);

/* ---- introspection (host-side bookkeeping; no GPU work unless stated) ---- */
int rlkv_length(const rlkv_cache* cache, int layer, int* len_out);
/* Bytes of K and V rows the next rlkv_decode_attention on `layer` must read:
 * batch * sum over KV heads of min(length, rows the head retains) * 2 * head_dim * 2
 * (the cost model of Section 4.3: (1-s) + s*W/L of the full-cache bytes). */
int rlkv_step_bytes(const rlkv_cache* cache, int layer, uint64_t* kv_bytes_out);
/* Copies one head's physical rows to the host (synchronises the device).  k_host, v_host: bf16
 * [rows][head_dim] where rows = max_len for a full head, sink+window for a compressed head;
 * token_of_slot_host: int32[rows], the token held by each row or -1 if the row is empty. */
int rlkv_debug_export_head(rlkv_cache* cache, int layer, int batch_row, int kv_head, void* k_host,
                           void* v_host, int* rows_out, int32_t* token_of_slot_host);
/* Synchronises the device and reads the kernels' status word: 0 = no kernel ever gave up on a
 * bounded wait; otherwise a code identifying the wait that ran out (results are then invalid). */
int rlkv_kernel_status(rlkv_cache* cache, int* status_out);
/* Number of kernels this cache has launched so far. */
int rlkv_launch_count(const rlkv_cache* cache, uint64_t* launches_out);
/* Tuning knobs of the decode kernel: persistent CTAs per SM (1 or 2), TMA pipeline stages (2..8, a
 * multiple of the consumer groups), groups of four consumer warps that take tiles in turn (1..3),
 * and the size in 64-row tiles of the smallest work items the K/V scan is cut into (2..1024; a
 * launch too small to give every CTA one such item uses smaller ones).
 * 0 keeps the current value (stages: lowered if the new shape no longer fits).  RLKV_EINVAL if the
 * shape does not fit in shared memory.  Defaults: 1 CTA per SM, 2 groups, as many stages as fit,
 * 32 tiles inside rlkv_step (whose launches overlap) and 8 tiles for a launch on its own.  Results do not depend on these knobs beyond floating-point summation order. */
int rlkv_set_decode_config(rlkv_cache* cache, int ctas_per_sm, int stages, int consumer_groups,
                           int item_tiles);
/* Debug trace of the decode kernel.  enable != 0: later decode launches record, per CTA, 40
 * 64-bit words: [0..3] %globaltimer (ns) at CTA start, when its first tile landed, when its last
 * segment was handed off and at CTA end; [4..6] work items, tiles and partial segments it
 * processed; [7] %globaltimer when its epilogue warps finished; [8..10] SM cycles its first consumer
 * warp waited for work items, for tiles and for a free hand-off buffer; [11] cycles its epilogue
 * warps were idle; [12..13] %globaltimer when the CTA's stream had ended and how many split units
 * it then merged; [14..15] cycles its producer waited for the next work item's number, and for a
 * free descriptor (low half) and a free stage (high half); [16..26] for its first 11 work items,
 * (%globaltimer << 16) | (item & 0xffff) when the consumers started it; [27] cycles the producer
 * ran; [28..31] %globaltimer stamps inside the final merge; [32..36] producer cycles spent arming
 * barriers, issuing tile copies, issuing query copies, publishing items and locating segments;
 * [37..39] %globaltimer when the producer issued its first tile copy, when the CTA's set-up was done
 * and when the producer entered its loop.
 * words_host != NULL: first synchronises the device and copies the words of the most recent launch
 * to words_host (host, 40 * 320 words) and the CTA capacity (320) to *ctas_out; then the switch is
 * applied. */
int rlkv_debug_trace(rlkv_cache* cache, int enable, unsigned long long* words_host, int* ctas_out);
/* The work schedule of the decode kernel, host arithmetic only (no GPU).  full_units units of
 * tiles_full 64-row tiles and comp_units units of tiles_comp tiles are laid out as one flat tile
 * space (in bands: the first half of every full unit, then half of the rest, ... then the rest and
 * the compressed units) and cut for `ctas` CTAs into *n_items_out contiguous work items whose sizes
 * shrink geometrically down to item_tiles; *n_slots_out is the number of partial-result records a
 * launch of this shape may write.  whole_step != 0: the schedule rlkv_step uses for one launch over
 * all layers instead (most full units whole, unit after unit, in one equal item per CTA; the rest and
 * the compressed units unit after unit in items of item_tiles tiles, fewer where the step is small;
 * whole_step == 2: the form rlkv_paged_step uses for sequences of unequal lengths, whose whole units
 * are handed out one by one instead of in one equal item per CTA).  Optional outputs (host; `cap` = ints available in starts_out
 * and 4-int records available in tile_map_out): starts_out[k] = first flat tile of item k, then
 * the total; tile_map_out[4x..4x+3] = unit, tile inside the unit, consecutive tiles of the unit
 * from x on, partial record of the segment holding flat tile x.  RLKV_EKERNEL if the schedule's
 * own maps disagree with each other (a self-check; never expected). */
int rlkv_debug_schedule(int full_units, int tiles_full, int comp_units, int tiles_comp, int ctas,
                        int item_tiles, int whole_step, int* n_items_out, int* n_slots_out,
                        int* starts_out, int* tile_map_out, int cap);

/* Measurement aid (synchronous; no cache involved): reads `bytes` of device memory at device_buf
 * (16-byte aligned, at least 32 KiB; contents irrelevant) `launches` times with the mechanism the
 * decode kernel's producer uses -- bulk asynchronous copies into a ring of shared-memory stages, one
 * persistent CTA per SM -- and nobody consuming the data.  *ms_out = mean time of one pass in
 * milliseconds (CUDA events, after one untimed pass): bytes / that is the read-only bandwidth the
 * decode kernel could at best reach on this GPU.  RLKV_EKERNEL if a wait inside the kernel ran out. */
int rlkv_debug_read_bandwidth(const void* device_buf, size_t bytes, int launches, float* ms_out);

/* Measurement and test aid: a stand-in for the kernels a model runs between two attention calls.
 * One launch on `stream` that (1) copies `bytes` bytes from src to dst (device buffers of the caller;
 * work that depends on nothing, like the weights a projection streams), then (2) waits for the kernel
 * before it, reads a word of `after` (device; may be NULL -- the attention output it would consume)
 * and copies produce_bytes bytes from produce_src to produce (device; the next call's q, k or v), so
 * that those are written at the very end of the kernel.  overlap != 0: launched with programmatic
 * stream serialization (it may start beside the kernel before it and lets the next one start early);
 * 0: an ordinary launch.  Sizes are multiples of 16, pointers 16-byte aligned. */
int rlkv_debug_standin(void* dst, const void* src, size_t bytes, const void* after, void* produce,
                       const void* produce_src, size_t produce_bytes, int overlap, void* stream);

/* How rlkv_step and rlkv_paged_step order the decode launches of one step, host arithmetic only (no
 * GPU).  For launch l of n_launches in a row (follows_append != 0: the first one directly follows the
 * step's append launch in the stream): overlap_out[l] = 1 if it is launched so that it may start
 * while launch l - 1 still runs; dep_wait_out[l] = what it waits for on the device before it lets
 * launch l + 1 start (0: nothing -- it is an ordinary launch, whose predecessor has completed before
 * it starts; 1: the append launch; 2: launch l - 1); scratch_copy_out[l] = which of the two copies
 * of the split-KV scratch it uses.  Launches l and l - 2 share a copy; they are never in flight
 * together because launch l - 1 holds launch l back until launch l - 2 has completed.  (host int
 * [n_launches] each) */
int rlkv_debug_step_plan(int n_launches, int follows_append, int* overlap_out, int* dep_wait_out,
                         int* scratch_copy_out);

/* The order in which the work items of rlkv_debug_schedule's schedule are handed out, host arithmetic
 * only: order_out[k] (host int[n_items]; `cap` = ints available) = the item CTA k starts with (k <
 * ctas) resp. the item the (k - ctas)-th run-time claim receives.  Items made of compressed units come
 * first among the claimed ones (many short segments: they must not be the launch's last items). */
int rlkv_debug_claim_order(int full_units, int tiles_full, int comp_units, int tiles_comp, int ctas,
                           int item_tiles, int whole_step, int* order_out, int cap);

const char* rlkv_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* RLKV_H */
