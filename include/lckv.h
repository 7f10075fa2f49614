/*
 * lckv.h - C ABI of the B200 (sm_100a) decode-step attention library for the
 * Layer-Condensed KV Cache (LCKV, arXiv 2405.10637).
 *
 * What the library computes (paper, Section 2.1).  In an LCKV decoder the
 * queries of every non-warmup layer are paired with the keys and values of
 * the TOP layer only, so one cache is shared by all those layers; a token does
 * not attend to itself there (the diagonal of the attention matrix is masked,
 * because the top layer's k,v of the current token do not exist yet while the
 * lower layers run), and a token that sees nothing attends to a zero dummy
 * key/value, i.e. its output is the zero vector.  The top w/2 and bottom w/2
 * layers ("warmup layers", sandwich placement) keep standard attention over
 * their own per-layer caches, including the current token.  Decoding proceeds
 * one token at a time, bottom layer to top layer (Section 2.2).
 *
 * Conventions common to every call
 *   - All tensor arguments are DEVICE pointers unless a name says "host".
 *   - bf16 tensors are raw 16-bit patterns (upper half of IEEE binary32),
 *     contiguous, 16-byte aligned.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Calls only enqueue work; none synchronises unless it says so.
 *   - The library allocates no device memory: the caller hands one device
 *     buffer to lckv_cache_alloc and keeps it alive until lckv_cache_free.
 *   - Every call returns an int status (LCKV_OK = 0).  Nothing aborts, throws
 *     or traps.  On any non-zero status nothing was enqueued and no length
 *     changed, unless stated otherwise.
 *   - A cache object is not thread-safe; use it from one host thread and one
 *     stream at a time (kernels of one cache share its workspace).
 */
#ifndef LCKV_H
#define LCKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    LCKV_OK = 0,
    LCKV_EINVAL = 1,    /* null pointer, bad shape, odd w, batch > max_batch, bad slot or mode  */
    LCKV_ECAPACITY = 2, /* a sequence would exceed max_seq rows                                */
    LCKV_ENOMEM = 3,    /* caller's buffer too small or not 256-byte aligned                   */
    LCKV_ECUDA = 4,     /* a CUDA runtime/driver call failed; see lckv_last_cuda_error         */
    LCKV_ETIMEOUT = 5,  /* a bounded device-side wait gave up (reported by lckv_cache_status)  */
    LCKV_ESTATICLIMIT = 6 /* lckv_decode_attention_static: batch or GPU beyond its fixed scratch */
};

enum {
    LCKV_MODE_CONDENSED = 0, /* visible positions j <  len[b]: diagonal masked (Section 2.1) */
    LCKV_MODE_STANDARD = 1   /* visible positions j <= len[b]: warmup layers  (Section 2.1)  */
};

typedef struct lckv_cache lckv_cache_t; /* opaque host object */

/* Plain-old-data description of a layer stack and its caches. */
typedef struct {
    uint32_t struct_size;  /* sizeof(lckv_config_t), for versioning                          */
    int32_t n_layers;      /* L >= 1, layer 0 = bottom                                       */
    int32_t n_warmup;      /* w: even with 0 <= w < L, or w == L (standard transformer)      */
    int32_t n_q_heads;     /* H_q                                                            */
    int32_t n_kv_heads;    /* H_kv, H_q % H_kv == 0; q head h reads kv head h / (H_q/H_kv)   */
    int32_t head_dim;      /* d_h: 64 or 128                                                 */
    int32_t max_batch;     /* B_max >= 1                                                     */
    int32_t max_seq;       /* T_cap >= 1 rows per sequence per cache                         */
    float softmax_scale;   /* 0 => 1/sqrt(d_h)                                               */
    int32_t top_variant;   /* which layer feeds the shared cache, see lckv_plan              */
    int32_t out_dtype;     /* 0 = bf16 outputs, 1 = fp32 outputs                             */
    int32_t host_staging;  /* 1: reserve device staging for lckv_layer_stack_step_host       */
    int32_t use_graph;     /* 1: lckv_layer_stack_step replays a CUDA graph when the argument
                              pointers repeat from the previous call (needs a stream other
                              than the legacy default stream; otherwise plain launches)      */
    int32_t stream_sink;   /* 0 = off.  s >= 1: StreamingLLM-style caches (paper Section 3.3): every
                              slot keeps the first s tokens ("attention sinks") and the most
                              recent max_seq - s tokens; token t >= max_seq overwrites row
                              s + (t - s) mod (max_seq - s).  Lengths keep counting all tokens;
                              LCKV_ECAPACITY is never returned.  Needs 1 <= s < max_seq.     */
    int32_t page_rows;     /* 0 = each slot is one [B_max, H_kv, T_cap, d_h] tensor.  P > 0 (a power of
                              two >= 64): paged slots [n_pages, H_kv, P, d_h]; a sequence owns
                              ceil(len / P) pages taken from a pool, so ragged batches pay for the
                              rows they hold, not for B_max * T_cap.  One page table
                              [B_max][ceil(T_cap / P)] serves every slot (all caches have the same
                              lengths).  Not combinable with stream_sink.                     */
    int32_t n_pages;       /* pool size per slot when page_rows > 0                            */
    int32_t kernel_kind;   /* 0 = choose (tensor-core kernel for query groups of 2 ... 7 and
                              multiples of 8, else the FP32-ALU kernel); 1 = force FP32-ALU  */
} lckv_config_t;

/* Facts about a built cache that a caller or a benchmark may want. */
typedef struct {
    int32_t n_slots;          /* distinct caches held (footprint in layers)                  */
    int32_t n_workers;        /* independent workers (warps) per attention launch            */
    int32_t rows_per_tile;    /* cache rows moved by one bulk copy                           */
    int32_t kernel_kind;      /* 1 = FP32-ALU kernel (one q head per pair),
                                 2 = tensor-core kernel (one kv head's query group per pair) */
    int32_t launches_per_step;/* kernels lckv_layer_stack_step enqueues                      */
    int32_t sm_count;
    uint64_t slot_bytes;      /* bytes of one K (or V) tensor of one slot                    */
    uint64_t workspace_bytes; /* lengths + plan tables + split-K partials + counters         */
} lckv_info_t;

/*
 * Layer plan (Section 2.1: the top w/2 layers and the bottom w/2 layers are
 * warmup layers; Section 4.2: w = L is the standard transformer).  Host only,
 * no GPU needed.  All output arrays have n_layers entries.
 *   is_warmup[l]     1 for warmup layers
 *   read_slot[l]     cache slot layer l attends to (slot 0 = the shared top-layer cache)
 *   mode[l]          LCKV_MODE_CONDENSED or LCKV_MODE_STANDARD
 *   write_slot[l]    slot that receives layer l's new k,v, or -1 (layer computes no K/V)
 *   write_before[l]  1: appended before layer l attends (standard layers see
 *                    their own token); 0: appended at the end of the step
 * top_variant 0 (paper-literal): slot 0 is the cache of layer L-1 itself; if
 *   that layer is a warmup layer it uses slot 0 with standard attention while
 *   the condensed layers below it see slot 0 without the current token.
 *   Footprint max(w,1) caches.
 * top_variant 1: slot 0 is fed by the topmost non-warmup layer L-1-w/2 and the
 *   w warmup layers own slots 1..w.  Footprint min(w+1, L) caches.
 * Errors: LCKV_EINVAL for null pointers, L < 1, odd w, w > L, bad variant.
 */
int lckv_plan(int32_t n_layers, int32_t n_warmup, int32_t top_variant, int32_t* is_warmup,
              int32_t* read_slot, int32_t* mode, int32_t* write_slot, int32_t* write_before,
              int32_t* n_slots);

/*
 * Device bytes lckv_cache_alloc needs for this configuration (caches for every
 * slot of the plan + lengths + workspace + optional staging), or 0 if the
 * configuration is invalid.  Needs a CUDA device (the workspace is sized from
 * the SM count of the current device).
 */
size_t lckv_cache_bytes(const lckv_config_t* cfg);

/*
 * Build a cache object over caller-owned device memory (Section 1: the KV
 * cache stores each layer's keys and values of past tokens; here only
 * max(w,1) or w+1 layers have one).
 *   dev_buf/dev_bytes  device buffer, 256-byte aligned, >= lckv_cache_bytes(cfg).
 *                      The caller owns it; the library never frees it.
 * Layout inside: per slot one K and one V tensor [B_max, H_kv, T_cap, d_h]
 * bf16, contiguous; one int32 length per sequence shared by all slots (all
 * caches advance together).  Lengths start at 0 and the workspace is cleared
 * (this call synchronises the device once).  Cache contents are NOT cleared.
 * Errors: EINVAL (bad config / null), ENOMEM (buffer small or misaligned),
 * ECUDA.
 */
int lckv_cache_alloc(lckv_cache_t** out, const lckv_config_t* cfg, void* dev_buf,
                     size_t dev_bytes);

/* Destroys the host object (and any CUDA graph it holds).  The device buffer stays the caller's. */
int lckv_cache_free(lckv_cache_t* cache);

/* Fills *info.  EINVAL on null. */
int lckv_cache_info(const lckv_cache_t* cache, lckv_info_t* info);

/*
 * Set per-sequence lengths (tokens already cached) from a HOST array, or all to
 * zero if host_lens is NULL; clears the split-K workspace and the device
 * status word.  Enqueued on `stream`; host_lens may be reused on return.
 * Errors: EINVAL (batch out of range, negative length), ECAPACITY (a length
 * > T_cap), ECUDA.
 */
int lckv_cache_reset(lckv_cache_t* cache, const int32_t* host_lens, int32_t batch, void* stream);

/* Copies the device lengths of the first `batch` sequences to host_out; SYNCHRONISES `stream`. */
int lckv_cache_lengths(const lckv_cache_t* cache, int32_t* host_out, int32_t batch, void* stream);

/*
 * Reads the device status word (0, or LCKV_ETIMEOUT if some kernel's bounded
 * wait on a copy gave up; the outputs of that launch are then undefined);
 * SYNCHRONISES `stream`.  lckv_cache_reset clears it.
 */
int lckv_cache_status(const lckv_cache_t* cache, int32_t* host_status, void* stream);

/*
 * Sets how many polls a device-side wait on a copy may take in the decode attention kernels
 * before the kernel gives up (default 2^18; one poll parks the warp for up to 20 us).  A wait that
 * runs out sets the status word to LCKV_ETIMEOUT, lets the copies still in flight land (a second,
 * fixed bound) and returns; that launch's outputs and the merge tickets are then undefined until
 * lckv_cache_reset.  0 makes the first wait of every worker give up at once: a way to exercise the
 * timeout path without anything actually hanging.  Takes effect from the next launch (a captured
 * step is dropped and captured again).  EINVAL on null.
 */
int lckv_cache_set_wait_limit(lckv_cache_t* cache, uint32_t polls);

/*
 * Diagnostic: lets the decode attention launches use only `workers` of the worker warps the cache was
 * laid out for (1 ... lckv_info_t.n_workers; 0 restores all).  The tile sequence of a launch is cut
 * into that many ranges instead, so pairs are split at other places and over other numbers of
 * workers: running one case at several limits exercises the split-K merge (paper-side this is
 * nothing but the log-sum-exp rule) at several split counts.  Results stay within the parity bounds
 * at any limit; they are bitwise repeatable only at equal limits.  Takes effect from the next launch (a
 * captured step is dropped and captured again).  EINVAL on null or a count out of range.
 */
int lckv_cache_set_worker_limit(lckv_cache_t* cache, int32_t workers);

/* Device pointers of slot `slot`'s K and V tensors [B_max, H_kv, T_cap, d_h] bf16 (for filling
 * a cache with a prompt's keys and values, or inspecting it).  EINVAL on bad slot / null. */
int lckv_cache_slot_ptrs(const lckv_cache_t* cache, int32_t slot, void** k, void** v);

/*
 * Paged caches only: copies the host mirror of the page table, [max_batch][*entries_per_seq] page
 * ids (-1 = no page), to host_out (may be NULL to query the width only).  Logical row r of
 * sequence b is row r % page_rows of page table[b][r / page_rows], i.e. element
 * [page, kv_head, r % page_rows, :] of a slot tensor.  Pages are assigned by lckv_cache_reset and,
 * as sequences grow, by the append / step calls; when the pool is exhausted those calls return
 * LCKV_ECAPACITY and change nothing.  EINVAL if the cache is not paged.
 */
int lckv_cache_page_table(const lckv_cache_t* cache, int32_t* host_out, int32_t* entries_per_seq);

/*
 * Append (Section 2.1: only the top layer and the warmup layers compute K/V):
 * writes k_new, v_new [batch, H_kv, d_h] bf16 as row len[b] of slot `slot` for
 * every b < batch; bit-exact copy.  If advance_len != 0 every len[b], b < batch,
 * grows by one afterwards (this advances ALL slots: they share the lengths).
 * Errors: EINVAL, ECAPACITY (some len[b] + 1 > T_cap, judged from the host
 * mirror of the lengths; nothing written), ECUDA.
 */
int lckv_append_kv(lckv_cache_t* cache, int32_t slot, const void* k_new, const void* v_new,
                   int32_t batch, int32_t advance_len, void* stream);

/*
 * Produce-and-append (Section 2.1: W_K and W_V map a hidden representation to
 * its key and value, and in the condensed model only the top layer and the
 * warmup layers still have them): for every b < batch computes
 *     k[b, f] = sum_c w_k[f, c] x[b, c],   v[b, f] = sum_c w_v[f, c] x[b, c]
 * on the tensor cores (bf16 inputs, fp32 accumulation, one rounding to bf16)
 * and stores them as row len[b] of slot `slot` - lckv_append_kv without the
 * round trip of k and v through device memory.
 *   x        [batch, d_model] bf16, device, 16-byte aligned, row-major
 *   w_k, w_v [H_kv * d_h, d_model] bf16, device, 16-byte aligned, row-major
 *            (row f = output feature = kv head f / d_h, dimension f % d_h)
 *   rope_cos, rope_sin  both NULL, or [rope_positions, d_h / 2] fp32 device
 *            tables (16-byte aligned): the key (never the value) is then rotated by the token's
 *            position p = len[b] in the half-split pairing
 *              k'[i]         = k[i] cos[p,i] - k[i + d_h/2] sin[p,i]
 *              k'[i + d_h/2] = k[i + d_h/2] cos[p,i] + k[i] sin[p,i],  i < d_h/2
 *            (rotary position embedding as Llama models apply it; the paper
 *            does not restate it, so it is optional and the tables - hence the
 *            frequencies - are the caller's).
 *   advance_len as in lckv_append_kv.
 * Requirements: d_model a multiple of 64, H_kv * d_h a multiple of 128.
 * Errors: EINVAL (null / misaligned pointer, bad shape, one table without the
 * other, rope_positions <= some len[b]), ECAPACITY as lckv_append_kv, ECUDA.
 * A device-side wait that runs out shows in lckv_cache_status (LCKV_ETIMEOUT).
 * The library keeps descriptors of x, w_k, w_v keyed by address and shape.
 */
int lckv_project_append_kv(lckv_cache_t* cache, int32_t slot, const void* x, int32_t d_model,
                           const void* w_k, const void* w_v, const float* rope_cos,
                           const float* rope_sin, int32_t rope_positions, int32_t batch,
                           int32_t advance_len, void* stream);

/*
 * Decode attention of one layer for one new token per sequence (Section 2.1):
 *   out[b,h] = sum_j softmax_j( scale * <q[b,h], K[b,kv(h),j]> ) * V[b,kv(h),j]
 * over the visible rows j of slot `slot`: j < len[b] (LCKV_MODE_CONDENSED,
 * diagonal masked) or j <= len[b] (LCKV_MODE_STANDARD; row len[b] must have
 * been appended without advancing).  A row that sees nothing (condensed mode,
 * len[b] == 0) gets the zero vector (zero dummy key/value) and lse 0.
 *   q    [batch, H_q, d_h] bf16
 *   out  [batch, H_q, d_h] bf16 (or fp32 if out_dtype == 1)
 *   lse  [batch, H_q] fp32 natural-log sum of exponentials of the scaled
 *        scores, or NULL
 * Arithmetic: fp32 scores, fp32 running max / sum / accumulators, split over
 * the sequence with a log-sum-exp merge of fp32 partials, one rounding to the
 * output type.  Rows >= the visible count are never read.
 * Errors: EINVAL, ECAPACITY (mode STANDARD with a full sequence), ECUDA.
 */
int lckv_decode_attention(lckv_cache_t* cache, int32_t slot, int32_t mode, const void* q,
                          void* out, float* lse, int32_t batch, void* stream);

/*
 * One decode step of the whole layer stack (Sections 2.1, 2.2), layers in
 * order as DEPENDENT launches on `stream` - layer l+1's query is a function of
 * layer l's output in a real model, so queries of different layers are never
 * batched into one pass.  For l = 0..L-1, following lckv_plan:
 *   write_before[l]: append k_new_layers[l], v_new_layers[l] to write_slot[l];
 *   attend q_layers[l] over read_slot[l] in mode[l] into out_layers[l];
 * then append the feeder layer's k,v to slot 0 if not done yet, then
 * len[b] += 1 for b < batch.
 *   q_layers, out_layers            HOST arrays of L device pointers
 *   k_new_layers, v_new_layers      HOST arrays of L device pointers; entries of
 *                                   layers with write_slot[l] < 0 are ignored
 * Errors: EINVAL (null array, null required entry, batch), ECAPACITY (some
 * sequence is full; nothing enqueued), ECUDA.
 */
int lckv_layer_stack_step(lckv_cache_t* cache, const void* const* q_layers,
                          void* const* out_layers, const void* const* k_new_layers,
                          const void* const* v_new_layers, int32_t batch, void* stream);

/*
 * The same step for callers whose activations live in HOST memory (pinned for
 * real overlap): copies every layer's q (and the k,v of layers that have them)
 * host->device into the cache's staging area, runs the step, copies every
 * layer's output device->host.  Asynchronous: the step is ordered after the work
 * already queued on `stream`, and `stream` ends up waiting for the last copy, so
 * synchronise `stream` before reading the outputs.  The copies themselves run
 * on two streams the cache creates on the first such call (no device memory is
 * allocated): the layers are cut into up to 8 chunks, a chunk's layers start
 * when its queries have arrived and its outputs leave while later chunks
 * compute.  Needs host_staging = 1 at alloc.  When the layers' host buffers are
 * contiguous in memory (one allocation sliced per layer) a chunk is a single
 * pitched copy per direction instead of one copy per layer.
 * Array arguments are HOST arrays of L HOST pointers with the shapes above.
 */
int lckv_layer_stack_step_host(lckv_cache_t* cache, const void* const* q_layers_host,
                               void* const* out_layers_host,
                               const void* const* k_new_layers_host,
                               const void* const* v_new_layers_host, int32_t batch,
                               void* stream);

/*
 * Prompt encoding (Section 2.3: the prompt is encoded by m + b parallel
 * iterations; Section 2.2.1 defines one iteration: all tokens in parallel, the
 * condensed layers paired with the top-layer k,v of the PREVIOUS iteration -
 * zero vectors before the first one - and the diagonal masked).  These calls
 * are the attention and cache-write operations of one such iteration.  They
 * require lengths already set to the prompt lengths (lckv_cache_reset) and do
 * not change them; n_max >= every len[b] of the batch is the token stride of
 * the token-major tensors.  Not available with stream_sink > 0.
 *
 * lckv_prefill_write_kv: rows [0, len[b]) of slot `slot` <- k, v
 *   [batch, n_max, H_kv, d_h] bf16 (bit-exact copies; other rows untouched).
 * lckv_prefill_attention: for every token i < len[b] and head h,
 *   out[b,i,h] = softmax-weighted sum over rows j < i (LCKV_MODE_CONDENSED) or
 *   j <= i (LCKV_MODE_STANDARD) of the slot; a token that sees nothing gets
 *   the zero vector.  q, out: [batch, n_max, H_q, d_h] (out bf16 or fp32 per
 *   out_dtype); rows i >= len[b] of out are not written.  Tensor-core kernel,
 *   fp32 accumulation, probabilities rounded to bf16 for the second product.
 * lckv_prefill_iteration: one iteration over the whole stack in plan order
 *   (write_before layers store their k,v and attend causally; condensed layers
 *   attend slot 0, which still holds the previous iteration's top-layer k,v;
 *   at the end the feeder layer's k,v replace them).  Before the first
 *   iteration the caller zero-fills slot 0 (the dummy zero k,v).  Array
 *   arguments as in lckv_layer_stack_step, tensors token-major as above.
 * Errors: EINVAL (null, bad slot/mode/batch, n_max < 1, a len[b] > n_max,
 * stream_sink > 0), ECUDA.
 */
int lckv_prefill_write_kv(lckv_cache_t* cache, int32_t slot, const void* k, const void* v,
                          int32_t n_max, int32_t batch, void* stream);
int lckv_prefill_attention(lckv_cache_t* cache, int32_t slot, int32_t mode, const void* q,
                           void* out, int32_t n_max, int32_t batch, void* stream);
int lckv_prefill_iteration(lckv_cache_t* cache, const void* const* q_layers,
                           void* const* out_layers, const void* const* k_layers,
                           const void* const* v_layers, int32_t n_max, int32_t batch,
                           void* stream);

/*
 * Decode attention without a cache object and without any allocation (the
 * paper has no counterpart: this is a packaging variant of
 * lckv_decode_attention for callers that cannot allocate).
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a
 * serving engine that has already handed all device memory to its own pool,
 * in a plugin whose host forbids allocation after initialisation, or on a
 * latency path where an allocation's implicit synchronisation is not
 * acceptable - and that also has nowhere to keep a workspace buffer for us.
 * The regular entry point needs a caller-provided workspace for its work plan,
 * split-K partials and merge tickets; this one keeps that scratch in a fixed
 * array compiled into the library's device image instead.
 *
 * Same computation and argument meaning as lckv_decode_attention, with the
 * cache described by plain pointers:
 *   k, v      [batch, H_kv, max_seq, d_h] bf16, rows [0, visible) of each
 *             (sequence, kv head) valid
 *   lens      [batch] int32 DEVICE array, tokens cached per sequence
 *   q, out, lse, mode, softmax_scale (0 => 1/sqrt(d_h)), out_dtype as above
 *   dev_status  optional DEVICE int32: receives LCKV_ETIMEOUT if a bounded
 *             device-side wait gave up (it is cleared to 0 first); NULL to ignore
 * Limits: batch <= LCKV_STATIC_MAX_BATCH and a GPU with at most
 * LCKV_STATIC_MAX_SMS multiprocessors, else LCKV_ESTATICLIMIT and nothing runs.
 * The scratch array is LCKV_STATIC_SCRATCH_BYTES of device memory that every
 * GPU loading this library holds until the process exits.
 *
 * Set-up: the first call on each device looks up the array's device address
 * and raises the kernel's shared-memory limit; make that first call outside
 * any stream capture (it is refused with EINVAL inside one); the set-up is
 * guarded, so first calls from several host threads are safe.  Later calls on that device only enqueue work.
 * Sharing: all calls on a device use the same scratch.  Calls are safe one
 * after another on one stream (the merge tickets are cleared at the start of
 * each call); calls that may overlap on the GPU - different streams, or a
 * cache-based call is unaffected but two static calls are - race on it and
 * give undefined results.  The lengths are read on the device, so a bad length
 * cannot be refused here: the visible count is clamped to [0, max_seq] (nothing
 * outside the tensors is read), but the result for such a sequence is not what
 * the caller meant; keep 0 <= lens[b] and lens[b] + mode <= max_seq.
 * This call performs no cudaMalloc/cudaFree and uses no allocating library.
 * Errors: EINVAL (null pointer; k, v, q or out not 16-byte aligned; lens, lse
 * or dev_status not 4-byte aligned; bad shape or mode; a first call on a device
 * made while `stream` is capturing), ESTATICLIMIT, ECUDA.  Argument errors are
 * found before any CUDA call is made.
 */
#define LCKV_STATIC_MAX_BATCH 4096
#define LCKV_STATIC_MAX_SMS 256
#define LCKV_STATIC_SCRATCH_BYTES (2304 * 1024)
int lckv_decode_attention_static(const void* k, const void* v, const int32_t* lens,
                                 const void* q, void* out, float* lse, int32_t* dev_status,
                                 int32_t batch, int32_t n_q_heads, int32_t n_kv_heads,
                                 int32_t head_dim, int64_t max_seq, int32_t mode,
                                 float softmax_scale, int32_t out_dtype, void* stream);

/*
 * Measurement helper (the paper has no counterpart): a read-only stream over `bytes` of device
 * memory at `src` (16-byte aligned), to learn the read bandwidth this GPU reaches when the bytes are
 * only read - the ceiling of the read-dominated attention kernels, which a read + write copy does
 * not show.  kind 0: independent 16-byte loads from every thread; kind 2: 32-byte loads
 * (src 32-byte aligned) marked evict-first; kind 1: 8 KB bulk copies into
 * per-warp shared-memory rings, the way the attention kernels stream K and V (bytes beyond the last
 * whole 8 KB are not read).  `repeats` >= 1 passes over the buffer are made in one launch: with a buffer
 * smaller than the L2 the passes after the first measure the L2's read bandwidth, the ceiling of a layer
 * that re-reads a cache the previous layer left there.  l2_keep in [0, 1] (kind 1 only) is the fraction of
 * lines the copies mark evict-last, as the attention kernels do for a cache that several layers read; the
 * rest is marked evict-first.  *dev_sum (device uint32, not cleared) receives a checksum so that the
 * reads cannot be optimised away: kinds 0 and 2 add the wrapped sum of all 32-bit words, kind 1 the first
 * word of every piece (each once per pass).  *dev_status (device int32) is set to LCKV_ETIMEOUT if a bounded wait of kind 1
 * runs out.  Time it with events on `stream`.  Errors: EINVAL, ECUDA.
 */
int lckv_read_stream_probe(const void* src, size_t bytes, int32_t kind, int32_t repeats, float l2_keep,
                           uint32_t* dev_sum, int32_t* dev_status, void* stream);

/* Short English name of a status code. */
const char* lckv_status_string(int status);

/* cudaError_t (as int) of the last failed CUDA call made by this library on this thread. */
int lckv_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* LCKV_H */
