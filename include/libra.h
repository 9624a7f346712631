/*
 * libra.h - C ABI of the B200 (sm_100a) paged GQA decode-attention library.
 *
 * The library implements the data-parallel core of one batched decode step of an agentic-RL
 * rollout: for every running sequence, one query token attends to all tokens of its paged
 * bf16 KV cache.  The paper this library accompanies ("Libra") characterises that step as
 * memory-bandwidth-bound and linear in sequence length (Section 1, Section 2.2) and removes
 * the stragglers caused by a few very long trajectories by bucketing requests by length and
 * giving longer buckets a higher parallel degree (Section 2.3, Section 4.3, Section 5).  The
 * planner below applies that idea inside one GPU: the "degree" of a sequence is the number of
 * thread blocks that share its KV range.
 *
 * Three steps make one call:
 *   P  libra_plan          host, integers only: bucket -> split count -> sorted work list
 *   D  split-KV decode     device: one pass over K and V, fp32 online softmax
 *   C  combine             device: log-sum-exp merge of the partial results of split sequences
 * D and C are launched by libra_decode_attn.
 *
 * Conventions
 *   - every function returns a libra_status_t (0 = OK) unless stated otherwise; nothing throws,
 *     aborts or traps; misuse that the host can see is rejected before any launch;
 *   - "device pointer" = memory of the handle's GPU, owned by the caller for the whole call and
 *     until the stream has finished with it; "host pointer" = ordinary host memory;
 *   - the library allocates host memory only (the handle and two small pinned staging buffers),
 *     except where a function says otherwise; all device memory, the workspace included, is the
 *     caller's;
 *   - streams are cudaStream_t passed as void*; all device work is asynchronous on that stream;
 *   - one handle serves one stream at a time (no internal locking).
 *
 * Data layout
 *   q, out        bf16 [batch, num_q_heads, head_dim], row-major, contiguous; q 4-byte, out 8-byte aligned
 *   k_pages,
 *   v_pages       bf16, two separate pools indexed by the same page ids; element (page, head,
 *                 token, c) lives at  page*kv_stride_page + head*kv_stride_head +
 *                 token*kv_stride_token + c  (strides in elements, head_dim contiguous).
 *                 "HND" = [num_pages, num_kv_heads, page_size, head_dim] (the default when all
 *                 three strides are 0), "NHD" = [num_pages, page_size, num_kv_heads, head_dim].
 *                 Pool base addresses must be 16-byte aligned and strides multiples of 8 elements.
 *   block_table   int32 [batch, block_table_ld]; entry i of row b = page id of tokens
 *                 [P i, P i + P) of sequence b (P = page_size); entries past the last page are ignored
 *   seq_lens      int32 [batch]; number of cached tokens INCLUDING the current one; the kernel
 *                 appends nothing; 0 is allowed (output row = 0)
 *   GQA map       query head h reads KV head h / (num_q_heads / num_kv_heads)
 *   Slots past seq_len in a sequence's last page, and pages no sequence owns, may hold anything
 *   (NaN included); they never influence a result.
 */
#ifndef LIBRA_H_
#define LIBRA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LIBRA_OK = 0,
  LIBRA_INVALID_ARGUMENT = 1,   /* null pointer, negative size, batch > max_batch ...            */
  LIBRA_UNSUPPORTED_SHAPE = 2,  /* head_dim not 64/128, page_size not 16/32/64, group size > 16  */
  LIBRA_WORKSPACE_TOO_SMALL = 3,
  LIBRA_NOT_PLANNED = 4,        /* libra_decode_attn before a successful libra_plan              */
  LIBRA_CUDA_ERROR = 5,         /* a CUDA call failed; see libra_last_cuda_error                 */
  LIBRA_DEVICE_FLAGGED = 6      /* a kernel recorded a problem; see libra_debug_error_word       */
} libra_status_t;

/* bits of the device error word */
#define LIBRA_ERR_WAIT_TIMEOUT 1u   /* a bounded wait on a copy barrier ran out                  */
#define LIBRA_ERR_BAD_PAGE_ID 2u    /* block-table entry outside [0, num_pages)                  */
#define LIBRA_ERR_SEQ_LEN_MISMATCH 4u /* device seq_lens differ from the lengths that were planned */
#define LIBRA_ERR_PLAN_OVERFLOW 8u  /* device-side planner: too many sequences or work items, or a length
                                       longer than a block-table row can describe; nothing was computed */

/* Planner constants (Section 4.3 of the paper: degrees are powers of two, work sorted by length,
 * min-max objective).  A zero field takes its default. */
typedef struct {
  int32_t n_sm;           /* SMs to plan for; 0 = the device's count (148 on B200)               */
  int32_t ctas_per_sm;    /* resident decode blocks per SM the plan assumes; default 1, and 2 where
                             a KV head serves more than 8 rows of q (query heads per KV head x
                             libra_set_max_query_tokens) or the pools are E4M3: those steps run
                             two blocks per SM                                                   */
  int32_t items_per_slot; /* target work units per resident block; default 1                    */
  int32_t chunk_align;    /* A: chunk lengths are multiples of this many tokens (itself a
                             multiple of 16); default 256                                       */
  int32_t min_chunk;      /* C_min: lower bound of the base chunk length; default 512           */
  int32_t max_splits;     /* S_max: cap of the split degree (power of two <= 64); default 64     */
  int32_t refine;         /* 0 or 1 (default): a plan of fewer than one and a half waves of
                             n_sm * ctas_per_sm blocks whose base chunk is 4096 tokens or longer is
                             made again for twice as many slots; -1 = never                      */
} libra_plan_params_t;

typedef struct {
  int32_t num_q_heads;
  int32_t num_kv_heads;        /* must divide num_q_heads; group size <= 16                      */
  int32_t head_dim;            /* 64 or 128                                                      */
  int32_t page_size;           /* 16, 32 or 64 tokens per page                                   */
  int64_t num_pages;           /* pages in each pool                                             */
  int32_t max_batch;           /* upper bound of `batch` in libra_plan; at most 262144 (2^18)    */
  int32_t block_table_ld;      /* row pitch of block_table in entries                            */
  int64_t kv_stride_page;      /* in elements; all three 0 = HND                                 */
  int64_t kv_stride_head;
  int64_t kv_stride_token;
  float sm_scale;              /* softmax scale; 0 = 1/sqrt(head_dim)                            */
  int32_t device;              /* CUDA device ordinal                                            */
  libra_plan_params_t plan;
} libra_config_t;

typedef struct libra_handle_s* libra_handle_t;

/* Read-only host view of the last plan of a handle; the arrays belong to the handle and stay
 * valid until the next libra_plan or libra_destroy. */
typedef struct {
  int32_t batch;
  int32_t chunk_target;        /* C, the base bucket length of this batch                        */
  int32_t num_items;
  int32_t num_combine;
  int32_t num_empty;
  const int32_t* bucket;       /* [batch] log2 of the split degree, -1 for an empty sequence     */
  const int32_t* num_splits;   /* [batch] non-empty chunks n_b                                   */
  const int32_t* chunk_len;    /* [batch]                                                        */
  const int32_t* item_offset;  /* [batch] exclusive prefix sum of n_b                            */
  const int32_t* items;        /* [num_items][4] = (b, j, kv_begin, kv_end), longest first       */
  const int32_t* combine;      /* [num_combine] sequences with n_b > 1, batch order              */
  const int32_t* empty;        /* [num_empty] sequences with length 0, batch order               */
} libra_plan_view_t;

/* Library version, major*10000 + minor*100 + patch. */
int libra_version(void);

/* Text for a status code; never NULL; static storage. */
const char* libra_status_string(int status);

/* Create a handle for one shape on cfg->device.  Queries the SM count, checks that the device is
 * compute capability 10.x and validates the shape.  Errors: INVALID_ARGUMENT (null, non-positive
 * sizes, num_q_heads not a multiple of num_kv_heads, bad strides), UNSUPPORTED_SHAPE, CUDA_ERROR
 * (no usable device).  On error *handle is set to NULL. */
int libra_create(libra_handle_t* handle, const libra_config_t* cfg);

/* Free the handle and its pinned staging buffers.  NULL is allowed.  The caller must have
 * synchronised the streams that used it. */
int libra_destroy(libra_handle_t handle);

/* Bytes of device workspace that libra_plan / libra_decode_attn need for any batch <= max_batch.
 * The workspace holds the device error word, arrival counters, the fp32 partial results of split
 * sequences and room for a plan too large for the kernel parameters.  It must be 256-byte aligned.
 * The handle remembers the address of the workspace it cleared last and does not clear it again on later
 * plans (the kernels leave the counters at zero).  If that memory was meanwhile used for anything else - freed and
 * handed out again by an allocator at the same address, say - call libra_workspace_invalidate before the next plan.
 * A handle is not thread-safe: one host thread at a time per handle; different handles are independent. */
int libra_workspace_size(libra_handle_t handle, size_t* bytes);

/* Forget which workspace was cleared last: the next libra_plan / libra_plan_device clears the control words and
 * arrival counters of its workspace again, on its stream.  The current plan is dropped.  Errors: INVALID_ARGUMENT. */
int libra_workspace_invalidate(libra_handle_t handle);

/* The planner constants the handle uses, defaults resolved (n_sm = the device's SM count). */
int libra_get_plan_params(libra_handle_t handle, libra_plan_params_t* out);

/* Several query tokens per sequence (default 1).  Lays the workspace out for up to `max_q_len` query tokens
 * per sequence in libra_decode_attn_multi: the partial buffers grow by that factor, so ask
 * libra_workspace_size again afterwards; the current plan is dropped.  A KV head's score tile has at most
 * 16 columns: max_q_len * (num_q_heads / num_kv_heads) <= 16, else UNSUPPORTED_SHAPE.  Past 8 columns the default of
 * ctas_per_sm becomes 2 (see libra_plan_params_t; libra_get_plan_params shows what is in force). */
int libra_set_max_query_tokens(libra_handle_t handle, int32_t max_q_len);

/* Storage type of the KV pools (default LIBRA_KV_BF16).  LIBRA_KV_E4M3: the pools hold 8-bit floating-point
 * codes (1 sign, 4 exponent, 3 mantissa bits, bias 7, no infinities, one NaN per sign), one byte per element,
 * with one scale per tensor: key = k_scale * value of the code, value = v_scale * value of the code; the
 * attention is the same definition on those keys and values, q and out stay bf16.  The strides given at
 * creation keep their meaning (elements, now bytes) and must be multiples of 16; k_scale and v_scale must be
 * positive and finite (ignored for BF16).
 * Halving the bytes per cached token halves what the step has to read.  With E4M3 pools the rows given to
 * libra_decode_attn_append (k_new, v_new: [batch, num_kv_heads, head_dim]) and the dense buffers of
 * libra_kv_gather / libra_kv_scatter hold codes too, one byte per element; libra_decode_attn_host returns
 * UNSUPPORTED_SHAPE.  The workspace does not depend on the type; the plan does where the default of ctas_per_sm does
 * (see libra_plan_params_t): there the call voids the plan (NOT_PLANNED until the next plan call). */
#define LIBRA_KV_BF16 0
#define LIBRA_KV_E4M3 1
int libra_set_kv_dtype(libra_handle_t handle, int32_t dtype, float k_scale, float v_scale);

/* Tuning knob: shape of the decode thread block: `warps` warps that each own `stages` shared-memory
 * stages of one K page plus one V page.  Only the compiled-in shapes are accepted (UNSUPPORTED_SHAPE
 * otherwise); the default is the tuned one (8 x 3; 4 x 2, three blocks per SM, when no unit of a host plan exceeds
 * 1024 tokens, and 2 x 2, seven per SM, when none exceeds 256; 6 x 2, two blocks per SM, when a KV head serves more than
 * 8 rows of q and the plan has two slots per SM (the default then), 12 x 2 on a one-slot plan; with an E4M3 cache,
 * whose tiles are half the size, 8 x 3 / 6 x 4 for one / two column tiles, two blocks per SM, on a two-slot plan (the
 * default), 16 x 3 / 8 x 6 on a one-slot plan, 4 x 2 / 2 x 4 for short units).  Results do not depend on the stage count; the warp
 * count changes the order of the per-unit merge and hence the last bits of the result. */
int libra_set_variant(libra_handle_t handle, int32_t warps, int32_t stages);

/* Programmatic dependent launch, on by default: the decode kernel is launched so that its blocks may
 * become resident while the kernel before it in the stream drains (and the separate combine kernel
 * likewise after the decode kernel); inside, they wait for that kernel to finish before they read any
 * input, so ordering and results are exactly those of ordinary launches - only the launch latency
 * and block start-up overlap the predecessor's tail.  on = 0 makes every launch an ordinary one. */
int libra_set_dependent_launch(libra_handle_t handle, int32_t on);

/* L2 warm-up at the start of a step, on by default (and only with dependent launches on).  The blocks of a step's
 * first wave become resident while the kernel before them in the stream drains, when DRAM is all but idle.  Before they
 * wait for that kernel they look up the page ids of their first tiles and ask for those tiles to be brought into L2
 * (a prefetch without destination); after the wait they read ids and tiles again, for real, so the results do not
 * depend on it: an id that the preceding kernel had not yet written only warms the wrong lines, and a line written
 * after it was warmed is updated in L2, where the copies read.  It needs no promise from the caller (unlike
 * libra_set_early_prefetch) but it does read block_table - as a hint - while the preceding kernel may still be writing
 * it, which a memory checker reports; on = 0 switches it off.  Worth 2 % on a 55 us step, nothing on long ones.
 * A plan that lies in the workspace (made by libra_plan_device, or too large for the kernel parameters) is warmed
 * from the second decode call on it onwards: the kernel or copy that wrote it is then known to have finished. */
int libra_set_cache_warmup(libra_handle_t handle, int32_t on);

/* Optional second output.  With a non-NULL lse_dev every later decode call (libra_decode_attn, _append, _multi,
 * _static) also writes, for every row of q, the natural logarithm of the sum of its exponentiated scores,
 * lse[b][row] = ln sum_t exp(s_t) with s_t = (q . k_t) * sm_scale, as float32 [batch, rows] (rows = q_len *
 * num_q_heads); -inf for an empty sequence or a query token that sees nothing.  Together with `out` this is what
 * merging the attention over several disjoint parts of one sequence needs (out = sum_i w_i out_i / sum_i w_i,
 * w_i = exp(lse_i - max lse)).  The buffer is the caller's and must stay valid while calls use it; NULL switches
 * the output off. */
int libra_set_lse_output(libra_handle_t handle, float* lse_dev);

/* Early prefetch, off by default: a PROMISE by the caller about the kernel that precedes each decode call in the
 * stream, namely that it writes none of: block_table, seq_lens (device), and the cached K/V rows of any token
 * other than each sequence's newest q_len + 1 tokens, counted by this call's seq_lens (a projection / rotary /
 * cache-write kernel for this step's tokens qualifies, and so does the previous step's
 * libra_decode_attn_append when the lengths grew by one; a kernel that moves or rewrites older pages does not).  With the promise, and dependent launch on, a decode block that
 * becomes resident while that kernel drains walks its block-table row and starts the copies of its first tiles
 * of old tokens before it waits for that kernel to finish; q, the newest rows, `out` and the workspace are
 * still touched only afterwards.  Results are bit-identical to the default.  Applies to plans that travel in
 * the kernel parameters (host plans of up to 768 entries); otherwise the setting has no effect. */
int libra_set_early_prefetch(libra_handle_t handle, int32_t on);

/* Where step C runs.  mode 1 (default): inside the decode kernel, by the block that publishes the last
 * partial result of a split sequence (one launch per step).  mode 0: as a separate combine kernel after
 * the decode kernel (two launches; the second is a programmatic dependent of the first).  The merge code
 * and its order of evaluation are the same, so both modes give bit-identical results. */
int libra_set_combine_mode(libra_handle_t handle, int32_t mode);

/* Step P as a pure host function (needs no GPU): the length-bucketed planner (Sections 2.3, 4.3
 * and 5 of the paper give the bucket properties it mirrors).  With W = n_sm * ctas_per_sm,
 * T = sum of lengths, cd = ceiling division, au(a,b) = cd(a,b)*b, p2 = next power of two:
 *   C       = max(min_chunk, au(cd(num_kv_heads * T, W * items_per_slot), chunk_align))
 *   s_b     = p2(cd(L_b, C)); if C < 4096 and s_b > 1 and 128 * L_b < 181 * (s_b / 2) * C: s_b = s_b / 2
 *             (short base chunks: the power of two nearer to L_b / C in ratio, 181 / 128 ~ sqrt 2; a work item
 *             costs ~4 us whatever its length, so fewer and longer items win there)
 *   s_b     = min(s_b, max_splits)                       bucket_b = log2 s_b
 *   chunk_b = au(cd(L_b, s_b), chunk_align)              n_b = cd(L_b, chunk_b)
 *   if refine and C >= 4096 and 2 * num_kv_heads * sum n_b < 3 * W   (fewer than one and a half waves of long blocks:
 *             the tail end of a rollout, a few long stragglers; so few blocks cannot pull the memory bandwidth):
 *             C = max(min_chunk, au(cd(num_kv_heads * T, 2 * W * items_per_slot), chunk_align)) and s_b, chunk_b, n_b
 *             are computed again with it
 *   items   = (b, j, j*chunk_b, min(L_b, (j+1)*chunk_b)) sorted by (length desc, b asc, j asc)
 * The number of items never exceeds max(2 * cd(W * items_per_slot, num_kv_heads) + batch,
 * 2 * cd(2 * W * items_per_slot, num_kv_heads) + min(batch, 3 * W / (2 * num_kv_heads))) (the second term only with
 * refine), which is what the workspace is sized for.  params->n_sm must be > 0 here.  All outputs are caller-allocated host arrays: the per-sequence
 * arrays hold `batch` entries, `items` holds items_capacity*4 entries.  Errors: INVALID_ARGUMENT
 * (null, negative length, bad params), WORKSPACE_TOO_SMALL (items_capacity too small; *num_items
 * then holds the number needed). */
int libra_plan_host(const libra_plan_params_t* params, int32_t num_kv_heads, const int32_t* seq_lens,
                    int32_t batch, int32_t* chunk_target, int32_t* bucket, int32_t* num_splits,
                    int32_t* chunk_len, int32_t* item_offset, int32_t* items, int32_t items_capacity,
                    int32_t* num_items, int32_t* combine, int32_t* num_combine, int32_t* empty,
                    int32_t* num_empty);

/* Step P for a handle: plan `batch` sequences from host lengths.  The plan is kept in the handle
 * and travels to the GPU inside the kernel parameters of every later libra_decode_attn, so in the
 * usual case nothing is copied here.  Only a plan of more than 768 work items (or more than 256 split
 * sequences) is uploaded into the workspace, with one asynchronous copy on `stream` from a pinned
 * staging buffer owned by the handle (two buffers alternate; one is reused only after its previous
 * upload finished).  The first plan into a given workspace also clears the workspace's control
 * words and arrival counters on `stream`.  seq_lens_host: host pointer, int32[batch].
 * Errors: INVALID_ARGUMENT, WORKSPACE_TOO_SMALL, CUDA_ERROR. */
int libra_plan(libra_handle_t handle, const int32_t* seq_lens_host, int32_t batch, void* workspace_dev,
               size_t workspace_bytes, void* stream);

/* Step P on the GPU: the same planning rule as libra_plan, evaluated by one thread block from the
 * DEVICE copy of the lengths (int32[batch]; negative values count as 0), enqueued on `stream`.  The
 * host never reads the lengths, so plan + libra_decode_attn can be enqueued back to back - or recorded
 * once and replayed - while the lengths change underneath (the paper re-plans as lengths drift:
 * Section 2.2, Section 4.3).  The plan is written into the workspace; later libra_decode_attn calls
 * launch grids sized for the worst case and the kernels read the real counts from the workspace.
 * Limits: batch <= 4096 (UNSUPPORTED_SHAPE otherwise); at most 4096 work items and no length beyond
 * block_table_ld * page_size, else the plan is empty and LIBRA_ERR_PLAN_OVERFLOW is set in the device error
 * word (checked on the device, since the host does not see the lengths).  The result equals
 * libra_plan's bit for bit (libra_plan_export reads it back).  The planning kernel is one more kernel on the stream's
 * critical path (about 6 us for 64 sequences, 8.5 us for 256, 12 us for 1024 and 21 us for 4096 work items); one plan
 * serves any number of decode calls on the same lengths - the attention layers of one generated token - so per call
 * the cost is a fraction of that.
 * Errors: INVALID_ARGUMENT, WORKSPACE_TOO_SMALL, UNSUPPORTED_SHAPE, CUDA_ERROR. */
int libra_plan_device(libra_handle_t handle, const int32_t* seq_lens_dev, int32_t batch, void* workspace_dev,
                      size_t workspace_bytes, void* stream);

/* A bound on the lengths of device-planned batches (0 = none, the default).  For a host plan the library sees the
 * longest work unit and picks the decode block's shape by it (small blocks, several per SM, when every unit is short:
 * up to 2.6 x faster on batches of short sequences); after libra_plan_device it cannot, and uses the large block.  A
 * caller who knows that no sequence of the coming batches is longer than max_seq_len tokens says so here, and the
 * same choice is made from that bound.  It is a hint: a longer sequence is still computed correctly, only on a block
 * shape that is slow for it.  Errors: INVALID_ARGUMENT (negative). */
int libra_set_length_hint(libra_handle_t handle, int32_t max_seq_len);

/* Host view of the last plan (see libra_plan_view_t); after libra_plan_device this copies the plan
 * back from the workspace and synchronises that call's stream.  Errors: NOT_PLANNED, CUDA_ERROR. */
int libra_plan_export(libra_handle_t handle, libra_plan_view_t* view);

/* Steps D and C: softmax(q K^T * sm_scale) V per query head over the pages of each sequence
 * (the rollout decode step of Section 1 / Section 2.2 of the paper; the attention itself is the
 * textbook definition).  All pointers are device pointers; the plan last uploaded by libra_plan
 * into `workspace` is used and `seq_lens` (device) must hold the planned lengths (a mismatch
 * sets LIBRA_ERR_SEQ_LEN_MISMATCH in the error word).  Launches the split-KV decode kernel (and, in
 * the two-launch combine mode, the combine kernel if any sequence is split) on `stream`;
 * returns without waiting.
 * Results are bit-reproducible run to run (fixed reduction order, no floating-point atomics).
 * The workspace also holds per-sequence arrival counters that the kernels leave at zero; a call that
 * is aborted (device reset, failed launch) may leave them dirty: plan into a different workspace, or
 * clear the workspace and create a new handle, after such a failure.
 * Errors: INVALID_ARGUMENT (null or misaligned pointer), NOT_PLANNED, CUDA_ERROR. */
int libra_decode_attn(libra_handle_t handle, const void* q, const void* k_pages, const void* v_pages,
                      const int32_t* block_table, const int32_t* seq_lens, void* out, void* stream);

/* The step for several query tokens per sequence: the last q_len tokens of every sequence are new in this
 * step (a tool return absorbed at once - Section 2.2: tool returns extend a trajectory mid-rollout - or a few
 * drafted tokens); their K and V rows are already in the cache and seq_lens counts them.  q and out are bf16
 * [batch, q_len, num_q_heads, head_dim].  Query token i attends causally to cached tokens
 * 0 .. L_b - q_len + i:  out[b, i, h] = softmax over those tokens of (q[b, i, h] . K_b[t]) * sm_scale, times V.
 * A query token with nothing to attend to (L_b - q_len + i < 0) gets a zero row.  The plan is the one
 * libra_plan made from seq_lens (it depends on the lengths only); all query tokens of a KV head's group share
 * one pass over K and V.  1 <= q_len <= the value given to libra_set_max_query_tokens; q_len = 1 is
 * libra_decode_attn.  Errors: as libra_decode_attn, INVALID_ARGUMENT for q_len out of range. */
int libra_decode_attn_multi(libra_handle_t handle, const void* q, int32_t q_len, const void* k_pages,
                            const void* v_pages, const int32_t* block_table, const int32_t* seq_lens, void* out,
                            void* stream);

/* The same step with the KV append fused in (the step before attention inside one decode step of
 * the rollout, Section 1 / Section 2.2 of the paper: the cache grows by one token per step).  k_new and
 * v_new are device pointers to the current token's key and value rows, bf16 [batch, num_kv_heads,
 * head_dim], 16-byte aligned; seq_lens still COUNTS that token.  For every sequence with L_b >= 1 the
 * rows are written into slot (L_b - 1) % P of page block_table[b][(L_b - 1) / P] of both pools (the
 * pools are therefore not const) and the attention result is exactly what libra_decode_attn returns on
 * the updated pools.  The block that owns the sequence's last page does both: it patches the staged copy
 * of that page in shared memory and stores the rows to the pools, so no ordering between the store and
 * the page reads is needed.  Errors: as libra_decode_attn. */
int libra_decode_attn_append(libra_handle_t handle, const void* q, const void* k_new, const void* v_new,
                             void* k_pages, void* v_pages, const int32_t* block_table, const int32_t* seq_lens,
                             void* out, void* stream);

/* Several query tokens with the append fused in: k_new and v_new hold the rows of the newest q_len tokens of every
 * sequence, [batch, q_len, num_kv_heads, head_dim] in the cache's element type (token i of the block is token
 * L_b - q_len + i of the sequence); they are written into their slots (which may lie in two pages) and the result
 * is libra_decode_attn_multi's on the updated pools.  Sequences shorter than q_len take only their last L_b rows
 * (the rows of block positions q_len - L_b .. q_len - 1).  Errors: as libra_decode_attn_multi. */
int libra_decode_attn_multi_append(libra_handle_t handle, const void* q, int32_t q_len, const void* k_new,
                                   const void* v_new, void* k_pages, void* v_pages, const int32_t* block_table,
                                   const int32_t* seq_lens, void* out, void* stream);

/* The same step for callers whose data lives in host memory: copies q, both pools, the block
 * table and the lengths to `staging_dev` (a caller-owned device region of at least
 * libra_host_staging_size bytes, 256-byte aligned), plans, runs D and C and copies `out` back
 * to out_host, all on `stream`; returns after synchronising the stream.  Host pointers should be
 * pinned for full copy speed.  `workspace_dev` as for libra_plan.  Pools must be in the handle's
 * layout.  Errors: as libra_plan and libra_decode_attn, plus DEVICE_FLAGGED if the error word is
 * non-zero afterwards. */
int libra_decode_attn_host(libra_handle_t handle, const void* q_host, const void* k_pages_host,
                           const void* v_pages_host, const int32_t* block_table_host,
                           const int32_t* seq_lens_host, int32_t batch, void* out_host, void* staging_dev,
                           size_t staging_bytes, void* workspace_dev, size_t workspace_bytes, void* stream);

/* Bytes of device staging libra_decode_attn_host needs for `batch` sequences. */
int libra_host_staging_size(libra_handle_t handle, int32_t batch, size_t* bytes);

/* The step as a serving loop sees it: the cache stays on the device (k_pages, v_pages: device pointers, bf16 or
 * E4M3 as set on the handle) and only what changes every step crosses the bus: q, the block table and the lengths
 * come from host memory, `out` goes back to it.  Copies them to `staging_dev` (at least libra_host_io_staging_size
 * bytes, 256-byte aligned), plans, runs D and C, copies the result to out_host, all on `stream`, and returns after
 * synchronising it.  Errors: as libra_decode_attn_host. */
int libra_decode_attn_host_io(libra_handle_t handle, const void* q_host, const void* k_pages, const void* v_pages,
                              const int32_t* block_table_host, const int32_t* seq_lens_host, int32_t batch,
                              void* out_host, void* staging_dev, size_t staging_bytes, void* workspace_dev,
                              size_t workspace_bytes, void* stream);
int libra_host_io_staging_size(libra_handle_t handle, int32_t batch, size_t* bytes);

/* Size of the scratch region built into the library for libra_decode_attn_static: 8 MiB of device
 * memory that every GPU holds from the moment it loads the library until the process exits. */
#define LIBRA_STATIC_SCRATCH_BYTES (8u << 20)

/* One whole step (P, D, C) without a caller-provided workspace and without any allocation.
 * (The paper has no counterpart to this entry point; it exists for integration reasons only.)
 *
 * Who needs it: code that runs where device memory cannot be obtained any more -- an inference
 * server that hands all free HBM to its KV-cache pool at start-up and runs with its allocator
 * closed, a plug-in called from inside someone else's step loop where a cudaMalloc would
 * synchronise the whole device and stall every stream, or a component that is simply not allowed to
 * own device memory.  Such a caller still passes its inputs and its output buffer (device pointers,
 * exactly as for libra_decode_attn, plus the host lengths that libra_plan takes); the workspace is
 * a fixed LIBRA_STATIC_SCRATCH_BYTES region inside the library image instead.
 *
 * The call plans `batch` sequences, clears the part of the region that must start at zero (control
 * words, arrival counters) on `stream`, and launches the same kernels as libra_decode_attn.  It calls
 * no cudaMalloc / cudaFree / cudaHostAlloc and no other allocating CUDA routine.
 *
 * Limits and rules:
 *  - the handle's shape must need no more than LIBRA_STATIC_SCRATCH_BYTES of workspace
 *    (libra_workspace_size); otherwise WORKSPACE_TOO_SMALL is returned and nothing is launched;
 *  - the first call on a device looks up the region's device address (once per device, kept for the
 *    life of the process); make that first call outside of any stream capture;
 *  - all handles and all calls on one device share the one region, which keeps the previous call's
 *    contents: two calls whose kernels can overlap on the GPU (different streams, no ordering)
 *    race on it and corrupt each other's results; issue them on one stream or order them with events;
 *  - a device error word left by the previous call is cleared by the next call: read it
 *    (libra_debug_error_word) in between if it matters.
 * Errors: as libra_plan and libra_decode_attn. */
int libra_decode_attn_static(libra_handle_t handle, const int32_t* seq_lens_host, int32_t batch, const void* q,
                             const void* k_pages, const void* v_pages, const int32_t* block_table,
                             const int32_t* seq_lens, void* out, void* stream);

/* Last CUDA error code (cudaError_t as int) seen by this handle, 0 if none. */
int libra_last_cuda_error(libra_handle_t handle);

/* Copy the device error word of the last planned workspace to *word (synchronises `stream` of the
 * last call first).  0 = no kernel recorded a problem.  The word accumulates over launches; reading
 * a non-zero word clears it.  Errors: NOT_PLANNED, CUDA_ERROR. */
int libra_debug_error_word(libra_handle_t handle, uint32_t* word);

/* KV migration, data movement (Section 5.3 of the paper: a paused request's KV cache is offloaded,
 * resharded along the attention-head dimension to the target bucket's tensor-parallel degree - a source
 * partition split into TP_tgt/TP_src shards, or TP_src/TP_tgt partitions concatenated - and reloaded).
 * The reshard is folded into the copies: both calls take a head range.
 *
 * libra_kv_gather copies, for each of `batch` sequences, tokens [0, seq_lens[b]) of KV heads
 * [head_begin, head_begin + head_count) from the handle's paged pools into dense buffers:
 *     k_dense[((token_offsets[b] + t) * head_count + (h - head_begin)) * head_dim + c]
 * libra_kv_scatter is the inverse: it writes the dense rows into the pages that `block_table` names, at
 * heads [head_begin, head_begin + head_count) of the handle's pools (slots past seq_lens[b] are left
 * untouched).  Splitting heads = several gathers with disjoint head ranges; concatenating = several
 * scatters into one pool at different head offsets.
 *
 * block_table, seq_lens (int32) and token_offsets (int64[batch], in tokens) are device pointers;
 * max_seq_len is an upper bound of the lengths (it sizes the grid; <= block_table_ld * page_size); the dense
 * buffers are 16-byte-aligned device memory or pinned host memory mapped into the device's address
 * space; error_word_dev points to a 32-bit device word that receives LIBRA_ERR_BAD_PAGE_ID if a page
 * id is outside the pool (that page is skipped).  The handle supplies the pool geometry only; no plan
 * and no workspace are needed.  Asynchronous on `stream`.  Errors: INVALID_ARGUMENT, CUDA_ERROR. */
int libra_kv_gather(libra_handle_t handle, const void* k_pages, const void* v_pages, const int32_t* block_table,
                    const int32_t* seq_lens, const int64_t* token_offsets, int32_t batch, int32_t max_seq_len,
                    int32_t head_begin, int32_t head_count, void* k_dense, void* v_dense, void* error_word_dev,
                    void* stream);
int libra_kv_scatter(libra_handle_t handle, const void* k_dense, const void* v_dense, const int32_t* block_table,
                     const int32_t* seq_lens, const int64_t* token_offsets, int32_t batch, int32_t max_seq_len,
                     int32_t head_begin, int32_t head_count, void* k_pages, void* v_pages, void* error_word_dev,
                     void* stream);

/* ---- the paper's rollout-side schedulers, host code only (no GPU) ------------------------------------ */

/* RolloutDP of the Global Resource Planner (Section 4.3, Algorithm 1): split `n_gpus` GPUs into inference
 * instances with tensor-parallel degrees from `tp_set` and give each a contiguous segment of the requests
 * sorted by length, minimising the largest instance time:
 *     dp[g][i] = min over tp in tp_set, tp <= g, 0 <= x <= i of max(dp[g - tp][i - x], Cost(tp, i-x+1, i))
 * with dp[0][0] = 0 and every GPU used ("exactly g GPUs").  Cost of an instance of degree tp_set[t] on a
 * segment: cost_coef[4t+0] * sum(L) + cost_coef[4t+1] * sum(L^2) + cost_coef[4t+2] * count +
 * cost_coef[4t+3], and 0 for an empty segment (the polynomial form of the paper's cost evaluator,
 * Section 4.6, with caller-supplied coefficients).  `lengths` may be in any order (sorted inside).
 * Outputs: *makespan (+inf if no partition uses exactly n_gpus GPUs) and the optimal partition recovered
 * by backtracking, instances in sorted-request order: degree, index of the first request in the sorted
 * list, number of requests.  Errors: INVALID_ARGUMENT, WORKSPACE_TOO_SMALL (inst_capacity too small;
 * *n_instances holds the number needed).  Ties go to the earlier degree of tp_set, then to the smaller x.
 * When no cost coefficient is negative the minimum over x is found by bisection (the first term of the max cannot
 * grow with x and the second cannot shrink, so the minimum sits where they cross); otherwise the states are relaxed
 * one by one.  Either way the result is the recurrence's, bit for bit. */
int libra_rollout_dp(int32_t n_gpus, const int32_t* lengths, int32_t n_requests, const int32_t* tp_set, int32_t n_tp,
                     const double* cost_coef, double* makespan, int32_t* inst_tp, int32_t* inst_first,
                     int32_t* inst_count, int32_t inst_capacity, int32_t* n_instances);

/* Causality-aware prefix tree (Section 5): a node is (prompt id, sequence of tool-return states); every
 * node keeps a histogram of the remaining trajectory length seen from that point, with bins aligned to
 * the buckets' length thresholds: bin k holds lengths <= bin_upper[k] (increasing), the last bin
 * everything above; n_thresholds + 1 bins in all. */
typedef struct libra_trie_s* libra_trie_t;
int libra_trie_create(libra_trie_t* trie, const int32_t* bin_upper, int32_t n_thresholds);
int libra_trie_destroy(libra_trie_t trie);

/* Phase 3 / profile phase: insert one finished trajectory.  states[k] is the label of the k-th tool return
 * (tool type x payload size class x success/failure, encoded by the caller); residual_lengths[0] is the
 * trajectory's remaining length at the start and residual_lengths[k+1] the remaining length after the
 * k-th tool return (n_states + 1 values).  Child nodes are created as needed. */
int libra_trie_insert(libra_trie_t trie, int64_t prompt_id, const int32_t* states, int32_t n_states,
                      const int32_t* residual_lengths);

/* Phase 2 look-up: walk down from the prompt's root along `states`; at an unseen state stay at the parent
 * (back-off).  hist[n_thresholds + 1] receives the node's empirical distribution (all zero for an unknown
 * prompt), *depth_reached how many states were matched (-1: unknown prompt), *samples the node's count.
 * depth_reached and samples may be NULL. */
int libra_trie_lookup(libra_trie_t trie, int64_t prompt_id, const int32_t* states, int32_t n_states, double* hist,
                      int32_t* depth_reached, int64_t* samples);

/* Phase 2 routing: B* = argmin_B ( sum_k p_k * decode_cost[B][k] + migration_cost[B] ), p from the
 * look-up above, decode_cost [n_buckets][n_thresholds + 1] row-major, migration_cost[B] the cost of
 * moving from the current bucket to B (0 for the current one).  Ties go to the lower bucket index.
 * best_cost may be NULL. */
int libra_trie_route(libra_trie_t trie, int64_t prompt_id, const int32_t* states, int32_t n_states,
                     int32_t n_buckets, const double* decode_cost, const double* migration_cost,
                     int32_t* best_bucket, double* best_cost);

/* ---- Data plane of the inter-replica ring all-reduce (Section 6, "Decoupled communication domains"; appendix
 * "Decoupled Communication Domain") ----------------------------------------------------------------------------
 * In the paper the CPU owns membership, transport and flow control of the gradient exchange between replicas; the
 * GPU runs only the copy / reduce steps of a ring ReduceScatter + AllGather, polls a host-pinned arrival flag with a
 * software timeout instead of blocking, and uses 2 SMs.  libra_ring_step enqueues ONE such step on `stream` of
 * `device` (a one-thread kernel that waits and writes the verdict, then the copy / reduce kernel, which acts on it):
 *   wait until *ready_flag >= expected (ready_flag: host-pinned mapped memory or device memory, 4-byte aligned; the
 *   producer writes the chunk first, then the flag), for at most timeout_us microseconds (1 .. 10,000,000);
 *   then  own != NULL : dst[i] = own[i] + received[i]   (a ReduceScatter step; LIBRA_RING_F32: float32 addition;
 *                        LIBRA_RING_BF16: bfloat16 values added in float32, rounded to nearest even)
 *         own == NULL : dst[i] = received[i]            (an AllGather step)
 * over `bytes` bytes (a multiple of 16; all buffers 16-byte aligned; dst may equal own).  num_blocks thread blocks of
 * 512 threads do the work (0 = the default of 2; at most 64).  *status_dev (device memory) receives 0 when the step
 * ran and 1 when the wait ran out, in which case nothing else was written and the context stays usable.  Everything
 * around the step - who sends what to whom, chunking, membership - is the caller's.
 * Errors: INVALID_ARGUMENT, CUDA_ERROR. */
#define LIBRA_RING_F32 0
#define LIBRA_RING_BF16 1
int libra_ring_step(int32_t device, void* dst, const void* own, const void* received, size_t bytes, int32_t dtype,
                    const uint32_t* ready_flag, uint32_t expected, uint32_t timeout_us, uint32_t* status_dev,
                    int32_t num_blocks, void* stream);

/* ---- The ring's host side: membership descriptor and schedule (same passages of the paper) ---------------------
 * libra_ring_t is the metadata the CPU control plane owns: the live replicas in ring order (members[i] sends to
 * members[(i + 1) % n_members]).  A replica that died or leaves is taken out with libra_ring_remove - the order of
 * the others stays, its neighbours become each other's neighbours - and one that joins is put in at any position
 * with libra_ring_insert; both are plain edits of this struct (no GPU state, no allocation) and bump `epoch`, so a
 * data plane can tell that its peer list is stale.  Ids are the caller's (any distinct int32 values).
 * Errors: INVALID_ARGUMENT (null, duplicate or unknown id, position out of range, more than 64 members). */
#define LIBRA_RING_MAX_MEMBERS 64
typedef struct {
  int32_t n_members;
  int32_t members[LIBRA_RING_MAX_MEMBERS];   /* unused entries are -1 */
  uint32_t epoch;                            /* number of edits since libra_ring_init */
} libra_ring_t;
int libra_ring_init(libra_ring_t* ring, const int32_t* ids, int32_t n);
int libra_ring_remove(libra_ring_t* ring, int32_t id);
int libra_ring_insert(libra_ring_t* ring, int32_t id, int32_t position);
int libra_ring_neighbors(const libra_ring_t* ring, int32_t id, int32_t* predecessor, int32_t* successor);

/* What member `id` does in one all-reduce of a vector of `bytes` bytes (a multiple of 16) over the ring as it stands:
 * the ReduceScatter steps 0 .. n-2 followed by the AllGather steps 0 .. n-2, every step cut into pipeline pieces of
 * at most piece_bytes (a multiple of 16; the paper pipelines 16 MB pieces).  The vector is cut into n segments of
 * whole 16-byte units, equal parts with the first (bytes / 16) % n one unit longer; the member at ring position p
 *   ReduceScatter step s : sends segment (p - s) mod n to its successor, adds what its predecessor sends into its
 *                          own segment (p - 1 - s) mod n       (so segment c is summed starting at position c)
 *   AllGather step s     : sends segment (p + 1 - s) mod n, overwrites its segment (p - s) mod n with what arrives.
 * ops[] receives, in the order they are to be issued, one record per piece: kind, phase (0 ReduceScatter, 1
 * AllGather), step, segment, piece index, the peer's id and the byte range [offset, offset + bytes) of the vector.
 * A receive record is one libra_ring_step (dst = own = vector + offset for RECV_REDUCE, own = NULL for RECV_COPY).
 * *n_ops = records needed; WORKSPACE_TOO_SMALL if capacity is less (the first `capacity` are written).  A ring of
 * one member has no steps.  Errors: INVALID_ARGUMENT. */
#define LIBRA_RING_OP_SEND 0
#define LIBRA_RING_OP_RECV_REDUCE 1
#define LIBRA_RING_OP_RECV_COPY 2
typedef struct {
  int32_t kind, phase, step, segment, piece, peer;
  int64_t offset, bytes;
} libra_ring_op_t;
int libra_ring_schedule(const libra_ring_t* ring, int32_t id, int64_t bytes, int64_t piece_bytes, libra_ring_op_t* ops,
                        int32_t capacity, int32_t* n_ops);

/* The whole ReduceScatter + AllGather over n_members vectors that live on ONE device (bufs[i] = the vector of the
 * member at ring position i, `bytes` each, 16-byte aligned), every receive record of every member's schedule enqueued
 * on `stream` as one libra_ring_step, step by step: within a step no member reads a range that another member's
 * record of the same step writes, so the launches of a step may run in any order.  This is the data plane of several
 * replicas hosted on one GPU, and the way the schedule is exercised where there is one GPU; between real GPUs the
 * same records are issued by each rank for itself, with the transport delivering `received` and setting the flag.
 * ready_flag / expected / timeout_us / status_dev / num_blocks as for libra_ring_step (the same flag guards every
 * step here; *status_dev holds the verdict of the last step).  Results are bit-identical to the ring's definition:
 * segment c is summed in the order position c, c + 1, ..., in the element type.
 * Errors: INVALID_ARGUMENT (also: n_members < 1 or > 64), CUDA_ERROR. */
int libra_ring_all_reduce_local(int32_t device, void* const* bufs, int32_t n_members, size_t bytes, int32_t dtype,
                                size_t piece_bytes, const uint32_t* ready_flag, uint32_t expected, uint32_t timeout_us,
                                uint32_t* status_dev, int32_t num_blocks, void* stream);

/* Merge of attention results over disjoint parts of the same sequences: the one exchange step of cutting a
 * sequence's TOKENS across GPUs (the paper's tensor parallelism cuts the cache by attention head, Section 5.3, and
 * needs none; this is the remaining way to shard the step).  Each holder of a part runs the decode call with
 * libra_set_lse_output; once the (out, lse) pairs are gathered,
 *     M = max_i lse_i,  w_i = exp(lse_i - M),  out = sum_i w_i out_i / sum_i w_i,  lse = M + ln sum_i w_i
 * gives the attention over the whole sequence (the rule of step C).  parts_out: bf16 [n_parts][rows][head_dim],
 * parts_lse: float32 [n_parts][rows] (-inf = that part holds no token for the row; its out row is ignored), out:
 * bf16 [rows][head_dim], lse_out: float32 [rows] or NULL; device pointers on `device`, 16-byte aligned, out not
 * overlapping the inputs; rows = batch * q_len * num_q_heads in any order common to all parts; head_dim 64 or 128;
 * 1 <= n_parts <= 64.  A row whose parts are all empty gets zeros and lse = -inf.  Parts are added in index order
 * in float32: bit-reproducible.  Asynchronous on `stream`.
 * Errors: INVALID_ARGUMENT, UNSUPPORTED_SHAPE (head_dim), CUDA_ERROR. */
int libra_merge_parts(int32_t device, const void* parts_out, const float* parts_lse, int32_t n_parts, int64_t rows,
                      int32_t head_dim, void* out, float* lse_out, void* stream);

/* Self-test of the kernels' bounded waits: enqueues a one-warp kernel that waits, with a limit of a few
 * milliseconds, on a copy barrier that nothing completes.  It must return (no hang, no trap) and leave
 * LIBRA_ERR_WAIT_TIMEOUT in the device error word of the last planned workspace, which is how a real
 * timeout inside the decode kernel would surface.  Errors: NOT_PLANNED, CUDA_ERROR. */
int libra_debug_wait_selftest(libra_handle_t handle, void* stream);

/* Two read ceilings to set the decode kernel's rate against (the step is bound by one pass over K and V,
 * Section 2.1); both only read, neither computes attention.
 * libra_debug_stream_read: one kernel that streams `bytes` (>= 16; the tail past a multiple of 16 is not
 *   read) of the contiguous device buffer `buf_dev` (16-byte aligned) with plain vector loads.
 * libra_debug_gather_read: the decode kernel's measurement build - same arguments, plan, grid, block-table
 *   walk and tiled page copies as libra_decode_attn with the default block shape, but a staged page is only
 *   touched, not computed on.  `out` and the partial buffers receive meaningless values; the device error
 *   word is updated as usual.
 * Both are asynchronous on `stream` and need a plan (the stream read only for its workspace).
 * Errors: INVALID_ARGUMENT, NOT_PLANNED, CUDA_ERROR. */
int libra_debug_stream_read(libra_handle_t handle, const void* buf_dev, size_t bytes, void* stream);
int libra_debug_gather_read(libra_handle_t handle, const void* q, const void* k_pages, const void* v_pages,
                            const int32_t* block_table, const int32_t* seq_lens, void* out, void* stream);

/* Per-kernel timing for benchmarks.  After libra_profile_begin, every libra_decode_attn records
 * CUDA events around the decode kernel and the combine kernel on the call's stream (at most
 * 4096 calls are kept).  libra_profile_end synchronises those events, returns the summed device
 * times in milliseconds and the number of calls they cover, and switches recording off.  Any of
 * the output pointers may be NULL. */
int libra_profile_begin(libra_handle_t handle);
int libra_profile_end(libra_handle_t handle, double* decode_ms, double* combine_ms, int32_t* calls);

/* Number of kernels launched through this handle since it was created. */
int libra_launch_count(libra_handle_t handle, int64_t* launches);

#ifdef __cplusplus
}
#endif
#endif /* LIBRA_H_ */
