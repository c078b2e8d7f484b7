/*
 * concur_attn -- paged-KV grouped-query decode attention for NVIDIA B200 (sm_100a).
 *
 * One call computes one decode step of one layer:  for every sequence b of the batch
 * and every query head h (KV head g = h / (Hq/Hkv), Hq/Hkv = 1 .. 8), over the n = seq_lens[b] tokens
 * cached for that sequence,
 *
 *     s_j   = scale * <q[b][h], K[token j of b][g]>
 *     out   = sum_j softmax(s)_j * V[token j of b][g]          (bf16, round-to-nearest-even)
 *     lse   = ln sum_j exp(s_j)                                  (fp32, natural log)
 *     n = 0:  out = 0, lse = -inf.
 *
 * This is the attention step of the batched autoregressive decoding of long reasoning
 * traces on which the ConCuR pipeline (arXiv 2510.07356) spends its generation time:
 * five samples for each of 18,162 tasks by a 32B GQA model (Sec. 3.3), ten per task in
 * evaluation (Sec. 4.2), traces of 4,000-8,500 tokens and more (Tables 3 and 4) under a
 * 32,768-token limit (Sec. 4.1).  The paper states no formula for it; the definition
 * above is the standard one.
 *
 * Method: a plan kernel cuts the batch's KV tiles into ranges of near-equal size
 * (split-KV), a partial kernel streams each K/V tile from HBM once for all query heads
 * of its GQA group with an fp32 online softmax, and a combine kernel merges the partial
 * results of sequences that were split, by their log-sum-exp.
 *
 * Memory layout (all device memory unless a parameter says otherwise; caller-owned):
 *     q            bf16  [batch][Hq][D]
 *     k_pages      bf16  [num_pages][Hkv][P][D]        one (page, head) tile is contiguous; or, with
 *                        kv_layout = CONCUR_KV_TOKEN_MAJOR, [num_pages][P][Hkv][D]
 *     v_pages      bf16  same shape; K and V of a token share page id and slot
 *     block_table  int32 [batch][block_table_stride]   logical page i of b -> physical page
 *     seq_lens     int32 [batch]
 *     out          bf16  [batch][Hq][D]
 *     lse          fp32  [batch][Hq]
 * Token j of sequence b is slot j % P of page block_table[b][j / P].  Table entries at
 * or beyond ceil(n/P), and slots at or beyond n in the last page, are never read into a
 * result (they may hold anything, NaN included).
 *
 * Conventions: every function returns CONCUR_OK (0) or a negative concur_status_t; none
 * throws, aborts or prints.  No pointer is retained after a call returns (concur_attn_plan
 * remembers the ADDRESS of seq_lens, to recognise the matching planned calls; it is never
 * dereferenced on the host).  The library has no CPU fallback: without a CUDA device every call
 * fails with CONCUR_ERR_CUDA.
 *
 * Host threads: a handle is not locked.  Calls on ONE handle (options, status and destroy included)
 * must not run at the same time in two host threads; order them yourself.  Calls on DIFFERENT
 * handles may run concurrently from different threads, and so may concur_attn_workspace_bytes,
 * concur_attn_create and concur_attn_strerror: the library's only process-wide state is the
 * one-time per-device set-up of its kernels, which is safe to race.  concur_decode_attn_static may be
 * called from several threads as far as the host is concerned, but its calls share one device
 * array per GPU and must not overlap ON THE GPU (see there).
 */
#ifndef CONCUR_ATTN_H_
#define CONCUR_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CONCUR_OK = 0,
    CONCUR_ERR_INVALID_ARG = -1,   /* null / misaligned pointer, negative size, unknown option   */
    CONCUR_ERR_UNSUPPORTED = -2,   /* geometry outside what the kernels are built for             */
    CONCUR_ERR_TOO_LARGE = -3,     /* batch, table stride or workspace beyond the handle's limits */
    CONCUR_ERR_CUDA = -4,          /* a CUDA runtime or driver call failed (no device, launch)    */
    CONCUR_ERR_OOM = -5            /* device allocation failed                                     */
} concur_status_t;

/* Sticky device-side condition bits reported by concur_attn_status. */
#define CONCUR_FLAG_BAD_PAGE_ID 1u  /* a used block-table entry was outside [0, num_pages): clamped    */
#define CONCUR_FLAG_BAD_SEQ_LEN 2u  /* a seq_lens entry was outside [0, stride*P]: clamped             */
#define CONCUR_FLAG_WAIT_LIMIT  4u  /* an in-kernel wait gave up; results of that call are invalid, and so
                                       are those of later calls on the handle until concur_attn_status
                                       has reported the flag (it then re-initialises the handle's counters) */
#define CONCUR_FLAG_BAD_GROUP   8u  /* cascade step: group_start was not 0 <= g[0] <= g[1] <= ... <= batch;
                                       the call then shared nothing and computed the plain step          */

#define CONCUR_FLAG_BOUNDS     16u  /* only from the checked build of the library (compiled with -DCONCUR_BOUNDS,
                                       `python -m paper_2510_07356_b200.build --bounds`): an index the
                                       kernels computed fell outside its buffer; the access was skipped    */

/* Option keys for concur_attn_set_option (tuning and tests; defaults are chosen per call). */
#define CONCUR_OPT_KERNEL      1    /* 0 = tensor-core partial kernel (default), 1 = scalar-FMA kernel */
#define CONCUR_OPT_NUM_RANGES  2    /* force the number of split-KV ranges; 0 = heuristic              */
#define CONCUR_OPT_GRID_CTAS   3    /* force the partial kernel's grid size; 0 = one wave of the GPU    */
#define CONCUR_OPT_RANGES_PER_CTA 4 /* heuristic's target ranges per CTA; 0 = built-in default: 1, or 2 for a
                                       skewed batch (longest sequence >= 4 x the mean) whose ranges then
                                       still have 64 tiles or more                                       */
#define CONCUR_OPT_MIN_RANGE_TILES 5/* heuristic's smallest range, in 64-token tiles; 0 = default (2)   */
#define CONCUR_OPT_EVENT_BEFORE_PARTIAL 6 /* a cudaEvent_t (as an integer) recorded on the call's stream
                                             just before the partial kernel; 0 = none.  For timing
                                             that kernel alone; the event stays the caller's.  In the
                                             cascade step the two events bracket the prefix-pass kernel. */
#define CONCUR_OPT_EVENT_AFTER_PARTIAL  7 /* likewise, just after the partial kernel                    */
#define CONCUR_OPT_FUSE_COMBINE 8   /* tensor-core kernel: 1 (default) = the CTA that finishes a unit's last
                                       partial merges the unit in-kernel; 0 = separate combine kernel   */
#define CONCUR_OPT_CLAIM_AHEAD  9   /* tiles before a range's end at which a CTA claims its next range
                                       (default: at the range's first tile; 0 = when the range is done) */

#define CONCUR_OPT_PREFIX_KERNEL 10 /* shared-prefix pass of the cascade step: 0 (default) = tcgen05 kernel with
                                       TMEM accumulators, 1 = warp-level mma.sync kernel                 */

#define CONCUR_OPT_SMALL_PAGE_COPY 11 /* tensor-core partial kernel with 16- or 32-token pages: 1 (default) = the
                                        producer warp copies tiles 16 bytes per lane, 0 = one TMA box per
                                        (page, head) chunk                                               */

#define CONCUR_OPT_WAIT_LIMIT_NS 12 /* tensor-core partial kernel: nanoseconds after which a warp's wait for
                                       another role of its CTA (a tile to land, a ring stage to be freed, a
                                       partial to merge) gives up.  The kernel then records
                                       CONCUR_FLAG_WAIT_LIMIT, every warp of that CTA returns once the copies it
                                       has in flight have landed, and the call's results are invalid; nothing
                                       faults and the handle stays usable.  0 = default (2 s; 60 s at most).
                                       No correct run comes near the default; the option exists so that the
                                       give-up path can be exercised                                       */

#define CONCUR_OPT_OVERLAP_CALLS 13 /* 1 = a decode call that is a single kernel launch (see concur_decode_attn) may
                                       start while the kernel ahead of it on the stream drains, if that kernel
                                       is such a call too: its CTAs take over the SMs the earlier call's CTAs
                                       leave and fill their rings, and write nothing before the earlier call
                                       has finished.  The caller promises that q, the pools, block_table and
                                       seq_lens of a call are not written by the call right ahead of it (true
                                       of the layers of a model, whose calls differ in q, pools and out).
                                       0 (default) = calls run strictly one after the other              */
#define CONCUR_OPT_PREFILL_KERNEL 14 /* concur_prefill_attn: 0 (default) = blocks of 32 query tokens, two tiles
                                       of 128 accumulator rows per CTA over 128-token steps of K and V;
                                       1 = blocks of 16 query tokens, one tile over 64-token tiles (the
                                       pipeline the shared-prefix pass uses)                             */

/* Layouts of the K and V pools (concur_attn_config_t.kv_layout). */
#define CONCUR_KV_HEAD_MAJOR  0   /* [num_pages][Hkv][P][D]: one (page, head) tile is contiguous (default) */
#define CONCUR_KV_TOKEN_MAJOR 1   /* [num_pages][P][Hkv][D]: one token's rows of all KV heads are contiguous */

typedef struct concur_attn concur_attn_t;   /* opaque; owns its workspace and nothing else */

typedef struct {
    int32_t num_q_heads;        /* Hq; supported: Hkv x (1 .. 8), e.g. 64 or 40 over 8 KV heads          */
    int32_t num_kv_heads;       /* Hkv; supported: 1 .. 8.  A rank of a model that is tensor-parallel over
                                   its KV heads passes the heads it holds: 8 query over 1 KV head at
                                   8 ranks of the 64 / 8 geometry, with its own slice of every page     */
    int32_t head_dim;           /* D; supported: 128                                            */
    int32_t page_size;          /* P; supported: 16, 32, 64, 128 tokens                         */
    int32_t max_batch;          /* largest `batch` any call will pass (1 .. 65536)              */
    int32_t max_pages_per_seq;  /* largest `block_table_stride` any call will pass             */
    int32_t device;             /* CUDA device ordinal                                          */
    int32_t kv_layout;          /* CONCUR_KV_HEAD_MAJOR (0, default) or CONCUR_KV_TOKEN_MAJOR   */
    void*   workspace;          /* optional device memory (256-byte aligned) of at least
                                   concur_attn_workspace_bytes(); NULL: the library allocates  */
    size_t  workspace_bytes;    /* size of `workspace`; ignored when it is NULL                */
} concur_attn_config_t;

/*
 * Bytes of device workspace a handle with this configuration needs (split-KV partial
 * results, the plan's tables, counters).  Host function, no CUDA call.  Returns 0 for an
 * invalid or unsupported configuration.
 */
size_t concur_attn_workspace_bytes(const concur_attn_config_t* cfg);

/*
 * Creates a handle on cfg->device.  Checks the geometry (CONCUR_ERR_UNSUPPORTED), the
 * limits (CONCUR_ERR_INVALID_ARG), takes or allocates the workspace (CONCUR_ERR_OOM,
 * CONCUR_ERR_TOO_LARGE if a caller-supplied one is too small) and clears it on the
 * device's default stream (synchronously).  *handle is written only on success.
 */
int concur_attn_create(const concur_attn_config_t* cfg, concur_attn_t** handle);

/*
 * One decode-attention step, enqueued on `cuda_stream` (a cudaStream_t; NULL = default
 * stream).  Asynchronous: returns after the launches are queued, never synchronises, and
 * reads seq_lens / block_table on the device only.  Calls on one handle must be
 * stream-ordered with each other (they share the workspace).
 *
 *   q, k_pages, v_pages, out   device, 16-byte aligned, layouts as in the file header
 *   block_table, seq_lens      device, 4-byte aligned
 *   scale                      multiplies q.k before the softmax (1/sqrt(D) usually)
 *   batch                      0 <= batch <= max_batch   (0: nothing is launched)
 *   num_pages                  pages in each pool, >= 1
 *   block_table_stride         int32 elements per table row, 1 .. max_pages_per_seq
 *
 * Launches: one kernel for batches of up to 511 sequences (the partial kernel works the plan out for
 * itself from seq_lens, merges split sequences itself and leaves the workspace ready for the next
 * call); a plan kernel and the partial kernel beyond that, unless the plan was made ahead with
 * concur_attn_plan; a third (combine) kernel only with the scalar kernel or CONCUR_OPT_FUSE_COMBINE 0.
 *
 * Errors: CONCUR_ERR_INVALID_ARG (null or misaligned pointer, bad size),
 * CONCUR_ERR_TOO_LARGE (batch or stride above the handle's limits), CONCUR_ERR_CUDA
 * (launch failure).  Bad *contents* never fault: a page id outside [0, num_pages) or a
 * length outside [0, stride*P] is clamped and recorded (see concur_attn_status); the
 * affected sequences' results are then unspecified but finite memory is all that is read.
 */
int concur_decode_attn(concur_attn_t* handle,
                       const void* q, const void* k_pages, const void* v_pages,
                       const int32_t* block_table, const int32_t* seq_lens,
                       float scale, void* out, float* lse,
                       int32_t batch, int32_t num_pages, int32_t block_table_stride,
                       void* cuda_stream);

/*
 * Plan once per token step, attend once per layer.  All layers of a model see the same seq_lens in a
 * decode step, so the split-KV plan (tile counts, ranges) is the same for each of them.  (The paper's
 * generation runs, Sec. 3.3 and 4.2, are such loops over the layers of 32B models; the paper does not
 * describe them.)
 *
 *   concur_attn_plan             computes the plan of (seq_lens, batch, block_table_stride) into the
 *                                handle's workspace: one small kernel on `cuda_stream`.
 *   concur_decode_attn_planned   concur_decode_attn as ONE kernel launch, using that plan.  It must
 *                                follow, on the same stream, a concur_attn_plan call with the same
 *                                seq_lens pointer, batch and stride, with no other call on the handle
 *                                in between except further concur_decode_attn_planned and concur_kv_append
 *                                calls; seq_lens' contents must be what the plan call saw (so: append all
 *                                layers' rows with lengths advanced once, or plan after the append).
 *                                Otherwise CONCUR_ERR_INVALID_ARG.  Batches of up to 511 sequences need
 *                                no plan call at all (concur_decode_attn is already one launch there)
 *                                and are accepted without one.
 * Arguments, asynchrony and other errors as for concur_decode_attn.
 */
int concur_attn_plan(concur_attn_t* handle, const int32_t* seq_lens, int32_t batch,
                     int32_t block_table_stride, void* cuda_stream);
int concur_decode_attn_planned(concur_attn_t* handle,
                               const void* q, const void* k_pages, const void* v_pages,
                               const int32_t* block_table, const int32_t* seq_lens,
                               float scale, void* out, float* lse,
                               int32_t batch, int32_t num_pages, int32_t block_table_stride,
                               void* cuda_stream);

/*
 * The same step when sequences share a cached prefix (cascade decode).  In the paper's
 * workload every task is sampled 5 times for synthesis and 10 times for evaluation from one
 * fixed prompt (Sec. 3.3, Sec. 4.2, App. C), so the samples of a task have their whole
 * prompt in common; with a paged cache they can point at the same physical pages.
 *
 *   group_start   device, int32 [num_groups + 1]: group i is sequences group_start[i] ..
 *                 group_start[i+1]-1 (consecutive); group_start[0] = 0, last entry = batch
 *   prefix_lens   device, int32 [num_groups]: the caller's promise that the first
 *                 prefix_lens[i] tokens of all sequences of group i are the same cached
 *                 tokens, i.e. their block-table rows agree on the pages that hold them
 *
 * The result is defined exactly as for concur_decode_attn on the same tables (sharing
 * changes how often the shared tiles are read, never what is computed): the shared tiles
 * are streamed once per group and KV head and multiplied with the query rows of up to 10
 * sharing sequences on the tensor cores; every sequence's remaining tokens are handled as
 * in the plain step; the partial results are merged by log-sum-exp.  Only whole 64-token
 * tiles are shared (the rest of the prefix is read per sequence), a group's sequences
 * beyond the tenth read everything themselves, and a prefix longer than the group's
 * shortest sequence is cut to it and recorded as CONCUR_FLAG_BAD_SEQ_LEN.  If the promise
 * is broken the shared part is read through the group's first sequence's table.  A group_start
 * array that is not non-decreasing within [0, batch] never faults either: the call then shares
 * nothing, computes what concur_decode_attn computes, and records CONCUR_FLAG_BAD_GROUP.
 *
 * Needs max_batch <= 4096 (CONCUR_ERR_UNSUPPORTED otherwise).  The first cascade call on a
 * handle allocates the cascade workspace (cudaMalloc; CONCUR_ERR_OOM); make it outside any
 * stream capture.  Other arguments, asynchrony and errors as for concur_decode_attn.
 */
int concur_decode_attn_cascade(concur_attn_t* handle,
                               const void* q, const void* k_pages, const void* v_pages,
                               const int32_t* block_table, const int32_t* seq_lens,
                               const int32_t* group_start, const int32_t* prefix_lens,
                               float scale, void* out, float* lse,
                               int32_t batch, int32_t num_groups, int32_t num_pages,
                               int32_t block_table_stride, void* cuda_stream);

/*
 * Prefill: causal attention of several new query tokens per sequence against the cache -- the
 * step that runs once per prompt before its samples are decoded (in the paper's pipeline every
 * task's prompt, the fixed template of App. C around the task's program, is processed once and
 * then sampled 5 or 10 times, Sec. 3.3 / 4.2), or once per chunk of a long prompt.  The paper
 * states no formula; per query token the definition is that of the decode step:
 *
 *   sequence b has q_len = q_start[b+1] - q_start[b] query tokens, rows q_start[b] .. of q, out
 *   and lse.  They are the LAST q_len of the seq_lens[b] cached tokens (their K and V must
 *   already be in the cache): query token i sits at position pos = seq_lens[b] - q_len + i and
 *   attends to the cached tokens 0 .. pos of its sequence, exactly as concur_decode_attn would
 *   for a sequence of length pos + 1.
 *
 *   q, out        device, bf16 [total_q][Hq][D], 16-byte aligned
 *   lse           device, fp32 [total_q][Hq]
 *   q_start       device, int32 [batch + 1], non-decreasing, q_start[0] = 0, q_start[batch] = total_q
 *   other arguments as for concur_decode_attn
 *
 * Runs on the 5th-generation tensor cores: a unit is 32 query tokens x the query heads of one
 * KV head (two tiles of up to 128 accumulator rows in tensor memory) streaming that KV head's
 * tokens once, 128 at a time (CONCUR_OPT_PREFILL_KERNEL 1: 16 query tokens, one tile, 64 at a time).
 * Asynchronous on `cuda_stream`.  q_len > seq_lens[b] is cut to seq_lens[b] and recorded as
 * CONCUR_FLAG_BAD_SEQ_LEN (the rows beyond are then not written).  Errors as for
 * concur_decode_attn; total_q < 0 or a null q_start is CONCUR_ERR_INVALID_ARG.
 */
int concur_prefill_attn(concur_attn_t* handle,
                        const void* q, const void* k_pages, const void* v_pages,
                        const int32_t* block_table, const int32_t* seq_lens, const int32_t* q_start,
                        float scale, void* out, float* lse,
                        int32_t batch, int32_t total_q, int32_t num_pages, int32_t block_table_stride,
                        void* cuda_stream);

/*
 * The write path of the paged cache, run once per decode step before the attention call:
 * for every sequence b, the new token's rows k_new[b][g][:], v_new[b][g][:] (g = 0..Hkv-1)
 * are stored at position pos = seq_lens[b], i.e. slot pos % P of page
 * block_table[b][pos / P], and seq_lens[b] becomes pos + 1.  (The generation loop whose
 * attention step this library implements -- Sec. 3.3 / 4.2 of the paper -- appends one
 * token per sequence per step; the paper does not describe the cache.)
 *
 *   k_new, v_new   device, bf16 [batch][Hkv][D], 16-byte aligned
 *   k_pages, v_pages, block_table   as for concur_decode_attn (the pools are written)
 *   seq_lens       device, int32 [batch], read and advanced
 *
 * Asynchronous on `cuda_stream`.  A sequence whose position is outside [0, stride*P) or
 * whose page id is outside [0, num_pages) is left untouched (nothing written, length not
 * advanced) and CONCUR_FLAG_BAD_SEQ_LEN / CONCUR_FLAG_BAD_PAGE_ID is recorded.  The page
 * must already be allocated in the block table: page allocation is the caller's.
 * Errors as for concur_decode_attn.
 */
int concur_kv_append(concur_attn_t* handle, const void* k_new, const void* v_new,
                     void* k_pages, void* v_pages, const int32_t* block_table, int32_t* seq_lens,
                     int32_t batch, int32_t num_pages, int32_t block_table_stride,
                     void* cuda_stream);

/*
 * The same write for the further layers of a model.  A model keeps one pair of pools per layer and one
 * set of lengths for all of them, so only the step's first append may advance the lengths:
 *   advance = 1   exactly concur_kv_append: rows go to position seq_lens[b], which becomes seq_lens[b] + 1;
 *   advance = 0   rows go to position seq_lens[b] - 1 -- the slot the step's first append opened -- and
 *                 seq_lens is only read.  A length of 0 (no slot opened) is flagged like any position
 *                 outside the table row and nothing is written.
 * Any other `advance` is CONCUR_ERR_INVALID_ARG; everything else as for concur_kv_append.
 */
int concur_kv_append_layer(concur_attn_t* handle, const void* k_new, const void* v_new,
                           void* k_pages, void* v_pages, const int32_t* block_table, int32_t* seq_lens,
                           int32_t batch, int32_t num_pages, int32_t block_table_stride, int32_t advance,
                           void* cuda_stream);

/*
 * concur_kv_append_layer(advance = 0) and concur_decode_attn in one: the K / V rows of every sequence's
 * newest token -- position seq_lens[b] - 1, which the step's first append has already counted -- are
 * passed in, used for the attention, and stored into their pool slot by the kernel itself.  One launch
 * per layer instead of two (for up to 511 sequences), and, with CONCUR_OPT_OVERLAP_CALLS, layer after
 * layer may overlap, which an append kernel between two attention kernels prevents.  The paper has no
 * counterpart (it implies the generation loop, Sec. 3.3, and describes none of it).
 *
 *   k_new, v_new   device, bf16 [batch][Hkv][D], 16-byte aligned: rows of the token at seq_lens[b] - 1
 *   k_pages, v_pages   as for concur_decode_attn, but WRITTEN: slot (seq_lens[b] - 1) % P of page
 *                  block_table[b][(seq_lens[b] - 1) / P] receives the rows; whatever that slot held before
 *                  is ignored
 *   other arguments, result, asynchrony as for concur_decode_attn (seq_lens is only read)
 *
 * A sequence with seq_lens[b] = 0 has no newest token: nothing is stored, its result is that of an empty
 * sequence.  A bad page id for the slot is flagged (CONCUR_FLAG_BAD_PAGE_ID) and nothing is stored.
 * Needs the tensor-core kernel with the fused merge (the defaults): CONCUR_ERR_UNSUPPORTED otherwise.
 */
int concur_decode_attn_append(concur_attn_t* handle, const void* q, const void* k_new, const void* v_new,
                              void* k_pages, void* v_pages, const int32_t* block_table,
                              const int32_t* seq_lens, float scale, void* out, float* lse,
                              int32_t batch, int32_t num_pages, int32_t block_table_stride,
                              void* cuda_stream);

/*
 * The same step for callers whose tensors live in HOST memory (pinned memory gives
 * asynchronous copies).  Every pointer is a host pointer with the layouts above; the
 * library copies the inputs into device staging buffers that it owns (allocated on first
 * use and grown when a call needs more: cudaMalloc inside this call), runs the three
 * kernels, copies out / lse back and synchronises the stream before returning.
 * Errors as for concur_decode_attn, plus CONCUR_ERR_OOM.
 */
int concur_decode_attn_host(concur_attn_t* handle,
                            const void* q, const void* k_pages, const void* v_pages,
                            const int32_t* block_table, const int32_t* seq_lens,
                            float scale, void* out, float* lse,
                            int32_t batch, int32_t num_pages, int32_t block_table_stride,
                            void* cuda_stream);

/*
 * Synchronises `cuda_stream` and returns, in *flags (host pointer), the OR of the
 * CONCUR_FLAG_* conditions seen by any call on this handle since the last status call;
 * the device word is then cleared.  If CONCUR_FLAG_WAIT_LIMIT is among them the handle's workspace
 * counters are re-initialised as well, so that the next call starts clean.
 */
int concur_attn_status(concur_attn_t* handle, void* cuda_stream, uint32_t* flags);

/* Sets a CONCUR_OPT_* value for later calls on this handle.  Unknown key or a value out
 * of range: CONCUR_ERR_INVALID_ARG. */
int concur_attn_set_option(concur_attn_t* handle, int32_t key, int64_t value);

/*
 * For tests and load-balance reports: copies the plan of the most recent call to the
 * host (synchronises `cuda_stream`).  *num_ranges and *total_tiles receive the split-KV
 * range count and the number of (KV head, 64-token tile) units; range_start (host,
 * capacity `cap` int32s, may be NULL) receives min(cap, num_ranges+1) range boundaries.
 */
int concur_attn_last_plan(concur_attn_t* handle, void* cuda_stream, int32_t* num_ranges,
                          int32_t* total_tiles, int32_t* range_start, int32_t cap);

/*
 * The same decode-attention step for callers that cannot allocate device memory.  (The
 * paper has no counterpart to this entry point; it exists for integration only.)
 *
 * Who needs it: a process that gave its whole device-memory budget to its own arena at
 * start-up and treats later driver allocations as errors; code that runs inside another
 * runtime's callback, where cudaMalloc is not permitted; a latency path that cannot risk
 * the device-wide synchronisation an allocation or a free may cause.  Such callers cannot
 * create a handle (a handle owns or borrows a workspace).  Here the workspace is a fixed
 * array inside the library's device image -- about 4.3 MB that every GPU which loads the
 * library holds until the process exits -- and there is no handle at all.
 *
 * Arguments and layouts are those of concur_decode_attn for 64 query heads and 8 KV heads, plus
 * `page_size` (16, 32 or 64);
 * the work is enqueued on `cuda_stream` of the CURRENT device and the call returns without
 * synchronising.  It performs no cudaMalloc / cudaFree and calls no allocating library
 * routine.  Limits: batch <= CONCUR_STATIC_MAX_BATCH (more: CONCUR_ERR_TOO_LARGE, nothing
 * is launched); the plan uses at most CONCUR_STATIC_MAX_RANGES split-KV ranges, so very
 * large batches balance a little more coarsely than through a handle.  Other errors as for
 * concur_decode_attn.  Device-side conditions are handled as in concur_decode_attn (a bad page
 * id or length is clamped; a bounded in-kernel wait that gives up ends the kernel, whose results
 * are then invalid) but this entry point has no handle to report them through: none of the
 * CONCUR_FLAG_* bits, CONCUR_FLAG_WAIT_LIMIT included, can be read back by its callers.
 *
 * The first call on each device resolves the array's device address
 * (cudaGetSymbolAddress) and reads the SM count; make that first call outside any stream
 * capture.  All calls on a device share the one array, which keeps the previous call's
 * contents: each call re-initialises what it reads, but two calls whose kernels overlap on
 * the GPU (different streams without ordering, or different host threads) race on it.
 * Order them on one stream or with events.
 */
#define CONCUR_STATIC_MAX_BATCH  1024
#define CONCUR_STATIC_MAX_RANGES 512
int concur_decode_attn_static(const void* q, const void* k_pages, const void* v_pages,
                              const int32_t* block_table, const int32_t* seq_lens,
                              float scale, void* out, float* lse,
                              int32_t batch, int32_t num_pages, int32_t block_table_stride,
                              int32_t page_size, void* cuda_stream);

/*
 * Merges finished attention results by their log-sum-exp: `parts` results of the SAME query rows, each
 * over a different part of the keys, into the result over all of them --
 *     L = ln sum_s exp(lse_s),  out = sum_s exp(lse_s - L) out_s;  a part with lse = -inf (no keys) weighs 0;
 *     every part empty: out = 0, lse = -inf.
 * It is the merge of the split-KV method (exact up to rounding: a re-association of the softmax sums) applied
 * ACROSS calls: when the cache of very long sequences is spread over several GPUs by token range (context
 * sharding), each GPU runs concur_decode_attn on its range, the (out, lse) pairs are gathered -- 260 bytes per
 * query row and GPU -- and every GPU calls this.  The paper has no counterpart.
 *
 *   outs   device, bf16 [parts][rows][D], 16-byte aligned      rows = batch x Hq, D = 128
 *   lses   device, fp32 [parts][rows], natural log, as concur_decode_attn returns it
 *   out    device, bf16 [rows][D], 16-byte aligned;   lse  device, fp32 [rows]
 * No handle, no workspace, no allocation; asynchronous on `cuda_stream` of the current device.  Because the
 * parts arrive rounded to bf16, the merged result carries their rounding (2^-9 relative each) as well as its own.
 * Errors: CONCUR_ERR_INVALID_ARG (parts < 1, rows < 0, null or misaligned pointer), CONCUR_ERR_CUDA.
 */
int concur_lse_merge(const void* outs, const float* lses, int32_t parts, int64_t rows,
                     void* out, float* lse, void* cuda_stream);

/* Frees the handle and any memory the library allocated for it.  NULL is accepted. */
int concur_attn_destroy(concur_attn_t* handle);

/* Static, never-NULL description of a status code. */
const char* concur_attn_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* CONCUR_ATTN_H_ */
