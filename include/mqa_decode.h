/*
 * mqa_decode.h -- C ABI of the B200 (sm_100a) decode-attention library.
 *
 * One incremental-decoding attention step as stated in "Fast Transformer Decoding: One
 * Write-Head is All You Need" (arXiv 1911.02150): for each sequence of a batch, h query
 * heads attend over that sequence's key/value cache,
 *
 *     logits[b,h,j] = sum_c q[b,h,c] * K[..,j,c]          (no 1/sqrt(k) factor: the note
 *     w[b,h,:]      = softmax_j(logits[b,h,:])             closing Section 2.2 folds it
 *     o[b,h,c]      = sum_j w[b,h,j] * V[..,j,c]           into the projections)
 *
 * with j running over the valid prefix of the cache.  The multi-query form (Section 3)
 * keeps ONE cache per sequence, K[b,m,k], V[b,m,v], shared by all heads; the multi-head
 * form (Section 2.4) keeps one per head, K[b,h,m,k], V[b,h,m,v].  The new token's key and
 * value row is appended to the cache in place before the step attends.
 *
 * Conventions for every entry point
 *   - Every pointer is a DEVICE pointer owned by the caller unless said otherwise; tensors
 *     are dense, row-major, innermost axis last.  q, K, V, k_new, v_new, o and the workspace
 *     must be 16-byte aligned; lens and status 4-byte aligned.
 *   - K, V, q, k_new, v_new hold bf16; o holds fp32; lens holds int32.
 *   - k == v == 128 is the only supported head width; h >= 1.  Many query rows per sequence (many heads;
 *     or beams x heads over one shared memory, passed as h = beams * heads) run on the tensor cores too:
 *     more than 32 rows on a kernel that puts the query rows on the rows of its tiles (128 rows per
 *     CTA; more as row tiles over the same cache rows).
 *   - `stream` is a cudaStream_t passed as a plain pointer (NULL = the legacy default stream).
 *     Calls only enqueue work on it: they never synchronise, never allocate device memory and
 *     never free anything.  The launch configuration is chosen from the integer arguments and
 *     the current device alone, never from device data.
 *   - Return value: MQA_OK (0) or one of the positive codes below.  Arguments, sizes and the
 *     workspace are checked before anything is enqueued: with every code except MQA_ERR_CUDA no
 *     kernel or copy has been launched and no buffer has been touched.  MQA_ERR_CUDA reports a
 *     failed launch or copy; in a call that enqueues several, the earlier ones are then already
 *     on the stream.
 *   - Cache rows at or beyond lens[b] are don't-care: they may hold anything (NaN, Inf) and
 *     do not influence o.  lens[b] outside [0, m_max] is clamped into it for the attention
 *     and reported through `status`; nothing is read or written out of bounds.
 *   - lens[b] == 0 gives o[b,:,:] = 0 (the paper's flow never produces an empty prefix, since
 *     the append precedes the attention).
 *   - Results are deterministic: the same inputs on the same device give the same bits.
 *   - `status` (optional, may be NULL) is one int32 word on the device that kernels OR bits
 *     into; the caller clears it.  Bits: MQA_STATUS_*.
 */
#ifndef MQA_DECODE_H_
#define MQA_DECODE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef void* mqa_stream_t; /* a cudaStream_t */

enum {
    MQA_OK = 0,
    MQA_ERR_INVALID_ARG = 1,         /* null or misaligned pointer, non-positive dimension   */
    MQA_ERR_UNSUPPORTED = 2,         /* k or v != 128, or a size the launch grid cannot hold */
    MQA_ERR_WORKSPACE_TOO_SMALL = 3, /* workspace_bytes < mqa_workspace_bytes(...)           */
    MQA_ERR_CUDA = 4,                /* the CUDA runtime reported an error at launch         */
    MQA_ERR_STATIC_SCRATCH_TOO_SMALL = 5 /* mqa_decode_step_noalloc: these sizes need more scratch
                                            than the library's built-in MQA_NOALLOC_SCRATCH_BYTES */
};

enum {
    MQA_STATUS_APPEND_CACHE_FULL = 1,   /* kv_cache_append: some lens[b] >= m_max, that sequence skipped */
    MQA_STATUS_APPEND_NEGATIVE_LEN = 2, /* kv_cache_append: some lens[b] < 0, that sequence skipped      */
    MQA_STATUS_LEN_CLAMPED = 4,         /* decode step: some lens[b] outside [0, m_max] was clamped       */
    MQA_STATUS_PIPELINE_TIMEOUT = 8     /* decode step: a bounded wait on an on-chip copy ran out; the
                                           affected outputs are not valid                              */
};

/*
 * kv_cache_append -- the concatenation of the new key/value row on the memory axis in the
 * incremental functions of Sections 2.4 (multi-head) and 3 (multi-query), done in place in
 * a cache padded to m_max rows.
 *
 *   K, V          [b, kv_heads, m_max, k], [b, kv_heads, m_max, v] bf16, read-write.
 *                 kv_heads = 1 for the multi-query cache ([b, m_max, k]), h for multi-head.
 *   k_new, v_new  [b, kv_heads, k], [b, kv_heads, v] bf16: the new token's rows.
 *   lens          [b] int32: rows valid BEFORE the call; row lens[b] is the one written.
 *   advance       non-zero: lens[b] += 1 on the device after the write (for written rows).
 *   status        optional; CACHE_FULL / NEGATIVE_LEN when a sequence cannot take a row
 *                 (that sequence is skipped: nothing written, lens[b] unchanged).
 * The rows are copied as 16-bit words and never interpreted as numbers: bit-exact.
 */
int kv_cache_append(void* K, void* V, const void* k_new, const void* v_new,
                    int32_t* lens, int advance, int32_t* status,
                    int b, int kv_heads, int m_max, int k, int v, mqa_stream_t stream);

/*
 * mqa_decode_step -- the three attention lines of the incremental multi-query function
 * (Section 3): logits = einsum(bhk,bmk->bhm), softmax over m, o = einsum(bhm,bmv->bhv),
 * over the first lens[b] rows of each sequence's shared cache.
 *
 *   q      [b, h, k] bf16          K, V   [b, m_max, k], [b, m_max, v] bf16 (read only)
 *   lens   [b] int32: rows to attend over (i.e. AFTER the append)
 *   o      [b, h, v] fp32, written
 *   workspace, workspace_bytes   scratch for the per-piece partial results; at least
 *          mqa_workspace_bytes(b, h, m_max, k, v) bytes.  It may hold anything on entry (never
 *          cleared, never assumed clear) and its contents on return are unspecified.  Two calls
 *          that may overlap on the GPU need two workspaces.  May be NULL when
 *          mqa_workspace_bytes(...) is 0.
 *   status optional; LEN_CLAMPED, PIPELINE_TIMEOUT.
 * The memory axis is cut into pieces that run in parallel, each keeping a maximum and a sum
 * (an exact re-association of the same softmax); shared K/V rows are read from HBM once and
 * used for all h heads.  For large batches (every SM takes an equal share of all valid rows)
 * the pieces of a sequence are merged inside the same kernel by the CTA that finishes the
 * sequence's last piece: one launch.  The bookkeeping for that lives at the head of the workspace
 * under a per-call epoch that the kernel itself moves on -- one epoch per workspace, whatever the
 * sizes of the calls that share it -- so nothing has to be initialised, CUDA-graph replays are
 * safe, and a workspace may serve calls of different shapes one after the other.  A call that
 * reported PIPELINE_TIMEOUT moves the epoch on as well: the workspace needs no repair afterwards.
 * Between two calls the caller may overwrite the whole workspace or leave it alone, but must not
 * restore an older copy of it.  Other sizes use a second kernel to combine the pieces.
 */
int mqa_decode_step(const void* q, const void* K, const void* V, const int32_t* lens, float* o,
                    void* workspace, size_t workspace_bytes, int32_t* status,
                    int b, int h, int m_max, int k, int v, mqa_stream_t stream);

/*
 * mha_decode_step -- the same three lines of the incremental multi-head function
 * (Section 2.4): logits = einsum(bhk,bhmk->bhm), softmax over m, o = einsum(bhm,bhmv->bhv).
 * Arguments as mqa_decode_step except K, V are [b, h, m_max, k], [b, h, m_max, v] (one
 * cache per head); lens[b] is shared by the h heads of a sequence.
 */
int mha_decode_step(const void* q, const void* K, const void* V, const int32_t* lens, float* o,
                    void* workspace, size_t workspace_bytes, int32_t* status,
                    int b, int h, int m_max, int k, int v, mqa_stream_t stream);

/*
 * mqa_decode_append_step -- one whole decoding step of the incremental multi-query function
 * (Section 3) in a single call: the new token's key/value row is concatenated to each
 * sequence's cache at row lens[b] (as kv_cache_append does), then the h heads attend over
 * the lens[b] + 1 rows (as mqa_decode_step does).  For batches large enough for the persistent
 * kernel (h <= 64) the whole step is one launch: the CTA that streams a sequence's last tile
 * writes the new row before it fetches that tile, the pieces of a sequence are merged by the
 * CTA that finishes the last one, and lens is advanced once every CTA has read it.  Other
 * sizes run the same step as separate launches (mqa_append_step_launches tells how many).
 *
 *   q, k_new, v_new   [b, h, k], [b, k], [b, v] bf16
 *   K, V              [b, m_max, k], [b, m_max, v] bf16, read-write (row lens[b] is written)
 *   lens              [b] int32: rows valid BEFORE the call.
 *   advance           bit flags.  MQA_STEP_ADVANCE (1): lens[b] += 1 on return for sequences that took a
 *                     row; without it lens is left as it was, although the row has been written and
 *                     attended over.  MQA_STEP_CHAINED (2): a promise by the caller about the work that
 *                     precedes this call on `stream` and may still be running when this call's kernel
 *                     starts (everything enqueued since the stream was last idle, or since the kernel
 *                     before the most recent kernel completed): apart from steps of this library, none
 *                     of it writes lens, and none of it writes rows of THIS cache below the last two
 *                     rows of each prefix.  Steps of this library on this or on other caches keep the
 *                     promise (a step writes one row per sequence at the end of its prefix and moves
 *                     lens on by one), and so do projections, a sampler, copies of q; other caches, o
 *                     and the workspace may be written freely.  The first step after something else
 *                     filled the cache (a prefill kernel) must not carry the flag.  With the promise
 *                     the persistent kernel starts fetching the cache, except each prefix's last rows,
 *                     while the kernel before it is still finishing, and reads q, the new rows, lens
 *                     and the workspace only after that kernel has completed.  What it fetches early
 *                     goes by lens as it reads then; should lens have moved by the time it may rely on
 *                     it, it fetches again.
 *                     MQA_STEP_TEST_WRONG_GUESS (4), for tests, with MQA_STEP_CHAINED: the early fetch is
 *                     deliberately the wrong one, so that this recovery runs; results are unchanged.
 *                     MQA_STEP_TEST_WITHHOLD_COPY (8), for tests: one on-chip copy of the first CTA is never
 *                     started, so that a bounded wait runs out (see mqa_set_wait_limit_cycles): the kernel
 *                     returns by itself, PIPELINE_TIMEOUT is flagged and o is not valid.
 *                     Any other bit: MQA_ERR_INVALID_ARG.
 *   o, workspace, workspace_bytes, status   as for mqa_decode_step.  A sequence with lens[b] == m_max
 *                     (or negative) takes no new row: APPEND_CACHE_FULL (APPEND_NEGATIVE_LEN) is flagged
 *                     and it attends over its existing rows.
 * Results are those of kv_cache_append followed by mqa_decode_step on the same inputs.
 */
#define MQA_STEP_ADVANCE 1
#define MQA_STEP_CHAINED 2
#define MQA_STEP_TEST_WRONG_GUESS 4
#define MQA_STEP_TEST_WITHHOLD_COPY 8
int mqa_decode_append_step(const void* q, void* K, void* V, const void* k_new, const void* v_new, int32_t* lens,
                           int advance, float* o, void* workspace, size_t workspace_bytes, int32_t* status,
                           int b, int h, int m_max, int k, int v, mqa_stream_t stream);

/*
 * The two phases of a step, separately (split then combine with the same arguments gives what
 * mqa_decode_step gives; likewise mha).  They exist so that a caller can time or schedule the
 * phases on their own.  *_split runs the pass over the cache (Section 3 / 2.4 lines, per piece)
 * and leaves partial results in the workspace -- or final results in o when the plan has a
 * single piece; *_combine merges the pieces into o with a second kernel (also where
 * mqa_decode_step itself would merge them inside its one launch) and is a no-op (no launch)
 * for a single piece.
 */
int mqa_decode_step_split(const void* q, const void* K, const void* V, const int32_t* lens, float* o,
                          void* workspace, size_t workspace_bytes, int32_t* status,
                          int b, int h, int m_max, int k, int v, mqa_stream_t stream);
int mqa_decode_step_combine(const int32_t* lens, float* o, const void* workspace, size_t workspace_bytes,
                            int b, int h, int m_max, int k, int v, mqa_stream_t stream);
int mha_decode_step_split(const void* q, const void* K, const void* V, const int32_t* lens, float* o,
                          void* workspace, size_t workspace_bytes, int32_t* status,
                          int b, int h, int m_max, int k, int v, mqa_stream_t stream);
int mha_decode_step_combine(const int32_t* lens, float* o, const void* workspace, size_t workspace_bytes,
                            int b, int h, int m_max, int k, int v, mqa_stream_t stream);

/*
 * mqa_workspace_bytes -- bytes of scratch that mqa_decode_step and mha_decode_step need for
 * these sizes on the current device (an upper bound valid for both; 0 if the arguments are
 * not valid).  Host-only; touches no device memory.
 */
size_t mqa_workspace_bytes(int b, int h, int m_max, int k, int v);

/*
 * mqa_plan_splits -- the launch plan for these sizes on the current device (`multi_query`
 * non-zero: mqa_decode_step, zero: mha_decode_step).  Returns the number of pieces one
 * sequence's memory axis may be cut into (1 = no second pass), and through *chunk_rows
 * (optional) the rows of one piece: the fixed split length, or, when the persistent kernel is
 * used (every SM takes an equal share of the valid rows of the whole batch), the rows one SM
 * streams when every cache is full.  Returns 0 for invalid arguments.  Informational; host-only.
 */
int mqa_plan_splits(int multi_query, int b, int h, int m_max, int k, int v, int* chunk_rows);

/*
 * mqa_plan_kernel_name -- the name of the kernel that does the pass over the cache for these sizes on
 * the current device (`multi_query` as for mqa_plan_splits; `whole_step` non-zero: as launched by
 * mqa_decode_append_step with MQA_STEP_CHAINED, zero: as launched by mqa_decode_step).  A static string,
 * "" for invalid arguments.  Informational (benchmarks and profiles name what they timed); host-only.
 */
const char* mqa_plan_kernel_name(int multi_query, int whole_step, int b, int h, int m_max, int k, int v);

/*
 * mqa_decode_step_noalloc -- mqa_decode_step for callers that cannot allocate.  (The paper has
 * no counterpart to this entry point; it computes exactly what mqa_decode_step computes.)
 *
 * Some callers of a decode step cannot give it a workspace: a plugin or custom op that runs
 * inside a host framework whose device memory was planned and reserved at start-up has no
 * allocator to ask, and cudaMalloc is either forbidden there (it stalls the whole device while
 * it runs) or bound to fail (the framework already holds all the memory).  This entry point
 * takes only inputs and outputs.  Its scratch is a fixed array of MQA_NOALLOC_SCRATCH_BYTES
 * bytes of device global memory inside the library image, which every GPU that loads the
 * library keeps reserved until the process exits.
 *
 *   Arguments: as mqa_decode_step, without workspace and workspace_bytes.
 *   Returns MQA_ERR_STATIC_SCRATCH_TOO_SMALL, and launches nothing, when
 *   mqa_workspace_bytes(b, h, m_max, k, v) exceeds MQA_NOALLOC_SCRATCH_BYTES; otherwise whatever
 *   mqa_decode_step returns for the same arguments.
 *   Allocation: none.  The call uses no cudaMalloc, cudaFree or other allocating routine.
 *   First call on a device: looks up the array's device address (cudaGetSymbolAddress, with
 *   that device current) and remembers it; make this first call during set-up, before any
 *   stream capture is begun on that device.
 *   Sharing: every call on a device uses the same array, which still holds whatever the last
 *   call left in it, of whatever shape that call was.  Nothing has to be cleared, not even
 *   after a call that reported PIPELINE_TIMEOUT -- a call reads only what the same call has
 *   written, or what carries its own epoch -- but two calls whose kernels may overlap on the
 *   GPU (different streams, no ordering between them) race on it and corrupt each other's
 *   results.  Calls on one stream are safe.
 */
#define MQA_NOALLOC_SCRATCH_BYTES (8u * 1024u * 1024u)
int mqa_decode_step_noalloc(const void* q, const void* K, const void* V, const int32_t* lens, float* o,
                            int32_t* status, int b, int h, int m_max, int k, int v, mqa_stream_t stream);

/*
 * mqa_append_step_launches -- how many kernels one call of mqa_decode_append_step launches for these
 * sizes on the current device when lens is advanced (0 for invalid arguments).  Informational;
 * host-only.
 */
int mqa_append_step_launches(int b, int h, int m_max, int k, int v);

/*
 * mqa_decode_append_step_host -- mqa_decode_append_step for a caller whose per-token inputs and result live in
 * HOST memory (the decoder's other layers, a sampler): q, k_new, v_new are copied to the device, the step runs,
 * o is copied back, all enqueued on `stream` (nothing is synchronised: wait on the stream before reading o_host).
 * The cache, lens, workspace and status stay on the device as in mqa_decode_append_step.
 *
 *   q_host, k_new_host, v_new_host   HOST pointers, [b, h, k], [b, k], [b, v] bf16.  Where all three are pinned memory
 *                     that the device can address (cudaHostAlloc, cudaHostRegister), a kernel of this library fetches
 *                     them into the staging buffer and the attention kernel behind it sets itself up and asks for its
 *                     first stages of the cache meanwhile; they must then stay unchanged until the stream has passed
 *                     this call's work.  Any other host memory goes by cudaMemcpyAsync (asynchronous for pinned
 *                     memory; one copy when the three are packed back to back with each part padded to a multiple
 *                     of 256 bytes, else three).
 *   o_host            HOST pointer, [b, h, v] fp32.  Pinned memory that the device can address (cudaHostAlloc,
 *                     cudaHostRegister) is written by the step's kernels themselves, with no copy after them;
 *                     any other host memory is filled by a copy from the staging buffer.  Either way it is
 *                     complete once the stream has passed this call's work.
 *   staging           DEVICE scratch of at least mqa_host_staging_bytes(b, h, k, v) bytes (the device copies of the
 *                     above); owned by the caller, one per call that may be in flight
 * Other arguments and errors as for mqa_decode_append_step; MQA_ERR_WORKSPACE_TOO_SMALL also for a small staging.
 */
int mqa_decode_append_step_host(const void* q_host, const void* k_new_host, const void* v_new_host, float* o_host,
                                void* K, void* V, int32_t* lens, int advance, void* staging, size_t staging_bytes,
                                void* workspace, size_t workspace_bytes, int32_t* status,
                                int b, int h, int m_max, int k, int v, mqa_stream_t stream);
size_t mqa_host_staging_bytes(int b, int h, int k, int v);

/*
 * mqa_decode_local_step -- one decoding step of multi-query attention restricted to a local neighbourhood
 * (Section 4.1: the current position and the previous window - 1 positions; Section 4.3: the memory tensors
 * padded to the window size).  The cache is a ring of `window` rows per sequence: the new token's key/value row
 * is written to row pos[b] % window and the h heads attend over the min(pos[b] + 1, window) rows that hold tokens
 * (the order of the rows in the ring does not matter to a softmax).
 *
 *   q, k_new, v_new   [b, h, k], [b, k], [b, v] bf16
 *   K, V              [b, window, k], [b, window, v] bf16, read-write
 *   pos               [b] int32: tokens of the sequence before this step (0 for the first); advance != 0: pos[b] += 1
 *   o                 [b, h, v] fp32, written;  status optional (APPEND_NEGATIVE_LEN for pos[b] < 0: no row, zeros)
 * One launch; no workspace.  One warp per sequence, eight sequences per CTA, any number of heads (16 at a time),
 * windows of up to 4096 rows (the paper's is 32; MQA_ERR_UNSUPPORTED beyond).
 */
int mqa_decode_local_step(const void* q, void* K, void* V, const void* k_new, const void* v_new, int32_t* pos,
                          int advance, float* o, int32_t* status, int b, int h, int window, int k, int v,
                          mqa_stream_t stream);

/*
 * mqa_layer_decode_step -- the whole incremental multi-query layer of Section 3
 * (MultiquerySelfAttentionIncremental) for one new token per sequence: the projections
 * q = einsum(bd,hdk->bhk)(x, P_q), k_new = einsum(bd,dk->bk)(x, P_k), v_new = einsum(bd,dv->bv)(x, P_v),
 * then what mqa_decode_append_step does with them (the new row is concatenated to the cache at row
 * lens[b], the h heads attend over lens[b] + 1 rows), then y = einsum(bhv,hdv->bd)(o, P_o).
 *
 *   x                [b, d] bf16                 P_q  [h, d, k] bf16        P_k, P_v  [d, k], [d, v] bf16
 *   P_o              [h, d, v] bf16              K, V, lens, advance, status   as for mqa_decode_append_step
 *   y                [b, d] fp32, written
 *   workspace        at least mqa_layer_workspace_bytes(b, h, d, m_max, k, v) bytes; may hold anything on entry.
 *                    It carries q, k_new, v_new (bf16), o (fp32) and the attention step's own workspace.
 * d must be a multiple of 128 (MQA_ERR_UNSUPPORTED otherwise), k = v = 128.  The products run on the tensor
 * cores in bf16 with fp32 accumulation; q, k_new and v_new are rounded to bf16 where the step and the cache
 * take them, o is rounded to bf16 as an operand of the output product; y is summed over head groups in a fixed
 * order (no float atomics: results are reproducible bit for bit).  Kernels: projections in, the step (one
 * launch for large batches), projection out (its head groups are one thread-block cluster of up to 16 CTAs, which
 * sum y through distributed shared memory).
 */
int mqa_layer_decode_step(const void* x, const void* P_q, const void* P_k, const void* P_v, const void* P_o,
                          void* K, void* V, int32_t* lens, int advance, float* y,
                          void* workspace, size_t workspace_bytes, int32_t* status,
                          int b, int h, int d, int m_max, int k, int v, mqa_stream_t stream);

/* mqa_layer_workspace_bytes -- scratch mqa_layer_decode_step needs (0 for invalid or unsupported sizes). Host-only. */
size_t mqa_layer_workspace_bytes(int b, int h, int d, int m_max, int k, int v);

/*
 * mqa_prefill_attention -- the three attention lines of the batched multi-query function of Section 3
 * (MultiqueryAttentionBatched: logits = einsum(bhnk,bmk->bhnm), weights = softmax(logits + mask),
 * O = einsum(bhnm,bmv->bhnv)) for n query positions per sequence at once, under the mask that Section 2.3
 * gives for an autoregressive model: -inf where a query would look at a position after its own.
 *
 *   Q      [b, h, n, k] bf16                    K, V   [b, m_max, k], [b, m_max, v] bf16 (read only)
 *   start  [b] int32 or NULL (all zero): the memory position of each sequence's first query.  Query t of
 *          sequence b is memory position start[b] + t and attends over rows 0 .. start[b] + t of that sequence's
 *          K and V (so start[b] + n <= m_max must hold; with start = 0 and n rows in the cache this is the
 *          paper's M = X case, the processing of a whole prompt).  A negative start[b] is taken as an empty memory
 *          for that sequence (zeros) and flagged LEN_CLAMPED, like a bad lens.
 *   O      [b, h, n, v] fp32, written           status   optional; LEN_CLAMPED, PIPELINE_TIMEOUT
 *   workspace   at least mqa_prefill_workspace_bytes(b, h, n, m_max, k, v) bytes (see below).
 * One launch of a persistent kernel made for this form (mqa_prefill_kernel: a CTA per SM walks the units of work).  A
 * unit is 128 consecutive positions of two heads of a sequence -- the heads share K and V, so each staged 128-row K/V tile serves 256 query rows -- with the query
 * rows as the rows of the tensor-core tiles (one thread owns one query row's logits, maximum and sum), the weights
 * handed to the second product through tensor memory, and cache rows beyond a tile's last position never fetched.
 * Any n >= 1 (the last tile of a head may be partly filled); k = v = 128 (MQA_ERR_UNSUPPORTED otherwise, and for
 * n > m_max).  A memory that would pass m_max (start[b] + n > m_max) is cut at m_max and flagged LEN_CLAMPED.  The
 * workspace is not touched by the present kernel; the argument stays in the interface (pass at least
 * mqa_prefill_workspace_bytes() bytes, which is small and non-zero for supported sizes, 0 otherwise).
 */
int mqa_prefill_attention(const void* Q, const void* K, const void* V, const int32_t* start, float* O,
                          void* workspace, size_t workspace_bytes, int32_t* status,
                          int b, int h, int n, int m_max, int k, int v, mqa_stream_t stream);
size_t mqa_prefill_workspace_bytes(int b, int h, int n, int m_max, int k, int v);

/*
 * mqa_set_wait_limit_cycles -- how long, in SM clock cycles, a kernel of this library waits for one of its own
 * on-chip copies or products before it gives up, flags MQA_STATUS_PIPELINE_TIMEOUT and returns (no kernel here
 * waits without a bound, and none traps).  The default, restored by cycles <= 0, is about one second; tests
 * shorten it to see a wait run out within milliseconds.  Sets a variable on the current device, for kernels
 * launched afterwards; unlike the step calls this one is synchronous (it waits for the device to take the value).
 */
int mqa_set_wait_limit_cycles(long long cycles);

/*
 * mqa_set_test_withhold_copy -- for tests of the bounded waits of mqa_prefill_attention (which takes no flags): while
 * on != 0, the kernel of the batched form never starts one on-chip copy of its first CTA's second stage, so that a
 * wait runs out, MQA_STATUS_PIPELINE_TIMEOUT is flagged and the kernel returns by itself (O of that call is not
 * valid).  Sets a variable on the current device, for kernels launched afterwards; synchronous, like
 * mqa_set_wait_limit_cycles.  Off (0) by default.
 */
int mqa_set_test_withhold_copy(int on);

/* mqa_status_string -- a static, human-readable name for a return code. */
const char* mqa_status_string(int code);

#ifdef __cplusplus
}
#endif
#endif /* MQA_DECODE_H_ */
