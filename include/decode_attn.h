/*
 * decode_attn.h -- C ABI of the B200 (sm_100a) paged GQA decode-attention library.
 *
 * The operation.  For every sequence b of a batch and every query head h, one
 * query vector (the token being decoded) attends over that sequence's cached
 * keys and values, which live in fixed-size pages addressed through a block
 * table:
 *
 *     L  = seq_lens[b]            (the current token's K/V are already cached)
 *     lo = (window > 0 && window < L) ? L - window : 0
 *     g  = h / (Hq / Hkv)         (consecutive query heads share one KV head)
 *     s_t = scale * <q[b,h,:], K[block_table[b][t/P], g, t%P, :]>     lo <= t < L
 *     out[b,h,:] = sum_t softmax(s)_t * V[block_table[b][t/P], g, t%P, :]
 *     lse[b,h]   = ln sum_t exp(s_t)
 *     L <= 0:  out = 0, lse = -inf.
 *
 * Where it comes from.  The paper's agent loop is bound by calls to a central
 * LLM inference service (Sec. 3.2, last paragraph of "Large-scale runs"; Sec. 4
 * sets a 131,072-token context, up to 15 calls x 3 sessions per operator,
 * hundreds of sessions at once).  Per generated token and layer that service
 * runs exactly this step.  The paper gives no internals for it; its pointer to
 * the computation is the FlashAttention line of work cited in Sec. 5 ("Kernel
 * Research"), which evaluates softmax attention exactly by tiling, online
 * softmax and split-K with a log-sum-exp merge.  Those three are the stages
 * behind decode_attn(): a plan kernel (split schedule), a partition kernel
 * (page gather by TMA, QK^T, online fp32 softmax, PV on tensor cores) and a
 * merge kernel (log-sum-exp combine).
 *
 * Conventions.  Every function returns a da_status (0 = ok) and never throws,
 * aborts or synchronises unless it says so.  Pointers inside da_tensor are
 * DEVICE pointers unless a function says HOST.  The library allocates no
 * memory: scratch comes from the caller through decode_attn_set_workspace()
 * (one entry point, decode_attn_static_scratch(), uses a fixed array inside the
 * library image instead).  Work is
 * enqueued on the given CUDA stream and the call returns at once (the cascade
 * calls may run part of their work on two streams of the library's own, created
 * with three events at the first such call on a device and ordered inside the
 * given stream by a fork and a join: option "cascade_overlap").  Arguments a
 * host can check (NULL, dtype, shape, stride, alignment, workspace size) are
 * rejected before anything is launched.  Errors that depend on device data are
 * found on the device (never a trap, never an unbounded wait); a status record
 * is set, decode_attn_read_device_status() returns it, and the affected rows
 * are marked in the result:
 *   - a block-table entry outside [0, num_pages): that page is not read, and
 *     out and lse of every (sequence, query head) whose KV head needed it are
 *     NaN (in decode_attn_cascade(), a bad entry inside the shared prefix makes
 *     every row NaN, since every row attends it);
 *   - a length below 0, beyond its block-table row, or below what the call
 *     requires (the shared prefix, the new tokens of an extend call): the
 *     sequence is treated as empty, out = 0 and lse = -inf.
 * Other sequences of the batch are not affected.
 */
#ifndef DECODE_ATTN_H_
#define DECODE_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DA_OK = 0,
    DA_ERR_NULL = 1,         /* a required pointer is NULL                              */
    DA_ERR_SHAPE = 2,        /* ranks or extents disagree                               */
    DA_ERR_DTYPE = 3,        /* wrong element type                                      */
    DA_ERR_STRIDE_ALIGN = 4, /* last dim not contiguous, or a stride/base not 16-B aligned */
    DA_ERR_UNSUPPORTED = 5,  /* head_dim != 128, page size not in {16,32,64,128}, group > 16 */
    DA_ERR_WORKSPACE = 6,    /* no workspace registered for this device, or too small   */
    DA_ERR_CUDA = 7          /* a CUDA call failed; see decode_attn_last_cuda_error()   */
} da_status;

typedef enum { DA_BF16 = 1, DA_F32 = 2, DA_I32 = 3, DA_FP8_E4M3 = 4 /* one byte per element */ } da_dtype;

/* Device-side status codes (first word of the status record). */
typedef enum {
    DA_DEV_OK = 0,
    DA_DEV_BAD_PAGE = 1,   /* block-table entry outside [0, num_pages); that load was skipped */
    DA_DEV_BAD_SEQLEN = 2, /* seq_len < 0 or > max_pages * P; the sequence was treated as empty */
    DA_DEV_TIMEOUT = 3,    /* a bounded wait inside a kernel ran out; results are invalid  */
    DA_DEV_BOUNDS = 4      /* diagnostic build only: a kernel formed an index outside one of its own
                              arrays; record = {4, site, index, extent}; that access was skipped    */
} da_dev_status;

/* A strided view.  `stride` is in ELEMENTS.  Nothing is owned. */
typedef struct da_tensor {
    void *data;
    int32_t dtype; /* da_dtype */
    int32_t ndim;
    int64_t shape[4];
    int64_t stride[4];
} da_tensor;

/*
 * decode_attn -- the whole hot path (plan, partition, merge) on `stream`.
 *
 *   q            bf16 [B, Hq, D]          D = 128, last dim contiguous, rows 4-B aligned
 *   k_pages      bf16 [num_pages, Hkv, P, D]   any strides with a contiguous last dim; base and
 *                                         every stride a multiple of 16 bytes (so both
 *                                         [page][head][token][d] and [page][token][head][d]
 *                                         memory orders are accepted); P in {16, 32, 64, 128}
 *   v_pages      same shape and rules as k_pages (a separate pool; strides may differ)
 *   block_table  i32 [B, max_pages], last dim contiguous; entry i of row b is the physical page
 *                holding tokens [i*P, (i+1)*P) of sequence b; entries at index >= ceil(L/P) are
 *                never read
 *   seq_lens     i32 [B]; includes the token being decoded
 *   window       <= 0: attend everything; else attend the last `window` tokens, the current one
 *                included (window >= L is the same as 0)
 *   scale        multiplies q.k before the softmax
 *   out          f32 or bf16 [B, Hq, D], last dim contiguous
 *   lse          f32 [B, Hq] (natural log of the sum of exp of the scaled scores); may be NULL
 *   stream       cudaStream_t (NULL = the legacy default stream)
 *
 * Rows of K/V past a sequence's end inside its last page, pages that no block table references
 * and block-table padding may hold anything (NaN included); they do not reach the result.
 * Hq % Hkv == 0 and Hq / Hkv <= 16 are required.  The registered workspace is read and written:
 * two calls that share it must not overlap on the GPU (use one stream, or order them).
 */
int decode_attn(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages,
                const da_tensor *block_table, const da_tensor *seq_lens, int32_t window, float scale,
                da_tensor *out, da_tensor *lse, void *stream);

/*
 * decode_attn_fp8kv -- decode_attn() over a cache stored in 8 bits per element: half the bytes per
 * attended token, which is the only way past the HBM roofline of the bf16 cache.  The paper does
 * not fix a cache precision; the reading taken is the usual serving one: K and V hold FP8 E4M3
 * codes (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities, S.1111.111 = NaN,
 * largest finite value 448; "FP8 Formats for Deep Learning", Sec. 3) with one fp32 factor per KV
 * head:  K[page,g,r,:] = k_scale[g] * e4m3(k_pages[page,g,r,:]),  V likewise with v_scale[g].
 * The result is the attention of decode_attn() over those dequantised values.
 *
 *   k_pages, v_pages  DA_FP8_E4M3 [num_pages, Hkv, P, 128]; last dim contiguous, base and every
 *                     stride a multiple of 16 bytes; P in {16, 32, 64, 128}
 *   k_scale, v_scale  DEVICE float[Hkv]; NULL means all factors are 1
 *   q                 bf16, finite
 *   other arguments, workspace, status and error conventions: as decode_attn().
 *
 * Arithmetic: the codes are widened to f16 in registers (exact: every E4M3 value is an f16
 * value) and both products run as f16 tensor-core mma with fp32 accumulation.  A head's query is
 * scaled by a power of two so that its largest magnitude lies in [2^14, 2^15) and rounded to f16,
 * which is exact for every element within 2^-28 of the head's largest; the softmax runs in fp32 as in
 * decode_attn(); every weight enters the PV product as an f16 high part plus an f16 low part
 * (about 22 bits).  Observed error against the fp64 oracle: ~1e-6 on N(0,1)-like data.
 */
int decode_attn_fp8kv(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages,
                      const float *k_scale, const float *v_scale, const da_tensor *block_table,
                      const da_tensor *seq_lens, int32_t window, float scale, da_tensor *out,
                      da_tensor *lse, void *stream);

/*
 * decode_attn_cascade -- decode_attn() (full attention, no window) for a batch whose sequences all
 * START WITH THE SAME PAGES: entries 0 .. shared_prefix_tokens / P - 1 are identical in every row of
 * the block table (the sessions of the paper's agent share one long initial prompt: task rules,
 * output format and three reference kernels; Sec. 3.2 "Generate Kernel" and App. B).  The result
 * is the same as decode_attn's; only the schedule differs.  The prefix is not streamed once per
 * sequence: all B * Hq query vectors attend it together, as a (B * Hq/Hkv) x prefix score matrix
 * per KV head on the tcgen05 tensor cores (the prefix kernel), each sequence's own tokens past the
 * prefix go through the plan / partition / merge kernels as usual, and a last kernel folds the two
 * with the log-sum-exp rule.
 *
 *   shared_prefix_tokens  a multiple of 128, at most max_pages * P; <= 0 means no shared prefix
 *                         (plain decode_attn).  Every seq_lens[b] must be >= shared_prefix_tokens
 *                         (a shorter one sets DA_DEV_BAD_SEQLEN in the device status and is treated
 *                         as empty: out = 0, lse = -inf).
 *   The page ids of the prefix are read from row 0 of the block table; that the other rows agree
 *   is the caller's promise and is not checked.
 * Other arguments, results, workspace and error conventions: as decode_attn().
 */
int decode_attn_cascade(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages,
                        const da_tensor *block_table, const da_tensor *seq_lens,
                        int32_t shared_prefix_tokens, float scale, da_tensor *out, da_tensor *lse,
                        void *stream);

/*
 * decode_attn_fp8kv_cascade -- decode_attn_cascade() over the 8-bit cache of decode_attn_fp8kv(): the sessions'
 * shared initial prompt (paper Sec. 3.2 "Generate Kernel", App. B) is the largest block of cache a server
 * would keep in 8 bits.  Same result as decode_attn_fp8kv() without a window.  The tokens past the prefix go
 * through the streaming kernels' 8-bit instances; the prefix's E4M3 codes are first widened -- exactly, every
 * E4M3 value is a bf16 value -- into a bf16 copy in `prefix_scratch`, which the tensor-core kernel then
 * attends once for the whole batch, with k_scale[g] folded into the score scale and v_scale[g] into the
 * result, so no rounding is added to the dequantised values.
 *
 *   prefix_scratch        DEVICE, caller-owned, 256-byte aligned, at least
 *                         decode_attn_fp8kv_cascade_scratch_bytes(shared_prefix_tokens, Hkv, P) bytes
 *                         (= 2 x prefix tokens x Hkv x 128 x 2: K copy, then V copy); rewritten by every call,
 *                         so calls that share it must not overlap on the GPU.  Too small: DA_ERR_WORKSPACE.
 * Other arguments, requirements on shared_prefix_tokens, results, workspace and error conventions: as
 * decode_attn_cascade() and decode_attn_fp8kv().
 */
int decode_attn_fp8kv_cascade(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages,
                              const float *k_scale, const float *v_scale, const da_tensor *block_table,
                              const da_tensor *seq_lens, int32_t shared_prefix_tokens, float scale, da_tensor *out,
                              da_tensor *lse, void *prefix_scratch, size_t prefix_scratch_bytes, void *stream);
size_t decode_attn_fp8kv_cascade_scratch_bytes(int32_t shared_prefix_tokens, int32_t Hkv, int32_t P);

/*
 * decode_attn_append -- the step that precedes decode_attn() in each layer of a decoding loop:
 * writes the new token's key and value vectors into the paged cache (the per-token growth of the
 * sessions' contexts; paper Sec. 3.2, the dialog that every FSM iteration extends).
 *
 *   k_new, v_new  bf16 [B, Hkv, 128], last dim contiguous, base and strides multiples of 16 bytes
 *   k_pages, v_pages, block_table, seq_lens   as in decode_attn(); the pools are WRITTEN
 * seq_lens already counts the new token: its rows go to position L-1, i.e. page
 * block_table[b][(L-1)/P], row (L-1) % P, of every KV head.  L <= 0 writes nothing; L < 0 or a
 * position beyond the block-table row sets DA_DEV_BAD_SEQLEN, a page id outside the pool sets
 * DA_DEV_BAD_PAGE, and that sequence is skipped.  Needs a registered workspace (for the status
 * record).  One kernel on `stream`; no RoPE or other transform is applied to the vectors.
 */
int decode_attn_append(const da_tensor *k_new, const da_tensor *v_new, da_tensor *k_pages, da_tensor *v_pages,
                       const da_tensor *block_table, const da_tensor *seq_lens, void *stream);

/*
 * decode_attn_append_fp8kv -- decode_attn_append() for the 8-bit cache of decode_attn_fp8kv(): the
 * new token's bf16 K and V rows are quantised and their E4M3 codes written to position L-1:
 *     code = nearest_e4m3( x / k_scale[g] )      (v_scale[g] for V)
 * with the quotient taken in fp32 (one correctly rounded division), ties to the even mantissa,
 * magnitudes beyond 448 saturating to +-448 and NaN giving the code 0x7F.
 *   k_new, v_new      bf16 [B, Hkv, 128] as in decode_attn_append()
 *   k_pages, v_pages  DA_FP8_E4M3 pools as in decode_attn_fp8kv(); WRITTEN
 *   k_scale, v_scale  DEVICE float[Hkv], or NULL for 1
 * Status, errors and workspace as decode_attn_append().
 */
int decode_attn_append_fp8kv(const da_tensor *k_new, const da_tensor *v_new, da_tensor *k_pages,
                             da_tensor *v_pages, const float *k_scale, const float *v_scale,
                             const da_tensor *block_table, const da_tensor *seq_lens, void *stream);

/*
 * decode_attn_extend -- attention for Lq NEW tokens per sequence at once, causal among them, over
 * the same paged cache: the step that ingests a multi-thousand-token feedback prompt (compiler
 * log, tensor summary; paper Sec. 3.2 "Feedback") into an existing context, or verifies a few
 * speculated tokens.  The new tokens' K/V are already in the cache (seq_lens counts them); query
 * qi of sequence b sits at position L_b - Lq + qi and attends tokens 0 .. L_b - Lq + qi:
 *
 *     out[b,qi,h,:] = sum_{t <= L_b-Lq+qi} softmax(scale * <q[b,qi,h], K[.., t]>)_t V[.., t]
 *
 * which for Lq = 1 is decode_attn() without a window.  Two schedules, same result: with at most 16
 * query rows per KV head (Lq * Hq / Hkv <= 16: a few speculated tokens) the rows ride through the
 * plan / partition / merge kernels of decode_attn() as one wider head group, each column with its own
 * causal limit, at the HBM rate; longer query blocks run on the tcgen05 tensor cores (the same kernel
 * as the cascade's prefix pass: 128 (query, head) rows of one KV group per thread block).  Option
 * "extend_stream_rows" (0 .. 48, default 16) moves the switch; 0 always takes the tensor-core kernel.
 *
 *   q      bf16 [B, Lq, Hq, 128], last dim contiguous
 *   out    f32 or bf16 [B, Lq, Hq, 128], last dim contiguous
 *   lse    f32 [B, Lq, Hq] or NULL
 *   every seq_lens[b] must be >= Lq, or 0 (then out = 0, lse = -inf); otherwise DA_DEV_BAD_SEQLEN
 *   is set and the sequence is treated as empty.  No window.  Other arguments, workspace and
 *   conventions as decode_attn().
 */
int decode_attn_extend(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages,
                       const da_tensor *block_table, const da_tensor *seq_lens, float scale, da_tensor *out,
                       da_tensor *lse, void *stream);

/*
 * decode_attn_fp8kv_extend -- decode_attn_extend() over the 8-bit cache of decode_attn_fp8kv(), for a
 * few new tokens per sequence (speculated tokens): Lq * Hq / Hkv must not exceed 48 (else
 * DA_ERR_UNSUPPORTED: longer query blocks need the tensor-core kernel, which reads a bf16 cache; see
 * decode_attn_fp8kv_extend_wide() below).
 * Runs on the streaming kernels with per-column causal limits.  Arguments as decode_attn_extend()
 * and decode_attn_fp8kv().
 */
int decode_attn_fp8kv_extend(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages,
                             const float *k_scale, const float *v_scale, const da_tensor *block_table,
                             const da_tensor *seq_lens, float scale, da_tensor *out, da_tensor *lse,
                             void *stream);

/*
 * decode_attn_fp8kv_extend_wide -- decode_attn_fp8kv_extend() for query blocks of any length (a
 * multi-thousand-token feedback prompt ingested into a context whose cache is kept in 8 bits; Sec. 3.2,
 * "Feedback").  Up to 48 query rows per KV head it is decode_attn_fp8kv_extend().  Beyond that the pages
 * every sequence attends are first widened, exactly (every E4M3 value is a bf16 value), into a bf16 copy in
 * `scratch` -- page i of sequence b becomes page b * max_pages + i of the copy -- and the tensor-core kernel
 * of decode_attn_extend() runs over that copy; the per-KV-head factors enter in that kernel (k_scale with
 * the score scale, v_scale with the result), so the result is extend attention over the dequantised cache.
 *   scratch        DEVICE, 256-byte aligned, caller-owned.
 *                  decode_attn_fp8kv_extend_wide_scratch_bytes(B, max_pages, Hkv, P) bytes
 *                  (= 2 * B * max_pages * Hkv * P * 256: the bf16 size of what the block table can name;
 *                  pages past a sequence's end are not written or read) serve all B sequences at once; with
 *                  less, down to one sequence's share (that figure for B = 1), the sequences are served in
 *                  groups of as many as fit, one group after the other on the stream.  Less than one
 *                  sequence's share: DA_ERR_WORKSPACE; NULL: DA_ERR_NULL; misaligned: DA_ERR_STRIDE_ALIGN;
 *                  all before any launch.  May be reused by the next call on the same stream.
 * A page id outside the pool fills that page of the copy with NaN (DA_DEV_BAD_PAGE); the rows that attend
 * it come out NaN.  Other arguments and conventions as decode_attn_fp8kv_extend().
 */
int decode_attn_fp8kv_extend_wide(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages,
                                  const float *k_scale, const float *v_scale, const da_tensor *block_table,
                                  const da_tensor *seq_lens, float scale, da_tensor *out, da_tensor *lse,
                                  void *scratch, size_t scratch_bytes, void *stream);
size_t decode_attn_fp8kv_extend_wide_scratch_bytes(int32_t B, int64_t max_pages, int32_t Hkv, int32_t P);

/*
 * decode_attn_host_io -- the same call for a caller whose per-step tensors are in HOST memory.
 * q, block_table, seq_lens, out and lse are HOST views (pinned memory makes the copies
 * asynchronous; they must stay valid until the stream reaches the end of the call); k_pages and
 * v_pages stay DEVICE views (the cache is resident state).  The inputs are staged into the
 * registered workspace with cudaMemcpyAsync, decode_attn() runs on the staged copies, and out/lse
 * are copied back, all on `stream`, without synchronising.  Host views must be contiguous.  Pinned,
 * mapped input buffers are gathered into the staging area by one kernel instead of three copies.  If out
 * and lse are pinned memory that is mapped into the device's address space (cudaHostAlloc /
 * cudaHostRegister under unified addressing, which is what torch's pin_memory() gives), the kernels
 * write them directly instead of going through staging and a copy; the results are complete when
 * the stream reaches the end of the call either way.
 */
int decode_attn_host_io(const da_tensor *q_host, const da_tensor *k_pages, const da_tensor *v_pages,
                        const da_tensor *block_table_host, const da_tensor *seq_lens_host,
                        int32_t window, float scale, da_tensor *out_host, da_tensor *lse_host,
                        void *stream);

/* The same for the 8-bit cache of decode_attn_fp8kv(): k_pages / v_pages and the factors stay on the DEVICE. */
int decode_attn_fp8kv_host_io(const da_tensor *q_host, const da_tensor *k_pages, const da_tensor *v_pages,
                              const float *k_scale, const float *v_scale, const da_tensor *block_table_host,
                              const da_tensor *seq_lens_host, int32_t window, float scale,
                              da_tensor *out_host, da_tensor *lse_host, void *stream);

/*
 * decode_attn_static_scratch -- decode_attn() for callers that cannot allocate device memory.
 * (The paper has no counterpart; this is a packaging variant of the same kernels.)
 *
 * Who needs it: an inference server that hands every free byte of HBM to its KV-cache pool at
 * start-up has nothing left for a later cudaMalloc, and a caller in the middle of a decode step
 * cannot afford cudaMalloc's device-wide synchronisation; neither may have an allocator whose
 * buffer it could register with decode_attn_set_workspace().  This entry point needs no registered
 * workspace and calls no cudaMalloc, cudaFree or any allocating routine: the plan arrays, the
 * split partials and the status record live in one fixed 6 MiB array that is part of the library
 * image (every GPU that loads the library holds those 6 MiB until the process exits).
 *
 * Arguments and results are those of decode_attn(), plus
 *   dev_status4  DEVICE int32[4], may be NULL: receives the device status record of THIS call
 *                ({da_dev_status code, sequence, block-table index, value}; all zero = clean),
 *                copied on `stream` after the kernels.
 * Limits: B <= 4096 sequences and at most 320 thread blocks in the partition kernel (the default
 * of two per SM on a B200 is 296); beyond either, or if the layout would exceed the 6 MiB, the
 * call returns DA_ERR_WORKSPACE and launches nothing.  To keep the split partials inside the
 * array, the work is cut into one static range per thread block only (as with "tail_units" 0).
 *
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 * that device current); make that first call outside any stream capture.  When the 6 MiB are
 * reserved: when the CUDA runtime loads this library's device code on that device -- with lazy
 * module loading that is the first library call on it that launches a kernel or looks up a
 * symbol, not process start.  A server that sizes its KV pool from "all the memory that is free" should therefore
 * make one library call on each device (this one with B = 0 will do) BEFORE it measures free memory,
 * or that first call can itself fail with an out-of-memory error.  All calls on a device
 * share the one array, which still holds the previous call's contents when the next one starts
 * (the call clears the only part that must start at zero, its status record): two calls that
 * overlap on the GPU race on it, so keep them on one stream or order them yourself.
 */
int decode_attn_static_scratch(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages,
                               const da_tensor *block_table, const da_tensor *seq_lens, int32_t window,
                               float scale, da_tensor *out, da_tensor *lse, int32_t *dev_status4,
                               void *stream);

/*
 * Scratch.  decode_attn_workspace_bytes() says how much device memory a call with these extents
 * needs on the current device with the current launch options (split partials, the plan, a status
 * record, and staging room for decode_attn_host_io).  decode_attn_set_workspace() registers a
 * caller-owned, 256-B aligned device buffer for the current device (one per device, process-wide)
 * and clears its status record with a cudaMemsetAsync on the legacy default stream followed by a
 * synchronize.  Passing NULL unregisters.
 */
size_t decode_attn_workspace_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t D, int32_t P,
                                   int64_t max_pages);
int decode_attn_set_workspace(void *dev_ptr, size_t bytes);

/*
 * decode_attn_read_device_status -- synchronises `stream`, copies the 4-word status record
 * {da_dev_status code, sequence index, block-table index, page id or length} of the current
 * device's workspace to HOST memory and clears it on the device.  All zero = clean.
 */
int decode_attn_read_device_status(void *stream, int32_t *host_status4);

/*
 * decode_attn_plan -- runs only the plan kernel (the split schedule of the partition kernel) and
 * copies it to HOST arrays, synchronising `stream`.  A debugging and test aid: it shows which
 * token ranges each work unit covers.  Units 0 .. num_static-1 are the ranges the thread blocks
 * of the partition kernel start on; the others are handed out through a ticket counter as blocks
 * finish.
 *   seq_lens        DEVICE i32 [B] view
 *   host_seq_info   HOST int32 [B][4]: {lo, L, first_tile, num_tiles}; a tile is tile_tokens
 *                   consecutive tokens starting at a multiple of tile_tokens
 *   host_unit_work  HOST int32 [capacity][4]: {b, kv_head, first tile of that pair relative to its
 *                   first_tile, number of tiles}; a unit walks forward from there through
 *                   (b, kv_head) pairs in row-major order
 *   num_units       HOST in: capacity of host_unit_work in rows (8192 always suffices);
 *                   out: units in use
 *   num_static      HOST out: the partition kernel's grid size
 *   tile_tokens     HOST out
 */
int decode_attn_plan(const da_tensor *seq_lens, int32_t window, int32_t Hkv, int32_t P,
                     int64_t max_pages, int32_t *host_seq_info, int32_t *host_unit_work,
                     int32_t *num_units, int32_t *num_static, int32_t *tile_tokens, void *stream);

/*
 * Launch options, for tests and tuning.  Every setting gives the same result up to fp32 rounding;
 * they change how sequences are split.
 *   "grid_blocks"  thread blocks of the partition kernel (0 = two per SM, at most 4096)
 *   "tail_units"   work units per thread block that are handed out by ticket after the static
 *                  ranges (0 .. 64, default 4; 0 = static ranges only)
 *   "static_frac"  share of the work, in 1/256, covered by the static ranges (default 224)
 *   "extend_stream_rows"  decode_attn_extend(): most query rows per KV head that go through the
 *                  streaming kernels instead of the tensor-core kernel (0 .. 48, default 16; beyond 16 rows
 *                  the thread blocks carry a second set of consumer warps for the further columns)
 *   "fold_pairs"   a (sequence, KV head) pair that the own ranges of two neighbouring thread blocks cut in
 *                  two can be folded by the partition kernel itself -- by whichever of the two blocks finishes
 *                  its piece second -- instead of by the merge kernel after the last block.  0 never, 1 always,
 *                  2 (default) in the host-buffer calls only: on the device the two ways take the same time,
 *                  but results that cross PCIe then leave while the batch is still streaming instead of
 *                  all at the end (c2 from host buffers: 0.376 -> 0.358 ms).
 *   "cascade_overlap"  decode_attn_cascade / decode_attn_fp8kv_cascade: whether the tensor-core pass over
 *                  the shared prefix runs BESIDE the HBM-bound pass over the sequences' own tokens -- the prefix
 *                  kernel on about a third of the SMs ("cascade_prefix_sms", 0 = a third), the other kernels on
 *                  the rest, joined by the prefix kernel's SMs when it ends -- or before it on all SMs.  Side
 *                  by side, the second pass is launched on a stream of the library's own (made, with two
 *                  events, at the first such call on a device: the one thing the library creates besides its
 *                  kernels), forked from `stream` at the start of the call and joined to it before the final
 *                  merge, so the call is still ordered on `stream` like any other and can be captured into a
 *                  CUDA graph.  0 never; 1 (default) when (row tiles x KV heads) fits half of the SMs and the
 *                  host's estimate says the second pass lasts at least as long as the first on its share (the
 *                  host cannot see the lengths: it assumes a sequence's own part is half of what its
 *                  block-table row can hold beyond the prefix); 2 whenever the shapes allow.  A caller whose
 *                  sequences are much shorter than their block-table rows should say 0.  While "grid_blocks"
 *                  is not 0, or profile events are set, the passes run one after the other.
 *   "direct_path"  1 (default): a call small enough that every (sequence, KV head) pair, cut into at most
 *                  eight pieces of at most eight tiles, fits one wave of thread blocks (judged from B, the
 *                  block table's width and the window, since the lengths are on the device) runs as ONE
 *                  kernel: each block derives its piece from seq_lens itself and the block that finishes a
 *                  pair last folds the pieces.  0: always plan + partition + merge.  Only taken while
 *                  "grid_blocks" is 0.
 *   "kv_evict_first"  L2 priority of the K and V page loads: 1 = "evict first" (pages that are read
 *                  once do not push the query rows, block table, plan and partial results out of L2),
 *                  0 = normal (better when sequences share pages, which are then re-read from L2),
 *                  2 = chosen per call on the device (default): normal when at least a quarter of the
 *                  non-empty sequences start on the same physical page as the first sequence or as
 *                  their predecessor in the batch, else evict first.  Results do not depend on it.
 * The diagnostic build of the library (the same sources compiled with -DDA_TIMELINE -DDA_DIAG
 * -DDA_BOUNDS_CHECK into a second shared object; the normal library knows none of these names) adds
 *   "diag_wait_limit_us"  how long a bounded wait inside a kernel lasts before it gives up with
 *                  DA_DEV_TIMEOUT (default 2,000,000 = the normal build's fixed 2 s)
 *   "diag_withhold_partition_tile", "diag_withhold_prefix_tile"   tile number (counted per thread
 *                  block, from 0) whose copies AND barrier arrival the loader of thread block 0 leaves
 *                  out in the partition / prefix kernel; -1 (default) = none.  Nothing is issued for that
 *                  tile, so the warps waiting for it run into the limit above and the kernel leaves
 *                  through its give-up path: a way to test that path without faulting or hanging the
 *                  device.  The results of such a call are invalid; the next call is unaffected.
 * and checks every index its kernels form into their own arrays (DA_DEV_BOUNDS).
 * Returns DA_ERR_UNSUPPORTED for an unknown name or a value out of range.
 */
int decode_attn_set_option(const char *name, int64_t value);
int64_t decode_attn_get_option(const char *name);

/*
 * decode_attn_set_profile_events -- timing aid.  While both handles are non-NULL, every
 * decode_attn() call records `before` (a cudaEvent_t) on its stream just before the partition
 * kernel's launch and `after` just after it, so that a benchmark can time that kernel alone
 * (decode_attn_cascade() brackets its prefix kernel instead).
 * Pass NULL, NULL to stop.  The events stay owned by the caller.
 */
int decode_attn_set_profile_events(void *before, void *after);

/*
 * decode_attn_timeline -- diagnostic build only (the same sources compiled with -DDA_TIMELINE,
 * -DDA_DIAG and -DDA_BOUNDS_CHECK into a second library; the normal library returns
 * DA_ERR_UNSUPPORTED and keeps no stamps).  In that build the plan, partition and merge kernels leave global-timer stamps (ns) of
 * their most recent launch in a device table; this call waits for the device, copies the table to
 * `host_out` and, if `clear` is non-zero, zeroes it.
 *   host_out   HOST, DECODE_ATTN_TIMELINE_ROWS x DECODE_ATTN_TIMELINE_COLS values, row-major:
 *              rows 0..1023 = thread blocks of the partition kernel (columns: 0 entry, 1 past the wait
 *              for the plan, 2 first tile ready, 3 last tile consumed, 4 exit, 5 tiles consumed,
 *              6 (sequence, KV head) items finished); rows 1024..1031 = the merge kernel's first eight
 *              blocks (0 resident, 1 released, 2 exit); row 1032 column 2 = the last merge block's
 *              exit; rows 1036..1051 = the plan kernel's blocks (0 entry, 1 exit, 2 past the wait for the
 *              kernel before it in the stream, 3 lengths scanned, 4 cut made, 5 units written);
 *              rows 1052..1057 = thread block 0 of the prefix kernel (decode_attn_cascade, decode_attn_extend),
 *              CYCLES one warp of each role spent in its phases, summed over the block's tiles: 1052 a softmax
 *              warp (0 waiting for scores, 1 loading them and agreeing on row maxima, 2 weights, 3 storing P,
 *              4 after the last tile, 5 tiles, 6 cycles entry to end, 7 the same span in ns), 1053 the score
 *              MMA warp (0 waiting for the PV products, 1 for K, 2 issuing), 1054 / 1055 the PV MMA warps
 *              (0 waiting for P, 1 for V, 2 issuing), 1056 / 1057 the K / V loader warps (0 waiting for a
 *              free buffer, 1 issuing copies)
 *   capacity   values `host_out` can hold; DA_ERR_SHAPE if fewer than rows x cols
 */
#define DECODE_ATTN_TIMELINE_ROWS 1064
#define DECODE_ATTN_TIMELINE_COLS 8
int decode_attn_timeline(unsigned long long *host_out, int64_t capacity, int32_t clear);

const char *decode_attn_strerror(int status);
int decode_attn_last_cuda_error(void); /* cudaError_t of the last failing CUDA call, else 0 */
int decode_attn_version(void);
/* Kernel launches issued by this library since load (a counter for benchmarks). */
int64_t decode_attn_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* DECODE_ATTN_H_ */
