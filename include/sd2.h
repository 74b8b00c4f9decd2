/*
 * sd2.h -- C ABI of libsd2: decode-time sparse linears of an SD^2 draft model
 * on one NVIDIA B200 (sm_100a).
 *
 * The operation.  A fine-grained-sparse drafter keeps, for every decoder-block
 * linear (q, k, v, o, gate, up, down), a weight W of shape (C_out, C_in) =
 * [M x K] and a fixed binary mask; pruned weights are exactly zero and stay so
 * (paper, Section "Sparse fine-tuning"; W's shape: Appendix "Non-uniform
 * layer-wise sparsity distributions").  Turning that sparsity into latency
 * needs "efficient sparse representations and kernels" (Section "Compressed
 * sparse drafters"); the paper specifies neither, so both are designed here.
 * Every entry point below computes, or prepares,
 *
 *        Y[n, m] = sum over kept k of  W[m, k] * X[n, k]        (Y = X (W.*mask)^T)
 *
 * with bf16 inputs, fp32 accumulation and one rounding at the output.
 *
 * Conventions
 *  - All matrices are row-major and dense in memory: W [M*K], mask [M*K],
 *    X [N*K], Y [N*M].  bf16 values are passed as their 16-bit patterns.
 *  - "host" / "device" on a pointer says where the memory must live.
 *  - Every call returns an sd2_status; nothing throws or aborts.  Output
 *    arguments are written only on SD2_OK.
 *  - The caller owns every buffer it passes.  The library owns a handle's
 *    memory (host and device) from sd2_compress / sd2_load_blob to sd2_free.
 *  - sd2_spmm, sd2_spmm_fused and sd2_block_step are asynchronous on the given
 *    stream, allocate nothing, never synchronise, overwrite their outputs
 *    (beta = 0, no bias) and may run concurrently on different streams.  A launch
 *    failure is reported as SD2_ERR_CUDA by the call that made it.
 *  - sd2_compress, sd2_load_blob, sd2_decompress and sd2_free may synchronise.
 *  - There is no CPU fallback: without a CUDA device the device entry points
 *    return SD2_ERR_CUDA.  sd2_pack_host / sd2_unpack_host need no device.
 */
#ifndef SD2_H
#define SD2_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sd2_handle_s* sd2_handle;   /* opaque; one compressed weight; owned by the library */
typedef struct sd2_drafter_s* sd2_drafter; /* opaque; a chain of drafter blocks; owned by the library */

typedef enum {
    SD2_OK = 0,
    SD2_ERR_INVALID_ARG = -1, /* NULL pointer, bad option, dead or unknown handle        */
    SD2_ERR_SHAPE = -2,       /* non-positive or inconsistent dimensions                 */
    SD2_ERR_ALLOC = -3,       /* host or device allocation failed                        */
    SD2_ERR_CUDA = -4,        /* CUDA runtime error (no device, launch failure, ...)     */
    SD2_ERR_UNSUPPORTED = -5, /* valid request this build cannot serve (e.g. huge K)     */
    SD2_ERR_CORRUPT = -6,     /* a blob failed validation                                */
    SD2_ERR_TIMEOUT = -7      /* a bounded device-side wait ran out (sd2_stream_check)   */
} sd2_status;

/* Compressed formats.  Both are lossless; "compressed bytes" always counts every
 * byte the kernels must read for W: values, position metadata and row offsets. */
enum {
    SD2_FORMAT_AUTO = 0,    /* library picks (currently SD2_FORMAT_GAP4 when it applies)    */
    SD2_FORMAT_BITMASK = 1, /* 1 bit per dense slot + packed kept values + row offsets    */
    SD2_FORMAT_GAP4 = 2,    /* 4-bit column gaps + packed kept values in 8-entry chunks,  */
                            /* rows cut into column strips, 32 strips to a tile (the fast */
                            /* path; column strips wider than 496 are not supported)      */
    SD2_FORMAT_GAP4_PAIRED = 3,/* as an option of sd2_pack_host / sd2_compress only: GAP4 */
                            /* whose rows 2i and 2i+1 stay next to each other in a tile   */
                            /* (for a stack that interleaves gate row i and up row i; M   */
                            /* even and at least two rows per tile, else UNSUPPORTED).    */
                            /* The blob and the handle report SD2_FORMAT_GAP4.            */
    SD2_FORMAT_GAP4_MMA = 4 /* for panels of N >= 16 activation rows: 128 x 128 blocks    */
                            /* whose 4-bit gaps run in the order of a tensor-core operand */
                            /* tile; sd2_spmm expands each block in shared memory and     */
                            /* multiplies it on the tensor cores (tcgen05.mma, fp32       */
                            /* accumulators in tensor memory).  Any N is accepted (rows   */
                            /* are taken 64 at a time, padded to a multiple of 16); never */
                            /* picked by AUTO; not accepted by sd2_block_step or a        */
                            /* drafter.  Calls on one handle must not overlap on the GPU: */
                            /* they share the handle's partial-sum buffer.                */
};

enum { SD2_DTYPE_BF16 = 0, SD2_DTYPE_F32 = 1 };

typedef struct {
    int32_t format;  /* SD2_FORMAT_*                                  */
    int32_t y_dtype; /* SD2_DTYPE_*: element type of Y for this weight */
} sd2_options;

/* ---- format builder on the host (no device needed) ----------------------------------- */

/* Encode W.*mask into a self-describing byte blob (the exact image sd2_compress uploads).
 *   weight_bf16 : host, [M*K] bf16 patterns.
 *   mask        : host, [M*K] bytes, non-zero = kept; NULL = keep every weight that is
 *                 not +0/-0.  The mask is authoritative: a kept weight may be zero, NaN or
 *                 Inf and survives bit for bit; a masked-out weight never takes part.
 *   opt         : NULL = {AUTO, BF16}.
 *   blob, blob_bytes : out; release with sd2_blob_free.
 * Errors: INVALID_ARG (NULL weight/out, unknown format), SHAPE (M or K < 1, or a size
 * that overflows the format's 32-bit offsets), ALLOC. */
sd2_status sd2_pack_host(const void* weight_bf16, const uint8_t* mask, int64_t M, int64_t K,
                         const sd2_options* opt, void** blob, int64_t* blob_bytes);

/* Validate a blob and decode it.  dense_bf16_out (host, [M*K]) may be NULL to only query;
 * every other out pointer may be NULL.  Decoding yields W with masked-out entries +0.
 * Errors: INVALID_ARG, CORRUPT (bad magic, sizes, offsets, checksum or metadata). */
sd2_status sd2_unpack_host(const void* blob, int64_t blob_bytes, void* dense_bf16_out,
                           int64_t* M, int64_t* K, int64_t* nnz, int64_t* compressed_bytes,
                           int32_t* format);

sd2_status sd2_blob_free(void* blob);

/* ---- handles ------------------------------------------------------------------------- */

/* Compress once per weight (the topology is static), copy to the current device.
 * weight_bf16 and mask may each be host or device memory. */
sd2_status sd2_compress(const void* weight_bf16, const uint8_t* mask, int64_t M, int64_t K,
                        const sd2_options* opt, sd2_handle* out);

/* Make a handle from a blob produced by sd2_pack_host (host memory). */
sd2_status sd2_load_blob(const void* blob, int64_t blob_bytes, sd2_handle* out);

/* Read the device copy back and decode it: dense_bf16_out ([M*K], host or device)
 * receives W.*mask bit-exactly (masked-out entries +0). */
sd2_status sd2_decompress(sd2_handle h, void* dense_bf16_out);

/* Any out pointer may be NULL. */
sd2_status sd2_info(sd2_handle h, int64_t* M, int64_t* K, int64_t* nnz,
                    int64_t* compressed_bytes, int32_t* format);

/* NULL, unknown or already freed handle -> SD2_ERR_INVALID_ARG (no crash). */
sd2_status sd2_free(sd2_handle h);

/* ---- the hot path -------------------------------------------------------------------- */

/* Y = X (W.*mask)^T.   X: device bf16 [N*K].   Y: device [N*M], bf16 or fp32 per the
 * handle's y_dtype.  N = 0 is a no-op; more than 8 rows (GAP4: fewer where the staged rows of a
 * wide layer would crowd the weight ring out of shared memory, e.g. 4 for K = 8192) are processed
 * in panels of at most that many rows of X (the weight is re-read for each panel).  cuda_stream is a
 * cudaStream_t (NULL = default stream).  X and Y need only their natural alignment; all
 * activations are expected to be finite (a filler entry of the GAP4 format multiplies +0 by
 * the activation of a masked-out column). */
sd2_status sd2_spmm(sd2_handle h, const void* X, void* Y, int64_t N, void* cuda_stream);

/* Same-input fusion (q|k|v, gate|up): count <= 4 weights with equal K share one staged X
 * and one launch.  Y[i] is device [N*M_i] with handle i's y_dtype. */
sd2_status sd2_spmm_fused(const sd2_handle* h, int32_t count, const void* X, void* const* Y,
                          int64_t N, void* cuda_stream);

/* One drafter block's seven linears in dependency order, h = {q,k,v,o,gate,up,down}
 * (a block is a self-attention module followed by a feed-forward module: Section "Layer
 * pruning").  Only the linears are on this path; the glue between them is a documented
 * stub, every intermediate rounded to bf16 (round-to-nearest-even):
 *     q = Wq x, k = Wk x, v = Wv x        (one fused launch; k, v stay in the workspace)
 *     a = q                                (attention stub: identity)
 *     hdn = Wo a
 *     g = Wg hdn, u = Wu hdn               (one fused launch)
 *     t = bf16(silu(g) * u)                (silu in fp32)
 *     y = Wd t
 * x: device bf16 [N*hidden]; y: device [N*M_down] in h[6]'s y_dtype.
 * workspace: device, sd2_block_workspace_bytes bytes, 256-byte aligned; after the call it
 * holds, in this order and each [N*dim] bf16, 256-byte aligned: q, k, v, hdn, g, u, t.
 * With seven GAP4 weights the block is ONE launch: a persistent CTA per SM runs the stages
 * one after another, separated by grid-wide barriers, while a producer warp keeps copying the
 * coming stages' weights into shared memory.  Such launches take every SM; two of them should
 * not be put on different streams in the hope of overlap.
 * Errors: SHAPE if the seven shapes do not chain, or N outside [0, 65536].  Any N in that range
 * is served: rows are independent and go through the block in panels of at most 8. */
sd2_status sd2_block_step(const sd2_handle* h, const void* x, void* y, int64_t N,
                          void* workspace, void* cuda_stream);

sd2_status sd2_block_workspace_bytes(const sd2_handle* h, int64_t N, int64_t* bytes);

/* Byte offsets of q, k, v, hdn, g, u, t inside the workspace (offsets[7]). */
sd2_status sd2_block_workspace_layout(const sd2_handle* h, int64_t N, int64_t* offsets);

/* sd2_block_step for callers that must not allocate device memory and have no workspace
 * to hand over.  (No counterpart in the paper: it exists for hosts such as a serving loop
 * that runs under a fixed memory plan, a plugin inside another runtime's allocator, or code
 * on a path where cudaMalloc's implicit device synchronisation is not acceptable.)  The
 * block's intermediates (q, k, v, hdn, g, u, t) and the grid-barrier words live in an array
 * built into the library image: 1 MiB + 256 bytes that every GPU which loads the library
 * keeps until the process exits.  Same result as sd2_block_step, same stub glue; x: device
 * bf16 [N*hidden], y: device [N*M_down] in h[6]'s y_dtype, N >= 0.
 *  - all seven weights must be GAP4 (SD2_ERR_UNSUPPORTED otherwise), live on the current device;
 *  - sd2_block_workspace_bytes(h, N) must not exceed 1 MiB, else SD2_ERR_UNSUPPORTED and
 *    nothing is launched (e.g. a Llama-3.2-3B block fits up to N = 16);
 *  - the first call on each device looks up the array's device address; make that call
 *    before any stream capture;
 *  - the call itself enqueues a 256-byte clear of the barrier words and then the launches;
 *    it calls no allocation routine;
 *  - every call uses the same array, and the intermediates of the previous call stay in it
 *    until overwritten: two calls that overlap on the GPU (different streams, no ordering)
 *    race on it.  Keep calls on one stream or order them with events.  The intermediates
 *    cannot be read back through this entry point. */
sd2_status sd2_block_step_static(const sd2_handle* h, const void* x, void* y, int64_t N, void* cuda_stream);

/* ---- a whole drafter: L blocks chained, one launch per panel of activation rows --------- */

/* h: 7 * L live GAP4 handles on the current device, block by block in the order q,k,v,o,gate,
 * up,down; block b+1 reads block b's output (rounded to bf16), so out(b) must equal
 * hidden(b+1).  n_max in [1, 64] sizes the intermediate buffers, which the drafter owns.
 * The handles must outlive the drafter.  May synchronise; allocates device memory.
 * Where the shapes allow it the drafter keeps its own paired copy of every block's gate and up
 * (one stacked GAP4 matrix, gate row i and up row i side by side, as large as the two
 * together), built here on the host from the handles' decoded contents, so that a step forms
 * t = silu(g) * u where g and u are produced.  That copy is device memory on top of the handles'
 * (about 55 % more for a Llama-shaped block: gate and up are most of its weights);
 * sd2_drafter_query reports what the drafter holds and what a step streams.
 * Errors: INVALID_ARG, SHAPE (shapes do not chain, L or n_max out of range), UNSUPPORTED (a
 * handle is not GAP4, or a layer is too wide for shared memory), ALLOC. */
sd2_status sd2_drafter_create(const sd2_handle* h, int32_t L, int64_t n_max, sd2_drafter* out);

/* One token step through all L blocks: x device bf16 [N*hidden], y device [N*out] in the
 * last down projection's y_dtype, 0 <= N <= n_max.  Same stub glue as sd2_block_step.
 * Asynchronous on the stream, allocates nothing.  Steps of one drafter must not overlap in
 * time (they share its buffers): keep them on one stream. */
sd2_status sd2_drafter_step(sd2_drafter d, const void* x, void* y, int64_t N, void* cuda_stream);

/* Facts about a drafter and a step of N rows (1 <= N <= n_max), out[6]:
 *   out[0] kernel launches the step makes (one per panel of rows), out[1] rows of the widest panel,
 *   out[2] device bytes the drafter owns (paired stacks, intermediates, tagged words, stage table),
 *   out[3] bytes of compressed weights one launch reads (paired stacks in place of the gate and up
 *          handles they replace), out[4] stages of a launch, out[5] kept weights of all handles. */
sd2_status sd2_drafter_query(sd2_drafter d, int64_t N, int64_t* out);

/* Device addresses of block `block`'s buffers after a step, ptrs[8] = q, k, v, hdn, g, u, t and
 * the block's bf16 output (not written for the last block, whose output goes to y).  Each is
 * [n_max rows capacity] with row n at n * width. */
sd2_status sd2_drafter_buffers(sd2_drafter d, int32_t block, void** ptrs);

sd2_status sd2_drafter_free(sd2_drafter d);

/* Wait for the stream and report device-side trouble: kernels bound every wait on an
 * asynchronous copy; one that runs out raises an error word instead of hanging.  Returns
 * SD2_ERR_TIMEOUT (and clears the word) if that happened since the last check, SD2_ERR_CUDA
 * if the stream itself failed, SD2_OK otherwise.  Synchronises; not for the hot loop. */
sd2_status sd2_stream_check(void* cuda_stream);

/* Diagnostic for the bounded waits (the paper has no counterpart): launches one warp that waits
 * on a barrier nothing ever signals, with the budget every device-side wait of this library has
 * (2 s of SM clock, or SD2_WAIT_MS milliseconds from the environment).  The wait runs out, the
 * kernel ends normally and the next sd2_stream_check returns SD2_ERR_TIMEOUT once.  Asynchronous. */
sd2_status sd2_selftest_timeout(void* cuda_stream);

/* ---- glue of a whole decode step (the parts of a drafter forward pass that are not sparse linears) ----
 *
 * The paper prunes the decoder blocks and leaves the embedding and the LM head dense (Section
 * "Results"); a block is a self-attention module and a feed-forward module (Section "Layer
 * pruning").  What those compute is not restated there: the calls below follow the published
 * definitions of the Llama / Qwen family.  All tensors are device memory, bf16 bit patterns unless
 * said otherwise, row-major; fp32 arithmetic, one rounding per output.  Asynchronous on the stream,
 * no allocation.  Errors: INVALID_ARG (NULL pointer), SHAPE (non-positive or inconsistent sizes),
 * UNSUPPORTED (limits named per call), CUDA. */

/* y[n, :] = x[n, :] / sqrt(mean(x[n, :]^2) + eps) * w.   x, y [N*H]; w [H].  y may be x. */
sd2_status sd2_rmsnorm(const void* x, const void* w, void* y, int64_t N, int64_t H, float eps, void* cuda_stream);

/* The residual connection and the norm that follows it, in one launch: sum = a + b (rounded to bf16), y = the
 * sd2_rmsnorm of sum with gain w.  a, b, sum, y [N*H]; sum may be a or b; y must not overlap sum. */
sd2_status sd2_add_rmsnorm(const void* a, const void* b, void* sum, const void* w, void* y, int64_t N, int64_t H, float eps,
                           void* cuda_stream);

/* Rotary embedding of one new token per row at position `pos` (pairs (i, i + head_dim/2) of a head
 * turn by pos * theta^(-2i/head_dim)), and the cache append: q [N, heads_q, head_dim] is rotated in
 * place; the rotated k and the plain v ([N, heads_kv, head_dim]) are written to position `pos` of
 * row n's cache, k_cache / v_cache [N, T_max, heads_kv, head_dim].  head_dim even, pos < T_max.
 * UNSUPPORTED: head_dim > 128.  The angles are computed on the host (fp64) at the call. */
sd2_status sd2_rope_cache(void* q, const void* k, const void* v, void* k_cache, void* v_cache, int64_t N, int64_t heads_q,
                          int64_t heads_kv, int64_t head_dim, int64_t pos, int64_t T_max, double theta, void* cuda_stream);

/* Grouped-query attention of one new token per row over the first T cached positions (its own
 * included): query head h reads key/value head h / (heads_q / heads_kv); scores q.k / sqrt(head_dim),
 * softmax over the T positions, out = sum of weights times values.  q, out [N, heads_q, head_dim].
 * UNSUPPORTED: head_dim > 128 or T > 8192. */
sd2_status sd2_attention_decode(const void* q, const void* k_cache, const void* v_cache, void* out, int64_t N, int64_t heads_q,
                                int64_t heads_kv, int64_t head_dim, int64_t T, int64_t T_max, void* cuda_stream);

/* sd2_rope_cache followed by sd2_attention_decode over positions 0..pos, in one launch: q is rotated in place, the
 * rotated k and v are appended at `pos`, out [N, heads_q, head_dim] is the attention output.  Same limits as the two. */
sd2_status sd2_rope_attention(void* q, const void* k, const void* v, void* k_cache, void* v_cache, void* out, int64_t N,
                              int64_t heads_q, int64_t heads_kv, int64_t head_dim, int64_t pos, int64_t T_max, double theta,
                              void* cuda_stream);

/* y = a + b over `count` elements (residual connection).  y may be a or b. */
sd2_status sd2_add(const void* a, const void* b, void* y, int64_t count, void* cuda_stream);

/* x[n, :] = table[tokens[n], :].  tokens: device int32 [N]; table [V*H]; a token outside [0, V) gives a zero row. */
sd2_status sd2_embedding(const int32_t* tokens, const void* table, void* x, int64_t N, int64_t V, int64_t H, void* cuda_stream);

/* Dense LM head: logits[n, v] = sum over h of w_out[v, h] * x[n, h] (fp32 out, device [N*V]), and, if
 * tokens is not NULL (device int32 [N]), the greedy token of each row: the index of the largest logit,
 * the lowest index among equals.  w_out [V*H] bf16, 16-byte aligned.  UNSUPPORTED: H not a multiple of 8. */
sd2_status sd2_lm_head(const void* x, const void* w_out, float* logits, int32_t* tokens, int64_t N, int64_t V, int64_t H,
                       void* cuda_stream);

/* One whole decoder block for one new token per row:
 *     x1 = x  + Wo attention(rope(Wq n), cache + rope(Wk n), cache + Wv n),   n = rmsnorm(x,  norm_attn)
 *     y  = x1 + Wd (silu(Wg m) * Wu m),                                        m = rmsnorm(x1, norm_ffn)
 * h[7] = q, k, v, o, gate, up, down handles.  With seven GAP4 handles the block is four launches: q|k|v with
 * the first norm folded into their activation staging; rotation, cache append and attention; o, gate|up and
 * down as one persistent launch with the residual and the second norm folded into gate|up's staging; the last
 * residual.  Other formats take one launch per operation (8 per block).  Every intermediate is rounded to bf16.  x, y [N*hidden]; caches as in sd2_rope_cache; the
 * block writes position `pos` of them and attends over positions 0..pos.  workspace: device, 256-byte
 * aligned, sd2_decoder_workspace_bytes(h, N) bytes; it holds, in this order, q, k, v, o-projection,
 * gate, up, t (offsets of sd2_block_workspace_layout), then n/m, x1, the attention output and the down
 * projection (each rounded up to 256 bytes), which tests read back. */
sd2_status sd2_decoder_workspace_bytes(const sd2_handle* h, int64_t N, int64_t* bytes);
sd2_status sd2_decoder_block_step(const sd2_handle* h, const void* norm_attn, const void* norm_ffn, const void* x, void* y,
                                  void* k_cache, void* v_cache, int64_t N, int64_t heads_q, int64_t heads_kv, int64_t pos,
                                  int64_t T_max, float eps, double theta, void* workspace, void* cuda_stream);

/* Failure injection for tests (the paper has no counterpart): the next `skip` allocations the library makes
 * for itself (host blobs and staging copies, handle and drafter objects, device memory) succeed, the `fail`
 * after them fail as if memory had run out; (0, 0) switches it off.  A call that meets a failed allocation
 * returns SD2_ERR_ALLOC and releases what it had taken.  Process-wide, not meant for concurrent use. */
sd2_status sd2_debug_fail_allocations(int64_t skip, int64_t fail);

/* Static string for a status code. */
const char* sd2_status_string(sd2_status s);

#ifdef __cplusplus
}
#endif
#endif /* SD2_H */
