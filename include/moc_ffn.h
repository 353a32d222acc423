/*
 * moc_ffn.h -- C ABI of the B200 (sm_100a) Mixture-of-Channels FFN operator.
 *
 * The operator (paper Section 3.2, Eqs. (Moc-1), the Top-K mask, (MoC-2)):
 *     G = X W_gate,  M = TopK_row(G),  S' = SiLU(G) . M,  Z' = S' . U on M (U = X W_up),  D = Z' W_down
 * Only the K selected channels of every token are formed, and only the compact triple
 * (channel index, gate value, up value) is kept for the backward pass (Section 4, Table 1,
 * column "MoC+GCP": G.M, U.M and M stored; S.M and Z.M recomputed).
 *
 * Conventions that hold for every entry point
 * -------------------------------------------
 * Pointers   All data pointers are DEVICE pointers on the current CUDA device, 16-byte aligned;
 *            `desc` is a HOST pointer; `cuda_stream` is a cudaStream_t passed as void* (NULL = the
 *            legacy default stream).  The caller owns every buffer, including the workspace.  The
 *            library allocates no device memory.
 * Layouts    x, out, grad_out, grad_x : [tokens, d_model] row-major.
 *            w_gate, w_up, w_down and their gradients : CHANNEL-MAJOR [d_ff_ld, d_model] row-major,
 *            row j = the d_model-vector of channel j.  For gate/up that is column j of the paper's
 *            W in R^{d x d_ffn}; for down it is row j of the paper's W_down in R^{d_ffn x d}.  Rows
 *            d_ff .. d_ff_ld-1 are padding: never selected, never read as channels, and their
 *            gradient rows are written as zero.
 *            topk_idx [tokens, k] int16, ascending within a token; topk_gate / topk_up [tokens, k]
 *            in the storage dtype: the pre-SiLU gate value g and the up value u of each kept channel.
 * Selection  The K channels with the largest SIGNED pre-SiLU gate values, compared on the fp32
 *            accumulator of the gate projection.  Ties at the K-th value go to the lower channel;
 *            -0.0 equals +0.0; NaN orders as -infinity.
 * Arithmetic Storage dtype per `dtype`; every contraction accumulates in fp32.
 * Async      Calls enqueue work on `cuda_stream` and return without synchronising.  Errors the host
 *            can see (bad descriptor, NULL or misaligned pointer, workspace too small) are returned
 *            as a negative status BEFORE anything is launched.  Conditions only the device can see
 *            (a saved index outside [0, d_ff), a bounded wait that expired) make the kernel skip the
 *            offending work without touching out-of-range memory and raise a sticky per-device status
 *            word that moc_last_device_status() reports.
 * Weights    The kernels of moc_ffn_decode, and of moc_ffn_forward for batches of up to 256 tokens, are chained with
 *            programmatic dependent launch and start fetching WEIGHTS before they synchronise with earlier work of
 *            the stream (activations and the workspace are touched only after that synchronisation).  Weights are
 *            therefore expected to be settled when the call is enqueued: a kernel that writes them and itself
 *            releases its dependents early must be followed by an event or stream synchronisation first.
 * Threads    Entry points may be called from several host threads on different streams as long as
 *            their buffers (workspace included) do not overlap.
 * Workspace  A workspace serves one call at a time: the next call that names it may be enqueued on the same stream
 *            behind the first, or anywhere once the first has completed.  Its contents between calls are the
 *            caller's (nothing in it outlives a call).  For batches of up to 32 tokens the library keeps three
 *            counters per workspace ADDRESS in its own statically allocated device memory (they are left zero by
 *            every call that completes, so a call can start without clearing them); 1024 addresses per device are
 *            served that way, further ones by the kernels that need no such state.
 * Co-op      Two kernels are launched cooperatively (cudaLaunchCooperativeKernel: their CTAs wait on one another, so
 *            all must be resident): the one-kernel forms of moc_ffn_decode / moc_ffn_forward for one or two tokens
 *            and for up to 32 tokens that keep nothing.  On a device or in a context that cannot launch them
 *            (no cooperative launch, SMs partly reserved) the multi-kernel forms run instead.
 */
#ifndef MOC_FFN_H_
#define MOC_FFN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(_WIN32)
#define MOC_API
#else
#define MOC_API __attribute__((visibility("default")))
#endif

typedef enum {
    MOC_OK = 0,
    MOC_ERR_INVALID_ARG = -1, /* NULL/misaligned pointer, k outside [1, d_ff], negative sizes ...   */
    MOC_ERR_UNSUPPORTED = -2, /* d_ff > 32768 (int16 indices), d_model % 8 != 0, decode tokens > 256 */
    MOC_ERR_WORKSPACE = -3,   /* workspace pointer NULL or smaller than moc_ffn_workspace_bytes()    */
    MOC_ERR_CUDA = -4,        /* a CUDA runtime call or a launch failed                             */
    MOC_ERR_TIMEOUT = -5,     /* device status: a bounded wait inside a kernel expired              */
    MOC_ERR_BAD_INDEX = -6,   /* device status: a saved channel index was outside [0, d_ff)         */
    MOC_ERR_STATIC_LIMIT = -7 /* problem larger than the built-in scratch of moc_ffn_decode_static   */
} moc_status;

typedef enum { MOC_F32 = 0, MOC_BF16 = 1 } moc_dtype;

typedef enum { MOC_OP_FORWARD = 0, MOC_OP_BACKWARD = 1, MOC_OP_DECODE = 2, MOC_OP_DECODE_BLOCK = 3 } moc_op;

/* bit 0 of moc_ffn_desc.flags: add into grad_w_* instead of overwriting them */
#define MOC_FLAG_ACCUMULATE_WGRAD 1u
/* bit 1: grouped mask, MoC 2:8 (Section 4, "MoC with structured 2:8 sparsity"; Theorem 1 states the a:b form):
 * instead of the K largest gate values of the whole row, the 2 largest of every group of 8 consecutive channels are
 * kept (signed pre-SiLU values, equal values: the lower channel, NaN as -inf).  Requires d_ff % 8 == 0 and
 * k == d_ff / 4; the kept channels of group q occupy slots 2q and 2q + 1 of topk_idx / topk_gate / topk_up.
 * Honoured by moc_ffn_forward, moc_ffn_decode and moc_ffn_decode_static.  For moc_ffn_backward the flag is a PROMISE
 * about the saved indices (they came from a forward call with the flag: at most 2 kept channels in every 4 consecutive
 * ones); the library may then form grad_x on the 2:4-sparse tensor-core MMA, as the forward call does for the down
 * projection (bf16, d_model >= 1024; for grad_x only with MOC_FFN_SPARSE_DX=1 in the environment: compressing the two
 * operands costs what the shorter contraction saves).  A saved row that breaks the promise raises MOC_ERR_BAD_INDEX in
 * the device status word and its surplus channels are left out of grad_x; without the flag the backward pass takes the
 * indices as they are. */
#define MOC_FLAG_SELECT_2_OF_8 2u
/* bit 2: the Top-K operator placed AFTER the activation (Section 6.5, "Effect of top-K position": the ablation whose
 * other arm is the default): the K channels with the largest SiLU(g) are kept instead of those with the largest g.
 * The two agree whenever a token has at least K positive gate values (SiLU is increasing there and negative below
 * zero); they differ on tokens with fewer, where SiLU's minimum near g = -1.28 reorders the negative values.  Keys
 * are SiLU(g) evaluated in fp32; equal keys: the lower channel; a NaN key (a NaN or -inf gate value) orders as -inf.
 * What is saved and what the backward pass computes do not change (the mask is taken as saved).  Not combinable with
 * MOC_FLAG_SELECT_2_OF_8.  This variant runs the exact gathered kernels for every dtype and batch size (it exists
 * for ablations, not for speed); moc_ffn_decode_block does not take it. */
#define MOC_FLAG_SELECT_POST_SILU 4u

typedef struct moc_ffn_desc {
    int64_t tokens;   /* T = batch * seq, >= 0 (0 is a no-op)                                   */
    int32_t d_model;  /* d, multiple of 8                                                        */
    int32_t d_ff;     /* F, logical channel count, 1 <= F <= 32768                               */
    int32_t d_ff_ld;  /* rows allocated in each weight array, >= d_ff                            */
    int32_t k;        /* channels kept per token, 1 <= k <= d_ff; k == d_ff is dense SwiGLU      */
    int32_t dtype;    /* moc_dtype of x, weights, out, topk_gate/topk_up and all gradients       */
    uint32_t flags;   /* MOC_FLAG_*                                                              */
} moc_ffn_desc;

/*
 * Bytes of caller-provided workspace that `op` needs for this descriptor (0 on an invalid
 * descriptor).  The workspace holds transient buffers only (gate projection of a token chunk,
 * per-channel token lists for the weight gradients ...); nothing in it outlives the call.
 */
MOC_API size_t moc_ffn_workspace_bytes(const moc_ffn_desc *desc, int op);

/*
 * Forward, Eqs. (Moc-1), mask, (MoC-2).
 *   in : x [T,d], w_gate / w_up / w_down [d_ff_ld, d]
 *   out: out [T,d]; topk_idx [T,k] int16, topk_gate [T,k], topk_up [T,k] -- the compact saved
 *        activations of Table 1 ("MoC+GCP").  The three saved outputs may all be NULL (inference:
 *        nothing is kept); passing only some of them is MOC_ERR_INVALID_ARG.
 * Returns MOC_OK or a negative moc_status; nothing is launched on error.
 */
MOC_API int moc_ffn_forward(const moc_ffn_desc *desc, const void *x, const void *w_gate, const void *w_up,
                            const void *w_down, void *out, int16_t *topk_idx, void *topk_gate, void *topk_up,
                            void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Backward, Eqs. (bp-1)..(bp-5), from the saved compact activations (S' and Z' are recomputed
 * element-wise from topk_gate / topk_up; the mask is a constant, no gradient flows through it).
 *   in : x, weights, topk_idx / topk_gate / topk_up as written by moc_ffn_forward, grad_out [T,d]
 *   out: grad_x [T,d]; grad_w_gate / grad_w_up / grad_w_down [d_ff_ld, d].  Any of the four may be
 *        NULL (skipped).  Weight gradients are overwritten unless MOC_FLAG_ACCUMULATE_WGRAD is set.
 * A saved index outside [0, d_ff) is skipped and reported through moc_last_device_status().
 */
MOC_API int moc_ffn_backward(const moc_ffn_desc *desc, const void *x, const void *w_gate, const void *w_up,
                             const void *w_down, const int16_t *topk_idx, const void *topk_gate,
                             const void *topk_up, const void *grad_out, void *grad_x, void *grad_w_gate,
                             void *grad_w_up, void *grad_w_down, void *workspace, size_t workspace_bytes,
                             void *cuda_stream);

/*
 * moc_ffn_backward for data-parallel training: Eqs. (bp-1) and (bp-4) are sums over tokens, so when a batch is
 * sharded by tokens over several GPUs (weights replicated) each GPU's grad_w_* is a partial sum and the job adds
 * them with one all-reduce of 3 d_ffn d elements, while Eq. (bp-5), grad_x, stays local.  This variant lets that
 * all-reduce overlap the grad_x kernel: `wgrad_done_event` (a cudaEvent_t passed as void*, created by the caller;
 * NULL = plain moc_ffn_backward) is recorded on `cuda_stream` at the point where every kernel that writes
 * grad_w_gate / grad_w_up / grad_w_down has been enqueued and before the grad_x kernel where the plan orders them
 * that way (the tensor-core plan; on the gathered plan the weight gradients come last, so the event marks the end of
 * the call).  A second stream that waits on the event may read the weight gradients at once.  It is recorded on
 * every successful return, also when no weight gradient was asked for.  Everything else as moc_ffn_backward.
 */
MOC_API int moc_ffn_backward_overlap(const moc_ffn_desc *desc, const void *x, const void *w_gate, const void *w_up,
                                     const void *w_down, const int16_t *topk_idx, const void *topk_gate,
                                     const void *topk_up, const void *grad_out, void *grad_x, void *grad_w_gate,
                                     void *grad_w_up, void *grad_w_down, void *workspace, size_t workspace_bytes,
                                     void *cuda_stream, void *wgrad_done_event);

/*
 * The up values of the kept channels again: topk_up[t, k] = x[t, :] . w_up[topk_idx[t, k], :], rounded to the
 * storage dtype.  For callers that keep only (topk_idx, topk_gate) between forward and backward -- the
 * recomputation idea of Section 4 (Table 1, the "+GCP" columns) taken one step further: 2 K + K e instead of
 * 2 K + 2 K e bytes per token are held, and the backward pass pays one more up projection (2 T d d_ffn flops on
 * the tensor-core plan, 2 T K d on the gathered plan).  The result feeds moc_ffn_backward as topk_up.
 *   in : x [T,d], w_up [d_ff_ld, d], topk_idx [T,k] as written by moc_ffn_forward
 *   out: topk_up [T,k]
 * workspace: moc_ffn_workspace_bytes(desc, MOC_OP_BACKWARD) bytes (the same buffer moc_ffn_backward takes next).
 * A saved index outside [0, d_ff) yields 0 and is reported through moc_last_device_status().
 */
MOC_API int moc_ffn_recompute_up(const moc_ffn_desc *desc, const void *x, const void *w_up, const int16_t *topk_idx,
                                 void *topk_up, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Small-batch inference (Section 5): the same forward with nothing saved, for tokens <= 256
 * (more: MOC_ERR_UNSUPPORTED; use moc_ffn_forward).  Up to 16 tokens it is organised so that only the
 * gate matrix and the selected rows of w_up / w_down are read from HBM (d d_ffn + 2 K d weight
 * elements per token instead of 3 d d_ffn).  From 17 tokens on the union of the tokens' channel sets
 * covers nearly every channel (from 5 tokens on nearly half of them at K = d_ff / 8), and all three matrices are
 * streamed once through tensor-core kernels whose tiles are shaped for a few dozen tokens;
 * moc_ffn_forward takes the same path for such batches.
 * In both forms the partial sums of the down projection meet in an fp32 accumulator in an order that
 * is not fixed, so the last bit of `out` can differ from run to run.
 */
MOC_API int moc_ffn_decode(const moc_ffn_desc *desc, const void *x, const void *w_gate, const void *w_up,
                           const void *w_down, void *out, void *workspace, size_t workspace_bytes,
                           void *cuda_stream);

/*
 * The FFN half of a pre-norm Transformer layer for small batches (Section 2, "LLM structure", with the items
 * "RMSNorm" and "Residual connections" of its activation list): out = h + MoC_FFN(RMSNorm(h)), where
 * RMSNorm(h) = h / sqrt(mean(h^2) + rms_eps) . rms_weight per token, rounded to bf16 as the layer's input, and the
 * sum h + D is formed in fp32 from the layer's unrounded output and rounded once.  The normalisation and the
 * residual addition ride on the decode kernels instead of being two more launches around them: with one or two
 * tokens both happen inside the one cooperative kernel; otherwise a one-CTA-per-token kernel chained in front writes
 * the normalised rows and the last step of the down projection adds h.
 *
 *   h           [tokens, d_model] bf16, device: the residual stream
 *   rms_weight  [d_model] bf16, device
 *   rms_eps     >= 0
 *   out         [tokens, d_model] bf16, device; may be h itself (update in place)
 *   workspace   moc_ffn_workspace_bytes(desc, MOC_OP_DECODE_BLOCK) bytes
 * bf16 only, tokens <= 256, d_model a multiple of 8, and a d_ff that the small-batch selector holds in shared
 * memory (moc_ffn_workspace_bytes returns 0 otherwise and the call MOC_ERR_UNSUPPORTED).  Weights, stream,
 * ownership and the status word as for moc_ffn_decode.
 */
MOC_API int moc_ffn_decode_block(const moc_ffn_desc *desc, const void *h, const void *rms_weight, float rms_eps,
                                 const void *w_gate, const void *w_up, const void *w_down, void *out,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * moc_ffn_decode for callers that must not allocate.  (The paper has no counterpart: this is a
 * packaging variant of the decode path, not a different computation.)
 *
 * Who needs it: code that runs where device allocation is off the table -- an inference server
 * that handed all free HBM to its KV-cache pool at start-up, so a cudaMalloc in the decode loop
 * would fail; a latency-critical loop that cannot afford cudaMalloc/cudaFree because they
 * synchronise the whole device; a plug-in that is handed tensors but no allocator.  Such callers
 * still pass their inputs and the output buffer, but no workspace: the transient buffers (the fp32
 * gate projection of the batch and its channel indices) live in an array that is part of the
 * library image, MOC_STATIC_SCRATCH_BYTES long.  Every GPU that loads the library holds that array
 * from load until the process exits, whether or not this entry point is ever called.
 *
 * Kernels bf16 problems whose decode-plan buffers fit the array (the LLaMA-7B layer at 16 tokens does) run the
 *         same HBM-streaming kernels as moc_ffn_decode with its decode plan; everything else the limits admit
 *         runs the exact gathered kernels (correct, but milliseconds rather than tens of microseconds).
 * Limits  tokens <= MOC_STATIC_MAX_TOKENS and d_ff <= MOC_STATIC_MAX_DFF; anything larger returns
 *         MOC_ERR_STATIC_LIMIT and launches nothing (use moc_ffn_decode with a workspace instead).
 *         All other argument rules are those of moc_ffn_decode.
 * Set-up  The first call on each device looks up the device address of the array (no allocation,
 *         but a runtime query): make that first call during start-up, before any stream capture.
 * Sharing All calls on a device use the SAME array.  Calls on one stream are ordered and safe;
 *         calls whose kernels can overlap on the GPU (different streams or host threads without an
 *         ordering between them) race on it and give undefined results.  The array keeps whatever
 *         the previous call left; nothing in it needs to start at zero, because each call writes
 *         the whole region it later reads.
 * It calls neither cudaMalloc nor cudaFree nor any allocating library routine.
 */
#define MOC_STATIC_MAX_TOKENS 16
#define MOC_STATIC_MAX_DFF 16384
#define MOC_STATIC_SCRATCH_BYTES \
    ((size_t)MOC_STATIC_MAX_TOKENS * MOC_STATIC_MAX_DFF * (sizeof(float) + sizeof(int16_t)) + 512)
MOC_API int moc_ffn_decode_static(const moc_ffn_desc *desc, const void *x, const void *w_gate,
                                  const void *w_up, const void *w_down, void *out, void *cuda_stream);

/*
 * The Top-K selector alone (the mask definition of Section 3.2), exposed so that it can be checked
 * bit-exactly: gate [rows, n_ld] fp32 on the device, only the first n columns of a row are channels;
 * idx_out [rows, k] int16 ascending.  Needs no workspace.  As in the plans, up to 256 rows are handled by
 * the selector that gives a whole CTA to each row (decode and small-batch plans), more rows by the
 * selector of the gathered plan; both are exact.
 */
MOC_API int moc_topk_select(int64_t rows, int32_t n, int32_t n_ld, int32_t k, const float *gate,
                            int16_t *idx_out, void *cuda_stream);

/*
 * The row Top-K selector of the tensor-core plan (the one moc_ffn_forward runs on training-sized bf16 batches) alone,
 * on caller-supplied fp32 gate rows, so that the mask definition of Section 3.2 can be checked bit-exactly on it too.
 * Which kernel form runs depends on the row length and k exactly as in moc_ffn_forward: teams of two or four warps per
 * row with the row staged in shared memory, the same with one buffer for the gate and the up row (long rows), or one
 * CTA per row (rows too long for a team's slice); `*variant` (host, may be NULL) receives which:
 * 0 CTA per row, 1 teams of two, 2 teams of four, 3 teams of four with a shared buffer.
 *   gate     [rows, n_ld] fp32, device; n_ld a multiple of 8 with n <= n_ld <= n rounded up to 128
 *   idx_out  [rows, k] int16, device, ascending
 *   bracket  host pointer to {center, half width} of the threshold bracket the launch starts from (what the previous
 *            launch of a forward pass would have left in the workspace), or NULL for the state of a first call; the
 *            bracket is a hint only: any value, however wrong, must give the same exact result
 *   workspace  moc_topk_select_tc_workspace_bytes(rows, n, n_ld, k) bytes (0 = shape not served by this selector:
 *            (n + k) * 4 bytes must fit 170 KiB)
 */
MOC_API size_t moc_topk_select_tc_workspace_bytes(int64_t rows, int32_t n, int32_t n_ld, int32_t k);
MOC_API int moc_topk_select_tc(int64_t rows, int32_t n, int32_t n_ld, int32_t k, const float *gate, int16_t *idx_out,
                               const float *bracket, int *variant, void *workspace, size_t workspace_bytes,
                               void *cuda_stream);

/*
 * The one-kernel form of moc_ffn_decode for one or two bf16 tokens (MOC_ERR_UNSUPPORTED where the problem or the
 * device does not admit that kernel; it runs here for every k, also where moc_ffn_decode would prefer another form),
 * which additionally reports the mask it applied: kept [tokens, d_ff] bytes on the device,
 * 1 for a kept channel.  In that kernel no SM ever holds a token's whole gate row (the K-th largest value is found
 * through a histogram and a candidate list shared by all SMs), so this is the only way to see its selection directly.
 * A test that makes x a one-hot row e_i reads G[t, j] = w_gate[j, i] exactly and can so put any bf16 gate row in front
 * of the selection.  workspace: moc_ffn_decode_probe_workspace_bytes(desc) bytes.  Arguments otherwise as
 * moc_ffn_decode.
 */
MOC_API size_t moc_ffn_decode_probe_workspace_bytes(const moc_ffn_desc *desc);
MOC_API int moc_ffn_decode_probe(const moc_ffn_desc *desc, const void *x, const void *w_gate, const void *w_up,
                                 const void *w_down, void *out, uint8_t *kept, void *workspace, size_t workspace_bytes,
                                 void *cuda_stream);

/*
 * The dense bf16 contraction used for the gate projection G = X W_gate of Eq. (Moc-1) and for every
 * other contraction of the tensor-core plan, exposed so that it can be checked on its own:
 *     C[m, n] (fp32, row-major, leading dimension ldc) = sum_k A(m, k) * B(n, k),  fp32 accumulation.
 * A is stored [m, k] row-major (lda >= k) when a_mn_major == 0, or [k, m] row-major (lda >= m) when
 * a_mn_major != 0; B likewise as [n, k] or [k, n].  lda and ldb are in elements and multiples of 8.
 * Runs on the tcgen05 tensor cores (one persistent CTA per SM, TMA-fed, TMEM accumulators).
 */
MOC_API int moc_tc_gemm_bf16(int64_t m, int64_t n, int64_t k, const void *a, int a_mn_major, int64_t lda,
                             const void *b, int b_mn_major, int64_t ldb, float *c, int64_t ldc,
                             void *cuda_stream);

/*
 * The 2:4-sparse bf16 contraction on the sparse tensor-core MMA (tcgen05.mma.sp), exposed so that it can be checked on
 * its own.  Section 4 ("MoC with structured 2:8 sparsity") keeps 2 of every 8 consecutive channels, so every 4
 * consecutive channels of the masked hidden state hold at most 2 non-zero values: a row is a valid 2:4-sparse operand.
 *     C[m, n] (fp32, row-major, ldc) = sum_k A(m, k) * B(n, k)
 *   a_compressed  [m, k / 2] bf16, device: of every 4 consecutive contraction elements of a row of A the 2 kept ones,
 *                 in order (k a multiple of 16)
 *   metadata      device, ceil(m / 128) * ceil(k / 128) * 128 * 4 32-bit words: for tile row block i and block j of 128
 *                 contraction elements, lane l (0..127), column c (0..3) the word at ((i * kb + j) * 128 + l) * 4 + c
 *                 holds, for the 32 contraction elements 32 c .. 32 c + 31 of the block, the nibbles (position of the
 *                 first kept element | position of the second << 2, positions 0..3 inside their group of 4) of rows
 *                 r = (l % 8) + 16 * (l / 16) (bits 0..15) and r + 8 (bits 16..31), groups 4 * ((l / 8) % 2) .. + 3 of
 *                 the 8 groups, four bits each in ascending order -- the arrangement tensor memory wants
 *   b             as in moc_tc_gemm_bf16: [n, k] (b_mn_major == 0) or [k, n]
 */
MOC_API int moc_tc_gemm_sp_bf16(int64_t m, int64_t n, int64_t k, const void *a_compressed, const void *metadata,
                                const void *b, int b_mn_major, int64_t ldb, float *c, int64_t ldc, void *cuda_stream);

/*
 * The same contraction the way the operator uses it: A is given DENSE ([m, k] bf16 row-major, lda, at most 2 non-zero
 * values in every 4 consecutive elements of a row); the library compresses it (values + metadata, into the workspace)
 * and runs the sparse MMA on CTA pairs.  b is [k, n] with n contiguous (the layout of the weight matrices in the
 * down projection), c is bf16 [m, ldc]; accumulate != 0 adds the previous content of c before rounding.
 * Groups of 4 with more than 2 non-zero values keep their first 2; *overflow_count (host, may be NULL; asking for it
 * synchronises the stream) receives how many values were left out.
 */
MOC_API size_t moc_tc_gemm_sp_dense_workspace_bytes(int64_t m, int64_t k);
MOC_API int moc_tc_gemm_sp_dense_bf16(int64_t m, int64_t n, int64_t k, const void *a_dense, int64_t lda, const void *b,
                                      int64_t ldb, void *c, int64_t ldc, int accumulate, int64_t *overflow_count,
                                      void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Test hook for the time-out path every kernel of the library shares: launches one warp that waits, with the
 * library's bounded wait, on a barrier nothing completes.  After `limit_cycles` SM clock cycles (1 .. 4e9) the wait
 * gives up, the kernel raises MOC_ERR_TIMEOUT in the device status word and returns normally; nothing traps or
 * faults, and the context stays usable.  Returns MOC_OK when the launch was enqueued.  (The paper has no
 * counterpart: it is how the error behaviour stated above is checked.)
 */
MOC_API int moc_test_bounded_wait(int64_t limit_cycles, void *cuda_stream);

/*
 * Test hook for the time-out path of the one kernel in which CTAs wait on one another through global memory (the
 * cooperative small-batch forward for up to 32 tokens): the call is moc_ffn_decode's, except that the selector CTAs
 * are told to wait for one streamer more than exists, and that every wait gives up after `limit_cycles` SM clock
 * cycles (1 .. 4e9) instead of the library's two seconds.  Every CTA then runs into a wait that nothing completes,
 * raises MOC_ERR_TIMEOUT and returns normally; `out` is not written; nothing traps or faults, the context stays usable,
 * and the next call on the same workspace finds no "clean" mark and prepares its counters itself.  Arguments, layouts
 * and host-side errors as moc_ffn_decode; MOC_ERR_UNSUPPORTED where that kernel would not run (more than 32 tokens,
 * the 2-of-8 mask, no cooperative launch).  (The paper has no counterpart.)
 */
MOC_API int moc_test_small_batch_stall(const moc_ffn_desc *desc, const void *x, const void *w_gate, const void *w_up,
                                       const void *w_down, void *out, void *workspace, size_t workspace_bytes,
                                       int64_t limit_cycles, void *cuda_stream);

/*
 * Synchronises `cuda_stream`, then returns and clears the current device's sticky status word:
 * MOC_OK, MOC_ERR_TIMEOUT or MOC_ERR_BAD_INDEX (MOC_ERR_CUDA if the synchronisation itself failed).
 */
MOC_API int moc_last_device_status(void *cuda_stream);

/* Bytes per token that stay alive between forward and backward: k * (2 + 2 * sizeof(dtype)). */
MOC_API size_t moc_ffn_saved_bytes_per_token(const moc_ffn_desc *desc);

/*
 * Diagnostics (no counterpart in the paper; they exist so that a benchmark can attribute device
 * time to kernels without a profiler attached).  Not thread-safe against concurrent entry-point
 * calls: open a window, run the calls to be measured on ONE stream, collect, read.
 *   moc_launch_count          kernels launched by this library in this process so far.
 *   moc_profile_enable(1)     opens a window and clears the accumulators; while it is open every
 *                             kernel launch is bracketed by a pair of CUDA events on its stream
 *                             (at most 8192 launches per collect; later ones are not recorded).
 *   moc_profile_enable(0)     closes the window.
 *   moc_profile_collect       synchronises `cuda_stream`, folds the recorded pairs into per-kernel
 *                             totals; returns the number of launches that were not recorded (>= 0)
 *                             or a negative moc_status.
 *   moc_profile_kernel_count / _name / _read   enumerate kernels and read launches + total ms.
 */
MOC_API int64_t moc_launch_count(void);
/*   moc_profile_stream_read   a bare streaming read of up to three device byte ranges (sizes multiples of 16, 0 = unused):
 *                             every byte is brought into shared memory once by bulk copies, nothing is computed.  The time
 *                             of this kernel for the bytes a decode call has to read (Section 5: the gate matrix and the
 *                             selected rows of the other two) is the floor under any schedule for that call; a benchmark
 *                             times it with the call's own protocol and reports the call against it. */
MOC_API int moc_profile_stream_read(const void *a, size_t a_bytes, const void *b, size_t b_bytes, const void *c,
                                    size_t c_bytes, void *cuda_stream);
MOC_API int moc_profile_enable(int on);
MOC_API int moc_profile_collect(void *cuda_stream);
MOC_API int moc_profile_kernel_count(void);
MOC_API const char *moc_profile_kernel_name(int id);
MOC_API int moc_profile_read(int id, int64_t *launches, double *total_ms);

/* Static, NUL-terminated description of a moc_status value. */
MOC_API const char *moc_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* MOC_FFN_H_ */
