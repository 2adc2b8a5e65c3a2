/*
 * based.h — C ABI of the B200 (sm_100a) implementation of the Based sequence
 * mixers (arXiv 2402.18668): causal linear attention with the 2nd-order Taylor
 * feature map, its recurrent decode step, and exact sliding-window softmax
 * attention.
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers to contiguous row-major arrays, owned
 *     by the caller, 16-byte aligned (else BASED_ERR_ALIGNMENT).  `cuda_stream` is a
 *     cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Launches are asynchronous on the given stream; no entry point synchronises
 *     except based_poll_error.  Arguments are validated before anything is launched.
 *   - The library never falls back to another implementation: an unsupported shape
 *     or dtype returns BASED_ERR_UNSUPPORTED.
 *   - No entry point allocates device memory, except where stated otherwise.
 *   - Errors are returned as based_status; nothing throws, aborts or exits.
 *
 * Notation: B batch, H heads, L sequence length, d_feat = d' (width of q, k, 16),
 * d_v head dimension of v, D = 1 + d_feat + d_feat^2 (= 273) expanded feature size.
 *
 * State layout (ABI-visible): kv_state [B, H, D, d_v] fp32 with d_v contiguous,
 * z_state [B, H, D] fp32.  Feature index 0 is the constant term, 1..d_feat the
 * linear terms x_m / d'^(1/4), and 1 + d_feat + m*d_feat + n the product
 * x_m x_n / (sqrt(2) sqrt(d')) (the concatenation order of the feature-map module
 * in the paper's App. B.1 listing).  Rows are not padded.
 */
#ifndef BASED_H_
#define BASED_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BASED_OK = 0,
    BASED_ERR_INVALID_ARG = 1,    /* NULL pointer, non-positive size, bad enum value */
    BASED_ERR_UNSUPPORTED = 2,    /* valid request outside the supported set */
    BASED_ERR_ALIGNMENT = 3,      /* a pointer is not 16-byte aligned */
    BASED_ERR_CUDA = 4,           /* a CUDA runtime/driver call failed */
    BASED_ERR_DEVICE_TIMEOUT = 5, /* a bounded on-device wait gave up (reported by based_poll_error) */
    BASED_ERR_WORKSPACE = 6       /* workspace missing or smaller than based_prefill_workspace_bytes */
} based_status;

typedef enum { BASED_F32 = 0, BASED_BF16 = 1 } based_dtype;

/* flags of based_prefill */
enum {
    BASED_STATE_ZERO_INIT = 0, /* start from the empty state */
    BASED_STATE_CONTINUE = 1,  /* start from the state held in kv_state / z_state */
    BASED_STATE_SYM = 2,       /* OR-ed in: kv_state / z_state use the 153-row symmetric format
                                  described at based_decode_step_sym ([B,H,153,d_v], [B,H,153]) */
    BASED_NUMERATOR_ONLY = 4   /* OR-ed in: out = sum_j w_ij v_j without the division by sum_j w_ij
                                  (what Algorithm 1 and the kernel micro-benchmarks of App. "IO Aware
                                  Implementations" compute); the state is updated as usual */
};

/*
 * Causal Taylor linear attention over whole sequences (Sec. 4.1, Eq. (2) with the
 * feature map of Eq. (3) scaled as in the App. B.1 listing; chunked evaluation as in
 * Sec. 5.2 / Algorithm 1, here with the normalising denominator included):
 *
 *   out[i] = sum_{j<=i} w_ij v_j / (sum_{j<=i} w_ij + 1e-12),
 *   w_ij   = phi(q_i).phi(k_j) = 1 + q_i.k_j/sqrt(d') + (q_i.k_j)^2 / (2 d')
 *
 * q, k      [B,H,L,d_feat]  io dtype          v, out  [B,H,L,d_v]  io dtype
 * kv_state  [B,H,D,d_v] fp32, z_state [B,H,D] fp32: both NULL (state not wanted) or
 *           both non-NULL.  With BASED_STATE_CONTINUE they are read as the state
 *           before token 0 (then they must be non-NULL); on return they hold the
 *           state after token L-1.  Accumulation and state are fp32 for both io dtypes.
 *           The rows of the products k_m k_n and k_n k_m hold equal values in every state a
 *           prefill or a decode step produces; the bf16 d_feat = 16 path relies on that and
 *           returns both as their mean when it continues from a state where they differ.
 * workspace device scratch of at least based_prefill_workspace_bytes(...) bytes
 *           (may be NULL when that size is 0); contents are undefined afterwards.
 * Supported: d_feat = 16; d_v in {64, 112, 128}; io in {F32, BF16}; any L >= 1.
 * d_feat in {8, 24, 32} (the other dimensions of the paper's feature-map ablation; state rows
 * D = 1 + d_feat + d_feat^2 = 73, 601, 1057) is served by the definition form: bf16 io from the
 * empty state on tensor cores (outputs and state), the other cases by fp32 FMA kernels; no
 * workspace, no BASED_STATE_SYM.
 * Batches of more than 65535 heads are cut into slabs of heads that run one after another on the stream.
 * out must not alias an input.
 */
based_status based_prefill(const void* q, const void* k, const void* v, void* out, float* kv_state,
                           float* z_state, int B, int H, int L, int d_feat, int d_v, based_dtype io,
                           int flags, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Scratch bytes based_prefill needs for these arguments (0 is possible). */
size_t based_prefill_workspace_bytes(int B, int H, int L, int d_feat, int d_v, based_dtype io);

/*
 * The recurrent state of a token block without its outputs (Sec. 4.1, recurrent view):
 *   kv_state (+)= sum_j phi(k_j) v_j^T,   z_state (+)= sum_j phi(k_j)
 * exactly what based_prefill leaves in kv_state / z_state for the same k, v, flags, at about a
 * third of its cost (no scores, no read-out).  k [B,H,L,d_feat], v [B,H,L,d_v] in the io dtype;
 * the state layouts are based_prefill's.  flags: BASED_STATE_ZERO_INIT or BASED_STATE_CONTINUE,
 * optionally BASED_STATE_SYM.  This is the first step of a prefill whose sequence is split across
 * GPUs: every rank computes its block's state, the states are exchanged and summed over the
 * earlier ranks, and based_prefill with BASED_STATE_CONTINUE produces the block's outputs.
 * Supported: d_feat in {8, 16, 24, 32}, d_v in {64, 112, 128}, io in {F32, BF16}; BASED_STATE_SYM
 * with d_feat = 16 and BF16 io only.  workspace: based_prefill_state_workspace_bytes (non-zero
 * for d_feat = 16 with BF16 io: partial states of sequence segments).
 */
based_status based_prefill_state(const void* k, const void* v, float* kv_state, float* z_state, int B, int H, int L,
                                 int d_feat, int d_v, based_dtype io, int flags, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream);
size_t based_prefill_state_workspace_bytes(int B, int H, int L, int d_feat, int d_v, based_dtype io);

/*
 * One recurrent step of the same mixer (Sec. 4.1 recurrences; App. B.2 step()
 * listing and Algorithm 2, here on raw q, k with the feature map applied on chip and
 * with the denominator): per (b, h), update then read,
 *
 *   kv_state += phi(k) v^T ;  z_state += phi(k) ;
 *   out = phi(q) kv_state / (phi(q).z_state + 1e-12)
 *
 * q, k [B,H,d_feat], v, out [B,H,d_v] in the io dtype; kv_state / z_state as above,
 * updated IN PLACE.  Supported: d_feat = 16; d_v in {64, 112, 128}; io in {F32, BF16}; also
 * d_feat in {8, 24, 32} with D = 1 + d_feat + d_feat^2 state rows (plain streaming kernel).
 */
based_status based_decode_step(const void* q, const void* k, const void* v, float* kv_state, float* z_state,
                               void* out, int B, int H, int d_feat, int d_v, based_dtype io,
                               void* cuda_stream);

/*
 * The same step on a symmetric state (opt-in format).  The outer product x (x) x has equal
 * entries (m,n) and (n,m); keeping one feature per unordered pair leaves
 * BASED_D_SYM = 1 + 3d'/2 + d'^2/2 = 153 rows (the feature count of the paper's appendix
 * "Computing Recurrent State Size" and of its feature-map ablation table) instead of 273,
 * with the same outputs and 44 % fewer state bytes read and written per step:
 *
 *   psi(x) = [1, x/2, {x_m^2 / (4 sqrt 2)} , {x_m x_n / 4 : m < n}]     psi(q).psi(k) = phi(q).phi(k)
 *
 * Row order: 0 the constant, 1..16 the linear terms, then the pairs m <= n in row-major order
 * of the upper triangle ((0,0), (0,1), ..., (0,15), (1,1), ...).
 * kv_sym [B,H,153,d_v] fp32 and z_sym [B,H,153] fp32 are updated IN PLACE; everything else as in
 * based_decode_step.
 */
#define BASED_D_SYM 153
based_status based_decode_step_sym(const void* q, const void* k, const void* v, float* kv_sym, float* z_sym,
                                   void* out, int B, int H, int d_feat, int d_v, based_dtype io,
                                   void* cuda_stream);

/*
 * based_decode_step with flags: 0, BASED_STATE_SYM (the state has the symmetric format, as
 * based_decode_step_sym), BASED_NUMERATOR_ONLY (out = phi(q) kv_state, no division), or both.
 */
based_status based_decode_step_flags(const void* q, const void* k, const void* v, float* kv_state, float* z_state,
                                     void* out, int B, int H, int d_feat, int d_v, based_dtype io, int flags,
                                     void* cuda_stream);

/*
 * Conversions between the 273-row state of based_prefill / based_decode_step and the symmetric
 * one.  to_sym: row (m,n), m < n, = (S_mn + S_nm) / sqrt 2, the other rows are copied.
 * from_sym: rows (m,n) and (n,m) = S_sym / sqrt 2 (exact inverse on states built by the
 * recurrences, which are symmetric).  Input and output must not alias; all device pointers, fp32.
 */
based_status based_state_to_sym(const float* kv_state, const float* z_state, float* kv_sym, float* z_sym, int B,
                                int H, int d_feat, int d_v, void* cuda_stream);
based_status based_state_from_sym(const float* kv_sym, const float* z_sym, float* kv_state, float* z_state, int B,
                                  int H, int d_feat, int d_v, void* cuda_stream);

/*
 * Exact causal softmax attention in a sliding window (Eq. (1) of Sec. 2 restricted as
 * in Sec. 4.2: query i attends keys max(0, i-window+1) .. i):
 *
 *   out[i] = sum_j softmax_j(scale * q_i.k_j) v_j
 *
 * q, k, v, out [B,H,L,d] in the io dtype.  softmax_scale <= 0 selects 1/sqrt(d).
 * Supported: d = 64; 1 <= window <= 128; io in {F32, BF16}; any L >= 1.
 */
based_status swa_forward(const void* q, const void* k, const void* v, void* out, int B, int H, int L, int d,
                         int window, float softmax_scale, based_dtype io, void* cuda_stream);

/*
 * One generation step of the sliding-window mixer on a rolling cache of the last `window` keys
 * and values (the sliding-window PyTorch listing and Algorithm 3 of App. B.2; the cache update,
 * which the paper's micro-benchmark leaves out, is part of the call):
 *
 *   k_cache[pos % window] = k ;  v_cache[pos % window] = v ;
 *   out = sum_j softmax_j(scale * q.k_cache[j]) v_cache[j]   over the cached positions
 *         max(0, pos-window+1) .. pos
 *
 * q, k, v, out [B,H,d]; k_cache, v_cache [B,H,window,d], all in the io dtype; the caches are
 * ring buffers updated IN PLACE: the token at absolute position t lives in slot t % window, and
 * slots of positions that have not occurred yet are never read.  `pos` is the absolute position
 * of the new token (the same for the whole batch).  softmax_scale <= 0 selects 1/sqrt(d).
 * Supported: d = 64; 1 <= window <= 128; io in {F32, BF16}.
 */
based_status swa_decode_step(const void* q, const void* k, const void* v, void* k_cache, void* v_cache, void* out,
                             int B, int H, int d, int window, int pos, float softmax_scale, based_dtype io,
                             void* cuda_stream);

/*
 * Backward pass of based_prefill from the empty state (the paper calls prefill "the forward pass
 * during training" but gives no backward algorithm: this is the chain rule on the definition
 * form of Eq. (2), Sec. 4.1).  With dout the gradient of the loss with respect to out,
 *
 *   a_i = dout_i / D_i,  b_i = -(dout_i . out_i) / D_i,  D_i = sum_{j<=i} w_ij + 1e-12,
 *   ds_ij = (a_i . v_j + b_i)(1/4 + q_i.k_j / 16),
 *   dq_i = sum_{j<=i} ds_ij k_j,  dk_j = sum_{i>=j} ds_ij q_i,  dv_j = sum_{i>=j} w_ij a_i.
 *
 * q, k, dq, dk [B,H,L,d_feat]; v, dout, dv [B,H,L,d_v], all in the io dtype; arithmetic in fp32
 * (the forward output is not an argument: out_i is recomputed in fp32, because a_i.v_j + b_i
 * cancels almost completely for short prefixes and a rounded out would dominate the result).
 * flags: 0, or BASED_NUMERATOR_ONLY for the backward of the numerator-only forward.
 * workspace: at least based_prefill_backward_workspace_bytes(B, H, L, d_v, io) bytes of device scratch.
 * Supported: d_feat = 16 with io in {F32, BF16}, d_feat in {8, 24, 32} with BF16 io (w = 1 + s/sqrt(d') +
 * s^2/(2 d'), so ds_ij = (a_i . v_j + b_i)(1/sqrt(d') + q_i.k_j / d')); d_v in {64, 112, 128}.
 * Both paths evaluate the quadratic form, O(L^2) per head, on 128 x 128 (bf16 io: tcgen05 tensor
 * cores, bf16 operands, fp32 accumulation) or 64 x 64 (fp32 io: fp32 FMAs) tiles of (query, key)
 * pairs; with bf16 io and d_feat = 16 longer sequences take the block-wise path described at
 * based_prefill_backward_with_out (the forward output that it needs is recomputed into the workspace:
 * one forward pass more).  Gradient outputs must not alias inputs.
 */
based_status based_prefill_backward(const void* q, const void* k, const void* v, const void* dout, void* dq,
                                    void* dk, void* dv, int B, int H, int L, int d_feat, int d_v, based_dtype io,
                                    int flags, void* workspace, size_t workspace_bytes, void* cuda_stream);
size_t based_prefill_backward_workspace_bytes(int B, int H, int L, int d_v, based_dtype io);

/*
 * The same backward pass for a caller that kept the forward output (training: autograd saves it).
 * out [B,H,L,d_v], io dtype: what based_prefill returned for these q, k, v from the empty state with
 * the same flags.  Results and arguments as based_prefill_backward.  With bf16 io the row statistics
 * and dq then take one sweep over the keys instead of two: dq_i = X_i / D_i + (m_i / D_i + b_i) Y_i
 * with X_i = sum_j w'_ij (dout_i.v_j - m_i) k_j and Y_i = sum_j w'_ij k_j needs neither D_i nor b_i
 * while the keys are swept, and m_i = dout_i . out_i, the weighted mean of dout_i . v_j up to the
 * rounding of out, keeps the cancellation against b_i in fp32.  out is used for this centring
 * only: D_i and dout_i . N_i are still recomputed in fp32.  fp32 io ignores out's values.
 * out must not alias a gradient output.
 *
 * Block-wise path (bf16 io, d_feat = 16; L >= 768 at d_v 64, L >= 1024 to 1536 at d_v 112 / 128): O(L) per
 * head, the recurrent view of Sec. 4.1 applied to the gradients.  The sequence is cut into blocks of
 * W = 256 tokens (512 for long sequences of few heads at d_v 128).  Pairs inside a block go through
 * the tiles above.  All earlier blocks reach a query through their summed state S = sum_j phi(k_j) v_j^T, z = sum_j phi(k_j):
 *   sum_j w'_ij (dout_i.v_j - m_i) k_j = J(q_i)^T (S dout_i - m_i z),   D_i += phi(q_i) . z
 * (J the Jacobian of phi), and all later blocks reach a key through R = sum_i phi(q_i) (dout_i / D_i)^T
 * and R_b = sum_i b_i phi(q_i):  dk_j += J(k_j)^T (R v_j + R_b),  dv_j += R^T phi(k_j).
 * The block states are fp32 sums, rounded once to bf16 as tensor-core operands, like the state copy of
 * the forward pass; the products S dout_i and m_i z cancel in fp32 after the product, so the error
 * relative to the gradient grows with |mean v| / std v over the earlier blocks (1.5e-2 at mean 3,
 * std 1; 3e-3 for centred values; the gradients do not depend on a common offset of the values, so a
 * caller with such an offset can subtract it first).  Four launches instead of two (six below 64 heads, where the block
 * states come from one CTA per head and block plus a scan instead of one CTA walking each head).
 */
based_status based_prefill_backward_with_out(const void* q, const void* k, const void* v, const void* out,
                                             const void* dout, void* dq, void* dk, void* dv, int B, int H, int L,
                                             int d_feat, int d_v, based_dtype io, int flags, void* workspace,
                                             size_t workspace_bytes, void* cuda_stream);

/*
 * Which path a backward call with these arguments takes: the block length W of the block-wise path, or 0
 * for the tile path (fp32 io, d_feat other than 16, short sequences).  with_out: nonzero for
 * based_prefill_backward_with_out with out non-null; without the forward output (and without
 * BASED_NUMERATOR_ONLY) the block-wise path starts at somewhat longer sequences.
 * Host only; for callers that account the work of a call (benchmarks).
 */
int based_prefill_backward_block_tokens(int B, int H, int L, int d_feat, int d_v, based_dtype io, int flags,
                                        int with_out);

/*
 * The gated short convolution at the core of the BaseConv layer (App. "Extended Architecture
 * Details", paragraph "Convolution": y = ((u W1 + b1) (.) SiLU(h * (u W2) + b2)) W3 + b3).
 * The three projections are plain matrix products and stay with the caller; this call is the
 * fused middle:
 *
 *   out[b,i,c] = a[b,i,c] * SiLU( sum_{j < width, j <= i} h[j,c] * g[b,i-j,c] + b2[c] )
 *
 * a = u W1 + b1, g = u W2, out: [B,N,C] in the io dtype; h [width,C] fp32, a causal depthwise
 * filter whose row 0 is the tap on the current token; b2 [C] fp32.  SiLU(x) = x / (1 + exp(-x)).
 * Supported: 1 <= width <= 4 (the paper uses 3); C a multiple of 8; io in {F32, BF16}.
 * out may alias a; it must not alias g.
 */
based_status baseconv_gate_forward(const void* a, const void* g, const float* h, const float* b2, void* out, int B,
                                   int N, int C, int width, based_dtype io, void* cuda_stream);

/*
 * The same for one new token per sequence (generation): a, g, out [B,C]; conv_state
 * [B,width-1,C] in the io dtype holds the previous rows of g (row j = the token j+1 steps back,
 * zeros before the sequence start) and is updated IN PLACE (shifted, g stored in row 0).
 * conv_state may be NULL when width = 1.
 */
based_status baseconv_gate_step(const void* a, const void* g, const float* h, const float* b2, void* conv_state,
                                void* out, int B, int C, int width, based_dtype io, void* cuda_stream);

/*
 * Loads the kernels of the generation step (based_decode_step, based_decode_step_sym,
 * swa_decode_step, swa_decode_step_at, the state conversions) into the current device's
 * context and resolves the library's device symbols, so that their first use may happen inside
 * a stream capture.  Launches nothing.
 */
based_status based_preload_decode(void);

/*
 * The same step with the position read from device memory (one int, >= 0) when the kernel runs,
 * so that a launch captured into a CUDA graph (as the paper does for next-token prediction,
 * Sec. 6 "Efficiency Benchmarks") can be replayed while the sequence grows: the caller advances
 * *pos_device between replays, e.g. with a node of the same graph.
 */
based_status swa_decode_step_at(const void* q, const void* k, const void* v, void* k_cache, void* v_cache,
                                void* out, int B, int H, int d, int window, const int* pos_device,
                                float softmax_scale, based_dtype io, void* cuda_stream);

/*
 * The same step for a batch whose sequences have different lengths (Algorithm 3 takes one position; a
 * serving batch does not share one): pos_per_sequence is an array of B ints in device memory, the
 * position of sequence b's new token (>= 0); every head of sequence b uses slot pos[b] % window of its
 * cache and attends to min(pos[b] + 1, window) keys.  The caller advances the positions.
 */
based_status swa_decode_step_ragged(const void* q, const void* k, const void* v, void* k_cache, void* v_cache,
                                    void* out, int B, int H, int d, int window, const int* pos_per_sequence,
                                    float softmax_scale, based_dtype io, void* cuda_stream);

/*
 * The same step for a generation loop that is replayed as a CUDA graph: pos_state points to two
 * ints in device memory, {position, ticket} (ticket 0 before the first call).  The step reads the
 * position like swa_decode_step_at and stores position + 1 when it ends, so the loop needs no
 * separate kernel to advance the counter: every CTA takes a ticket at its end, and the one that
 * takes the last ticket, at which point all have read the position, resets the ticket and writes
 * the new position.  pos_state must be 8-byte aligned and is owned by the caller.
 */
based_status swa_decode_step_advance(const void* q, const void* k, const void* v, void* k_cache, void* v_cache,
                                     void* out, int B, int H, int d, int window, int* pos_state,
                                     float softmax_scale, based_dtype io, void* cuda_stream);

/*
 * One generated token through both mixers in ONE launch: based_decode_step (or its symmetric-state /
 * numerator-only forms, by flags: BASED_STATE_SYM, BASED_NUMERATOR_ONLY) on the linear-attention
 * layer's B x H heads (Sec. 4.1 recurrences, Algorithm 2) and swa_decode_step_advance on the
 * sliding-window layer's B x H_w heads (Algorithm 3, rolling cache, position read from and advanced in
 * device memory), the two kinds of CTA dealt out in turn within one grid so that the short window
 * step hides under the long state stream (the paper runs next-token prediction under CUDA graphs,
 * Sec. 6 "Efficiency Benchmarks"; as two kernels the steps run one after the other).
 * q, k [B,H,16], v, out [B,H,d_v], kv_state / z_state as in based_decode_step_flags (updated in
 * place); qw, kw, vw, out_w [B,H_w,64], k_cache, v_cache [B,H_w,window,64] as in swa_decode_step
 * (slot position % window is overwritten); pos_state: two ints in device memory, {position,
 * ticket}, 8-byte aligned (ticket 0 before the first call): position + 1 is stored when the step
 * ends.  All device pointers, io dtype for both mixers, results identical to the separate calls.
 * Supported: d_feat = 16, d_v in {64, 112, 128}, d_w = 64, window <= 128.  Errors as the separate
 * calls; nothing is launched when validation fails.
 */
based_status based_generation_step(const void* q, const void* k, const void* v, float* kv_state, float* z_state,
                                   void* out, const void* qw, const void* kw, const void* vw, void* k_cache,
                                   void* v_cache, void* out_w, int B, int H, int d_feat, int d_v, int H_w, int d_w,
                                   int window, int* pos_state, float softmax_scale, based_dtype io, int flags,
                                   void* cuda_stream);

/*
 * The same computation as based_prefill, for callers that cannot give the library scratch
 * memory.  (The paper has no counterpart: this is a deployment convenience.)  Some hosts
 * may not allocate device memory around a call at all - a serving process that has handed
 * the whole GPU to its own arena and exposes no allocator to plug-ins, a latency-critical
 * loop in which cudaMalloc's device-wide synchronisation is not acceptable, a sandbox that
 * forbids the allocation calls.  For them the scratch lives in a fixed array of
 * BASED_STATIC_SCRATCH_BYTES (8 MiB) of device memory inside the library image; every GPU
 * that loads the library holds that array until the process exits.  This entry point, and
 * everything it calls, allocates nothing.
 *
 * Arguments, layouts, supported set and results are those of based_prefill without the
 * workspace pair.  A request whose based_prefill_workspace_bytes exceeds the array (few heads
 * with a long sequence) is cut into fewer segments per head, as many as the array holds
 * partial states for, and is slower than based_prefill with a workspace of the full size;
 * the results are those of based_prefill up to the rounding order of the partial sums.
 * The first call on a device looks up the array's device address (one
 * cudaGetSymbolAddress, no allocation); make that first call outside any stream capture.
 * All calls on a device share the one array and it keeps the previous call's contents:
 * nothing in it needs clearing (each call overwrites what it later reads), but two calls
 * whose kernels can overlap on the GPU - different streams, or different threads - race on
 * it and must be serialised by the caller.
 */
#define BASED_STATIC_SCRATCH_BYTES (8u << 20)
based_status based_prefill_static_scratch(const void* q, const void* k, const void* v, void* out, float* kv_state,
                                          float* z_state, int B, int H, int L, int d_feat, int d_v, based_dtype io,
                                          int flags, void* cuda_stream);
size_t based_static_scratch_bytes(void);

/*
 * Synchronises the stream and returns the sticky device-side status: BASED_OK, or
 * BASED_ERR_DEVICE_TIMEOUT if a kernel abandoned a bounded wait (its outputs are then
 * undefined), or BASED_ERR_CUDA if the stream reported a CUDA error.  Clears the flag.
 */
based_status based_poll_error(void* cuda_stream);

/*
 * Diagnostic (no counterpart in the paper): launches a one-CTA kernel whose bounded wait is
 * made to run out after limit_ms (1..2000) - it waits on a barrier nothing signals - so the
 * error path "wait gives up -> sticky status word -> clean kernel exit" can be checked on a
 * live GPU without faulting or hanging it.  based_poll_error then returns
 * BASED_ERR_DEVICE_TIMEOUT once, and the context stays usable.
 */
based_status based_selftest_bounded_wait(unsigned int limit_ms, void* cuda_stream);

const char* based_status_string(based_status s);
int based_version(void);

/* Number of kernels this library has launched in this process (all entry points). */
unsigned long long based_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* BASED_H_ */
