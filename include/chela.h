/*
 * chela.h -- C ABI of the B200 (sm_100a) CHELA token-mixer hot path.
 *
 * The library evaluates, on one GPU, the forward pass of
 *   - the short depthwise causal convolution + SiLU            (Eq. 7, inner part),
 *   - the per-channel long convolution of length L via FFT       (Eq. 6, Sec. 2.2),
 *   - chunked ("tiled, divide-and-conquer") causal linear attention with a carried
 *     d_k x d_v state and a row normaliser                       (Eq. 2, Sec. 4.1),
 *   - their composition with the Q/K/V formation                 (Eqs. 8, 10-12).
 *
 * Conventions common to every entry point
 *   - Every data pointer is a DEVICE pointer owned by the caller; the library never frees or
 *     keeps it.  Pointers must be 16-byte aligned and the tensors contiguous in the stated
 *     row-major layout (last index fastest).
 *   - Work is enqueued on `stream`; calls return without synchronising the stream.
 *   - `workspace` is caller-provided device scratch of at least the size the matching
 *     `*_workspace_bytes` query returns (a query may return 0; then `workspace` may be NULL).
 *     Its contents are undefined before and after a call.  Two calls that share a workspace
 *     must be ordered on the GPU (same stream or an event).
 *   - The library allocates no device memory in these calls.
 *   - Return value: CHELA_OK or an error; arguments are validated before anything is
 *     launched, so an error return means no kernel ran.  Nothing throws or aborts.
 *   - dtype arguments take chela_dtype_t; bf16 tensors hold IEEE bfloat16 bit patterns.
 *     All arithmetic accumulates in fp32.
 */
#ifndef CHELA_H_
#define CHELA_H_

#include <stddef.h>
#include <cuda_runtime_api.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CHELA_OK = 0,
    CHELA_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, misaligned pointer          */
    CHELA_ERR_UNSUPPORTED = 2, /* valid but outside the supported set (see each function)     */
    CHELA_ERR_WORKSPACE = 3,   /* workspace missing or smaller than the query's answer        */
    CHELA_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed (launch, tensor map, ...) */
    CHELA_ERR_TIMEOUT = 5      /* a bounded device-side wait gave up (reported asynchronously) */
} chela_status_t;

/* CHELA_BF16_PAIR: a tensor stored as two bf16 planes of the same shape, the high plane first and the low
 * plane directly after it (numel elements later); its value is hi + lo (about 16 mantissa bits).
 * Accepted only where an entry point says so. */
typedef enum { CHELA_F32 = 0, CHELA_BF16 = 1, CHELA_BF16_PAIR = 2 } chela_dtype_t;

/* CHELA_NORM_RMS: o = r * (mean_j r_j^2 + eps)^(-1/2) over the d_v entries of one head's output
 * row, no learnable gain -- the library's reading of "Norm" in Eq. 2.  CHELA_NORM_NONE: o = r. */
typedef enum { CHELA_NORM_NONE = 0, CHELA_NORM_RMS = 1 } chela_norm_t;

const char *chela_status_string(chela_status_t status);
int chela_version(void);

/* Which linear-attention kernel a call with these arguments dispatches to:
 * 0 = none (unsupported), 1 = fp32 SIMT kernel, 2 = tcgen05/TMEM/TMA bf16 kernel. */
int chela_linattn_kernel_kind(int B, int H, int L, int d_k, int d_v, int chunk,
                              chela_dtype_t in_dtype, chela_dtype_t out_dtype);

/* How the tensor-core kernels share a sequence between CTAs when there are fewer (batch, head) pairs than SMs (host
 * logic only, no launch; the paper's tiling of Sec. 4.1 has no counterpart: it walks each sequence in one block).
 * bf16-pair inputs (in_dtype CHELA_BF16_PAIR, one CTA per SM) and d = 128: the sequence's 64-token chunks are divided
 * into *groups consecutive groups: the first of *first_chunks chunks, the others of *other_chunks (the last one what is
 * left); every group but the last is full and none is empty.  Plain bf16 with d = 64: *groups CTAs, CTA g owning the
 * chunks g, g + *groups, ...; *first_chunks = *other_chunks = 0 then (or the whole sequence when *groups = 1).
 * sms: SM count to plan for, <= 0 = the current device's.  Returns 1, or 0 for arguments no tensor-core kernel takes
 * (d not 64 or 128, null pointers). */
int chela_linattn_split_plan(int B, int H, int L, int d, chela_dtype_t in_dtype, int sms,
                             int *groups, int *first_chunks, int *other_chunks);

/*
 * Short depthwise causal convolution with optional SiLU (Eq. 7, inner part; Sec. 4.2):
 *   y[b,t,c] = act( bias[c] + sum_{j=0}^{width-1} w[c,j] * x[b,t-j,c] ),   x[b,t<0,c] = 0.
 * x, y : [B, L, D] of io_dtype (y may not alias x).  w : [D, width] fp32.  bias : [D] fp32 or NULL.
 * act : 0 = identity, 1 = SiLU.  Supported: 1 <= width <= 16, D a multiple of 8.
 */
chela_status_t chela_shortconv_fwd(const void *x, const float *w, const float *bias, void *y,
                                   int B, int L, int D, int width, int act,
                                   chela_dtype_t io_dtype, cudaStream_t stream);

/*
 * Structural re-parameterisation of parallel short kernels (Sec. 4.2): two depthwise causal kernels applied
 * to the same input and summed before the activation are one kernel whose taps are the zero-padded sum,
 *   conv(x; w1) + conv(x; w2) = conv(x; merged),  merged[c][j] = w1[c][j] (j < width1) + w2[c][j] (j < width2),
 * aligned at lag 0.  w1 : [D, width1], w2 : [D, width2], merged : [D, max(width1, width2)], all fp32 device
 * pointers.  chela_second_short_width gives the paper's length-dependent width 2 log10(L) + 1, rounded to the
 * nearest odd integer (the paper's value is not an integer in general) and clamped to [1, 15].
 */
int chela_second_short_width(int L);
chela_status_t chela_shortconv_reparam(const float *w1, int width1, const float *w2, int width2, float *merged, int D,
                                       cudaStream_t stream);

/*
 * Long convolution (Eq. 6, Sec. 2.2), optionally preceded by the short convolution + SiLU so
 * that the whole of Eq. 7 is one call:
 *   a = (w_short ? silu(shortconv(x; w_short)) : x) ;  z[b,t,c] = sum_{s=0}^{t} k_long[c,s] * a[b,t-s,c].
 * The product is evaluated with fp32 FFTs of size >= 2L (zero padded), so it is the causal
 * linear convolution, not the circular one.
 * x : [B, L, D] in_dtype.  k_long : [D, L] fp32.  w_short : [D, short_width] fp32 or NULL.
 * z : [B, L, D] out_dtype.  Supported: L <= 262144, D a multiple of 8.  Up to L = 16384 a row is transformed inside
 * one SM's shared memory; longer rows are cut into blocks of 16384 tokens whose spectra pass through the workspace
 * (2 x the row bytes more), one forward and one inverse transform per block and the block products in between.
 */
size_t chela_longconv_workspace_bytes(int B, int L, int D, chela_dtype_t in_dtype,
                                      chela_dtype_t out_dtype);
chela_status_t chela_longconv_fwd(const void *x, const float *k_long, const float *w_short,
                                  int short_width, void *z, int B, int L, int D,
                                  chela_dtype_t in_dtype, chela_dtype_t out_dtype,
                                  void *workspace, size_t workspace_bytes, cudaStream_t stream);

/*
 * Chunked causal linear attention forward (Eq. 2 with the causal mask; tiling of Sec. 4.1):
 *   r_t = scale * sum_{s<=t} <q_t, k_s> v_s ;   o_t = Norm(r_t)
 * evaluated chunk by chunk: inside a chunk the masked product (Q_i K_i^T . M) V_i, across chunks
 * Q_i S_{i-1} with the running state S_i = S_{i-1} + K_i^T V_i kept on chip in fp32.
 * q, k : [B, L, H, d_k] in_dtype.  v : [B, L, H, d_v] in_dtype.  o : [B, L, H, d_v] out_dtype.
 * L need not be a multiple of chunk.  The result does not depend on chunk beyond rounding.
 * Supported: d_k = d_v in {64, 128}, chunk in {64, 128}.
 * With fewer (batch, head) pairs than SMs a sequence is shared between several CTAs (plain bf16, d = 64: by stride,
 * each CTA accumulating the whole state) or split along L (the per-split states then live in `workspace`, fp32).
 */
size_t chela_linattn_workspace_bytes(int B, int H, int L, int d_k, int d_v, int chunk);
chela_status_t chela_linattn_fwd(const void *q, const void *k, const void *v, void *o,
                                 int B, int H, int L, int d_k, int d_v, int chunk,
                                 chela_dtype_t in_dtype, chela_dtype_t out_dtype,
                                 chela_norm_t norm, float norm_eps, float scale,
                                 void *workspace, size_t workspace_bytes, cudaStream_t stream);

/*
 * chela_linattn_fwd with the running state carried across calls, for segment-wise sequential evaluation
 * and decoding (Sec. 5, language modelling: segment-wise sequential evaluation; the state is the
 * intermediate variable of Sec. 4.1):
 *   S_{-1} = state_in (zero if NULL);  outputs as chela_linattn_fwd;  state_out = S after the last token.
 * Evaluating a sequence in consecutive segments with the state carried gives the result of one call over
 * the whole sequence (up to rounding).  state_in, state_out : [B, H, d_k, d_v] fp32, nullable, may alias
 * each other (the initial state is then read from a copy that the call takes on `stream` first, in `workspace`,
 * because several CTAs may work on one sequence).  Supported: everything chela_linattn_fwd supports.
 */
chela_status_t chela_linattn_carry_fwd(const void *q, const void *k, const void *v, void *o,
                                       const float *state_in, float *state_out,
                                       int B, int H, int L, int d_k, int d_v, int chunk,
                                       chela_dtype_t in_dtype, chela_dtype_t out_dtype,
                                       chela_norm_t norm, float norm_eps, float scale,
                                       void *workspace, size_t workspace_bytes, cudaStream_t stream);

/*
 * Decoding step: one new token per sequence against the carried state (recurrent form of Eq. 2; Sec. 5's
 * sequential evaluation taken to segments of one token):
 *   S <- S + k v^T  (in place),   r = scale * S^T q,   o = Norm(r) as in chela_linattn_fwd.
 * Equals chela_linattn_carry_fwd with L = 1 and state_in = state_out = state, without its per-call tile
 * machinery: the state is read and written once.
 * q, k : [B, H, d_k];  v, o : [B, H, d_v];  state : [B, H, d_k, d_v] fp32, updated in place; device pointers,
 * 16-byte aligned, owned by the caller.  Supported: d_k = d_v in {64, 128}; in_dtype F32 or BF16; out_dtype
 * F32 or BF16.  No workspace.  Errors: CHELA_ERR_INVALID_ARG (null pointer, B, H < 1), CHELA_ERR_UNSUPPORTED.
 */
chela_status_t chela_linattn_step(const void *q, const void *k, const void *v, void *o, float *state,
                                  int B, int H, int d_k, int d_v,
                                  chela_dtype_t in_dtype, chela_dtype_t out_dtype,
                                  chela_norm_t norm, float norm_eps, float scale, cudaStream_t stream);

/*
 * Backward of chela_linattn_fwd (gradients of Eq. 2 with the causal mask and the row normaliser; the
 * chunked evaluation of Sec. 4.1 run in both directions): given d_o = dLoss/do,
 *   dq_t = scale sum_{s<=t} <g_t,v_s> k_s,  dk_s = scale sum_{t>=s} <g_t,v_s> q_t,  dv_s = scale sum_{t>=s} <q_t,k_s> g_t,
 * with g_t = d_o[t] pulled back through the normaliser (g_t = d_o[t] for CHELA_NORM_NONE).  Nothing saved by the
 * forward pass is needed: the pre-normaliser output is recomputed.
 * q, k, v, d_o : [B, L, H, d] in_dtype (F32 or BF16).  dq, dk, dv : [B, L, H, d] fp32.
 * Supported: d_k = d_v in {64, 128}.  bf16 inputs run on the tensor cores: the three gradients are
 * linear attentions with the operands' roles exchanged, evaluated by the forward kernel (two of them in its
 * anti-causal mode) on g rounded to bf16; everything else runs on an fp32 SIMT kernel.  The workspace word 0 is
 * the asynchronous status of the tensor-core launches (chela_async_status).
 */
size_t chela_linattn_bwd_workspace_bytes(int B, int H, int L, int d_k, int d_v);
chela_status_t chela_linattn_bwd(const void *q, const void *k, const void *v, const void *d_o,
                                 float *dq, float *dk, float *dv, int B, int H, int L, int d_k, int d_v,
                                 chela_dtype_t in_dtype, chela_norm_t norm, float norm_eps, float scale,
                                 void *workspace, size_t workspace_bytes, cudaStream_t stream);

/*
 * Dense projection with optional SiLU, the building block of the Q/K/V formation (Eq. 12; Eqs. 10-11 in
 * their dense form): y = act(a w + bias), fp32 accumulation.
 * a : [M, K], a_dtype in {F32, BF16, BF16_PAIR}.  w : [K, N] row-major, w_dtype in {F32, BF16}.
 * bias : [N] fp32 or NULL.  y : [M, N], y_dtype in {F32, BF16, BF16_PAIR}.  act : 0 identity, 1 SiLU, 2 sigmoid.
 * Tensor-core path (tcgen05): a BF16 or BF16_PAIR, w BF16, y BF16 or BF16_PAIR, K a multiple of 64, N a
 * multiple of 128.  Other combinations without a pair run on an fp32 SIMT kernel; pairs outside the
 * tensor-core path are CHELA_ERR_UNSUPPORTED.  The workspace holds the asynchronous status word
 * (chela_async_status).
 */
size_t chela_dense_workspace_bytes(void);
chela_status_t chela_dense_fwd(const void *a, const void *w, const float *bias, void *y, int M, int K, int N,
                               int act, chela_dtype_t a_dtype, chela_dtype_t w_dtype, chela_dtype_t y_dtype,
                               void *workspace, size_t workspace_bytes, cudaStream_t stream);

/*
 * Asynchronous status of the last chela_linattn_fwd / chela_mixer_fwd launch that used `workspace`.
 * Device-side waits in the tensor-core kernel are bounded; a wait that gives up makes its CTA stop
 * cleanly and records CHELA_ERR_TIMEOUT in the first word of the workspace.  This call synchronises
 * `stream`, copies that word to the host and returns it (CHELA_OK if nothing was recorded, or if the
 * launch used a kernel without device-side waits).  `workspace` must be the pointer given to the
 * launch (for the mixer: its own workspace pointer).
 */
chela_status_t chela_async_status(const void *workspace, cudaStream_t stream);

/*
 * Test hook for the bounded waits (the paper has no counterpart).  Every device-side wait of the tensor-core kernels
 * gives up after `limit_cycles` SM cycles (<= 0: the default, about one second) and then ends as chela_async_status
 * describes.  skip_arrival != 0 makes the first CTA of the d = 64 linear-attention kernels and of the tensor-core
 * projection leave out one mbarrier arrival, so that the role waiting for it runs into the limit: the kernel returns by
 * itself, records CHELA_ERR_TIMEOUT, and words 8..11 of the workspace header keep the site of the wait, the CTA, the
 * chunk and the grid size.  Process-wide, not thread-safe, read by every later launch: set it, launch, set it back.
 */
void chela_debug_wait_control(long long limit_cycles, int skip_arrival);

/*
 * Measurement aid (the paper has no counterpart): the SM clock as the hardware counts it.  Enqueues one CTA of one
 * thread on `stream` that spins for spin_cycles SM cycles (clamped to [10 000, 2 000 000]) and writes two 64-bit
 * integers to the device buffer `out16` (16 bytes, 8-byte aligned): the SM cycles that passed and the nanoseconds of
 * the GPU's global timer over the same interval.  cycles * 1000 / nanoseconds = MHz.  Run right after a timed region it
 * shows the clock that region ended at; the driver's management interface was seen to report the maximum clock while
 * this ratio read 1400 MHz after a few hundred milliseconds of load.
 */
chela_status_t chela_debug_sm_clock(void *out16, long long spin_cycles, cudaStream_t stream);

/*
 * chela_linattn_fwd without a caller-provided workspace and without any allocation.  (The paper has no
 * counterpart: this is a packaging variant of the entry point above, same kernels, same results.)
 *
 * For callers that cannot allocate device memory: a plug-in inside a server whose device memory was all
 * handed to another framework's pool at start-up, a latency-critical loop in which cudaMalloc (it may
 * synchronise the device) is forbidden once initialisation is over, a component that only ever receives
 * finished input and output buffers.  Inputs and outputs are still the caller's; only the scratch (the
 * asynchronous status word and, for sequences that are split along L, the per-group state sums) comes
 * from an 8 MiB array built into the library image.  Every GPU that loads the library holds those 8 MiB
 * until the process exits.
 *
 *   - Arguments as chela_linattn_fwd, minus workspace and workspace_bytes.
 *   - A call whose chela_linattn_workspace_bytes() exceeds 8 MiB returns CHELA_ERR_WORKSPACE and launches
 *     nothing (use chela_linattn_fwd with your own workspace).  Plain bf16 and fp32 calls with d = 64 need the
 *     512-byte header only.  d = 128 calls with few (batch, head) pairs keep one 64 KiB state sum per group of a
 *     split sequence, up to one group per SM: B*H = 1 with L above about 130 000 tokens needs more than 8 MiB on a
 *     148-SM part and is refused.
 *   - The first call on each device looks up the device address of the built-in array (with that device
 *     current) and caches it; make that first call during set-up.
 *   - The call itself calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - All calls on one GPU share the one array, which keeps the previous call's contents.  Nothing in it
 *     needs to start at zero except the status word, which each launch clears on `stream` itself.  Two
 *     calls that overlap on the GPU (different streams without an ordering event) race on it: order them.
 *   - The asynchronous status word lives inside the built-in array: chela_linattn_static_ws_status(stream)
 *     synchronises `stream` and returns it for the current device, like chela_async_status, without allocating.
 */
chela_status_t chela_linattn_fwd_static_ws(const void *q, const void *k, const void *v, void *o,
                                           int B, int H, int L, int d_k, int d_v, int chunk,
                                           chela_dtype_t in_dtype, chela_dtype_t out_dtype,
                                           chela_norm_t norm, float norm_eps, float scale,
                                           cudaStream_t stream);
chela_status_t chela_linattn_static_ws_status(cudaStream_t stream);

/*
 * Token mixer forward without the gates (Eq. 7, Eqs. 10-12, Eq. 8 without G_a):
 *   A = silu(shortconv(X));  Z = longconv(A)
 *   Q = Z W_q + b_q,  K = Z W_k + b_k            (qk_diag = 0: dense D x D weights)
 *   Q = w_q . Z + b_q,  K = w_k . Z + b_k         (qk_diag = 1: w_q, w_k are length-D scalers, Eqs. 10-11)
 *   V = act(X W_v + b_v), act = SiLU if v_silu else identity (Eq. 12)
 *   O = per-head Norm(causal linear attention), head h = columns [h*D/H, (h+1)*D/H), scale 1.
 * x, o : [B, L, D] (in_dtype / out_dtype).  Dense weights : [D_in, D_out] row-major, in_dtype.
 * qk_diag scalers : [D], in_dtype.  Biases : [D] fp32 or NULL.  w_short : [D, short_width] fp32.
 * k_long : [D, L] fp32.  Supported: D/H in {64, 128}, chunk in {64, 128}, L <= 262144.
 */
size_t chela_mixer_workspace_bytes(int B, int L, int D, int H, int chunk, chela_dtype_t in_dtype);
chela_status_t chela_mixer_fwd(const void *x, const float *w_short, int short_width,
                               const float *k_long, const void *w_q, const void *w_k,
                               const void *w_v, const float *b_q, const float *b_k,
                               const float *b_v, int qk_diag, int v_silu, void *o, int B, int L,
                               int D, int H, int chunk, chela_dtype_t in_dtype,
                               chela_dtype_t out_dtype, chela_norm_t norm, float norm_eps,
                               void *workspace, size_t workspace_bytes, cudaStream_t stream);

/*
 * Token mixer forward with the gates (Eqs. 8, 9, 13, 14): with O the output of chela_mixer_fwd,
 *   G_a = silu(Z W_a + b_a),  G_o = sigmoid(Z W_o + b_o),  U = O . G_a . G_o + X . (1 - G_o).
 * (Eq. 9 prints the gate weight with the same symbol as the value projection; it is read as a weight of
 * its own, w_a.)  w_a, w_o : [D, D] row-major, in_dtype.  b_a, b_o : [D] fp32 or NULL.  u : [B, L, D]
 * out_dtype.  Everything else as chela_mixer_fwd; the workspace is larger (three more [B, L, D] buffers).
 */
size_t chela_mixer_gated_workspace_bytes(int B, int L, int D, int H, int chunk, chela_dtype_t in_dtype);
chela_status_t chela_mixer_gated_fwd(const void *x, const float *w_short, int short_width,
                                     const float *k_long, const void *w_q, const void *w_k,
                                     const void *w_v, const float *b_q, const float *b_k,
                                     const float *b_v, const void *w_a, const float *b_a,
                                     const void *w_o, const float *b_o, int qk_diag, int v_silu,
                                     void *u, int B, int L, int D, int H, int chunk,
                                     chela_dtype_t in_dtype, chela_dtype_t out_dtype, chela_norm_t norm,
                                     float norm_eps, void *workspace, size_t workspace_bytes,
                                     cudaStream_t stream);

/*
 * The long convolution for weights that do not change between calls (Eq. 6: y = F^-1 D_K F u; D_K, the spectrum of
 * the zero-padded kernel, depends on the weights only).  chela_longconv_prepare writes the spectra of all D kernels
 * and the transform's twiddle table into a caller-owned device buffer of chela_longconv_spectrum_bytes(L, D) bytes
 * (16-byte aligned; 0 = unsupported L or D); the *_prepared_fwd calls take that buffer in place of k_long and skip
 * that part of the work, with results identical to the calls they stand for.  The buffer is only valid for the
 * (L, D) and the weights it was prepared for, and must not be written while a call that reads it is in flight.
 *   chela_longconv_prepared_fwd : chela_longconv_fwd with `spectrum` in place of k_long.
 *   chela_mixer_prepared_fwd    : chela_mixer_fwd (w_a = w_o = NULL) or chela_mixer_gated_fwd (both given, with the
 *                                 gated workspace size) with `spectrum` in place of k_long.
 */
size_t chela_longconv_spectrum_bytes(int L, int D);
chela_status_t chela_longconv_prepare(const float *k_long, int L, int D, void *spectrum, size_t spectrum_bytes,
                                      cudaStream_t stream);
chela_status_t chela_longconv_prepared_fwd(const void *x, const void *spectrum, const float *w_short, int short_width,
                                           void *z, int B, int L, int D, chela_dtype_t in_dtype, chela_dtype_t out_dtype,
                                           void *workspace, size_t workspace_bytes, cudaStream_t stream);
chela_status_t chela_mixer_prepared_fwd(const void *x, const float *w_short, int short_width, const void *spectrum,
                                        const void *w_q, const void *w_k, const void *w_v, const float *b_q,
                                        const float *b_k, const float *b_v, const void *w_a, const float *b_a,
                                        const void *w_o, const float *b_o, int qk_diag, int v_silu, void *o, int B,
                                        int L, int D, int H, int chunk, chela_dtype_t in_dtype, chela_dtype_t out_dtype,
                                        chela_norm_t norm, float norm_eps, void *workspace, size_t workspace_bytes,
                                        cudaStream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* CHELA_H_ */
