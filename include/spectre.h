/*
 * spectre.h - C ABI of the B200 (sm_100a) SPECTRE spectral-mixer library.
 *
 * The library implements the per-head spectral token mixer of SPECTRE
 * (arXiv 2502.18394): real FFT along the sequence axis, multiplication of the
 * floor(n/2)+1 bins by a content-adaptive complex gate, inverse real FFT
 * (Sec. 3.2, Eq. 1-4), the Prefix-FFT cache for decoding (Sec. 3.3, Eq. 5,
 * Alg. 1) and the optional Haar wavelet refinement (Sec. 3.5).
 *
 * Conventions
 *   - Every tensor argument is CALLER-OWNED DEVICE memory unless a comment says
 *     "host".  The library never allocates or frees device memory in the calls
 *     below (spectre_create owns one small device table); scratch is passed in as
 *     `workspace`, sized by the matching *_workspace_bytes query.
 *   - All work is enqueued on the caller's stream (`stream` is a cudaStream_t
 *     passed as void*; NULL = the default stream).  No call synchronises.
 *   - Activations are [B, L, H, D] with D contiguous; strides are in elements.
 *     The base pointer and every stride must keep each D-row 16-byte aligned.
 *   - Complex numbers are interleaved (re, im) float32.
 *   - n = n_fft is the transform length, K = n/2 + 1 (integer division) the
 *     number of bins.  Supported n: 2^a for 0 <= a <= 17, and any
 *     n = 2^a 3^b 5^c 7^e <= 2048.  D must be a multiple of 8.
 *   - Every function returns a spectre_status; nothing throws or aborts.
 *     Arguments are validated on the host before anything is launched.  There is
 *     no CPU fallback: without a CUDA device every compute call fails.
 */
#ifndef SPECTRE_H_
#define SPECTRE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SPECTRE_OK = 0,
  SPECTRE_ERR_INVALID_ARG = 1,   /* null / misaligned pointer, bad shape, bad dtype      */
  SPECTRE_ERR_UNSUPPORTED = 2,   /* valid request outside the supported set              */
  SPECTRE_ERR_WORKSPACE = 3,     /* workspace missing or smaller than the query result   */
  SPECTRE_ERR_CUDA = 4,          /* a CUDA runtime call or launch failed                 */
  SPECTRE_ERR_TIMEOUT = 5,       /* a bounded on-chip wait ran out (spectre_poll_status) */
  SPECTRE_ERR_RANGE = 6          /* a 16-bit tensor-core mixer overflowed (spectre_poll_status) */
} spectre_status;

/* Element types of activations and ring buffers; weights are SPECTRE_F32 or SPECTRE_BF16. */
typedef enum { SPECTRE_F32 = 0, SPECTRE_BF16 = 1, SPECTRE_F16 = 2 } spectre_dtype;

typedef struct spectre_ctx spectre_ctx;   /* opaque: device properties, launch limits */

/* Creates a context for CUDA device `device`.  Besides host memory it owns six small device
 * tables (the 64-point and 49-point DFT matrices of the tensor-core mixers, 32 KiB each; the
 * twiddles between two 64-point stages and a quarter-wave twiddle table, 16 KiB each; the twiddles
 * of the four-step splits n = 4096 R, 63 KiB; the DFT matrices of the tensor-core radix-32 ... 2
 * kernels, 320 KiB) and one pinned status word, all released by spectre_destroy.  No other
 * call allocates. */
int spectre_create(spectre_ctx** out, int device);
int spectre_destroy(spectre_ctx* ctx);
/* The tensor-core mixers record two kinds of trouble in a status word instead of failing on
 * the device.  (1) They hand tiles between their warps through on-chip barriers whose waits are
 * bounded; a wait that runs out makes the kernel finish early.  (2) Their intermediates are
 * fp16 (see spectre_mixer_forward for the amplitude range this allows); a call whose input
 * leaves that range ends in Inf / NaN outputs, which the last epilogue notices.  Call this
 * after synchronising the stream: SPECTRE_OK, or - the record is cleared - SPECTRE_ERR_TIMEOUT
 * if any kernel since the last poll gave up on a wait (its output is invalid), else
 * SPECTRE_ERR_RANGE if one produced non-finite values (rerun that call on the fp32 path:
 * environment variable SPECTRE_FORCE_PATH=alu). */
int spectre_poll_status(spectre_ctx* ctx);
/* Diagnostic (the paper has no counterpart): enqueues a one-warp kernel whose bounded wait
 * runs out by construction - a barrier nobody arrives on, 4096 polls, no copy or MMA in
 * flight - and which reports it the way the mixers do, so that the path wait -> status word ->
 * spectre_poll_status can be exercised without disturbing a real kernel.  After the stream
 * is synchronised the next spectre_poll_status returns SPECTRE_ERR_TIMEOUT once. */
int spectre_selftest_wait_timeout(spectre_ctx* ctx, void* stream);
/* Static description of a status code. */
const char* spectre_status_string(int status);
/* Text of the most recent failure on the calling thread ("" if none). */
const char* spectre_last_error(void);

/* A [B, L, H, D] activation; D contiguous; strides in elements. */
typedef struct {
  void* ptr;
  int32_t dtype;                 /* spectre_dtype */
  int32_t B, L, H, D;
  int64_t stride_b, stride_l, stride_h;
} spectre_act;

/* Parameters of the gate network (Sec. 3.2 step 3).  All arrays are per head
 * ([H, ...]); with shared_across_heads != 0 they hold a single head's worth
 * that every head uses (Sec. 3.6: gates shared across heads). */
typedef struct {
  int32_t wdtype;                /* spectre_dtype of W1 and W2                        */
  int32_t hidden;                /* MLP hidden width (1..1024)                        */
  int32_t toeplitz_r;            /* 0 = Toeplitz update off; else bandwidth 2r+1      */
  int32_t shared_across_heads;
  const float* ln_gamma;         /* [H, D]                                            */
  const float* ln_beta;          /* [H, D]                                            */
  float ln_eps;
  const void* W1;                /* [H, D, hidden]                                    */
  const float* b1;               /* [H, hidden]                                       */
  const void* W2;                /* [H, hidden, 2K]  (re, im) interleaved per bin     */
  const float* b2;               /* [H, 2K]                                           */
  const float* modrelu_bias;     /* [H, K] or NULL (= 0)                              */
  const float* toeplitz;         /* [H, 2r+1, 2] complex taps t_{-r..r}, or NULL      */
} spectre_gate_params;

/*
 * spectre_gate - content-adaptive spectral gate (Sec. 3.2 step 3; Sec. 3.3.2
 * steps c-d; Alg. 1 DecodeStep).
 *   (a) mu = inv_count * sum_i q_i ; q_bar = LayerNorm_D(mu) ;
 *       o = GELU(q_bar W1 + b1) W2 + b2 ; g_k = o_{2k} + j o_{2k+1}
 *   (b) if toeplitz_r > 0: g_k <- g_k + sum_{m=-r..r} t_m g_{k-m} (zero boundary)
 *   (c) modReLU: g_k <- max(|g_k| + bias_k, 0) g_k / |g_k|
 *   then the positional phase g_k <- g_k exp(+j 2 pi k p / n), p = shift_all +
 *   shift[b] ("Positional Awareness"; decode uses p = t).
 * Either `q` (a [B, L, H, D] activation: the sum over L is computed here, and
 * inv_count <= 0 means 1/L) or `sum_q` ([B, H, D] float32, e.g. the cache's
 * running sum with inv_count = 1/N_max) must be given, not both.  B, H, D are
 * always passed (and must match q when q is given).
 *   shift      [B] int64 on the DEVICE, or NULL
 *   g_out      [B, H, K, 2] float32
 *   qbar_out   [B, H, D] float32 or NULL (input of the wavelet level-gate MLP)
 *   workspace  16-byte aligned; spectre_gate_workspace_bytes(...) is the size at which the
 *              pooling runs fastest (16 partial copies of the [B, H, D] sums); any size down
 *              to one copy (4*B*H*D bytes of sums, 4*B*H*hidden of hidden activations, plus
 *              8*B*H*K with the Toeplitz update on, each rounded up to 256) is accepted;
 *              with sum_q given the sums part is still counted but unused
 */
size_t spectre_gate_workspace_bytes(const spectre_ctx* ctx, int32_t B, int32_t H, int32_t D,
                                    int32_t n_fft, int32_t toeplitz_r);
int spectre_gate(spectre_ctx* ctx, void* stream,
                 const spectre_act* q, const float* sum_q,
                 int32_t B, int32_t H, int32_t D, float inv_count,
                 const spectre_gate_params* params, int32_t n_fft,
                 const int64_t* shift, int64_t shift_all,
                 float* g_out, float* qbar_out,
                 void* workspace, size_t workspace_bytes);

/*
 * spectre_gate_static - spectre_gate for callers that cannot provide scratch.
 * (The paper has no counterpart; this is a deployment convenience.)
 *
 * Some hosts of this library may not allocate device memory at all at the point
 * where the gate runs: an inference-engine plugin whose enqueue hook is handed
 * inputs and outputs only and whose host owns every byte of the memory pool, a
 * serving loop that must stay free of the implicit device-wide synchronisation
 * cudaMalloc/cudaFree bring, or a process pinned to a fixed memory budget.  For
 * them this entry point computes exactly what spectre_gate computes, with the
 * same kernels, but keeps its scratch (the pooled sum of the queries and, with
 * the Toeplitz update on, the pre-update gate) in an array compiled into the
 * library: spectre_gate_static_max_bytes() bytes (1 MiB) of device memory that
 * every GPU which loads the library holds until the process exits.  It calls no
 * cudaMalloc, cudaFree or any allocating routine; inputs and outputs are still
 * the caller's.
 *
 *   - Shapes whose minimum gate scratch (one copy of the sums; see spectre_gate)
 *     exceeds the array are rejected with SPECTRE_ERR_UNSUPPORTED and a message
 *     that names both sizes (with the Toeplitz update off the need is 4*B*H*D
 *     plus 4*B*H*hidden bytes, each rounded up to 256).
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress); make that first call before starting any stream
 *     capture on that device.
 *   - All calls on a device share the one array.  Each call clears the part it
 *     accumulates into, so leftovers of earlier calls are harmless, but two calls
 *     whose kernels may overlap on the GPU (different streams, no dependency
 *     between them) race on it and give wrong gates: serialise them, or use
 *     spectre_gate with separate workspaces.
 * Arguments and results are those of spectre_gate without the workspace pair.
 */
size_t spectre_gate_static_max_bytes(void);
int spectre_gate_static(spectre_ctx* ctx, void* stream,
                        const spectre_act* q, const float* sum_q,
                        int32_t B, int32_t H, int32_t D, float inv_count,
                        const spectre_gate_params* params, int32_t n_fft,
                        const int64_t* shift, int64_t shift_all,
                        float* g_out, float* qbar_out);

/* Wavelet refinement parameters (Sec. 3.5).  Either level_gates is given, or it
 * is NULL and the gates are computed from qbar by the two-layer MLP
 * s = GELU(qbar Ww1 + bw1) Ww2 + bw2 (linear output). */
typedef struct {
  int32_t levels;                /* J >= 1; 2^J must divide L; J <= 10              */
  int32_t hidden;                /* MLP hidden width (1..1024)                       */
  int32_t wdtype;                /* spectre_dtype of Ww1, Ww2                        */
  int32_t shared_across_heads;
  const float* level_gates;      /* [B, H, J+1, D] order a_J, d_J, ..., d_1; or NULL */
  const float* qbar;             /* [B, H, D]                                        */
  const void* Ww1;               /* [H, D, hidden]                                   */
  const float* bw1;              /* [H, hidden]                                      */
  const void* Ww2;               /* [H, hidden, (J+1) D]                             */
  const float* bw2;              /* [H, (J+1) D]                                     */
  const int32_t* skip;           /* [B] on the device, or NULL: batch entries with a
                                    non-zero flag are passed through unrefined (the
                                    module is "applied conditionally", Sec. 3.5; the
                                    controller that sets the flags is the caller's)   */
} spectre_wavelet;

/*
 * spectre_mixer_forward - Y = R_n^{-1}( diag(g) R_n(V) ) per (batch, head)
 * (Sec. 3.2 steps 2 and 4, Eq. 1, 3, 4); heads are written side by side in
 * [B, L, H, D], which is the concatenation of step 4.
 *   v, y     activations of identical shape and dtype; y may alias v where the
 *            transform is one kernel (the workspace query returns 0, and the
 *            bf16 / fp16 tensor-core paths n_fft = 196 with D = 64 and
 *            n_fft = 8192); on a multi-pass path a call whose v and y overlap
 *            anywhere between their first and last byte is refused with
 *            SPECTRE_ERR_INVALID_ARG
 *   g        [B, H, K, 2] float32, K = n_fft/2 + 1; one gain per bin per head,
 *            applied to all D columns; Im of the DC / Nyquist gains is ignored
 *   n_fft    == L: exact circular transform of Eq. 1;  > L: rows L..n_fft-1 are
 *            zero (the pad(.) of Sec. 3.3.1) and only rows 0..L-1 are written
 *   wrm      NULL, or the wavelet refinement applied to Y afterwards (Sec. 3.5)
 *   workspace  >= spectre_mixer_workspace_bytes(...) bytes, 16-byte aligned
 *              (0 bytes / NULL allowed when the query returns 0).  For bf16 / fp16,
 *              n_fft = 196, D = 64 the workspace only holds the level gates that
 *              wrm's MLP produces for the refinement fused into the mixer kernel
 *              (B H 3 D floats): with less, the refinement runs as its own kernel
 * Amplitude range of the 16-bit paths.  bf16 / fp16 activations at n_fft = 196 (D = 64) and
 * n_fft = 4096 ... 131072 run on the tensor cores with fp16 operands between the stages and
 * fixed power-of-two stage scales (unitary overall), fp32 accumulation.  Noise-like data passes
 * at any plausible magnitude, but a column with a constant or periodic component of amplitude A
 * concentrates A sqrt(n_fft) in one bin: beyond A of about 250 at n_fft = 131072, 500 at 8192 and
 * 1000 at 196 an intermediate exceeds 65504, the outputs turn into Inf / NaN, and
 * spectre_poll_status reports SPECTRE_ERR_RANGE.  Data whose magnitude is below about 1e-3
 * gradually loses accuracy in fp16 subnormals, without a report.  f32 activations, and any
 * activations with the environment variable SPECTRE_FORCE_PATH=alu, take the fp32 path, which has
 * neither limit.
 */
size_t spectre_mixer_workspace_bytes(const spectre_ctx* ctx, int32_t B, int32_t L, int32_t H,
                                     int32_t D, int32_t n_fft, int32_t dtype);
int spectre_mixer_forward(spectre_ctx* ctx, void* stream,
                          const spectre_act* v, const float* g, const spectre_act* y,
                          int32_t n_fft, const spectre_wavelet* wrm,
                          void* workspace, size_t workspace_bytes);

/*
 * spectre_wavelet_refine - Y_out = Y_in + W^{-1}( s * W Y_in ) with the
 * orthonormal Haar transform W over aligned blocks of 2^J tokens (Sec. 3.5
 * steps a, c, d); y_out may alias y_in.
 */
int spectre_wavelet_refine(spectre_ctx* ctx, void* stream,
                           const spectre_act* y_in, const spectre_act* y_out,
                           const spectre_wavelet* wrm);

/* Prefix-FFT cache state (Alg. 1 "persistent state"), all caller-owned. */
typedef struct {
  int32_t B, H, D, N_max;
  int32_t buf_dtype;             /* spectre_dtype of V_buf, Q_buf and of the tokens */
  int32_t reserved;
  float* prefix_fft;             /* [B, H, K, D, 2] float32, K = N_max/2 + 1        */
  void* V_buf;                   /* [B, N_max, H, D] ring buffer                    */
  void* Q_buf;                   /* [B, N_max, H, D] ring buffer                    */
  float* sum_q;                  /* [B, H, D] float32 running sum of queries        */
} spectre_cache;

/*
 * spectre_prefix_cache_prefill - PreFill of Alg. 1 (Sec. 3.3.1):
 * prefix_fft = R_{N_max}(pad(V, N_max)) (unnormalised, Eq. 1), ring buffers
 * rows 0..L-1 <- tokens and rows L..N_max-1 <- 0, sum_q = sum_i q_i.
 * q, v: [B, L, H, D] with L <= N_max, dtype == buf_dtype.  N_max must be a
 * supported n.  workspace >= spectre_prefill_workspace_bytes(...) bytes.
 * The ring buffers are written by the passes that read q and v (q and v must
 * not overlap V_buf or Q_buf).
 */
size_t spectre_prefill_workspace_bytes(const spectre_ctx* ctx, int32_t B, int32_t H, int32_t D,
                                       int32_t N_max);
int spectre_prefix_cache_prefill(spectre_ctx* ctx, void* stream, const spectre_cache* cache,
                                 const spectre_act* q, const spectre_act* v,
                                 void* workspace, size_t workspace_bytes);

/*
 * spectre_prefix_cache_append - DecodeStep of Alg. 1, steps (a)-(b) of
 * Sec. 3.3.2: with i = t mod N_max and (v_old, q_old) = ring-buffer row i if
 * t >= N_max else 0, for every bin k
 *   prefix_fft[k] += (v_t - v_old) exp(-j 2 pi k t / N_max)            (Eq. 5)
 * then V_buf[i] <- v_t, Q_buf[i] <- q_t, sum_q += q_t - q_old.
 * q_t, v_t: [B, H, D] contiguous, dtype buf_dtype.  t >= 0 is the absolute
 * position of the new token; N_max may be any integer >= 2 here.
 */
int spectre_prefix_cache_append(spectre_ctx* ctx, void* stream, const spectre_cache* cache,
                                const void* q_t, const void* v_t, int64_t t);

/* Largest number of read-out rows one decode step returns. */
#define SPECTRE_DECODE_MAX_ROWS 4

/*
 * spectre_prefix_cache_decode_step - the whole DecodeStep of Alg. 1 for one
 * token (Sec. 3.3.2 steps a-e), returning selected rows of the read-out:
 *   (a)-(b) exactly what spectre_prefix_cache_append does for (q_t, v_t, t);
 *   (c)-(d) g = gate of sum_q / N_max with the positional phase p = t
 *           (spectre_gate with the cache's running sum, inv_count = 1/N_max);
 *   (e)     for each listed row r, the entry r of
 *           V~ = R^{-1}_{N_max}( diag(g) prefix_fft ) by its definition,
 *             V~[r] = (1/N) sum_k w_k Re( g_k prefix_fft[k] exp(+j 2 pi k r / N) ),
 *           w_0 = w_{N/2} = 1 and w_k = 2 otherwise (Im of the DC / Nyquist
 *           products drops out), N = N_max: O(K D) per row, the per-token cost
 *           quoted at the end of Sec. 3.3.2, instead of a full inverse transform.
 * The spectrum is read and written once: the rank-one update of Eq. 5 and the
 * row sums run in the same pass (the gate needs only sum_q, so it is computed
 * first).  With the phase p = t, row r of V~ is row (r + t) mod N_max of the
 * un-phased window, i.e. ring-buffer slot (r + t) mod N_max; Alg. 1 returns rows
 * N_max - L' .. N_max - 1.
 *   q_t, v_t  [B, H, D] contiguous, dtype buf_dtype (device)
 *   params    gate network; K = N_max/2 + 1 bins
 *   rows      HOST array of nrows indices in [0, N_max), 1 <= nrows <= SPECTRE_DECODE_MAX_ROWS
 *   y_rows    [B, nrows, H, D] contiguous, dtype buf_dtype (device), written
 *   g_out     [B, H, K, 2] float32 (device), written: the gate of this step
 *   workspace >= spectre_decode_workspace_bytes(...) bytes, 16-byte aligned
 * Errors: as spectre_prefix_cache_append and spectre_gate; a row outside the
 * window or nrows out of range is SPECTRE_ERR_INVALID_ARG before any launch.
 */
size_t spectre_decode_workspace_bytes(const spectre_ctx* ctx, int32_t B, int32_t H, int32_t D,
                                      int32_t N_max, int32_t nrows, int32_t toeplitz_r);
int spectre_prefix_cache_decode_step(spectre_ctx* ctx, void* stream, const spectre_cache* cache,
                                     const void* q_t, const void* v_t, int64_t t,
                                     const spectre_gate_params* params,
                                     const int32_t* rows, int32_t nrows, void* y_rows, float* g_out,
                                     void* workspace, size_t workspace_bytes);

/*
 * spectre_prefix_cache_readout - step (e) of Sec. 3.3.2 for the whole window:
 * y = R^{-1}_{N_max}( diag(g) prefix_fft ), rows 0..L-1 of it (L = y->L <= N_max;
 * Alg. 1 returns rows N_max - L' .. N_max - 1, so pass L = N_max and slice).
 * The inverse half of the mixer, entered with the cached half spectra instead of
 * a forward transform; Im of the DC / Nyquist products is dropped (App. B).
 *   g       [B, H, K, 2] float32, e.g. the g_out of spectre_prefix_cache_decode_step
 *   y       [B, L, H, D] activation, any supported dtype; written
 *   workspace >= spectre_readout_workspace_bytes(...) bytes, 16-byte aligned
 *           (0 / NULL allowed when the query returns 0)
 * N_max must be a supported transform length.  The same rows equal
 * spectre_mixer_forward(V_buf, g) because prefix_fft = R(V_buf); this entry
 * point does half the work and does not need the ring buffer.
 * bf16 / fp16 rows with N_max = 4096 * 2^r (r <= 5) and D <= 64 take the tensor
 * cores: the gated spectra become fp16 operand images and the inverse stages of
 * spectre_mixer_forward's long-sequence path run on them (same amplitude range and
 * SPECTRE_ERR_RANGE report as there; SPECTRE_FORCE_PATH=alu, fp32 rows, or a workspace
 * too small for the operand images of one (batch, head) keep the fp32 kernels).
 */
size_t spectre_readout_workspace_bytes(const spectre_ctx* ctx, int32_t B, int32_t H, int32_t D,
                                       int32_t N_max);
int spectre_prefix_cache_readout(spectre_ctx* ctx, void* stream, const spectre_cache* cache,
                                 const float* g, const spectre_act* y,
                                 void* workspace, size_t workspace_bytes);

/*
 * spectre_mixer_backward - gradients of <dy, Y> for Y = spectre_mixer_forward(v, g)
 * (Eq. 3-4 are real-linear in V and in (Re g, Im g); Sec. 3.7 "fully differentiable").
 * With Vhat = R_n(pad v), Ghat = R_n(pad dy), w_0 = w_{n/2} = 1 and w_k = 2 otherwise:
 *   dv   = R_n^{-1}( conj(g) Ghat ), rows 0..L-1        (the mixer on dy with the conjugate gate)
 *   dg_k = dL/dRe g_k + j dL/dIm g_k = (w_k / n) sum_c conj(Vhat_{k,c}) Ghat_{k,c}
 * v, dy, dv: activations of identical shape and dtype; dv may alias dy where
 * spectre_mixer_forward allows y to alias v.  dv or dg may be NULL to skip that
 * gradient (not both).  dg: [B, H, K, 2] float32.  dv runs on the same kernels as
 * the forward pass; dg uses two forward-only fp32 transforms and a reduction.
 * workspace >= spectre_mixer_backward_workspace_bytes(...), 16-byte aligned; any size
 * down to the conjugate gate + the forward workspace + two (batch, head) slabs of
 * spectrum (n_fft * D/2 * 8 bytes each) is accepted.
 */
size_t spectre_mixer_backward_workspace_bytes(const spectre_ctx* ctx, int32_t B, int32_t L, int32_t H,
                                              int32_t D, int32_t n_fft, int32_t dtype);
int spectre_mixer_backward(spectre_ctx* ctx, void* stream,
                           const spectre_act* v, const spectre_act* dy, const float* g,
                           const spectre_act* dv, float* dg, int32_t n_fft,
                           void* workspace, size_t workspace_bytes);

/*
 * spectre_project_qv - token projections of Sec. 3.2 step 1 (Eq. 2), per head:
 *   Q = X W^(q),  V = X W^(v),  X the head's [L, D] slice, W [D, D] (input channel first),
 * on the tensor cores (bf16 operands, fp32 accumulation), with the pooled query sum
 *   sum_q[b, h, :] = sum_t Q[b, t, h, :]   (fp32, taken from the accumulators)
 * of step 3a as a by-product, so that spectre_gate can be called with sum_q
 * (inv_count = 1/L) instead of reading Q again.
 *   x, q, v   [B, L, H, D] bf16 activations, D = 64, three distinct buffers
 *   Wq, Wv    [H, D, D] of dtype wdtype (SPECTRE_F32 or SPECTRE_BF16; rounded to bf16)
 *   sum_q     [B, H, D] float32, overwritten; or NULL
 *   workspace >= spectre_project_workspace_bytes(ctx, H, D) bytes, 16-byte aligned
 * Other dtypes or head widths: SPECTRE_ERR_UNSUPPORTED.
 */
size_t spectre_project_workspace_bytes(const spectre_ctx* ctx, int32_t H, int32_t D);
int spectre_project_qv(spectre_ctx* ctx, void* stream, const spectre_act* x,
                       const void* Wq, const void* Wv, int32_t wdtype,
                       const spectre_act* q, const spectre_act* v, float* sum_q,
                       void* workspace, size_t workspace_bytes);

#ifdef __cplusplus
}
#endif
#endif  /* SPECTRE_H_ */
