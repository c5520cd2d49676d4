// Wavelet refinement (Sec. 3.5): Y_out = Y + W^{-1}( s * W Y ), orthonormal Haar
// over aligned blocks of 2^J tokens, level gates s broadcast over each band.
// By linearity this equals W^{-1}( (1 + s) * W Y ), which is what the kernel
// evaluates: analysis, scale by 1 + s, synthesis, all in shared memory.
#include "common.cuh"

namespace spectre {

template <typename WT> __device__ __forceinline__ float wl(const WT* p);
template <> __device__ __forceinline__ float wl<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float wl<bf16>(const bf16* p) { return __bfloat162float(*p); }

struct WaveletParams {
  const void* src; void* dst;
  int64_t s_sb, s_sl, s_sh, d_sb, d_sl, d_sh;
  int B, L, H, D, J, rows, chunks;
  const float* level_gates;       // [B,H,J+1,D] or NULL
  const float* qbar; const void* Ww1; const float* bw1; const void* Ww2; const float* bw2;
  int hidden; size_t hs_w1, hs_b1, hs_w2, hs_b2;
  const int* skip;                // [B] or NULL: non-zero = pass this batch entry through
};

// Pass-through of one (batch, head) slab for a skipped batch entry (nothing to do in place).
template <typename T>
__device__ __forceinline__ void wavelet_pass_through(const WaveletParams& p, int b, int h, int r0, int nr) {
  if (p.src == p.dst && p.s_sb == p.d_sb && p.s_sl == p.d_sl && p.s_sh == p.d_sh) return;
  const T* src = reinterpret_cast<const T*>(p.src) + b * p.s_sb + h * p.s_sh;
  T* dst = reinterpret_cast<T*>(p.dst) + b * p.d_sb + h * p.d_sh;
  constexpr int V = 16 / sizeof(T);
  const int nv = p.D / V;
  for (int i = threadIdx.x; i < nr * nv; i += blockDim.x) {
    const int r = i / nv, c = (i - r * nv) * V;
    *reinterpret_cast<uint4*>(dst + (int64_t)(r0 + r) * p.d_sl + c) = *reinterpret_cast<const uint4*>(src + (int64_t)(r0 + r) * p.s_sl + c);
  }
}

template <typename T, typename WT>
__global__ void __launch_bounds__(256) wavelet_kernel(const WaveletParams p) {
  extern __shared__ float smw[];
  float* tile = smw;                               // [rows][D]
  float* sg = tile + (size_t)p.rows * p.D;         // [(J+1)][D]  holds 1 + s
  float* u = sg + (size_t)(p.J + 1) * p.D;         // [hidden]
  const int chunk = blockIdx.x % p.chunks;
  const int bh = blockIdx.x / p.chunks, b = bh / p.H, h = bh - b * p.H;
  const int D = p.D, J = p.J;
  const int r0 = chunk * p.rows;
  const int nr = min(p.rows, p.L - r0);
  if (p.skip && p.skip[b]) { wavelet_pass_through<T>(p, b, h, r0, nr); return; }
  // level gates (step b): given, or the two-layer MLP on q_bar
  if (p.level_gates) {
    for (int i = threadIdx.x; i < (J + 1) * D; i += blockDim.x) sg[i] = 1.0f + p.level_gates[(size_t)bh * (J + 1) * D + i];
  } else {
    const WT* W1 = reinterpret_cast<const WT*>(p.Ww1) + h * p.hs_w1;
    const WT* W2 = reinterpret_cast<const WT*>(p.Ww2) + h * p.hs_w2;
    const float* qb = p.qbar + (size_t)bh * D;
    for (int j = threadIdx.x; j < p.hidden; j += blockDim.x) {
      float acc = p.bw1[h * p.hs_b1 + j];
      for (int c = 0; c < D; ++c) acc = fmaf(qb[c], wl<WT>(W1 + (size_t)c * p.hidden + j), acc);
      u[j] = gelu_erf(acc);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < (J + 1) * D; i += blockDim.x) {
      float acc = p.bw2[h * p.hs_b2 + i];
      for (int j = 0; j < p.hidden; ++j) acc = fmaf(u[j], wl<WT>(W2 + (size_t)j * (J + 1) * D + i), acc);
      sg[i] = 1.0f + acc;
    }
  }
  // load the tile
  const T* src = reinterpret_cast<const T*>(p.src) + b * p.s_sb + h * p.s_sh;
  const int nv = D / 4;
  for (int i = threadIdx.x; i < nr * nv; i += blockDim.x) {
    int r = i / nv, c = (i - r * nv) * 4;
    float4 v = io<T>::load4(src + (int64_t)(r0 + r) * p.s_sl + c);
    *reinterpret_cast<float4*>(tile + (size_t)r * D + c) = v;
  }
  __syncthreads();
  const float s = 0.70710678118654752440f;
  // analysis, in place: after level l the slots i*2^l hold a_l, i*2^l + 2^(l-1) hold d_l
  for (int l = 1; l <= J; ++l) {
    const int span = 1 << l, hs = span >> 1;
    const int nwork = (nr / span) * D;
    for (int i = threadIdx.x; i < nwork; i += blockDim.x) {
      int blk = i / D, c = i - blk * D;
      float* x0 = tile + (size_t)(blk * span) * D + c;
      float* x1 = x0 + (size_t)hs * D;
      float a = *x0, d = *x1;
      *x0 = (a + d) * s;
      *x1 = (a - d) * s;
    }
    __syncthreads();
  }
  // modulate: slot p of a 2^J block is a_J (p = 0) or d_l with l = ctz(p) + 1
  const int mask = (1 << J) - 1;
  for (int i = threadIdx.x; i < nr * D; i += blockDim.x) {
    int r = i / D, c = i - r * D;
    int pos = r & mask;
    int lev = pos == 0 ? 0 : 1 + (J - (__ffs(pos)));     // gate order a_J, d_J, ..., d_1
    tile[i] *= sg[lev * D + c];
  }
  __syncthreads();
  // synthesis
  for (int l = J; l >= 1; --l) {
    const int span = 1 << l, hs = span >> 1;
    const int nwork = (nr / span) * D;
    for (int i = threadIdx.x; i < nwork; i += blockDim.x) {
      int blk = i / D, c = i - blk * D;
      float* x0 = tile + (size_t)(blk * span) * D + c;
      float* x1 = x0 + (size_t)hs * D;
      float a = *x0, d = *x1;
      *x0 = (a + d) * s;
      *x1 = (a - d) * s;
    }
    __syncthreads();
  }
  T* dst = reinterpret_cast<T*>(p.dst) + b * p.d_sb + h * p.d_sh;
  for (int i = threadIdx.x; i < nr * nv; i += blockDim.x) {
    int r = i / nv, c = (i - r * nv) * 4;
    io<T>::store4(dst + (int64_t)(r0 + r) * p.d_sl + c, *reinterpret_cast<float4*>(tile + (size_t)r * D + c));
  }
}


// Register-resident variant for J <= 4: a thread owns one aligned block of 2^J tokens of two
// adjacent channels (4-byte bf16 pairs / 8-byte fp32 pairs), so the refinement is a single
// streaming pass with no shared-memory tile.  CTA = (batch, head): the level gates are computed
// (or fetched) once into shared memory, then threads sweep the head's blocks.
template <typename T> struct pair_io;
template <> struct pair_io<bf16> {
  static __device__ __forceinline__ float2 load(const bf16* p) {
    const uint32_t u = *reinterpret_cast<const uint32_t*>(p);
    return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
  }
  static __device__ __forceinline__ void store(bf16* p, float2 v) {
    __nv_bfloat162 o = __floats2bfloat162_rn(v.x, v.y);
    *reinterpret_cast<uint32_t*>(p) = *reinterpret_cast<uint32_t*>(&o);
  }
};
template <> struct pair_io<f16> {
  static __device__ __forceinline__ float2 load(const f16* p) { return __half22float2(*reinterpret_cast<const __half2*>(p)); }
  static __device__ __forceinline__ void store(f16* p, float2 v) { *reinterpret_cast<__half2*>(p) = __floats2half2_rn(v.x, v.y); }
};
template <> struct pair_io<float> {
  static __device__ __forceinline__ float2 load(const float* p) { return *reinterpret_cast<const float2*>(p); }
  static __device__ __forceinline__ void store(float* p, float2 v) { *reinterpret_cast<float2*>(p) = v; }
};

template <typename T, typename WT, int J>
__global__ void __launch_bounds__(256) wavelet_reg_kernel(const WaveletParams p) {
  extern __shared__ float smw[];
  float* sg = smw;                                 // [(J+1)][D]  holds 1 + s
  float* u = sg + (size_t)(J + 1) * p.D;           // [hidden]
  const int bh = blockIdx.x, b = bh / p.H, h = bh - b * p.H;
  const int D = p.D;
  if (p.skip && p.skip[b]) { wavelet_pass_through<T>(p, b, h, 0, p.L); return; }
  if (p.level_gates) {
    for (int i = threadIdx.x; i < (J + 1) * D; i += blockDim.x) sg[i] = 1.0f + p.level_gates[(size_t)bh * (J + 1) * D + i];
  } else {
    const WT* W1 = reinterpret_cast<const WT*>(p.Ww1) + h * p.hs_w1;
    const WT* W2 = reinterpret_cast<const WT*>(p.Ww2) + h * p.hs_w2;
    const float* qb = p.qbar + (size_t)bh * D;
    for (int j = threadIdx.x; j < p.hidden; j += blockDim.x) {
      float acc = p.bw1[h * p.hs_b1 + j];
      for (int c = 0; c < D; ++c) acc = fmaf(qb[c], wl<WT>(W1 + (size_t)c * p.hidden + j), acc);
      u[j] = gelu_erf(acc);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < (J + 1) * D; i += blockDim.x) {
      float acc = p.bw2[h * p.hs_b2 + i];
      for (int j = 0; j < p.hidden; ++j) acc = fmaf(u[j], wl<WT>(W2 + (size_t)j * (J + 1) * D + i), acc);
      sg[i] = 1.0f + acc;
    }
  }
  __syncthreads();
  constexpr int S = 1 << J;
  const float r2 = 0.70710678118654752440f;
  const int npair = D / 2, nblk = p.L / S;
  const T* src = reinterpret_cast<const T*>(p.src) + b * p.s_sb + h * p.s_sh;
  T* dst = reinterpret_cast<T*>(p.dst) + b * p.d_sb + h * p.d_sh;
  for (int item = threadIdx.x; item < nblk * npair; item += blockDim.x) {
    const int blk = item / npair, c = 2 * (item - blk * npair);
    float2 x[S];
#pragma unroll
    for (int r = 0; r < S; ++r) x[r] = pair_io<T>::load(src + (int64_t)(blk * S + r) * p.s_sl + c);
    // analysis in place: after level l, slot i * 2^l holds a_l and slot i * 2^l + 2^(l-1) holds d_l
#pragma unroll
    for (int l = 1; l <= J; ++l) {
      const int span = 1 << l, hs = span >> 1;
#pragma unroll
      for (int i = 0; i < S; i += span) {
        const float2 a = x[i], d = x[i + hs];
        x[i] = make_float2((a.x + d.x) * r2, (a.y + d.y) * r2);
        x[i + hs] = make_float2((a.x - d.x) * r2, (a.y - d.y) * r2);
      }
    }
    // modulate: slot 0 is a_J, slot r > 0 is d_l with l = ctz(r) + 1; gate order a_J, d_J, ..., d_1
#pragma unroll
    for (int r = 0; r < S; ++r) {
      const int lev = r == 0 ? 0 : 1 + (J - (__ffs(r)));
      x[r].x *= sg[lev * D + c];
      x[r].y *= sg[lev * D + c + 1];
    }
#pragma unroll
    for (int l = J; l >= 1; --l) {
      const int span = 1 << l, hs = span >> 1;
#pragma unroll
      for (int i = 0; i < S; i += span) {
        const float2 a = x[i], d = x[i + hs];
        x[i] = make_float2((a.x + d.x) * r2, (a.y + d.y) * r2);
        x[i + hs] = make_float2((a.x - d.x) * r2, (a.y - d.y) * r2);
      }
    }
#pragma unroll
    for (int r = 0; r < S; ++r) pair_io<T>::store(dst + (int64_t)(blk * S + r) * p.d_sl + c, x[r]);
  }
}

template <typename T, typename WT>
static int launch_wavelet_reg(const WaveletParams& p, int J, unsigned grid, size_t smem, cudaStream_t st) {
  switch (J) {
    case 1: wavelet_reg_kernel<T, WT, 1><<<grid, 256, smem, st>>>(p); break;
    case 2: wavelet_reg_kernel<T, WT, 2><<<grid, 256, smem, st>>>(p); break;
    case 3: wavelet_reg_kernel<T, WT, 3><<<grid, 256, smem, st>>>(p); break;
    default: wavelet_reg_kernel<T, WT, 4><<<grid, 256, smem, st>>>(p); break;
  }
  SPECTRE_LAUNCH_OK("wavelet_reg_kernel");
  return SPECTRE_OK;
}

}  // namespace spectre

using namespace spectre;

extern "C" int spectre_wavelet_refine(spectre_ctx* ctx, void* stream, const spectre_act* y_in, const spectre_act* y_out,
                                      const spectre_wavelet* w) {
  if (!ctx) return fail(SPECTRE_ERR_INVALID_ARG, "ctx is NULL");
  if (!w) return fail(SPECTRE_ERR_INVALID_ARG, "wavelet parameters are NULL");
  int rc = check_act(y_in, "y_in");
  if (rc != SPECTRE_OK) return rc;
  rc = check_act(y_out, "y_out");
  if (rc != SPECTRE_OK) return rc;
  if (y_in->B != y_out->B || y_in->L != y_out->L || y_in->H != y_out->H || y_in->D != y_out->D ||
      y_in->dtype != y_out->dtype)
    return fail(SPECTRE_ERR_INVALID_ARG, "y_in and y_out differ in shape or dtype");
  const int J = w->levels, L = y_in->L, D = y_in->D;
  if (J < 1 || J > 10) return fail(SPECTRE_ERR_INVALID_ARG, "wavelet levels must be in 1..10");
  if (L % (1 << J)) return fail(SPECTRE_ERR_INVALID_ARG, "2^J must divide L");
  if (!w->level_gates) {
    if (!w->qbar || !w->Ww1 || !w->bw1 || !w->Ww2 || !w->bw2)
      return fail(SPECTRE_ERR_INVALID_ARG, "level_gates is NULL and the MLP inputs are incomplete");
    if (w->hidden < 1 || w->hidden > 1024) return fail(SPECTRE_ERR_UNSUPPORTED, "wavelet hidden width must be in 1..1024");
    if (w->wdtype != SPECTRE_F32 && w->wdtype != SPECTRE_BF16) return fail(SPECTRE_ERR_INVALID_ARG, "unknown weight dtype");
  }
  if (J <= 4) {                              // register-resident streaming kernel
    SPECTRE_CUDA_OK(cudaSetDevice(ctx->device));
    cudaStream_t st0 = reinterpret_cast<cudaStream_t>(stream);
    const int hidden0 = w->level_gates ? 0 : w->hidden;
    WaveletParams p0 = {};
    p0.src = y_in->ptr; p0.dst = y_out->ptr;
    p0.s_sb = y_in->stride_b; p0.s_sl = y_in->stride_l; p0.s_sh = y_in->stride_h;
    p0.d_sb = y_out->stride_b; p0.d_sl = y_out->stride_l; p0.d_sh = y_out->stride_h;
    p0.B = y_in->B; p0.L = L; p0.H = y_in->H; p0.D = D; p0.J = J;
    p0.level_gates = w->level_gates; p0.qbar = w->qbar; p0.Ww1 = w->Ww1; p0.bw1 = w->bw1; p0.Ww2 = w->Ww2; p0.bw2 = w->bw2;
    p0.hidden = hidden0; p0.skip = w->skip;
    const size_t one0 = w->shared_across_heads ? 0 : 1;
    p0.hs_w1 = one0 * (size_t)D * hidden0; p0.hs_b1 = one0 * hidden0;
    p0.hs_w2 = one0 * (size_t)hidden0 * (J + 1) * D; p0.hs_b2 = one0 * (size_t)(J + 1) * D;
    const size_t smem0 = ((size_t)(J + 1) * D + hidden0) * sizeof(float);
    const unsigned grid0 = (unsigned)((size_t)p0.B * p0.H);
    const bool wbf0 = w->wdtype == SPECTRE_BF16;
    SPECTRE_IO_DISPATCH(y_in->dtype, {
      if (wbf0) return launch_wavelet_reg<T, bf16>(p0, J, grid0, smem0, st0);
      return launch_wavelet_reg<T, float>(p0, J, grid0, smem0, st0);
    });
  }
  const int span = 1 << J;
  int rows = (8192 / D) / span * span;      // about 32 KB of fp32 per CTA
  if (rows < span) rows = span;
  if (rows > L) rows = L;
  const int hidden = w->level_gates ? 0 : w->hidden;
  size_t smem = ((size_t)rows * D + (size_t)(J + 1) * D + hidden) * sizeof(float);
  if (smem > (size_t)ctx->max_smem_optin) return fail(SPECTRE_ERR_UNSUPPORTED, "2^J * D exceeds the shared-memory tile");
  SPECTRE_CUDA_OK(cudaSetDevice(ctx->device));
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  WaveletParams p = {};
  p.src = y_in->ptr; p.dst = y_out->ptr;
  p.s_sb = y_in->stride_b; p.s_sl = y_in->stride_l; p.s_sh = y_in->stride_h;
  p.d_sb = y_out->stride_b; p.d_sl = y_out->stride_l; p.d_sh = y_out->stride_h;
  p.B = y_in->B; p.L = L; p.H = y_in->H; p.D = D; p.J = J; p.rows = rows; p.chunks = (L + rows - 1) / rows;
  p.level_gates = w->level_gates; p.qbar = w->qbar; p.Ww1 = w->Ww1; p.bw1 = w->bw1; p.Ww2 = w->Ww2; p.bw2 = w->bw2;
  p.hidden = hidden; p.skip = w->skip;
  const size_t one = w->shared_across_heads ? 0 : 1;
  p.hs_w1 = one * (size_t)D * hidden; p.hs_b1 = one * hidden;
  p.hs_w2 = one * (size_t)hidden * (J + 1) * D; p.hs_b2 = one * (size_t)(J + 1) * D;
  const unsigned grid = (unsigned)((size_t)p.B * p.H * p.chunks);
  const bool wbf = w->wdtype == SPECTRE_BF16;
#define SPECTRE_WAVELET_LAUNCH(T, WT)                                                                           \
  do {                                                                                                          \
    if (smem > 48 * 1024)                                                                                       \
      SPECTRE_CUDA_OK(cudaFuncSetAttribute(wavelet_kernel<T, WT>, cudaFuncAttributeMaxDynamicSharedMemorySize,  \
                                           (int)smem));                                                         \
    wavelet_kernel<T, WT><<<grid, 256, smem, st>>>(p);                                                          \
  } while (0)
  SPECTRE_IO_DISPATCH(y_in->dtype, {
    if (wbf) SPECTRE_WAVELET_LAUNCH(T, bf16);
    else SPECTRE_WAVELET_LAUNCH(T, float);
  });
#undef SPECTRE_WAVELET_LAUNCH
  SPECTRE_LAUNCH_OK("wavelet_kernel");
  return SPECTRE_OK;
}
