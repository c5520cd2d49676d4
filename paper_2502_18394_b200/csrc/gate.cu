// Content-adaptive spectral gate (Sec. 3.2 step 3; Sec. 3.3.2 steps c-d).
//   pool_kernel      sum of the query tokens over the sequence (bandwidth-bound)
//   gate_hidden_kernel LayerNorm + hidden layer once per (head, batch group), long transforms only
//   gate_out_kernel    LayerNorm + hidden layer (per CTA, short transforms) and the output layer as a
//                      stream over W2, 1-8 batch entries per pass; with the Toeplitz update off it also applies modReLU and
//                      the positional phase
//   gate_post_kernel Toeplitz update, modReLU, phase (only when r > 0)
#include "tc_common.cuh"

#include <atomic>
#include <string>
#include <type_traits>

namespace spectre {

// ---- pooled sum over the sequence --------------------------------------------
// Grid (groups of 32 vectors, slices of the sequence, B).  A lane owns one 8-channel vector of the
// [H*D] row, so a warp reads 512 contiguous bytes of a row; the CTA's 8 warps take rows 8 apart with
// up to 8 rows per thread in flight and four CTAs per SM.  The warps' partial sums meet in shared memory, and the CTA adds
// one value per channel with float atomics into copy (slice mod ncopy) of sums[ncopy][B,H,D] (zeroed
// by the caller on the same stream), which keeps the contention per address low; a CTA that holds the
// whole sequence stores its sums instead.
template <typename T> struct vec8;
template <> struct vec8<bf16> {
  typedef uint4 raw;
  static constexpr int kRows = 8;
  static __device__ __forceinline__ raw load(const bf16* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }
  static __device__ __forceinline__ raw zero() { return make_uint4(0u, 0u, 0u, 0u); }
  static __device__ __forceinline__ void add(const raw& r, float (&a)[8]) {
    const uint32_t u[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      a[2 * i] += __uint_as_float(u[i] << 16);
      a[2 * i + 1] += __uint_as_float(u[i] & 0xffff0000u);
    }
  }
};
template <> struct vec8<f16> {
  typedef uint4 raw;
  static constexpr int kRows = 8;
  static __device__ __forceinline__ raw load(const f16* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }
  static __device__ __forceinline__ raw zero() { return make_uint4(0u, 0u, 0u, 0u); }
  static __device__ __forceinline__ void add(const raw& r, float (&a)[8]) {
    const uint32_t u[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 v = __half22float2(*reinterpret_cast<const __half2*>(&u[i]));
      a[2 * i] += v.x;
      a[2 * i + 1] += v.y;
    }
  }
};
template <> struct vec8<float> {
  struct raw { float4 lo, hi; };
  static constexpr int kRows = 4;
  static __device__ __forceinline__ raw load(const float* p) {
    raw r;
    r.lo = __ldg(reinterpret_cast<const float4*>(p));
    r.hi = __ldg(reinterpret_cast<const float4*>(p) + 1);
    return r;
  }
  static __device__ __forceinline__ raw zero() {
    raw r;
    r.lo = make_float4(0.f, 0.f, 0.f, 0.f);
    r.hi = r.lo;
    return r;
  }
  static __device__ __forceinline__ void add(const raw& r, float (&a)[8]) {
    a[0] += r.lo.x; a[1] += r.lo.y; a[2] += r.lo.z; a[3] += r.lo.w;
    a[4] += r.hi.x; a[5] += r.hi.y; a[6] += r.hi.z; a[7] += r.hi.w;
  }
};

// RING: the rows also go, as loaded, into the dense copy ring[B][N][H][D]; rows L..N-1 of it are zeroed
// (the ring buffer of the Prefix-FFT cache, Alg. 1 PreFill), and the slices cover N rows instead of L.
template <typename T, bool RING>
__global__ void __launch_bounds__(256, 4) pool_kernel(const T* __restrict__ q, int64_t sb, int64_t sl, int64_t sh, int L,
                                                   int H, int D, int rows_per, int ncopy, size_t copy_stride,
                                                   float* __restrict__ sums, T* __restrict__ ring, int N) {
  __shared__ float red[8][8][32];                              // [warp][channel][lane]
  // the gate kernels behind this one may start early: they stream weights before they need the sums
  asm volatile("griddepcontrol.launch_dependents;");
  constexpr int R = vec8<T>::kRows;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int b = blockIdx.z;
  const int vec_per_head = D / 8, nvec = H * vec_per_head;
  const int vi = blockIdx.x * 32 + lane;
  const bool live = vi < nvec;
  const int h = live ? vi / vec_per_head : 0, c = live ? (vi - h * vec_per_head) * 8 : 0;
  const T* base = q + b * sb + h * sh + c;
  const int r0 = blockIdx.y * rows_per, r1 = min(L, r0 + rows_per), r2 = RING ? min(N, r0 + rows_per) : r1;
  float acc[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0.f;
  if (live) {
    T* out = RING ? ring + ((size_t)b * N * H + h) * D + c : nullptr;
    for (int r = r0 + warp; r < r2; r += 8 * R) {
      typename vec8<T>::raw v[R];
#pragma unroll
      for (int u = 0; u < R; ++u) v[u] = (r + 8 * u < r1) ? vec8<T>::load(base + (int64_t)(r + 8 * u) * sl) : vec8<T>::zero();
#pragma unroll
      for (int u = 0; u < R; ++u) {
        vec8<T>::add(v[u], acc);
        if (RING && r + 8 * u < r2) *reinterpret_cast<typename vec8<T>::raw*>(out + (size_t)(r + 8 * u) * H * D) = v[u];
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) red[warp][i][lane] = acc[i];
  __syncthreads();
  float s = 0.f;                                               // thread (channel = warp, lane) adds up the 8 warps
#pragma unroll
  for (int w = 0; w < 8; ++w) s += red[w][warp][lane];
  // with several slices the kernel runs as the programmatic dependent of the kernel that clears the sums:
  // everything above overlaps it, the additions wait for it (no effect in an ordinary launch)
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (live) {
    float* dst = sums + (size_t)(blockIdx.y % ncopy) * copy_stride + ((size_t)b * H + h) * D + c + warp;
    if (gridDim.y == 1) *dst = s;                              // the only slice: no other CTA adds to this address
    else atomicAdd(dst, s);
  }
}

// Clears the partial sums ahead of a pooling pass with several slices; lets that pass start at once.
__global__ void __launch_bounds__(256) pool_clear_kernel(float4* __restrict__ sums, size_t n4) {
  asm volatile("griddepcontrol.launch_dependents;");
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n4) sums[i] = make_float4(0.f, 0.f, 0.f, 0.f);
}

// Sums of q over the sequence into *ncopy_used <= ncopy_max partial copies (the consumer adds them up);
// with `ring`, also the copy of q into ring[B][N][H][D] (zero rows from L on).
static int pool_launch(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* q, float* sums, int ncopy_max,
                       int* ncopy_used, void* ring, int N) {
  const int rows = ring ? N : q->L;
  const size_t copy_stride = (size_t)q->B * q->H * q->D;
  const int groups = (q->H * (q->D / 8) + 31) / 32;
  if (q->B > 65535) return fail(SPECTRE_ERR_UNSUPPORTED, "B exceeds 65535");
  // one resident wave (four CTAs per SM) of equal slices, never a few CTAs more than fit at once;
  // at least 8 rows (one per warp) per CTA
  const long long per_slice = (long long)groups * q->B;
  long long slices = (4LL * ctx->sm_count) / per_slice;
  if (slices < 1) slices = 1;
  int rows_per = (int)((rows + slices - 1) / slices);
  if (rows_per < 8) rows_per = 8;
  const int nslice = (rows + rows_per - 1) / rows_per;
  int ncopy = (nslice + 15) / 16;                              // <= 16 CTAs add into one address
  if (ncopy > 8) ncopy = 8;                                    // one batch of loads for the consumer
  if (ncopy > ncopy_max) ncopy = ncopy_max;
  if (ncopy < 1) ncopy = 1;
  *ncopy_used = ncopy;
  // Several slices add into the same words: a small kernel clears them (D is a multiple of 8 and the sums are
  // 16-byte aligned: whole float4) and the pooling kernel, its programmatic dependent, reads its rows meanwhile.
  // A memset node in the stream instead costs the step 3.6 us at L = 8192.
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)groups, (unsigned)nslice, (unsigned)q->B);
  cfg.blockDim = dim3(256);
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 0;
  if (nslice > 1) {
    const size_t n4 = copy_stride * ncopy / 4;
    if ((reinterpret_cast<uintptr_t>(sums) & 15) || (copy_stride * ncopy) % 4) {
      SPECTRE_CUDA_OK(cudaMemsetAsync(sums, 0, copy_stride * ncopy * sizeof(float), st));
    } else {
      pool_clear_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(reinterpret_cast<float4*>(sums), n4);
      SPECTRE_LAUNCH_OK("pool_clear_kernel");
      cfg.numAttrs = 1;
    }
  }
  SPECTRE_IO_DISPATCH(q->dtype, {
    if (ring)
      SPECTRE_CUDA_OK(cudaLaunchKernelEx(&cfg, pool_kernel<T, true>, reinterpret_cast<const T*>(q->ptr), (int64_t)q->stride_b,
                                         (int64_t)q->stride_l, (int64_t)q->stride_h, (int)q->L, (int)q->H, (int)q->D, rows_per,
                                         ncopy, copy_stride, sums, reinterpret_cast<T*>(ring), N));
    else
      SPECTRE_CUDA_OK(cudaLaunchKernelEx(&cfg, pool_kernel<T, false>, reinterpret_cast<const T*>(q->ptr), (int64_t)q->stride_b,
                                         (int64_t)q->stride_l, (int64_t)q->stride_h, (int)q->L, (int)q->H, (int)q->D, rows_per,
                                         ncopy, copy_stride, sums, static_cast<T*>(nullptr), 0));
  });
  SPECTRE_LAUNCH_OK("pool_kernel");
  return SPECTRE_OK;
}

int pool_sum(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* q, float* sums, int ncopy_max, int* ncopy_used) {
  return pool_launch(ctx, st, q, sums, ncopy_max, ncopy_used, nullptr, 0);
}

// Prefill of the cache's query side in one pass over q: sum over the sequence into sums[B,H,D] and the ring copy.
int pool_sum_ring(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* q, float* sums, void* ring, int N) {
  int used = 1;
  return pool_launch(ctx, st, q, sums, 1, &used, ring, N);
}

// ---- MLP ---------------------------------------------------------------------
template <typename WT> __device__ __forceinline__ float wload(const WT* p);
template <> __device__ __forceinline__ float wload<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float wload<bf16>(const bf16* p) {
  return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p)) << 16);
}
template <typename WT> __device__ __forceinline__ float2 wload2(const WT* p);
template <> __device__ __forceinline__ float2 wload2<float>(const float* p) { return __ldg(reinterpret_cast<const float2*>(p)); }
template <> __device__ __forceinline__ float2 wload2<bf16>(const bf16* p) {
  unsigned r = __ldg(reinterpret_cast<const unsigned*>(p));
  return make_float2(__uint_as_float(r << 16), __uint_as_float(r & 0xffff0000u));
}

// q_bar = LN(inv_count * sum) into shared memory (Sec. 3.2 step 3a), then the hidden layer
// u = GELU(q_bar W1 + b1), for nb <= NB batch entries of one head at once: the means are spread over
// the CTA, a warp normalises one entry, then a thread takes one hidden unit for every g-th batch
// entry (g = threads / hidden groups), so a weight column is fetched once per group, not per entry.
// sums points at the first entry's [D] row, bstride is the distance between batch entries;
// u is written as [hidden][ustride] (batch entry fastest).
// STAGED: W1 points at a copy of the head's weights in shared memory (made before the wait on the
// producer of the sums), so the hidden layer adds no memory round trip behind the sums.
template <typename WT> __device__ __forceinline__ float wvalue(WT x);
template <> __device__ __forceinline__ float wvalue<float>(float x) { return x; }
template <> __device__ __forceinline__ float wvalue<bf16>(bf16 x) { return __bfloat162float(x); }
template <typename WT, bool STAGED> __device__ __forceinline__ float wget(const WT* p) {
  if constexpr (STAGED) return wvalue<WT>(*p);
  else return wload<WT>(p);
}

template <typename WT, int NB, bool STAGED>
__device__ __forceinline__ void descriptor_and_hidden(const float* __restrict__ sums, size_t bstride, int nb, int ncopy,
                                                      size_t copy_stride, float inv_count, int D, int hidden,
                                                      const float* __restrict__ gamma, const float* __restrict__ beta,
                                                      float eps, const WT* __restrict__ W1, const float* __restrict__ b1,
                                                      float* qbar, float* u, int ustride) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  if (NB > 1 && ncopy == 1) {                                // means, one copy: up to 4 channels per thread in flight
    for (int e0 = threadIdx.x; e0 < nb * D; e0 += 4 * blockDim.x) {
      float v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int e = e0 + u * (int)blockDim.x, bb = e / D, c = e - bb * D;
        v[u] = e < nb * D ? sums[(size_t)bb * bstride + c] : 0.f;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int e = e0 + u * (int)blockDim.x;
        if (e < nb * D) qbar[e] = v[u] * inv_count;
      }
    }
  } else {
    for (int e = threadIdx.x; e < nb * D; e += blockDim.x) {   // means: the whole CTA, one channel per thread
      const int bb = e / D, c = e - bb * D;
      const float* sb = sums + (size_t)bb * bstride + c;
      float m = 0.f;
      for (int k0 = 0; k0 < ncopy; k0 += 8) {                   // eight copies in flight at once
        float v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] = (k0 + k < ncopy) ? sb[(size_t)(k0 + k) * copy_stride] : 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) m += v[k];
      }
      qbar[e] = m * inv_count;
    }
  }
  __syncthreads();
  for (int bb = warp; bb < nb; bb += nw) {                    // statistics: one warp per batch entry
    float* qb = qbar + bb * D;
    float part = 0.f;
    for (int c = lane; c < D; c += 32) part += qb[c];
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    const float mean = part / (float)D;
    part = 0.f;
    for (int c = lane; c < D; c += 32) {
      float dlt = qb[c] - mean;
      part += dlt * dlt;
    }
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    const float rstd = 1.0f / sqrtf(part / (float)D + eps);
    for (int c = lane; c < D; c += 32) qb[c] = gamma[c] * (qb[c] - mean) * rstd + beta[c];
  }
  __syncthreads();
  if constexpr (NB == 1) {
    for (int jj = threadIdx.x; jj < hidden; jj += blockDim.x) {
      float acc = b1[jj];
      int c = 0;
      for (; c + 32 <= D; c += 32) {                // 32 independent loads in flight
        float wv[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) wv[i] = wget<WT, STAGED>(W1 + (size_t)(c + i) * hidden + jj);
#pragma unroll
        for (int i = 0; i < 32; ++i) acc = fmaf(qbar[c + i], wv[i], acc);
      }
      for (; c < D; ++c) acc = fmaf(qbar[c], wget<WT, STAGED>(W1 + (size_t)c * hidden + jj), acc);
      u[jj * ustride] = gelu_erf(acc);
    }
    __syncthreads();
    return;
  }
  int groups = (int)blockDim.x / hidden;
  groups = groups < 1 ? 1 : (groups > nb ? nb : groups);
  for (int item = threadIdx.x; item < groups * hidden; item += blockDim.x) {
    const int gi = item / hidden, jj = item - gi * hidden;
    float acc[NB];                                  // slot s: batch entry gi + s * groups
#pragma unroll
    for (int sl = 0; sl < NB; ++sl) acc[sl] = b1[jj];
    int c = 0;
    for (; c + 32 <= D; c += 32) {                  // 32 independent loads in flight
      float wv[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) wv[i] = wget<WT, STAGED>(W1 + (size_t)(c + i) * hidden + jj);
#pragma unroll
      for (int sl = 0; sl < NB; ++sl) {
        const int bb = gi + sl * groups;
        if (bb < nb) {
          const float* qb = qbar + bb * D + c;
#pragma unroll
          for (int i = 0; i < 32; ++i) acc[sl] = fmaf(qb[i], wv[i], acc[sl]);
        }
      }
    }
    for (; c < D; ++c) {
      const float wv = wget<WT, STAGED>(W1 + (size_t)c * hidden + jj);
#pragma unroll
      for (int sl = 0; sl < NB; ++sl) {
        const int bb = gi + sl * groups;
        if (bb < nb) acc[sl] = fmaf(qbar[bb * D + c], wv, acc[sl]);
      }
    }
#pragma unroll
    for (int sl = 0; sl < NB; ++sl) {
      const int bb = gi + sl * groups;
      if (bb < nb) u[jj * ustride + bb] = gelu_erf(acc[sl]);   // [hidden][ustride]: one row = all batch entries
    }
  }
  __syncthreads();
}

// 16-byte copy of a head's W1 into shared memory, two pieces per thread in flight
__device__ __forceinline__ void stage_weights(const void* src, void* dst, int bytes) {
  const uint4* s4 = reinterpret_cast<const uint4*>(src);
  uint4* d4 = reinterpret_cast<uint4*>(dst);
  const int n16 = bytes >> 4;
  for (int i0 = threadIdx.x; i0 < n16; i0 += 2 * blockDim.x) {
    const int i1 = i0 + (int)blockDim.x;
    const uint4 v0 = __ldg(s4 + i0);
    uint4 v1 = make_uint4(0u, 0u, 0u, 0u);
    if (i1 < n16) v1 = __ldg(s4 + i1);
    d4[i0] = v0;
    if (i1 < n16) d4[i1] = v1;
  }
}

// modReLU: max(|z| + b, 0) z / |z|   (0 at z = 0)
__device__ __forceinline__ float2 modrelu(float2 gk, float bias) {
  const float mag = sqrtf(fmaf(gk.x, gk.x, gk.y * gk.y));
  const float sc = mag > 0.f ? fmaxf(mag + bias, 0.f) / mag : 0.f;
  return cscale(gk, sc);
}
// positional phase exp(+j 2 pi k p / n), angle reduced in integers
// pm = shift mod n in [0, n)
__device__ __forceinline__ float2 phase_reduced(int k, int n, unsigned pm) {
  if (pm == 0u) return make_float2(1.f, 0.f);
  const unsigned kp = (unsigned)(((unsigned long long)k * (unsigned long long)pm) % (unsigned)n);
  const float2 w = twiddle_fwd(kp, (unsigned)n);  // exp(-j ...)
  return make_float2(w.x, -w.y);
}
__device__ __forceinline__ float2 phase_factor(int k, int n, long long shift) {
  long long pm = shift % n;
  if (pm < 0) pm += n;
  return phase_reduced(k, n, (unsigned)pm);
}
__device__ __forceinline__ float2 modrelu_phase(float2 gk, float bias, int k, int n, unsigned pm) {
  gk = modrelu(gk, bias);
  if (pm != 0u) gk = cmul(gk, phase_factor(k, n, (long long)pm));
  return gk;
}

struct GateMlpParams {
  const float* sums;      // [ncopy][B,H,D]
  int ncopy; size_t copy_stride;
  float inv_count;
  int B, H, D, hidden, n, K;
  size_t hs_ln, hs_w1, hs_b1, hs_w2, hs_b2, hs_mb;   // per-head strides (0 when shared)
  const float* gamma; const float* beta; float eps;
  const void* W1; const float* b1; const void* W2; const float* b2;
  const float* modrelu_bias;
  const long long* shift; long long shift_all;
  unsigned pm_all;        // shift_all mod n in [0, n), reduced on the host
  float2* g_out;          // final gate, or the raw MLP output when post != 0
  float* qbar_out;
  float* u_ws;            // [B,H,hidden] hidden activations (workspace)
  int post;               // 1: Toeplitz follows, skip modReLU/phase here
  int stage_w1;           // W1 of a head is copied to shared memory before the wait (size and alignment allow)
};

// raw (re, im) weight pair of one bin in one hidden row
template <typename WT> struct wraw;
template <> struct wraw<bf16> {
  typedef unsigned type;
  static __device__ __forceinline__ type load(const bf16* p) { return __ldg(reinterpret_cast<const unsigned*>(p)); }
  static __device__ __forceinline__ float2 cvt(type r) { return make_float2(__uint_as_float(r << 16), __uint_as_float(r & 0xffff0000u)); }
  static constexpr int kRows = 32;
};
template <> struct wraw<float> {
  typedef float2 type;
  static __device__ __forceinline__ type load(const float* p) { return __ldg(reinterpret_cast<const float2*>(p)); }
  static __device__ __forceinline__ float2 cvt(type r) { return r; }
  static constexpr int kRows = 16;
};

// Output layer: grid (ceil(K / threads), H * ceil(B / BB)), one bin per thread for BB batch
// entries of one head: W2 is shared by the batch, so a column fetched once serves all of them.
// A thread issues the loads of kRows hidden rows of its W2 column before it uses any of them
// (32 rows in bf16: two round trips for the usual 64-wide hidden layer) and needs few enough
// registers for four CTAs per SM, so that the grid of an 8k-token transform is resident at once;
// the kernel is a pure stream over W2.
// Hidden activations of BB batch entries of one head, once: grid H * ceil(B / BB).
template <typename WT, int BB>
__global__ void __launch_bounds__(256) gate_hidden_kernel(const GateMlpParams p) {
  extern __shared__ __align__(16) float u[];       // [hidden][BB], then q_bar [BB][D]
  const int nbg = (p.B + BB - 1) / BB;
  const int h = blockIdx.x / nbg, b0 = (blockIdx.x - h * nbg) * BB;
  const int nb = min(BB, p.B - b0);
  asm volatile("griddepcontrol.launch_dependents;");
  float* qbar = u + BB * p.hidden;
  const WT* W1 = reinterpret_cast<const WT*>(p.W1) + h * p.hs_w1;
  WT* w1s = reinterpret_cast<WT*>(u + ((BB * (p.hidden + p.D) + 3) & ~3));
  if (p.stage_w1) stage_weights(W1, w1s, p.D * p.hidden * (int)sizeof(WT));
  asm volatile("griddepcontrol.wait;" ::: "memory");        // the sums come from the kernel before
  if (p.stage_w1)
    descriptor_and_hidden<WT, BB, true>(p.sums + ((size_t)b0 * p.H + h) * p.D, (size_t)p.H * p.D, nb, p.ncopy, p.copy_stride,
                                        p.inv_count, p.D, p.hidden, p.gamma + h * p.hs_ln, p.beta + h * p.hs_ln, p.eps, w1s,
                                        p.b1 + h * p.hs_b1, qbar, u, BB);
  else
    descriptor_and_hidden<WT, BB, false>(p.sums + ((size_t)b0 * p.H + h) * p.D, (size_t)p.H * p.D, nb, p.ncopy, p.copy_stride,
                                         p.inv_count, p.D, p.hidden, p.gamma + h * p.hs_ln, p.beta + h * p.hs_ln, p.eps, W1,
                                         p.b1 + h * p.hs_b1, qbar, u, BB);
  for (int e = threadIdx.x; e < nb * p.hidden; e += blockDim.x) {
    const int bb = e / p.hidden, jj = e - bb * p.hidden;
    p.u_ws[((size_t)(b0 + bb) * p.H + h) * p.hidden + jj] = u[jj * BB + bb];
  }
  if (p.qbar_out)
    for (int e = threadIdx.x; e < nb * p.D; e += blockDim.x) {
      const int bb = e / p.D, c = e - bb * p.D;
      p.qbar_out[((size_t)(b0 + bb) * p.H + h) * p.D + c] = qbar[e];
    }
}

// ---- the output layer's stream over W2: blocks of rows of one column (bin) per thread ----
// rows j .. j + N - 1 (all present when FULL) held in wc[o .. o + N - 1], added to the sums of BB batch entries
template <typename WT, int BB, bool FULL, int N>
__device__ __forceinline__ void gate_use_rows(const typename wraw<WT>::type (&wc)[wraw<WT>::kRows], int o, int j, int hidden,
                                              const float* __restrict__ u, float2 (&acc)[BB],
                                              uint64_t (&ax)[BB >= 4 ? BB / 2 : 1], uint64_t (&ay)[BB >= 4 ? BB / 2 : 1]) {
  const int nr = FULL ? N : min(N, hidden - j);
#pragma unroll
  for (int i = 0; i < N; ++i) {
    if (FULL || i < nr) {
      const float2 wv = wraw<WT>::cvt(wc[o + i]);
      const float* ur = u + (j + i) * BB;                 // entries of absent batch rows hold stale values, never stored
      if (BB >= 4) {
        const uint64_t wx = pk2(wv.x, wv.x), wy = pk2(wv.y, wv.y);
#pragma unroll
        for (int v = 0; v < BB / 4; ++v) {
          const ulonglong2 t = *reinterpret_cast<const ulonglong2*>(ur + 4 * v);   // entries 4v .. 4v + 3
          ax[2 * v] = fma2(t.x, wx, ax[2 * v]);         ay[2 * v] = fma2(t.x, wy, ay[2 * v]);
          ax[2 * v + 1] = fma2(t.y, wx, ax[2 * v + 1]); ay[2 * v + 1] = fma2(t.y, wy, ay[2 * v + 1]);
        }
      } else {
#pragma unroll
        for (int bb = 0; bb < BB; ++bb) {
          acc[bb].x = fmaf(ur[bb], wv.x, acc[bb].x);
          acc[bb].y = fmaf(ur[bb], wv.y, acc[bb].y);
        }
      }
    }
  }
}
template <typename WT, bool FULL, int N>
__device__ __forceinline__ void gate_fetch_rows(typename wraw<WT>::type (&wc)[wraw<WT>::kRows], int o, const WT* __restrict__ col,
                                                size_t ld, int j, int hidden) {
  const int nr = FULL ? N : min(N, hidden - j);
#pragma unroll
  for (int i = 0; i < N; ++i)
    if (FULL || i < nr) wc[o + i] = wraw<WT>::load(col + (size_t)(j + i) * ld);
}
// w holds rows 0 .. R - 1 on entry.  One batch entry per pass: a block of R rows is requested when the
// one before it has been used.  Several entries per pass (a thread then spends long enough on a row for
// the latency of a whole block to show): the two halves of w alternate, each refilled with the rows R
// further on as soon as it has been used, so R / 2 to R rows are in flight throughout.
template <typename WT, int BB, bool FULL>
__device__ __forceinline__ void gate_stream(typename wraw<WT>::type (&w)[wraw<WT>::kRows], const WT* __restrict__ col, size_t ld,
                                            int hidden, const float* __restrict__ u, float2 (&acc)[BB],
                                            uint64_t (&ax)[BB >= 4 ? BB / 2 : 1], uint64_t (&ay)[BB >= 4 ? BB / 2 : 1]) {
  constexpr int R = wraw<WT>::kRows, Hf = R / 2;
  if (BB >= 4) {
    for (int j = 0; j < hidden; j += R) {
      gate_use_rows<WT, BB, FULL, Hf>(w, 0, j, hidden, u, acc, ax, ay);
      if (j + R < hidden) gate_fetch_rows<WT, FULL, Hf>(w, 0, col, ld, j + R, hidden);
      if (j + Hf < hidden) gate_use_rows<WT, BB, FULL, Hf>(w, Hf, j + Hf, hidden, u, acc, ax, ay);
      if (j + R + Hf < hidden) gate_fetch_rows<WT, FULL, Hf>(w, Hf, col, ld, j + R + Hf, hidden);
    }
  } else {
    for (int j = 0; j < hidden; j += R) {
      if (j > 0) gate_fetch_rows<WT, FULL, R>(w, 0, col, ld, j, hidden);
      gate_use_rows<WT, BB, FULL, R>(w, 0, j, hidden, u, acc, ax, ay);
    }
  }
}

// PRE: the hidden activations were computed once per (head, batch entry) by gate_hidden_kernel
// (long transforms: hundreds of CTAs per head would otherwise repeat that work).
template <typename WT, int BB, bool PRE>
__global__ void __launch_bounds__(256, BB == 1 ? 4 : 2) gate_out_kernel(const GateMlpParams p) {
  extern __shared__ __align__(16) float u[];       // [hidden][BB], then q_bar [BB][D]
  // a kernel launched behind this one as a programmatic dependent may do its set-up meanwhile
  asm volatile("griddepcontrol.launch_dependents;");
  constexpr int R = wraw<WT>::kRows;
  const int nbg = (p.B + BB - 1) / BB;
  const int h = blockIdx.y / nbg, b0 = (blockIdx.y - h * nbg) * BB;
  const int nb = min(BB, p.B - b0);
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  const bool live = k < p.K;
  const WT* col = reinterpret_cast<const WT*>(p.W2) + h * p.hs_w2 + 2 * (size_t)(live ? k : 0);
  const size_t ld = 2 * (size_t)p.K;
  WT* w1s = reinterpret_cast<WT*>(u + ((BB * (p.hidden + p.D) + 3) & ~3));
  if (!PRE && p.stage_w1) stage_weights(reinterpret_cast<const WT*>(p.W1) + h * p.hs_w1, w1s, p.D * p.hidden * (int)sizeof(WT));
  typename wraw<WT>::type w[R];
  const int n0 = min(R, p.hidden);
  if (live) {
#pragma unroll
    for (int i = 0; i < R; ++i)
      if (i < n0) w[i] = wraw<WT>::load(col + (size_t)i * ld);
  }
  // everything above reads only weights; the sums / hidden activations come from the kernel before
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (PRE) {
    for (int e = threadIdx.x; e < nb * p.hidden; e += blockDim.x) {
      const int bb = e / p.hidden, jj = e - bb * p.hidden;
      u[jj * BB + bb] = p.u_ws[((size_t)(b0 + bb) * p.H + h) * p.hidden + jj];
    }
    __syncthreads();
  } else {
    // LayerNorm + hidden layer, repeated by every CTA of the head (a few thousand FLOPs per batch
    // entry, two short round trips) while this thread's W2 column is already on its way
    float* qbar = u + BB * p.hidden;   // [BB][D]
    const WT* W1 = reinterpret_cast<const WT*>(p.W1) + h * p.hs_w1;
    if (p.stage_w1)
      descriptor_and_hidden<WT, BB, true>(p.sums + ((size_t)b0 * p.H + h) * p.D, (size_t)p.H * p.D, nb, p.ncopy, p.copy_stride,
                                          p.inv_count, p.D, p.hidden, p.gamma + h * p.hs_ln, p.beta + h * p.hs_ln, p.eps, w1s,
                                          p.b1 + h * p.hs_b1, qbar, u, BB);
    else
      descriptor_and_hidden<WT, BB, false>(p.sums + ((size_t)b0 * p.H + h) * p.D, (size_t)p.H * p.D, nb, p.ncopy, p.copy_stride,
                                           p.inv_count, p.D, p.hidden, p.gamma + h * p.hs_ln, p.beta + h * p.hs_ln, p.eps, W1,
                                           p.b1 + h * p.hs_b1, qbar, u, BB);
    if (p.qbar_out && blockIdx.x == 0)
      for (int e = threadIdx.x; e < nb * p.D; e += blockDim.x) {
        const int bb = e / p.D, c = e - bb * p.D;
        p.qbar_out[((size_t)(b0 + bb) * p.H + h) * p.D + c] = qbar[e];
      }
  }
  if (!live) return;
  const float* b2 = p.b2 + h * p.hs_b2;
  float2 acc[BB];
#pragma unroll
  for (int bb = 0; bb < BB; ++bb) acc[bb] = make_float2(b2[2 * k], b2[2 * k + 1]);
  // BB >= 4: the sums of two batch entries share a packed fp32 pair (one instruction per pair and
  // component; each half rounds like a scalar fmaf, so the results do not change)
  constexpr int NP = BB >= 4 ? BB / 2 : 1;
  uint64_t ax[NP], ay[NP];
#pragma unroll
  for (int pp = 0; pp < NP; ++pp) { ax[pp] = pk2(acc[0].x, acc[0].x); ay[pp] = pk2(acc[0].y, acc[0].y); }
  if (p.hidden % R == 0) gate_stream<WT, BB, true>(w, col, ld, p.hidden, u, acc, ax, ay);
  else gate_stream<WT, BB, false>(w, col, ld, p.hidden, u, acc, ax, ay);
  if (BB >= 4) {
#pragma unroll
    for (int pp = 0; pp < NP; ++pp) {
      upk2(ax[pp], acc[2 * pp].x, acc[2 * pp + 1].x);
      upk2(ay[pp], acc[2 * pp].y, acc[2 * pp + 1].y);
    }
  }
  const float bias = (!p.post && p.modrelu_bias) ? p.modrelu_bias[h * p.hs_mb + k] : 0.f;
  // one positional phase for the whole batch unless per-entry shifts are given
  float2 ph = make_float2(1.f, 0.f);
  if (!p.post && !p.shift) ph = phase_reduced(k, p.n, p.pm_all);
#pragma unroll
  for (int bb = 0; bb < BB; ++bb) {
    if (bb < nb) {
      const int b = b0 + bb;
      float2 a = acc[bb];
      if (!p.post) {
        if (p.modrelu_bias) a = modrelu(a, bias);         // without a bias modReLU is the identity (|z| z / |z| = z, exactly, in this arithmetic too)
        a = cmul(a, p.shift ? phase_factor(k, p.n, p.shift_all + p.shift[b]) : ph);
      }
      p.g_out[((size_t)b * p.H + h) * p.K + k] = a;
    }
  }
}

struct GatePostParams {
  const float2* g_raw; float2* g_out;
  const float2* taps; size_t hs_t; int r;
  const float* modrelu_bias; size_t hs_mb;
  const long long* shift; long long shift_all;
  int H, K, n;
};

// Toeplitz update along the bin axis ('same' window, zero boundary, reads the
// pre-update gate), then modReLU and phase (Sec. 3.2 steps 3b-3c).
__global__ void __launch_bounds__(256) gate_post_kernel(const GatePostParams p) {
  asm volatile("griddepcontrol.launch_dependents;");
  const int bh = blockIdx.y, b = bh / p.H, h = bh - b * p.H;
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= p.K) return;
  const float2* g = p.g_raw + (size_t)bh * p.K;
  const float2* t = p.taps + h * p.hs_t;
  float2 acc = g[k];
  for (int m = -p.r; m <= p.r; ++m) {
    int src = k - m;
    if (src >= 0 && src < p.K) acc = cadd(acc, cmul(t[m + p.r], g[src]));
  }
  long long sh = p.shift_all + (p.shift ? p.shift[b] : 0);
  long long pm = sh % p.n; if (pm < 0) pm += p.n;
  float bias = p.modrelu_bias ? p.modrelu_bias[h * p.hs_mb + k] : 0.f;
  p.g_out[(size_t)bh * p.K + k] = modrelu_phase(acc, bias, k, p.n, (unsigned)pm);
}

constexpr int kPoolCopies = 16;      // partial copies of the pooled sum in a full-size workspace

// Layout: [raw gate (Toeplitz only)] [hidden activations] [ncopy x pooled sums].  ncopy = 1 is the minimum.
static size_t gate_ws_layout(int B, int H, int D, int n_fft, int r, int hidden, int ncopy, size_t* u_off,
                             size_t* sums_off) {
  size_t raw = r > 0 ? align_up((size_t)B * H * (n_fft / 2 + 1) * sizeof(float2), 256) : 0;
  *u_off = raw;
  *sums_off = raw + align_up((size_t)B * H * hidden * sizeof(float), 256);
  return *sums_off + align_up((size_t)ncopy * B * H * D * sizeof(float), 256);
}

}  // namespace spectre

using namespace spectre;

namespace spectre {
// Smallest gate scratch (one copy of the sums, any hidden width); used by the decode step.
size_t gate_min_workspace(int B, int H, int D, int n_fft, int r) {
  size_t off, off2;
  return gate_ws_layout(B, H, D, n_fft, r, 1024, 1, &off, &off2);
}
}  // namespace spectre

extern "C" size_t spectre_gate_workspace_bytes(const spectre_ctx* ctx, int32_t B, int32_t H, int32_t D, int32_t n_fft,
                                               int32_t toeplitz_r) {
  (void)ctx;
  if (B < 1 || H < 1 || D < 1 || n_fft < 1 || toeplitz_r < 0) return 0;
  size_t off, off2;
  return gate_ws_layout(B, H, D, n_fft, toeplitz_r, 1024, kPoolCopies, &off, &off2);   // any hidden width
}

extern "C" int spectre_gate(spectre_ctx* ctx, void* stream, const spectre_act* q, const float* sum_q, int32_t B,
                            int32_t H, int32_t D, float inv_count, const spectre_gate_params* gp, int32_t n_fft,
                            const int64_t* shift, int64_t shift_all, float* g_out, float* qbar_out, void* workspace,
                            size_t workspace_bytes) {
  if (!ctx) return fail(SPECTRE_ERR_INVALID_ARG, "ctx is NULL");
  if (!gp) return fail(SPECTRE_ERR_INVALID_ARG, "gate parameters are NULL");
  if ((q != nullptr) == (sum_q != nullptr)) return fail(SPECTRE_ERR_INVALID_ARG, "give exactly one of q and sum_q");
  if (!g_out || (reinterpret_cast<uintptr_t>(g_out) & 7)) return fail(SPECTRE_ERR_INVALID_ARG, "g_out is NULL or misaligned");
  if (B < 1 || H < 1 || D < 1 || D > 1024) return fail(SPECTRE_ERR_INVALID_ARG, "B, H, D must be positive (D <= 1024)");
  if (n_fft < 1 || n_fft > (1 << 24)) return fail(SPECTRE_ERR_INVALID_ARG, "n_fft out of range");
  if (gp->hidden < 1 || gp->hidden > 1024) return fail(SPECTRE_ERR_UNSUPPORTED, "hidden width must be in 1..1024");
  if (gp->toeplitz_r < 0 || gp->toeplitz_r > 64) return fail(SPECTRE_ERR_UNSUPPORTED, "toeplitz_r must be in 0..64");
  if (gp->wdtype != SPECTRE_F32 && gp->wdtype != SPECTRE_BF16) return fail(SPECTRE_ERR_INVALID_ARG, "unknown weight dtype");
  if (!gp->ln_gamma || !gp->ln_beta || !gp->W1 || !gp->b1 || !gp->W2 || !gp->b2)
    return fail(SPECTRE_ERR_INVALID_ARG, "a gate parameter array is NULL");
  if (gp->toeplitz_r > 0 && !gp->toeplitz) return fail(SPECTRE_ERR_INVALID_ARG, "toeplitz taps are NULL");
  if (reinterpret_cast<uintptr_t>(gp->W2) & 7) return fail(SPECTRE_ERR_INVALID_ARG, "W2 not 8-byte aligned");
  if (!(gp->ln_eps >= 0.f)) return fail(SPECTRE_ERR_INVALID_ARG, "ln_eps must be >= 0");
  if (q) {
    int rc = check_act(q, "q");
    if (rc != SPECTRE_OK) return rc;
    if (q->B != B || q->H != H || q->D != D) return fail(SPECTRE_ERR_INVALID_ARG, "q shape differs from B, H, D");
    if (!(inv_count > 0.f)) inv_count = 1.0f / (float)q->L;
  } else if (!(inv_count > 0.f)) {
    return fail(SPECTRE_ERR_INVALID_ARG, "inv_count must be positive with sum_q");
  }
  const int K = n_fft / 2 + 1;
  const int r = gp->toeplitz_r;
  size_t sums_off, u_off;
  const size_t need = gate_ws_layout(B, H, D, n_fft, r, gp->hidden, 1, &u_off, &sums_off);   // one copy is enough
  const bool need_ws = true;
  if (need_ws) {
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 15))
      return fail(SPECTRE_ERR_WORKSPACE, "workspace is NULL or not 16-byte aligned");
    if (workspace_bytes < need) return fail(SPECTRE_ERR_WORKSPACE, "gate workspace too small");
  }
  SPECTRE_CUDA_OK(cudaSetDevice(ctx->device));
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const float* sums = sum_q;
  int ncopy = 1;
  if (q) {
    float* pooled = reinterpret_cast<float*>(reinterpret_cast<char*>(workspace) + sums_off);
    const size_t one_copy = (size_t)B * H * D * sizeof(float);
    size_t fit = (workspace_bytes - sums_off) / one_copy;
    int rc = pool_sum(ctx, st, q, pooled, fit > (size_t)kPoolCopies ? kPoolCopies : (int)fit, &ncopy);
    if (rc != SPECTRE_OK) return rc;
    sums = pooled;
  }
  const size_t one = gp->shared_across_heads ? 0 : 1;
  GateMlpParams mp = {};
  mp.sums = sums; mp.ncopy = ncopy; mp.copy_stride = (size_t)B * H * D; mp.inv_count = inv_count;
  mp.B = B; mp.H = H; mp.D = D; mp.hidden = gp->hidden; mp.n = n_fft; mp.K = K;
  mp.hs_ln = one * D; mp.hs_w1 = one * (size_t)D * gp->hidden; mp.hs_b1 = one * gp->hidden;
  mp.hs_w2 = one * (size_t)gp->hidden * 2 * K; mp.hs_b2 = one * 2 * (size_t)K; mp.hs_mb = one * K;
  mp.gamma = gp->ln_gamma; mp.beta = gp->ln_beta; mp.eps = gp->ln_eps;
  mp.W1 = gp->W1; mp.b1 = gp->b1; mp.W2 = gp->W2; mp.b2 = gp->b2;
  mp.modrelu_bias = gp->modrelu_bias;
  mp.shift = reinterpret_cast<const long long*>(shift); mp.shift_all = shift_all;
  {
    long long pm = shift_all % n_fft;
    if (pm < 0) pm += n_fft;
    mp.pm_all = (unsigned)pm;
  }
  mp.qbar_out = qbar_out;
  mp.u_ws = reinterpret_cast<float*>(reinterpret_cast<char*>(workspace) + u_off);
  mp.post = r > 0;
  float2* raw = r > 0 ? reinterpret_cast<float2*>(workspace) : nullptr;
  mp.g_out = r > 0 ? raw : reinterpret_cast<float2*>(g_out);
  // block sized to the bin count for short transforms (K = 99 does not need 256 threads)
  const int thr_out = K >= 256 ? 256 : ((K + 31) / 32 * 32 < 64 ? 64 : (K + 31) / 32 * 32);
  // batch entries per CTA: the weights of a head are fetched once for all of them
  const int BB = (gp->hidden > 256 || B < 2) ? 1 : (B < 4 ? 2 : (B < 8 ? 4 : 8));
  dim3 grid_out((K + thr_out - 1) / thr_out, (unsigned)(H * ((B + BB - 1) / BB)));
  if (grid_out.y > 65535) return fail(SPECTRE_ERR_UNSUPPORTED, "H * ceil(B / 8) exceeds 65535");
  const bool wb = gp->wdtype == SPECTRE_BF16;
  const size_t w1_bytes = (size_t)D * gp->hidden * (wb ? 2 : 4);
  mp.stage_w1 = w1_bytes <= 16384 && w1_bytes % 16 == 0 && !(reinterpret_cast<uintptr_t>(gp->W1) & 15);
  const size_t smem = (((size_t)BB * (D + gp->hidden) + 3) & ~(size_t)3) * sizeof(float) + (mp.stage_w1 ? w1_bytes : 0);
  const bool pre = grid_out.x >= 32;               // many CTAs per head: compute the hidden layer once
  // Programmatic dependent launch: the weight stream of the output layer may overlap the kernel
  // before it (the pooling pass here, or whatever produced sum_q); each kernel waits for its
  // predecessor (griddepcontrol.wait) before it touches the sums.
  cudaLaunchAttribute pdl[1];
  pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  pdl[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg_out = {}, cfg_hid = {};
  cfg_out.gridDim = grid_out; cfg_out.blockDim = dim3(thr_out, 1, 1); cfg_out.dynamicSmemBytes = smem; cfg_out.stream = st;
  cfg_out.attrs = pdl; cfg_out.numAttrs = 1;
  cfg_hid = cfg_out;
  cfg_hid.gridDim = dim3(grid_out.y, 1, 1); cfg_hid.blockDim = dim3(256, 1, 1);
#define SPECTRE_GATE_LAUNCH(WT, NB)                                                              \
  do {                                                                                           \
    if (pre) {                                                                                   \
      SPECTRE_CUDA_OK(cudaLaunchKernelEx(&cfg_hid, gate_hidden_kernel<WT, NB>, mp));             \
      SPECTRE_CUDA_OK(cudaLaunchKernelEx(&cfg_out, gate_out_kernel<WT, NB, true>, mp));          \
    } else {                                                                                     \
      SPECTRE_CUDA_OK(cudaLaunchKernelEx(&cfg_out, gate_out_kernel<WT, NB, false>, mp));         \
    }                                                                                            \
  } while (0)
  switch (BB) {
    case 8: if (wb) SPECTRE_GATE_LAUNCH(bf16, 8); else SPECTRE_GATE_LAUNCH(float, 8); break;
    case 4: if (wb) SPECTRE_GATE_LAUNCH(bf16, 4); else SPECTRE_GATE_LAUNCH(float, 4); break;
    case 2: if (wb) SPECTRE_GATE_LAUNCH(bf16, 2); else SPECTRE_GATE_LAUNCH(float, 2); break;
    default: if (wb) SPECTRE_GATE_LAUNCH(bf16, 1); else SPECTRE_GATE_LAUNCH(float, 1); break;
  }
#undef SPECTRE_GATE_LAUNCH
  SPECTRE_LAUNCH_OK("gate_out_kernel");
  if (r > 0) {
    GatePostParams pp = {};
    pp.g_raw = raw; pp.g_out = reinterpret_cast<float2*>(g_out);
    pp.taps = reinterpret_cast<const float2*>(gp->toeplitz); pp.hs_t = one * (2 * r + 1); pp.r = r;
    pp.modrelu_bias = gp->modrelu_bias; pp.hs_mb = one * K;
    pp.shift = mp.shift; pp.shift_all = shift_all;
    pp.H = H; pp.K = K; pp.n = n_fft;
    dim3 grid((K + 255) / 256, B * H);
    if (grid.y > 65535) return fail(SPECTRE_ERR_UNSUPPORTED, "B*H exceeds 65535");
    gate_post_kernel<<<grid, 256, 0, st>>>(pp);
    SPECTRE_LAUNCH_OK("gate_post_kernel");
  }
  return SPECTRE_OK;
}

// ---- gate without any caller- or library-side allocation -----------------------
// Scratch of spectre_gate_static: one fixed array per GPU that loads this library,
// resident until the process exits.  Host code must not hand this name to a kernel
// (on the host it is only a stand-in for the symbol); the device address is looked
// up once per device below.
#define SPECTRE_GATE_STATIC_BYTES (1u << 20)
static __device__ __align__(256) unsigned char g_gate_static_scratch[SPECTRE_GATE_STATIC_BYTES];

namespace spectre {
static const int kMaxDevices = 64;
static std::atomic<void*> g_static_ptr[kMaxDevices];     // device address of the array, per device ordinal

// With `device` current: resolves (once) the device address of the static scratch.  Host threads
// that race on the first call of a device each look the address up and store the same value.
static int static_scratch_address(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return fail(SPECTRE_ERR_UNSUPPORTED, "device ordinal beyond 63");
  void* p = g_static_ptr[device].load(std::memory_order_acquire);
  if (!p) {
    cudaError_t e = cudaGetSymbolAddress(&p, g_gate_static_scratch);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(gate static scratch)");
    if (!p) return fail(SPECTRE_ERR_CUDA, "static scratch has no device address");
    g_static_ptr[device].store(p, std::memory_order_release);
  }
  *out = p;
  return SPECTRE_OK;
}
}  // namespace spectre

extern "C" size_t spectre_gate_static_max_bytes(void) { return SPECTRE_GATE_STATIC_BYTES; }

extern "C" int spectre_gate_static(spectre_ctx* ctx, void* stream, const spectre_act* q, const float* sum_q, int32_t B,
                                   int32_t H, int32_t D, float inv_count, const spectre_gate_params* gp, int32_t n_fft,
                                   const int64_t* shift, int64_t shift_all, float* g_out, float* qbar_out) {
  if (!ctx) return fail(SPECTRE_ERR_INVALID_ARG, "ctx is NULL");
  if (!gp) return fail(SPECTRE_ERR_INVALID_ARG, "gate parameters are NULL");
  if (B < 1 || H < 1 || D < 1 || D > 1024) return fail(SPECTRE_ERR_INVALID_ARG, "B, H, D must be positive (D <= 1024)");
  if (n_fft < 1 || n_fft > (1 << 24)) return fail(SPECTRE_ERR_INVALID_ARG, "n_fft out of range");
  // the widths that size the scratch are range-checked before the size is computed from them
  if (gp->hidden < 1 || gp->hidden > 1024) return fail(SPECTRE_ERR_UNSUPPORTED, "hidden width must be in 1..1024");
  if (gp->toeplitz_r < 0 || gp->toeplitz_r > 64) return fail(SPECTRE_ERR_UNSUPPORTED, "toeplitz_r must be in 0..64");
  size_t off_a, off_b;
  const size_t need = gate_ws_layout(B, H, D, n_fft, gp->toeplitz_r, gp->hidden, 1, &off_a, &off_b);   // one copy of the sums
  if (need > SPECTRE_GATE_STATIC_BYTES)
    return fail(SPECTRE_ERR_UNSUPPORTED,
                "spectre_gate_static: this shape needs " + std::to_string(need) + " bytes of scratch, the built-in array holds " +
                    std::to_string((size_t)SPECTRE_GATE_STATIC_BYTES) + "; use spectre_gate with a workspace");
  SPECTRE_CUDA_OK(cudaSetDevice(ctx->device));
  void* scratch = nullptr;
  int rc = static_scratch_address(ctx->device, &scratch);
  if (rc != SPECTRE_OK) return rc;
  // Same kernels as spectre_gate; the pooled sum is cleared inside (on the caller's stream), so what an
  // earlier call left in the array does not matter.
  return spectre_gate(ctx, stream, q, sum_q, B, H, D, inv_count, gp, n_fft, shift, shift_all, g_out, qbar_out, scratch,
                      SPECTRE_GATE_STATIC_BYTES);
}
