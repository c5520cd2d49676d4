// Prefix-FFT cache (Sec. 3.3, Eq. 5, Alg. 1): prefill, per-token append, and the whole decode
// step with single-row read-out.
#include "common.cuh"

namespace spectre {

// from mixer.cu / gate.cu
int forward_decimated(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, int n, int slab0, int cnt,
                      float2* ws, int* N1_out, int* M_out, void* ring, int* ring_done);
bool transform_supported(const spectre_ctx* ctx, int n);
size_t transform_slab_bytes(int n, int D);
int pool_sum(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* q, float* sums, int ncopy_max, int* ncopy_used);
int pool_sum_ring(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* q, float* sums, void* ring, int N);
size_t gate_min_workspace(int B, int H, int D, int n_fft, int r);
size_t inverse_workspace_bytes(const spectre_ctx* ctx, int n, int D, int nslab);
int inverse_from_spectrum(const spectre_ctx* ctx, cudaStream_t st, const float* spec, const float* g, const spectre_act* y,
                          int n, void* ws, size_t ws_bytes);

// ---- prefill -----------------------------------------------------------------
// With Z = fft_n(a + jb) for each column pair (a, b), the half spectra of the two real columns follow
// from Hermitian symmetry (App. B):
//   A_k = (Z_k + conj(Z_{n-k})) / 2,   B_k = (Z_k - conj(Z_{n-k})) / (2j).
__device__ __forceinline__ void store_split(float* __restrict__ prefix, size_t slab, int K, int D, int k, int c, float2 z,
                                            float2 zm) {
  float4 out;
  out.x = 0.5f * (z.x + zm.x);
  out.y = 0.5f * (z.y - zm.y);
  out.z = 0.5f * (z.y + zm.y);
  out.w = -0.5f * (z.x - zm.x);
  *reinterpret_cast<float4*>(prefix + ((slab * K + k) * D + 2 * c) * 2) = out;
}

// Transforms that fit the on-chip kernel (N1 = 1) leave Z in ws[slab_local][k][D/2].  A thread takes
// kSplitBins consecutive bins of one column pair, all their loads in flight together.
constexpr int kSplitBins = 4;
__global__ void __launch_bounds__(256) split_kernel(const float2* __restrict__ ws, float* __restrict__ prefix, int n,
                                                    int K, int D, int slab0, int nslab) {
  const int half = D / 2;
  const int kblocks = (K + kSplitBins - 1) / kSplitBins;
  const size_t total = (size_t)nslab * kblocks * half;
  size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int c = (int)(idx % half);
  const size_t r = idx / half;
  const int k0 = (int)(r % kblocks) * kSplitBins;
  const int slab_local = (int)(r / kblocks);
  float2 z[kSplitBins], zm[kSplitBins];
#pragma unroll
  for (int u = 0; u < kSplitBins; ++u) {
    const int k = min(k0 + u, K - 1), km = (n - k) % n;
    z[u] = ws[((size_t)slab_local * n + k) * half + c];
    zm[u] = ws[((size_t)slab_local * n + km) * half + c];
  }
#pragma unroll
  for (int u = 0; u < kSplitBins; ++u) {
    const int k = k0 + u;
    if (k < K) store_split(prefix, (size_t)(slab0 + slab_local), K, D, k, c, z[u], zm[u]);
  }
}

// Longer transforms, n = N1 M with token t = N1 n2 + n1: the forward pass leaves the M-point spectra of the
// N1 decimated sequences, Y[n1][k2] in ws[slab_local][n1][k2][D/2], and the last radix-N1 step runs here,
//   Z[k2 + M k1] = sum_n1 W_N1^{n1 k1} ( W_n^{n1 k2} Y[n1][k2] ).
// Z[n - k] for k = k2 + M k1 is Z[(M - k2) + M (N1 - 1 - k1)] (k2 > 0), so the thread that owns k2 and
// M - k2 of one column pair holds both sides of every Hermitian pair it stores: the bins k2 + M k1 and
// (M - k2) + M k1 for k1 < N1/2 (and, at k2 = 0, bin n/2); the packed spectrum never goes back to memory.
template <int N1>
__global__ void __launch_bounds__(256) combine_split_kernel(const float2* __restrict__ ws, float* __restrict__ prefix, int n,
                                                            int K, int D, int M, int slab0, int nslab) {
  const int half = D / 2;
  const int nk2 = M / 2 + 1;
  const size_t total = (size_t)nslab * nk2 * half;
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int c = (int)(idx % half);
  const size_t r = idx / half;
  const int k2 = (int)(r % nk2);
  const int slab_local = (int)(r / nk2);
  const int m2 = (M - k2) % M;
  float2 xa[N1], xb[N1];
#pragma unroll
  for (int n1 = 0; n1 < N1; ++n1) {
    const size_t row = ((size_t)slab_local * N1 + n1) * M;
    xa[n1] = ws[(row + k2) * half + c];
    xb[n1] = ws[(row + m2) * half + c];
  }
  const float2 wa1 = twiddle_fwd((unsigned)k2, (unsigned)n), wb1 = twiddle_fwd((unsigned)m2, (unsigned)n);
  float2 wa[N1], wb[N1];
  wa[0] = wb[0] = make_float2(1.f, 0.f);
#pragma unroll
  for (int q = 1; q < N1; ++q) {
    wa[q] = (q == 1) ? wa1 : cmul(wa[q / 2], wa[q - q / 2]);
    wb[q] = (q == 1) ? wb1 : cmul(wb[q / 2], wb[q - q / 2]);
    xa[q] = cmul(xa[q], wa[q]);
    xb[q] = cmul(xb[q], wb[q]);
  }
  Dft<N1, false>::run(xa);
  Dft<N1, false>::run(xb);
  const size_t slab = (size_t)(slab0 + slab_local);
  const bool own = k2 == 0 || k2 == m2;       // k2 = 0 and k2 = M/2 are their own mirror
#pragma unroll
  for (int k1 = 0; k1 < N1 / 2; ++k1) {
    store_split(prefix, slab, K, D, k2 + M * k1, c, xa[k1], k2 == 0 ? xa[(N1 - k1) % N1] : xb[N1 - 1 - k1]);
    if (!own) store_split(prefix, slab, K, D, m2 + M * k1, c, xb[k1], xa[N1 - 1 - k1]);
  }
  if (k2 == 0) store_split(prefix, slab, K, D, M * (N1 / 2), c, xa[N1 / 2], xa[N1 / 2]);
}

template <int N1>
static void launch_combine_split(cudaStream_t st, const float2* ws, float* prefix, int n, int K, int D, int M, int slab0,
                                 int cnt) {
  const size_t total = (size_t)cnt * (M / 2 + 1) * (D / 2);
  combine_split_kernel<N1><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(ws, prefix, n, K, D, M, slab0, cnt);
}

// Ring buffers: rows 0..L-1 <- tokens, rows L..N-1 <- 0 (Alg. 1 PreFill).  A CTA copies kRingRows
// consecutive rows of one batch entry, a thread one 16-byte piece of each with all of them in flight.
constexpr int kRingRows = 8;
template <typename T>
__global__ void __launch_bounds__(256) ring_fill_kernel(const T* __restrict__ src, int64_t sb, int64_t sl, int64_t sh,
                                                        T* __restrict__ buf, int B, int N, int H, int D, int L) {
  constexpr int V = 16 / sizeof(T);
  const int vec_per_row = H * D / V;
  const int chunks = (N + kRingRows - 1) / kRingRows;
  const int b = blockIdx.x / chunks, r0 = (blockIdx.x - b * chunks) * kRingRows;
  for (int vi = threadIdx.x; vi < vec_per_row; vi += blockDim.x) {
    const int e = vi * V, h = e / D, c = e - h * D;
    const T* s = src + b * sb + h * sh + c;
    T* d = buf + (((size_t)b * N + r0) * H + h) * D + c;
    uint4 val[kRingRows];
#pragma unroll
    for (int u = 0; u < kRingRows; ++u)
      val[u] = (r0 + u < L) ? __ldcs(reinterpret_cast<const uint4*>(s + (int64_t)(r0 + u) * sl)) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int u = 0; u < kRingRows; ++u)
      if (r0 + u < N) __stcs(reinterpret_cast<uint4*>(d + (size_t)u * H * D), val[u]);
  }
}

// ---- append ------------------------------------------------------------------
// A warp owns 32 consecutive bins of one (batch, head): lane l evaluates the
// twiddle of bin k0 + l once, then the warp walks the 32 bins with every lane
// updating 2 channels (one 16-byte complex pair) of the bin's contiguous row.
template <typename T>
__global__ void __launch_bounds__(256) append_spectrum_kernel(float* __restrict__ prefix, const T* __restrict__ V_buf,
                                                              const T* __restrict__ v_t, int H, int D, int N, int K,
                                                              int slot, unsigned tm, int evict, int warps_per_slab,
                                                              size_t nwarps_total) {
  const size_t wid = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (wid >= nwarps_total) return;
  const int slab = (int)(wid / warps_per_slab);
  const int k0 = (int)(wid % warps_per_slab) * 32;
  const int b = slab / H, h = slab - b * H;
  // twiddle exp(-j 2 pi k t / N) of bin k0 + lane, angle reduced in integers
  float2 my = make_float2(1.f, 0.f);
  if (k0 + lane < K) {
    unsigned kk = (unsigned)(((unsigned long long)(k0 + lane) * tm) % (unsigned)N);
    my = twiddle_fwd(kk, (unsigned)N);
  }
  const int nb = min(32, K - k0);
  const int half = D / 2;
  float* base = prefix + (((size_t)slab * K + k0) * D) * 2;
  for (int c0 = 0; c0 < half; c0 += 32) {      // uniform trip count: every lane takes part in the shuffles
    const int c = c0 + lane;
    const bool live = c < half;
    float d0 = 0.f, d1 = 0.f;
    if (live) {
      d0 = io<T>::load1(v_t + (size_t)slab * D + 2 * c);
      d1 = io<T>::load1(v_t + (size_t)slab * D + 2 * c + 1);
      if (evict) {
        const T* old = V_buf + (((size_t)b * N + slot) * H + h) * D + 2 * c;
        d0 -= io<T>::load1(old);
        d1 -= io<T>::load1(old + 1);
      }
    }
    // four bins per round, their loads issued together (the compiler cannot move a load of this array
    // above the store before it)
    for (int i0 = 0; i0 < nb; i0 += 4) {
      float4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (live && i0 + u < nb) v[u] = *reinterpret_cast<const float4*>(base + ((size_t)(i0 + u) * D + 2 * c) * 2);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = min(i0 + u, 31);
        const float wr = __shfl_sync(0xffffffffu, my.x, i), wi = __shfl_sync(0xffffffffu, my.y, i);
        if (live && i0 + u < nb) {
          v[u].x = fmaf(d0, wr, v[u].x); v[u].y = fmaf(d0, wi, v[u].y);
          v[u].z = fmaf(d1, wr, v[u].z); v[u].w = fmaf(d1, wi, v[u].w);
          *reinterpret_cast<float4*>(base + ((size_t)(i0 + u) * D + 2 * c) * 2) = v[u];
        }
      }
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(256) append_ring_kernel(T* __restrict__ V_buf, T* __restrict__ Q_buf,
                                                          float* __restrict__ sum_q, const T* __restrict__ q_t,
                                                          const T* __restrict__ v_t, int B, int H, int D, int N,
                                                          int slot, int evict) {
  const int total = B * H * D;
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  int b = idx / (H * D), hd = idx - b * (H * D);
  size_t o = ((size_t)b * N + slot) * H * D + hd;
  float qn = io<T>::load1(q_t + idx);
  float qo = evict ? io<T>::load1(Q_buf + o) : 0.f;
  sum_q[idx] += qn - qo;
  Q_buf[o] = q_t[idx];
  V_buf[o] = v_t[idx];
}


// ---- decode step -------------------------------------------------------------
// Ring buffers and running sum as in the append, plus delta = v_t - v_old in fp32 for the
// spectrum pass (which then no longer needs the ring buffer).
template <typename T>
__global__ void __launch_bounds__(256) decode_ring_kernel(T* __restrict__ V_buf, T* __restrict__ Q_buf,
                                                          float* __restrict__ sum_q, float* __restrict__ delta,
                                                          const T* __restrict__ q_t, const T* __restrict__ v_t, int B,
                                                          int H, int D, int N, int slot, int evict) {
  const int total = B * H * D;
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  int b = idx / (H * D), hd = idx - b * (H * D);
  size_t o = ((size_t)b * N + slot) * H * D + hd;
  float qn = io<T>::load1(q_t + idx), vn = io<T>::load1(v_t + idx);
  float qo = evict ? io<T>::load1(Q_buf + o) : 0.f;
  float vo = evict ? io<T>::load1(V_buf + o) : 0.f;
  sum_q[idx] += qn - qo;
  delta[idx] = vn - vo;
  Q_buf[o] = q_t[idx];
  V_buf[o] = v_t[idx];
}

struct DecodeRows { int r[SPECTRE_DECODE_MAX_ROWS]; };

// One pass over the spectrum: P_k += delta exp(-j 2 pi k t / N) (Eq. 5) and, from the updated
// value, the NR read-out rows  V~[r] = (1/N) sum_k w_k Re(g_k P_k exp(+j 2 pi k r / N)),
// w_0 = w_{N/2} = 1, else 2 (Sec. 3.3.2 step e at one output index).  A CTA takes 256
// consecutive bins of one (batch, head), a warp 32 of them: lane l evaluates bin k0 + l's
// update twiddle and its NR read-out coefficients once, then the warp walks the 32 bins with
// every lane holding 2 channels.  Row sums are reduced over the CTA and written as one
// partial per (slab, bin block); decode_reduce_kernel adds the partials in a fixed order.
template <int NR>
__global__ void __launch_bounds__(256) decode_spectrum_kernel(float* __restrict__ prefix, const float* __restrict__ delta,
                                                              const float2* __restrict__ g, float* __restrict__ partial,
                                                              int D, int N, int K, unsigned tm, DecodeRows rows,
                                                              int nblk) {
  __shared__ float red[8][NR][64];
  const int slab = blockIdx.x / nblk, blk = blockIdx.x - slab * nblk;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int k0 = (blk * 8 + warp) * 32, k = k0 + lane;
  float2 my = make_float2(1.f, 0.f);
  float2 coef[NR];
#pragma unroll
  for (int r = 0; r < NR; ++r) coef[r] = make_float2(0.f, 0.f);
  if (k < K) {
    my = twiddle_fwd((unsigned)(((unsigned long long)k * tm) % (unsigned)N), (unsigned)N);
    const float2 gk = __ldg(g + (size_t)slab * K + k);
    const float wk = ((k == 0 || 2 * k == N) ? 1.0f : 2.0f) / (float)N;
#pragma unroll
    for (int r = 0; r < NR; ++r) {
      const float2 e = twiddle_fwd((unsigned)(((unsigned long long)k * (unsigned)rows.r[r]) % (unsigned)N), (unsigned)N);
      coef[r] = cscale(cmulc(gk, e), wk);               // g_k exp(+j theta) w_k / N
    }
  }
  const int nb = max(0, min(32, K - k0));
  const int half = D / 2;
  float* base = prefix + (((size_t)slab * K + k0) * D) * 2;
  for (int c0 = 0; c0 < half; c0 += 32) {               // uniform trip count: every lane takes part in the shuffles
    const int c = c0 + lane;
    const bool live = c < half;
    float d0 = 0.f, d1 = 0.f;
    if (live) {
      d0 = delta[(size_t)slab * D + 2 * c];
      d1 = delta[(size_t)slab * D + 2 * c + 1];
    }
    float acc[NR][2];
#pragma unroll
    for (int r = 0; r < NR; ++r) acc[r][0] = acc[r][1] = 0.f;
    // eight bins per round, their loads issued together (the compiler cannot move a load of this array
    // above the store before it)
    for (int i0 = 0; i0 < nb; i0 += 8) {
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (live && i0 + u < nb) v[u] = *reinterpret_cast<const float4*>(base + ((size_t)(i0 + u) * D + 2 * c) * 2);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int i = min(i0 + u, 31);
        const bool in = i0 + u < nb;                          // uniform over the warp
        const float wr = __shfl_sync(0xffffffffu, my.x, i), wi = __shfl_sync(0xffffffffu, my.y, i);
        if (live && in) {
          v[u].x = fmaf(d0, wr, v[u].x); v[u].y = fmaf(d0, wi, v[u].y);
          v[u].z = fmaf(d1, wr, v[u].z); v[u].w = fmaf(d1, wi, v[u].w);
          *reinterpret_cast<float4*>(base + ((size_t)(i0 + u) * D + 2 * c) * 2) = v[u];
        }
#pragma unroll
        for (int r = 0; r < NR; ++r) {
          const float cr = __shfl_sync(0xffffffffu, coef[r].x, i), ci = __shfl_sync(0xffffffffu, coef[r].y, i);
          if (in) {
            acc[r][0] = fmaf(cr, v[u].x, fmaf(-ci, v[u].y, acc[r][0]));
            acc[r][1] = fmaf(cr, v[u].z, fmaf(-ci, v[u].w, acc[r][1]));
          }
        }
      }
    }
#pragma unroll
    for (int r = 0; r < NR; ++r) {
      red[warp][r][2 * lane] = acc[r][0];
      red[warp][r][2 * lane + 1] = acc[r][1];
    }
    __syncthreads();
    for (int e = threadIdx.x; e < NR * 64; e += 256) {
      const int r = e >> 6, cc = e & 63;
      if (2 * c0 + cc < D) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) s += red[w][r][cc];
        partial[(((size_t)slab * nblk + blk) * NR + r) * D + 2 * c0 + cc] = s;
      }
    }
    __syncthreads();
  }
}

template <typename T>
__global__ void __launch_bounds__(256) decode_reduce_kernel(const float* __restrict__ partial, T* __restrict__ y, int B, int H,
                                                            int D, int nblk, int NR, int nrows) {
  const int total = B * nrows * H * D;
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  int c = idx % D, h = (idx / D) % H, r = (idx / (D * H)) % nrows, b = idx / (D * H * nrows);
  const float* p = partial + (((size_t)(b * H + h) * nblk) * NR + r) * D + c;
  float s = 0.f;
  for (int blk0 = 0; blk0 < nblk; blk0 += 16) {              // 16 partials in flight; the order of the sum is fixed
    float v[16];
#pragma unroll
    for (int u = 0; u < 16; ++u) v[u] = blk0 + u < nblk ? __ldg(p + (size_t)(blk0 + u) * NR * D) : 0.f;
#pragma unroll
    for (int u = 0; u < 16; ++u) s += v[u];
  }
  io<T>::store1(y + idx, s);
}

static int check_cache(const spectre_cache* c) {
  if (!c) return fail(SPECTRE_ERR_INVALID_ARG, "cache descriptor is NULL");
  if (c->B < 1 || c->H < 1 || c->D < 1 || c->N_max < 2) return fail(SPECTRE_ERR_INVALID_ARG, "cache extents");
  if (c->D % 8) return fail(SPECTRE_ERR_UNSUPPORTED, "cache D must be a multiple of 8");
  if (!is_io_dtype(c->buf_dtype)) return fail(SPECTRE_ERR_INVALID_ARG, "cache dtype");
  if (!c->prefix_fft || !c->V_buf || !c->Q_buf || !c->sum_q) return fail(SPECTRE_ERR_INVALID_ARG, "cache pointer is NULL");
  if ((reinterpret_cast<uintptr_t>(c->prefix_fft) | reinterpret_cast<uintptr_t>(c->V_buf) |
       reinterpret_cast<uintptr_t>(c->Q_buf)) & 15)
    return fail(SPECTRE_ERR_INVALID_ARG, "cache buffers must be 16-byte aligned");
  return SPECTRE_OK;
}

// Group size cap for the prefill scratch.  Larger groups measured faster (fewer, fuller launches; the partial
// spectra do not stay in L2 at any useful group size): 3.0 ms at 32-64 MB, 2.58 ms at 256 MB, 2.49 ms at 1 GiB, 2.47 ms
// with all 256 heads of the c4 window in one group (2.15 GB).
static const size_t kPrefillWsCap = (size_t)1 << 30;

}  // namespace spectre

using namespace spectre;

extern "C" size_t spectre_prefill_workspace_bytes(const spectre_ctx* ctx, int32_t B, int32_t H, int32_t D, int32_t N_max) {
  if (!ctx || B < 1 || H < 1 || D < 8 || !transform_supported(ctx, N_max)) return 0;
  size_t per = transform_slab_bytes(N_max, D);
  size_t g = kPrefillWsCap / per;
  if (g < 1) g = 1;
  if (g > (size_t)B * H) g = (size_t)B * H;
  return g * per;
}

extern "C" int spectre_prefix_cache_prefill(spectre_ctx* ctx, void* stream, const spectre_cache* cache,
                                            const spectre_act* q, const spectre_act* v, void* workspace,
                                            size_t workspace_bytes) {
  if (!ctx) return fail(SPECTRE_ERR_INVALID_ARG, "ctx is NULL");
  int rc = check_cache(cache);
  if (rc != SPECTRE_OK) return rc;
  rc = check_act(q, "q");
  if (rc != SPECTRE_OK) return rc;
  rc = check_act(v, "v");
  if (rc != SPECTRE_OK) return rc;
  const int B = cache->B, H = cache->H, D = cache->D, N = cache->N_max;
  if (q->B != B || q->H != H || q->D != D || v->B != B || v->H != H || v->D != D || q->L != v->L)
    return fail(SPECTRE_ERR_INVALID_ARG, "q / v shape differs from the cache");
  if (q->dtype != cache->buf_dtype || v->dtype != cache->buf_dtype)
    return fail(SPECTRE_ERR_INVALID_ARG, "q / v dtype differs from buf_dtype");
  if (v->L > N) return fail(SPECTRE_ERR_INVALID_ARG, "prompt longer than N_max");
  if (!transform_supported(ctx, N)) return fail(SPECTRE_ERR_UNSUPPORTED, "N_max outside the supported transform lengths");
  const size_t per = transform_slab_bytes(N, D);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 15))
    return fail(SPECTRE_ERR_WORKSPACE, "workspace is NULL or not 16-byte aligned");
  if (workspace_bytes < per) return fail(SPECTRE_ERR_WORKSPACE, "prefill workspace smaller than one (batch, head) slab");
  SPECTRE_CUDA_OK(cudaSetDevice(ctx->device));
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int nslab = B * H, K = N / 2 + 1;
  size_t gmax = workspace_bytes / per;
  if (gmax > (size_t)nslab) gmax = (size_t)nslab;
  const int ngroups = (nslab + (int)gmax - 1) / (int)gmax;
  const int group = (nslab + ngroups - 1) / ngroups;             // equal groups rather than full ones and a remainder
  float2* ws = reinterpret_cast<float2*>(workspace);
  int v_ring_done = 0;                 // the transform's load pass can fill V_buf on its way
  for (int s0 = 0; s0 < nslab; s0 += group) {
    int cnt = nslab - s0 < group ? nslab - s0 : group;
    int N1 = 1, M = N;
    rc = forward_decimated(ctx, st, v, N, s0, cnt, ws, &N1, &M, cache->V_buf, &v_ring_done);
    if (rc != SPECTRE_OK) return rc;
    switch (N1) {
      case 1: {
        size_t total = (size_t)cnt * ((K + kSplitBins - 1) / kSplitBins) * (D / 2);
        split_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(ws, cache->prefix_fft, N, K, D, s0, cnt);
        break;
      }
      case 2: launch_combine_split<2>(st, ws, cache->prefix_fft, N, K, D, M, s0, cnt); break;
      case 4: launch_combine_split<4>(st, ws, cache->prefix_fft, N, K, D, M, s0, cnt); break;
      case 8: launch_combine_split<8>(st, ws, cache->prefix_fft, N, K, D, M, s0, cnt); break;
      case 16: launch_combine_split<16>(st, ws, cache->prefix_fft, N, K, D, M, s0, cnt); break;
      default: return fail(SPECTRE_ERR_UNSUPPORTED, "outer factor not supported");
    }
    SPECTRE_LAUNCH_OK("split kernel");
  }
  const size_t nblocks = (size_t)B * ((N + kRingRows - 1) / kRingRows);
  if (nblocks > 0x7fffffffu) return fail(SPECTRE_ERR_UNSUPPORTED, "B * N_max too large for the ring copy");
  unsigned blocks = (unsigned)nblocks;
  if (!v_ring_done) {
    SPECTRE_IO_DISPATCH(cache->buf_dtype, {
      ring_fill_kernel<T><<<blocks, 256, 0, st>>>(reinterpret_cast<const T*>(v->ptr), v->stride_b, v->stride_l, v->stride_h,
                                                  reinterpret_cast<T*>(cache->V_buf), B, N, H, D, v->L);
    });
    SPECTRE_LAUNCH_OK("ring_fill_kernel");
  }
  // q is read once: its sum over the sequence and its ring copy come from the same pass
  return pool_sum_ring(ctx, st, q, cache->sum_q, cache->Q_buf, N);
}

extern "C" int spectre_prefix_cache_append(spectre_ctx* ctx, void* stream, const spectre_cache* cache, const void* q_t,
                                           const void* v_t, int64_t t) {
  if (!ctx) return fail(SPECTRE_ERR_INVALID_ARG, "ctx is NULL");
  int rc = check_cache(cache);
  if (rc != SPECTRE_OK) return rc;
  if (!q_t || !v_t) return fail(SPECTRE_ERR_INVALID_ARG, "token pointer is NULL");
  if (t < 0) return fail(SPECTRE_ERR_INVALID_ARG, "t must be >= 0");
  const int B = cache->B, H = cache->H, D = cache->D, N = cache->N_max;
  if ((size_t)B * H * D > (size_t)1 << 30) return fail(SPECTRE_ERR_UNSUPPORTED, "B*H*D too large");
  SPECTRE_CUDA_OK(cudaSetDevice(ctx->device));
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int K = N / 2 + 1;
  const int slot = (int)(t % N);
  const int evict = t >= N ? 1 : 0;
  const int wps = (K + 31) / 32;
  const size_t nwarps = (size_t)B * H * wps;
  const unsigned blocks = (unsigned)((nwarps * 32 + 255) / 256);
  const unsigned blocks2 = (unsigned)(((size_t)B * H * D + 255) / 256);
  SPECTRE_IO_DISPATCH(cache->buf_dtype, {
    append_spectrum_kernel<T><<<blocks, 256, 0, st>>>(cache->prefix_fft, reinterpret_cast<const T*>(cache->V_buf),
                                                      reinterpret_cast<const T*>(v_t), H, D, N, K, slot, (unsigned)slot,
                                                      evict, wps, nwarps);
    append_ring_kernel<T><<<blocks2, 256, 0, st>>>(reinterpret_cast<T*>(cache->V_buf), reinterpret_cast<T*>(cache->Q_buf),
                                                   cache->sum_q, reinterpret_cast<const T*>(q_t),
                                                   reinterpret_cast<const T*>(v_t), B, H, D, N, slot, evict);
  });
  SPECTRE_LAUNCH_OK("append kernels");
  return SPECTRE_OK;
}

static size_t round256(size_t x) { return (x + 255) & ~(size_t)255; }
static int decode_nr(int nrows) { return nrows <= 1 ? 1 : (nrows <= 2 ? 2 : SPECTRE_DECODE_MAX_ROWS); }

extern "C" size_t spectre_decode_workspace_bytes(const spectre_ctx* ctx, int32_t B, int32_t H, int32_t D, int32_t N_max,
                                                 int32_t nrows, int32_t toeplitz_r) {
  (void)ctx;
  if (B < 1 || H < 1 || D < 1 || N_max < 2 || nrows < 1 || nrows > SPECTRE_DECODE_MAX_ROWS || toeplitz_r < 0) return 0;
  const int K = N_max / 2 + 1, nblk = (K + 255) / 256;
  return round256((size_t)B * H * D * 4) + round256((size_t)B * H * nblk * decode_nr(nrows) * D * 4) +
         gate_min_workspace(B, H, D, N_max, toeplitz_r);
}

extern "C" int spectre_prefix_cache_decode_step(spectre_ctx* ctx, void* stream, const spectre_cache* cache, const void* q_t,
                                                const void* v_t, int64_t t, const spectre_gate_params* params,
                                                const int32_t* rows, int32_t nrows, void* y_rows, float* g_out,
                                                void* workspace, size_t workspace_bytes) {
  if (!ctx) return fail(SPECTRE_ERR_INVALID_ARG, "ctx is NULL");
  int rc = check_cache(cache);
  if (rc != SPECTRE_OK) return rc;
  if (!q_t || !v_t || !y_rows || !g_out) return fail(SPECTRE_ERR_INVALID_ARG, "token, output or gate pointer is NULL");
  if (!params) return fail(SPECTRE_ERR_INVALID_ARG, "gate parameters are NULL");
  if (t < 0) return fail(SPECTRE_ERR_INVALID_ARG, "t must be >= 0");
  if (!rows || nrows < 1 || nrows > SPECTRE_DECODE_MAX_ROWS)
    return fail(SPECTRE_ERR_INVALID_ARG, "rows is NULL or nrows outside 1..SPECTRE_DECODE_MAX_ROWS");
  const int B = cache->B, H = cache->H, D = cache->D, N = cache->N_max;
  for (int i = 0; i < nrows; ++i)
    if (rows[i] < 0 || rows[i] >= N) return fail(SPECTRE_ERR_INVALID_ARG, "read-out row outside [0, N_max)");
  if ((size_t)B * H * D > (size_t)1 << 30) return fail(SPECTRE_ERR_UNSUPPORTED, "B*H*D too large");
  const int K = N / 2 + 1, nblk = (K + 255) / 256, NR = decode_nr(nrows);
  if ((size_t)B * H * nblk > (size_t)0x7fffffff) return fail(SPECTRE_ERR_UNSUPPORTED, "B*H*K too large");
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 15))
    return fail(SPECTRE_ERR_WORKSPACE, "workspace is NULL or not 16-byte aligned");
  const size_t delta_bytes = round256((size_t)B * H * D * 4);
  const size_t part_bytes = round256((size_t)B * H * nblk * NR * D * 4);
  const size_t gate_bytes = gate_min_workspace(B, H, D, N, params->toeplitz_r < 0 ? 0 : params->toeplitz_r);
  if (workspace_bytes < delta_bytes + part_bytes + gate_bytes) return fail(SPECTRE_ERR_WORKSPACE, "decode workspace too small");
  SPECTRE_CUDA_OK(cudaSetDevice(ctx->device));
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  float* delta = reinterpret_cast<float*>(workspace);
  float* partial = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(workspace) + delta_bytes);
  void* gate_ws = reinterpret_cast<unsigned char*>(workspace) + delta_bytes + part_bytes;
  const int slot = (int)(t % N);
  const int evict = t >= N ? 1 : 0;
  // (a)-(b) ring buffers, running sum, delta
  const unsigned blocks_r = (unsigned)(((size_t)B * H * D + 255) / 256);
  SPECTRE_IO_DISPATCH(cache->buf_dtype,
                      decode_ring_kernel<T><<<blocks_r, 256, 0, st>>>(reinterpret_cast<T*>(cache->V_buf), reinterpret_cast<T*>(cache->Q_buf),
                                                                      cache->sum_q, delta, reinterpret_cast<const T*>(q_t),
                                                                      reinterpret_cast<const T*>(v_t), B, H, D, N, slot, evict));
  SPECTRE_LAUNCH_OK("decode_ring_kernel");
  // (c)-(d) gate from the running sum with phase p = t
  rc = spectre_gate(ctx, stream, nullptr, cache->sum_q, B, H, D, 1.0f / (float)N, params, N, nullptr, t, g_out, nullptr,
                    gate_ws, gate_bytes);
  if (rc != SPECTRE_OK) return rc;
  // (b) + (e) one pass over the spectrum
  DecodeRows dr;
  for (int i = 0; i < SPECTRE_DECODE_MAX_ROWS; ++i) dr.r[i] = rows[i < nrows ? i : nrows - 1];
  const unsigned blocks_s = (unsigned)((size_t)B * H * nblk);
  const float2* g2 = reinterpret_cast<const float2*>(g_out);
  if (NR == 1) decode_spectrum_kernel<1><<<blocks_s, 256, 0, st>>>(cache->prefix_fft, delta, g2, partial, D, N, K, (unsigned)slot, dr, nblk);
  else if (NR == 2) decode_spectrum_kernel<2><<<blocks_s, 256, 0, st>>>(cache->prefix_fft, delta, g2, partial, D, N, K, (unsigned)slot, dr, nblk);
  else decode_spectrum_kernel<SPECTRE_DECODE_MAX_ROWS><<<blocks_s, 256, 0, st>>>(cache->prefix_fft, delta, g2, partial, D, N, K, (unsigned)slot, dr, nblk);
  SPECTRE_LAUNCH_OK("decode_spectrum_kernel");
  const unsigned blocks_y = (unsigned)(((size_t)B * nrows * H * D + 255) / 256);
  SPECTRE_IO_DISPATCH(cache->buf_dtype,
                      decode_reduce_kernel<T><<<blocks_y, 256, 0, st>>>(partial, reinterpret_cast<T*>(y_rows), B, H, D, nblk, NR, nrows));
  SPECTRE_LAUNCH_OK("decode_reduce_kernel");
  return SPECTRE_OK;
}

extern "C" size_t spectre_readout_workspace_bytes(const spectre_ctx* ctx, int32_t B, int32_t H, int32_t D, int32_t N_max) {
  if (!ctx || B < 1 || H < 1 || D < 8 || !transform_supported(ctx, N_max)) return 0;
  return inverse_workspace_bytes(ctx, N_max, D, B * H);
}

extern "C" int spectre_prefix_cache_readout(spectre_ctx* ctx, void* stream, const spectre_cache* cache, const float* g,
                                            const spectre_act* y, void* workspace, size_t workspace_bytes) {
  if (!ctx) return fail(SPECTRE_ERR_INVALID_ARG, "ctx is NULL");
  int rc = check_cache(cache);
  if (rc != SPECTRE_OK) return rc;
  rc = check_act(y, "y");
  if (rc != SPECTRE_OK) return rc;
  if (!g || (reinterpret_cast<uintptr_t>(g) & 7)) return fail(SPECTRE_ERR_INVALID_ARG, "g is NULL or not 8-byte aligned");
  const int N = cache->N_max;
  if (y->B != cache->B || y->H != cache->H || y->D != cache->D || y->L > N || y->L < 1)
    return fail(SPECTRE_ERR_INVALID_ARG, "y shape differs from the cache (rows 0..L-1 of the window, L <= N_max)");
  if (!transform_supported(ctx, N)) return fail(SPECTRE_ERR_UNSUPPORTED, "N_max outside the supported transform lengths");
  SPECTRE_CUDA_OK(cudaSetDevice(ctx->device));
  return inverse_from_spectrum(ctx, reinterpret_cast<cudaStream_t>(stream), cache->prefix_fft, g, y, N, workspace,
                               workspace_bytes);
}
