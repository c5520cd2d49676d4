// Backward of the spectral mixer (Eq. 3-4 are real-linear in V and in (Re g, Im g); Sec. 3.7
// asks for differentiability).  With Vhat = R_n(pad V), Ghat = R_n(pad dY):
//   dV   = R_n^{-1}( conj(g) Ghat )              -> the forward mixer on dY with the conjugate gate
//   dg_k = (w_k / n) sum_c conj(Vhat_{k,c}) Ghat_{k,c},   w_0 = w_{n/2} = 1, else 2
// The gate gradient needs both spectra at once: two forward-only passes of the fp32 transform
// kernels into the workspace (pair-packed columns, Z = fft(a + jb)), then one reduction over the
// column pairs that uses  conj(A^V) A^G + conj(B^V) B^G = ( conj(Z^V_k) Z^G_k + Z^V_{n-k} conj(Z^G_{n-k}) ) / 2.
// Beyond one CTA's 2048 rows the passes leave the spectra of the N1 decimated sequences and the reduction
// runs the last radix-N1 step itself.
#include "common.cuh"

namespace spectre {

// from mixer.cu
int forward_decimated(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, int n, int slab0, int cnt,
                      float2* ws, int* N1_out, int* M_out, void* ring, int* ring_done);
bool transform_supported(const spectre_ctx* ctx, int n);
size_t transform_slab_bytes(int n, int D);

__global__ void __launch_bounds__(256) conj_gate_kernel(const float2* __restrict__ g, float2* __restrict__ gc, size_t total) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < total) {
    float2 v = g[i];
    gc[i] = make_float2(v.x, -v.y);
  }
}

// One warp per (slab, bin): lanes over the column pairs, both workspaces hold the spectrum itself,
// ws[slab_local][k][D/2] (transforms that fit one CTA).
__global__ void __launch_bounds__(256) gate_grad_kernel(const float2* __restrict__ wsV, const float2* __restrict__ wsG,
                                                        float2* __restrict__ dg, int n, int K, int D, int slab0, int nslab) {
  const size_t wid = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (wid >= (size_t)nslab * K) return;
  const int k = (int)(wid % K), slab_local = (int)(wid / K);
  const int km = (n - k) % n;
  const int half = D / 2;
  const size_t rk = ((size_t)slab_local * n + k) * half;
  const size_t rm = ((size_t)slab_local * n + km) * half;
  float2 acc = make_float2(0.f, 0.f);
  for (int c = lane; c < half; c += 32) {
    const float2 vk = wsV[rk + c], vm = wsV[rm + c], gk = wsG[rk + c], gm = wsG[rm + c];
    acc = cadd(acc, cmulc(gk, vk));          // conj(Z^V_k) Z^G_k
    acc = cadd(acc, cmulc(vm, gm));          // Z^V_{n-k} conj(Z^G_{n-k})
  }
  for (int o = 16; o > 0; o >>= 1) {
    acc.x += __shfl_xor_sync(0xffffffffu, acc.x, o);
    acc.y += __shfl_xor_sync(0xffffffffu, acc.y, o);
  }
  if (lane == 0) {
    const float w = ((k == 0 || 2 * k == n) ? 1.0f : 2.0f) * 0.5f / (float)n;
    dg[(size_t)(slab0 + slab_local) * K + k] = cscale(acc, w);
  }
}

// Longer transforms, n = N1 M with token t = N1 n2 + n1: the workspaces hold Y[n1][k2], the M-point spectra of
// the N1 decimated sequences (ws[slab_local][n1][k2][D/2]), and Z[k2 + M k1] = sum_n1 W_N1^{n1 k1} W_n^{n1 k2} Y[n1][k2].
// A warp (or half of one) per (slab, k2 <= M/2): it forms Z at k2 + M k1 and at (M - k2) + M k1 for both tensors — each
// family holds the mirror bins n - k of the other — and reduces the N1 (+1 at k2 = 0) bins k <= n/2 among them.
// KW bins k2 per warp, 32 / KW lanes each; a lane takes KW adjacent column pairs per load (KW = 2: 16-byte loads).
template <int N1, int KW>
__device__ __forceinline__ void combine_bins(const float2* __restrict__ ws, size_t row0, int M, int half, int c, int k2,
                                             int m2, const float2 (&wa)[N1], const float2 (&wb)[N1], float2 (&a)[KW][N1],
                                             float2 (&b)[KW][N1]) {
#pragma unroll
  for (int n1 = 0; n1 < N1; ++n1) {
    const float2* pa = ws + (row0 + (size_t)n1 * M + k2) * half + c;
    const float2* pb = ws + (row0 + (size_t)n1 * M + m2) * half + c;
    if (KW == 2) {
      const float4 ta = *reinterpret_cast<const float4*>(pa), tb = *reinterpret_cast<const float4*>(pb);
      a[0][n1] = make_float2(ta.x, ta.y); a[KW - 1][n1] = make_float2(ta.z, ta.w);
      b[0][n1] = make_float2(tb.x, tb.y); b[KW - 1][n1] = make_float2(tb.z, tb.w);
    } else {
      a[0][n1] = *pa;
      b[0][n1] = *pb;
    }
  }
#pragma unroll
  for (int v = 0; v < KW; ++v) {
#pragma unroll
    for (int q = 1; q < N1; ++q) {
      a[v][q] = cmul(a[v][q], wa[q]);
      b[v][q] = cmul(b[v][q], wb[q]);
    }
    Dft<N1, false>::run(a[v]);
    Dft<N1, false>::run(b[v]);
  }
}

template <int N1, int KW>
__global__ void __launch_bounds__(256) gate_grad_combine_kernel(const float2* __restrict__ wsV, const float2* __restrict__ wsG,
                                                                float2* __restrict__ dg, int n, int K, int D, int M,
                                                                int slab0, int nslab) {
  constexpr int LPK = 32 / KW;
  const size_t wid = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31, sub = lane % LPK;
  const int nk2 = M / 2 + 1, wpk = (nk2 + KW - 1) / KW;      // warps per slab
  if (wid >= (size_t)nslab * wpk) return;
  const int slab_local = (int)(wid / wpk);
  const int k2raw = (int)(wid % wpk) * KW + lane / LPK;
  const bool valid = k2raw < nk2;                               // the last warp of a slab may own one bin only
  const int k2 = valid ? k2raw : 0;
  const int m2 = (M - k2) % M;
  const int half = D / 2;
  const bool own = k2 == 0 || k2 == m2;        // k2 = 0 and k2 = M/2 are their own mirror
  float2 wa[N1], wb[N1];
  wa[0] = wb[0] = make_float2(1.f, 0.f);
#pragma unroll
  for (int q = 1; q < N1; ++q) {
    wa[q] = (q == 1) ? twiddle_fwd((unsigned)k2, (unsigned)n) : cmul(wa[q / 2], wa[q - q / 2]);
    wb[q] = (q == 1) ? twiddle_fwd((unsigned)m2, (unsigned)n) : cmul(wb[q / 2], wb[q - q / 2]);
  }
  float2 acc1[N1 / 2], acc2[N1 / 2], accn = make_float2(0.f, 0.f);
#pragma unroll
  for (int k1 = 0; k1 < N1 / 2; ++k1) acc1[k1] = acc2[k1] = make_float2(0.f, 0.f);
  const size_t row0 = (size_t)slab_local * N1 * M;
  for (int c = KW * sub; c < half; c += KW * LPK) {
    float2 va[KW][N1], vb[KW][N1], ga[KW][N1], gb[KW][N1];
    combine_bins<N1, KW>(wsV, row0, M, half, c, k2, m2, wa, wb, va, vb);
    combine_bins<N1, KW>(wsG, row0, M, half, c, k2, m2, wa, wb, ga, gb);
#pragma unroll
    for (int v = 0; v < KW; ++v) {
#pragma unroll
      for (int k1 = 0; k1 < N1 / 2; ++k1) {
        // bin k2 + M k1; its mirror is (N1 - k1) % N1 of the same family at k2 = 0, else N1 - 1 - k1 of the other
        const float2 vm = k2 == 0 ? va[v][(N1 - k1) % N1] : vb[v][N1 - 1 - k1];
        const float2 gm = k2 == 0 ? ga[v][(N1 - k1) % N1] : gb[v][N1 - 1 - k1];
        acc1[k1] = cadd(acc1[k1], cadd(cmulc(ga[v][k1], va[v][k1]), cmulc(vm, gm)));
        // bin (M - k2) + M k1, mirror N1 - 1 - k1 of the first family
        acc2[k1] = cadd(acc2[k1], cadd(cmulc(gb[v][k1], vb[v][k1]), cmulc(va[v][N1 - 1 - k1], ga[v][N1 - 1 - k1])));
      }
      // bin n/2 (k2 = 0 only), its own mirror
      accn = cadd(accn, cadd(cmulc(ga[v][N1 / 2], va[v][N1 / 2]), cmulc(va[v][N1 / 2], ga[v][N1 / 2])));
    }
  }
  float2* out = dg + (size_t)(slab0 + slab_local) * K;
  const float w2 = 1.0f / (float)n, w1 = 0.5f / (float)n;      // bins other than 0 and n/2 count twice
#pragma unroll
  for (int k1 = 0; k1 <= N1; ++k1) {
    float2 v = k1 < N1 / 2 ? acc1[k1 % (N1 / 2)] : (k1 < N1 ? acc2[k1 % (N1 / 2)] : accn);
#pragma unroll
    for (int o = LPK / 2; o > 0; o >>= 1) {
      v.x += __shfl_xor_sync(0xffffffffu, v.x, o);
      v.y += __shfl_xor_sync(0xffffffffu, v.y, o);
    }
    if (sub == 0 && valid) {
      if (k1 < N1 / 2) out[k2 + M * k1] = cscale(v, (k2 == 0 && k1 == 0) ? w1 : w2);
      else if (k1 < N1) { if (!own) out[m2 + M * (k1 - N1 / 2)] = cscale(v, w2); }
      else if (k2 == 0) out[M * (N1 / 2)] = cscale(v, w1);
    }
  }
}

template <int N1>
static void launch_gate_grad_combine(cudaStream_t st, const float2* wsV, const float2* wsG, float2* dg, int n, int K, int D,
                                     int M, int slab0, int cnt) {
  constexpr int KW = N1 <= 8 ? 2 : 1;
  const size_t nwarps = (size_t)cnt * ((M / 2 + 1 + KW - 1) / KW);
  gate_grad_combine_kernel<N1, KW><<<(unsigned)((nwarps * 32 + 255) / 256), 256, 0, st>>>(wsV, wsG, dg, n, K, D, M, slab0, cnt);
}

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }
static const size_t kSpectrumCap = (size_t)128 << 20;      // per spectrum buffer

static size_t spectrum_group(int n, int D, int nslab) {
  size_t per = transform_slab_bytes(n, D);
  size_t g = kSpectrumCap / per;
  if (g < 1) g = 1;
  if (g > (size_t)nslab) g = (size_t)nslab;
  return g;
}

}  // namespace spectre

using namespace spectre;

extern "C" size_t spectre_mixer_backward_workspace_bytes(const spectre_ctx* ctx, int32_t B, int32_t L, int32_t H, int32_t D,
                                                         int32_t n_fft, int32_t dtype) {
  if (!ctx || B < 1 || H < 1 || D < 8 || !transform_supported(ctx, n_fft)) return 0;
  const size_t K = (size_t)n_fft / 2 + 1;
  return align256((size_t)B * H * K * sizeof(float2)) +
         align256(spectre_mixer_workspace_bytes(ctx, B, L, H, D, n_fft, dtype)) +
         2 * spectrum_group(n_fft, D, B * H) * transform_slab_bytes(n_fft, D);
}

extern "C" int spectre_mixer_backward(spectre_ctx* ctx, void* stream, const spectre_act* v, const spectre_act* dy,
                                      const float* g, const spectre_act* dv, float* dg, int32_t n_fft, void* workspace,
                                      size_t workspace_bytes) {
  if (!ctx) return fail(SPECTRE_ERR_INVALID_ARG, "ctx is NULL");
  int rc = check_act(v, "v");
  if (rc != SPECTRE_OK) return rc;
  rc = check_act(dy, "dy");
  if (rc != SPECTRE_OK) return rc;
  if (dv) {
    rc = check_act(dv, "dv");
    if (rc != SPECTRE_OK) return rc;
    if (dv->B != v->B || dv->L != v->L || dv->H != v->H || dv->D != v->D || dv->dtype != v->dtype)
      return fail(SPECTRE_ERR_INVALID_ARG, "dv differs from v in shape or dtype");
  }
  if (dy->B != v->B || dy->L != v->L || dy->H != v->H || dy->D != v->D || dy->dtype != v->dtype)
    return fail(SPECTRE_ERR_INVALID_ARG, "dy differs from v in shape or dtype");
  if (!dv && !dg) return fail(SPECTRE_ERR_INVALID_ARG, "neither dv nor dg requested");
  if (!g || (reinterpret_cast<uintptr_t>(g) & 7)) return fail(SPECTRE_ERR_INVALID_ARG, "g is NULL or not 8-byte aligned");
  if (dg && (reinterpret_cast<uintptr_t>(dg) & 7)) return fail(SPECTRE_ERR_INVALID_ARG, "dg not 8-byte aligned");
  if (n_fft < v->L) return fail(SPECTRE_ERR_INVALID_ARG, "n_fft smaller than L");
  if (!transform_supported(ctx, n_fft)) return fail(SPECTRE_ERR_UNSUPPORTED, "n_fft outside the supported set");
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 15))
    return fail(SPECTRE_ERR_WORKSPACE, "workspace is NULL or not 16-byte aligned");
  const int B = v->B, H = v->H, D = v->D, nslab = B * H;
  const size_t K = (size_t)n_fft / 2 + 1;
  const size_t gc_bytes = align256((size_t)nslab * K * sizeof(float2));
  const size_t mix_bytes = align256(spectre_mixer_workspace_bytes(ctx, B, v->L, H, D, n_fft, v->dtype));
  const size_t per = transform_slab_bytes(n_fft, D);
  if (workspace_bytes < gc_bytes + mix_bytes + 2 * per) return fail(SPECTRE_ERR_WORKSPACE, "backward workspace too small");
  SPECTRE_CUDA_OK(cudaSetDevice(ctx->device));
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  unsigned char* base = reinterpret_cast<unsigned char*>(workspace);
  if (dv) {
    float2* gc = reinterpret_cast<float2*>(base);
    const size_t total = (size_t)nslab * K;
    conj_gate_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(reinterpret_cast<const float2*>(g), gc, total);
    SPECTRE_LAUNCH_OK("conj_gate_kernel");
    rc = spectre_mixer_forward(ctx, stream, dy, reinterpret_cast<const float*>(gc), dv, n_fft, nullptr,
                               mix_bytes ? base + gc_bytes : nullptr, mix_bytes);
    if (rc != SPECTRE_OK) return rc;
  }
  if (dg) {
    size_t group = (workspace_bytes - gc_bytes - mix_bytes) / (2 * per);
    if (group > (size_t)nslab) group = (size_t)nslab;
    float2* wsV = reinterpret_cast<float2*>(base + gc_bytes + mix_bytes);
    float2* wsG = reinterpret_cast<float2*>(base + gc_bytes + mix_bytes + group * per);
    for (int s0 = 0; s0 < nslab; s0 += (int)group) {
      const int cnt = nslab - s0 < (int)group ? nslab - s0 : (int)group;
      int N1 = 1, M = n_fft;
      int no_ring = 0;
      rc = forward_decimated(ctx, st, v, n_fft, s0, cnt, wsV, &N1, &M, nullptr, &no_ring);
      if (rc != SPECTRE_OK) return rc;
      rc = forward_decimated(ctx, st, dy, n_fft, s0, cnt, wsG, &N1, &M, nullptr, &no_ring);
      if (rc != SPECTRE_OK) return rc;
      float2* dgc = reinterpret_cast<float2*>(dg);
      switch (N1) {
        case 1: {
          const size_t nwarps = (size_t)cnt * K;
          gate_grad_kernel<<<(unsigned)((nwarps * 32 + 255) / 256), 256, 0, st>>>(wsV, wsG, dgc, n_fft, (int)K, D, s0, cnt);
          break;
        }
        case 2: launch_gate_grad_combine<2>(st, wsV, wsG, dgc, n_fft, (int)K, D, M, s0, cnt); break;
        case 4: launch_gate_grad_combine<4>(st, wsV, wsG, dgc, n_fft, (int)K, D, M, s0, cnt); break;
        case 8: launch_gate_grad_combine<8>(st, wsV, wsG, dgc, n_fft, (int)K, D, M, s0, cnt); break;
        case 16: launch_gate_grad_combine<16>(st, wsV, wsG, dgc, n_fft, (int)K, D, M, s0, cnt); break;
        default: return fail(SPECTRE_ERR_UNSUPPORTED, "outer factor not supported");
      }
      SPECTRE_LAUNCH_OK("gate_grad kernel");
    }
  }
  return SPECTRE_OK;
}
