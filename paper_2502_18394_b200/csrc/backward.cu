// Backward of the spectral mixer (Eq. 3-4 are real-linear in V and in (Re g, Im g); Sec. 3.7
// asks for differentiability).  With Vhat = R_n(pad V), Ghat = R_n(pad dY):
//   dV   = R_n^{-1}( conj(g) Ghat )              -> the forward mixer on dY with the conjugate gate
//   dg_k = (w_k / n) sum_c conj(Vhat_{k,c}) Ghat_{k,c},   w_0 = w_{n/2} = 1, else 2
// The gate gradient needs both spectra at once: two forward-only passes of the fp32 transform
// kernels into the workspace (pair-packed columns, Z = fft(a + jb)), then one reduction over the
// column pairs that uses  conj(A^V) A^G + conj(B^V) B^G = ( conj(Z^V_k) Z^G_k + Z^V_{n-k} conj(Z^G_{n-k}) ) / 2.
#include "common.cuh"

namespace spectre {

// from mixer.cu
int forward_spectrum(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, int n, int slab0, int cnt,
                     float2* ws, int* N1_out, int* M_out);
bool transform_supported(const spectre_ctx* ctx, int n);
size_t transform_slab_bytes(int n, int D);

__global__ void __launch_bounds__(256) conj_gate_kernel(const float2* __restrict__ g, float2* __restrict__ gc, size_t total) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < total) {
    float2 v = g[i];
    gc[i] = make_float2(v.x, -v.y);
  }
}

// One warp per (slab, bin): lanes over the column pairs, both workspaces laid out
// ws[slab_local][k1][kM][D/2] with bin k = k1 + N1 kM.
__global__ void __launch_bounds__(256) gate_grad_kernel(const float2* __restrict__ wsV, const float2* __restrict__ wsG,
                                                        float2* __restrict__ dg, int n, int K, int D, int N1, int M,
                                                        int slab0, int nslab) {
  const size_t wid = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (wid >= (size_t)nslab * K) return;
  const int k = (int)(wid % K), slab_local = (int)(wid / K);
  const int km = (n - k) % n;
  const int half = D / 2;
  const size_t rk = (((size_t)slab_local * N1 + (k % N1)) * M + k / N1) * half;
  const size_t rm = (((size_t)slab_local * N1 + (km % N1)) * M + km / N1) * half;
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
      rc = forward_spectrum(ctx, st, v, n_fft, s0, cnt, wsV, &N1, &M);
      if (rc != SPECTRE_OK) return rc;
      rc = forward_spectrum(ctx, st, dy, n_fft, s0, cnt, wsG, &N1, &M);
      if (rc != SPECTRE_OK) return rc;
      const size_t nwarps = (size_t)cnt * K;
      gate_grad_kernel<<<(unsigned)((nwarps * 32 + 255) / 256), 256, 0, st>>>(wsV, wsG, reinterpret_cast<float2*>(dg), n_fft, (int)K,
                                                                              D, N1, M, s0, cnt);
      SPECTRE_LAUNCH_OK("gate_grad_kernel");
    }
  }
  return SPECTRE_OK;
}
