// Context, status strings and host-side argument checks of the C ABI.
#include <cstdio>
#include <new>

#include "tc_common.cuh"

namespace spectre {

int build_dft64(__half* F, cudaStream_t st);   // mixer_tc.cu
int build_tw8192(float2* tab, cudaStream_t st);
int build_dft49(__half* F, cudaStream_t st);
int build_tw64x64(float2* tab, cudaStream_t st);
int build_tw_staged(float2* tab, cudaStream_t st);   // mixer_tc4k.cu
int build_dft32(void* mats, cudaStream_t st);        // mixer_tc32.cu

static thread_local std::string g_last_error;

int fail(int status, const std::string& msg) {
  g_last_error = msg;
  return status;
}

int cuda_fail(cudaError_t e, const char* what) {
  g_last_error = std::string(what) + ": " + cudaGetErrorString(e);
  return SPECTRE_ERR_CUDA;
}

bool is_pow2(int64_t x) { return x > 0 && (x & (x - 1)) == 0; }

int radix_plan(int n, int* radices) {
  if (n < 1) return -1;
  int cnt = 0;
  int rem = n;
  const int odd[3] = {7, 5, 3};
  for (int i = 0; i < 3; ++i) {
    while (rem % odd[i] == 0) {
      if (cnt >= 8) return -1;
      radices[cnt++] = odd[i];
      rem /= odd[i];
    }
  }
  if (!is_pow2(rem)) return -1;
  int a = 0;
  while ((1 << a) < rem) ++a;
  int q = a / 4, r = a % 4;
  if (r == 1 && q >= 1) {          // 16 * 2 -> 8 * 4 keeps the stages balanced
    for (int i = 0; i < q - 1; ++i) { if (cnt >= 8) return -1; radices[cnt++] = 16; }
    if (cnt + 2 > 8) return -1;
    radices[cnt++] = 8;
    radices[cnt++] = 4;
  } else {
    for (int i = 0; i < q; ++i) { if (cnt >= 8) return -1; radices[cnt++] = 16; }
    if (r > 0) { if (cnt >= 8) return -1; radices[cnt++] = 1 << r; }
  }
  return cnt;
}

int check_act(const spectre_act* a, const char* name) {
  std::string nm(name);
  if (!a) return fail(SPECTRE_ERR_INVALID_ARG, nm + ": descriptor is NULL");
  if (!a->ptr) return fail(SPECTRE_ERR_INVALID_ARG, nm + ": data pointer is NULL");
  if (!is_io_dtype(a->dtype)) return fail(SPECTRE_ERR_INVALID_ARG, nm + ": unknown dtype");
  if (a->B < 1 || a->L < 1 || a->H < 1 || a->D < 1) return fail(SPECTRE_ERR_INVALID_ARG, nm + ": non-positive extent");
  if (a->D % 8 != 0) return fail(SPECTRE_ERR_UNSUPPORTED, nm + ": D must be a multiple of 8");
  const int64_t es = io_elem_bytes(a->dtype);
  if (reinterpret_cast<uintptr_t>(a->ptr) & 15) return fail(SPECTRE_ERR_INVALID_ARG, nm + ": pointer not 16-byte aligned");
  if ((a->stride_b * es) % 16 || (a->stride_l * es) % 16 || (a->stride_h * es) % 16)
    return fail(SPECTRE_ERR_INVALID_ARG, nm + ": strides must keep rows 16-byte aligned");
  if (a->stride_h < a->D && a->H > 1) return fail(SPECTRE_ERR_INVALID_ARG, nm + ": head stride smaller than D");
  return SPECTRE_OK;
}

}  // namespace spectre

using namespace spectre;

extern "C" int spectre_create(spectre_ctx** out, int device) {
  if (!out) return fail(SPECTRE_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  int count = 0;
  cudaError_t e = cudaGetDeviceCount(&count);
  if (e != cudaSuccess) return cuda_fail(e, "cudaGetDeviceCount (no CUDA device: there is no CPU fallback)");
  if (device < 0 || device >= count) return fail(SPECTRE_ERR_INVALID_ARG, "device index out of range");
  cudaDeviceProp prop;
  SPECTRE_CUDA_OK(cudaGetDeviceProperties(&prop, device));
  if (prop.major < 10) return fail(SPECTRE_ERR_UNSUPPORTED, "built for sm_100a; this device is older");
  spectre_ctx* c = new (std::nothrow) spectre_ctx();
  if (!c) return fail(SPECTRE_ERR_INVALID_ARG, "out of host memory");
  c->device = device;
  c->sm_count = prop.multiProcessorCount;
  c->max_smem_optin = (int)prop.sharedMemPerBlockOptin;
  int cl = 0;
  cudaDeviceGetAttribute(&cl, cudaDevAttrClusterLaunch, device);
  c->cluster_ok = cl;
  c->l2_bytes = (size_t)prop.l2CacheSize;
  c->dft64 = nullptr;
  c->tw8192 = nullptr;
  c->dft49 = nullptr;
  c->tw64x64 = nullptr;
  c->tw_staged = nullptr;
  c->dft32 = nullptr;
  c->status_host = nullptr;
  c->status_dev = nullptr;
  cudaError_t e2 = cudaSetDevice(device);
  if (e2 == cudaSuccess) e2 = cudaMalloc(&c->dft64, 128 * 128 * sizeof(__half));
  if (e2 == cudaSuccess) e2 = cudaMalloc(&c->tw8192, 2049 * sizeof(float2));
  if (e2 == cudaSuccess) e2 = cudaMalloc(&c->dft49, 128 * 128 * sizeof(__half));
  if (e2 == cudaSuccess) e2 = cudaMalloc(&c->tw64x64, 2048 * sizeof(float2));
  if (e2 == cudaSuccess) e2 = cudaMalloc(&c->tw_staged, 63 * 128 * sizeof(float2));
  if (e2 == cudaSuccess) e2 = cudaMalloc(&c->dft32, 5 * 4 * 16384);
  if (e2 == cudaSuccess) e2 = cudaHostAlloc(reinterpret_cast<void**>(&c->status_host), sizeof(int), cudaHostAllocMapped);
  if (e2 == cudaSuccess) {
    *c->status_host = 0;
    e2 = cudaHostGetDevicePointer(reinterpret_cast<void**>(&c->status_dev), c->status_host, 0);
  }
  if (e2 == cudaSuccess) {
    int rc = build_dft64(reinterpret_cast<__half*>(c->dft64), 0);
    if (rc == SPECTRE_OK) rc = build_tw8192(reinterpret_cast<float2*>(c->tw8192), 0);
    if (rc == SPECTRE_OK) rc = build_dft49(reinterpret_cast<__half*>(c->dft49), 0);
    if (rc == SPECTRE_OK) rc = build_tw64x64(reinterpret_cast<float2*>(c->tw64x64), 0);
    if (rc == SPECTRE_OK) rc = build_tw_staged(reinterpret_cast<float2*>(c->tw_staged), 0);
    if (rc == SPECTRE_OK) rc = build_dft32(c->dft32, 0);
    if (rc == SPECTRE_OK) e2 = cudaStreamSynchronize(0);
    else e2 = cudaErrorUnknown;
  }
  if (e2 != cudaSuccess) {
    spectre_destroy(c);
    return cuda_fail(e2, "spectre_create: device table set-up");
  }
  *out = c;
  return SPECTRE_OK;
}

extern "C" int spectre_destroy(spectre_ctx* ctx) {
  if (ctx) {
    if (ctx->dft64) cudaFree(ctx->dft64);
    if (ctx->tw8192) cudaFree(ctx->tw8192);
    if (ctx->dft49) cudaFree(ctx->dft49);
    if (ctx->tw64x64) cudaFree(ctx->tw64x64);
    if (ctx->tw_staged) cudaFree(ctx->tw_staged);
    if (ctx->dft32) cudaFree(ctx->dft32);
    if (ctx->status_host) cudaFreeHost(ctx->status_host);
  }
  delete ctx;
  return SPECTRE_OK;
}

extern "C" int spectre_poll_status(spectre_ctx* ctx) {
  if (!ctx || !ctx->status_host) return fail(SPECTRE_ERR_INVALID_ARG, "ctx is NULL");
  int v = *reinterpret_cast<volatile int*>(ctx->status_host);
  if (v != 0) {
    *reinterpret_cast<volatile int*>(ctx->status_host) = 0;
    if (v & 1) return fail(SPECTRE_ERR_TIMEOUT, "a kernel gave up on a bounded on-chip wait; its outputs are undefined");
    return fail(SPECTRE_ERR_RANGE,
                "a tensor-core mixer produced non-finite values: its fp16 intermediates overflowed (input amplitude beyond "
                "the documented range); rerun that call with SPECTRE_FORCE_PATH=alu");
  }
  return SPECTRE_OK;
}

// One warp, one barrier nobody arrives on, a short poll limit: the wait runs out by construction (no copy,
// no MMA in flight), the kernel records it like the mixers do and returns normally.
__global__ void wait_selftest_kernel(int* status) {
  __shared__ __align__(8) uint64_t bar;
  const uint32_t b = (uint32_t)__cvta_generic_to_shared(&bar);
  if (threadIdx.x == 0) {
    mbar_init(b, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  const bool ok = mbar_wait_limit(b, 0, 4096);
  if (!ok && threadIdx.x == 0) report_timeout(status);
}

extern "C" int spectre_selftest_wait_timeout(spectre_ctx* ctx, void* stream) {
  if (!ctx) return fail(SPECTRE_ERR_INVALID_ARG, "ctx is NULL");
  SPECTRE_CUDA_OK(cudaSetDevice(ctx->device));
  wait_selftest_kernel<<<1, 32, 0, reinterpret_cast<cudaStream_t>(stream)>>>(ctx->status_dev);
  SPECTRE_LAUNCH_OK("wait_selftest_kernel");
  return SPECTRE_OK;
}

extern "C" const char* spectre_status_string(int status) {
  switch (status) {
    case SPECTRE_OK: return "ok";
    case SPECTRE_ERR_INVALID_ARG: return "invalid argument";
    case SPECTRE_ERR_UNSUPPORTED: return "unsupported configuration";
    case SPECTRE_ERR_WORKSPACE: return "workspace missing or too small";
    case SPECTRE_ERR_CUDA: return "CUDA error";
    case SPECTRE_ERR_TIMEOUT: return "device-side wait timed out";
    case SPECTRE_ERR_RANGE: return "input amplitude outside the range of the 16-bit tensor-core path";
    default: return "unknown status";
  }
}

extern "C" const char* spectre_last_error(void) { return g_last_error.c_str(); }
