// Shared device helpers for the SPECTRE kernels: status plumbing, I/O type
// conversion, complex arithmetic and in-register DFT butterflies.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>

#include "spectre.h"

struct spectre_ctx {
  int device;
  int sm_count;
  int max_smem_optin;     // bytes of dynamic shared memory a CTA may opt in to
  int cluster_ok;         // thread-block clusters usable on this device
  size_t l2_bytes;
  void* dft64;            // device: 64-point DFT matrix (fp16, MMA operand layout), 32 KiB
  void* dft49;            // device: 49-point DFT matrix, same format (n = 196 path), 32 KiB
  void* tw8192;           // device: (cos, sin)(2 pi r / 8192), r = 0..2048 (quarter wave), 16 KiB
  void* tw64x64;          // device: W_4096^{row d}, even columns d, in the epilogue threads' own order (float2), 16 KiB
  void* tw_staged;        // device: twiddles of the four-step split n = 4096 R, R = 1..32 (float2): rows R - 1 + k1 of
                          // 128 entries, W_n^{64 k1 t1} (t1 < 64) then W_n^{k1 t2} (t2 < 64); 63 KiB
  void* dft32;            // device: DFT matrices of the tensor-core radix-32 ... 2 kernels (MMA operand layout), 5 x 4 x 16 KiB
  int* status_host;       // pinned, device-mapped status word written by kernels whose waits ran out
  int* status_dev;
};

namespace spectre {

// ---- host-side error plumbing ------------------------------------------------
int fail(int status, const std::string& msg);          // records msg, returns status
int cuda_fail(cudaError_t e, const char* what);        // SPECTRE_ERR_CUDA with text
#define SPECTRE_CUDA_OK(expr)                                                   \
  do {                                                                          \
    cudaError_t e__ = (expr);                                                   \
    if (e__ != cudaSuccess) return ::spectre::cuda_fail(e__, #expr);            \
  } while (0)
#define SPECTRE_LAUNCH_OK(name)                                                 \
  do {                                                                          \
    cudaError_t e__ = cudaGetLastError();                                       \
    if (e__ != cudaSuccess) return ::spectre::cuda_fail(e__, name);             \
  } while (0)

int check_act(const spectre_act* a, const char* name);  // pointer, shape, alignment
bool is_pow2(int64_t x);
// Factorises n into radices from {16,8,4,2,7,5,3}; returns the number of
// stages (0 for n = 1) or -1 if n has another prime factor or needs > 8 stages.
int radix_plan(int n, int* radices);

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- device helpers --------------------------------------------------------
#ifdef __CUDACC__

typedef __nv_bfloat16 bf16;
typedef __half f16;

__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }
__device__ __forceinline__ float2 cmul(float2 a, float2 b) {
  return make_float2(fmaf(a.x, b.x, -a.y * b.y), fmaf(a.x, b.y, a.y * b.x));
}
// a * conj(b)
__device__ __forceinline__ float2 cmulc(float2 a, float2 b) {
  return make_float2(fmaf(a.x, b.x, a.y * b.y), fmaf(a.y, b.x, -a.x * b.y));
}
__device__ __forceinline__ float2 cscale(float2 a, float s) { return make_float2(a.x * s, a.y * s); }

// exp(-j 2 pi num / den) with the argument reduced exactly (0 <= num < den).
__device__ __forceinline__ float2 twiddle_fwd(unsigned num, unsigned den) {
  float s, c;
  sincospif(2.0f * (float)num / (float)den, &s, &c);
  return make_float2(c, -s);
}

// Full-spectrum value of a column pair (a, b) from their half spectra and the gate (read-out from a cached spectrum):
// Z_k = X^a_k + j X^b_k with X = g * P completed by Hermitian symmetry; at DC and Nyquist only
// the real parts of the two products survive the real inverse (App. B).
__device__ __forceinline__ float2 pair_from_half(float2 gk, float4 ab, int k, int kk, int n) {
  const float2 xa = cmul(gk, make_float2(ab.x, ab.y)), xb = cmul(gk, make_float2(ab.z, ab.w));
  if (k == 0 || 2 * k == n) return make_float2(xa.x, xb.x);
  if (kk == k) return make_float2(xa.x - xb.y, xa.y + xb.x);
  return make_float2(xa.x + xb.y, xb.x - xa.y);
}

// exp(-j 2 pi m / 8192) from the quarter-wave table (cos, sin)(2 pi r / 8192), r = 0..2048
__device__ __forceinline__ float2 twiddle8192(const float2* __restrict__ tab, unsigned m) {
  const unsigned q = (m >> 11) & 3u, r = m & 2047u;
  const float2 t = __ldg(tab + r);
  const float c = (q & 1u) ? -t.y : t.x, s = (q & 1u) ? t.x : t.y;    // rotate by q quarter turns
  return (q & 2u) ? make_float2(-c, s) : make_float2(c, -s);
}

// ---- loads / stores of 4 adjacent real columns as two complex pairs ----------
// (columns 2c and 2c+1 form the complex number a + jb; see mixer.cu)
template <typename T> struct io;
template <> struct io<float> {
  static __device__ __forceinline__ float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
  static __device__ __forceinline__ void store4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
  static __device__ __forceinline__ float load1(const float* p) { return *p; }
  static __device__ __forceinline__ void store1(float* p, float v) { *p = v; }
};
template <> struct io<bf16> {
  static __device__ __forceinline__ float4 load4(const bf16* p) {
    uint2 r = *reinterpret_cast<const uint2*>(p);
    float4 v;
    v.x = __uint_as_float(r.x << 16);
    v.y = __uint_as_float(r.x & 0xffff0000u);
    v.z = __uint_as_float(r.y << 16);
    v.w = __uint_as_float(r.y & 0xffff0000u);
    return v;
  }
  static __device__ __forceinline__ void store4(bf16* p, float4 v) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
    __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 r;
    r.x = *reinterpret_cast<unsigned*>(&lo);
    r.y = *reinterpret_cast<unsigned*>(&hi);
    *reinterpret_cast<uint2*>(p) = r;
  }
  static __device__ __forceinline__ float load1(const bf16* p) { return __bfloat162float(*p); }
  static __device__ __forceinline__ void store1(bf16* p, float v) { *p = __float2bfloat16_rn(v); }
};
template <> struct io<f16> {
  static __device__ __forceinline__ float4 load4(const f16* p) {
    const uint2 r = *reinterpret_cast<const uint2*>(p);
    const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&r.x));
    const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&r.y));
    return make_float4(lo.x, lo.y, hi.x, hi.y);
  }
  static __device__ __forceinline__ void store4(f16* p, float4 v) {
    const __half2 lo = __floats2half2_rn(v.x, v.y), hi = __floats2half2_rn(v.z, v.w);
    uint2 r;
    r.x = *reinterpret_cast<const unsigned*>(&lo);
    r.y = *reinterpret_cast<const unsigned*>(&hi);
    *reinterpret_cast<uint2*>(p) = r;
  }
  static __device__ __forceinline__ float load1(const f16* p) { return __half2float(*p); }
  static __device__ __forceinline__ void store1(f16* p, float v) { *p = __float2half_rn(v); }
};

// Runs the statement(s) with T bound to the element type of an activation dtype.
#define SPECTRE_IO_DISPATCH(dtype, ...)                                        \
  do {                                                                         \
    if ((dtype) == SPECTRE_BF16) { using T = ::spectre::bf16; __VA_ARGS__; }   \
    else if ((dtype) == SPECTRE_F16) { using T = ::spectre::f16; __VA_ARGS__; } \
    else { using T = float; __VA_ARGS__; }                                     \
  } while (0)
inline bool is_io_dtype(int d) { return d == SPECTRE_F32 || d == SPECTRE_BF16 || d == SPECTRE_F16; }
inline int io_elem_bytes(int d) { return d == SPECTRE_F32 ? 4 : 2; }

// ---- constant roots of unity -----------------------------------------------
// x * exp(-/+ j 2 pi J / R) for compile-time-foldable (J, R); INV conjugates.
template <bool INV>
__device__ __forceinline__ float2 mul_root(float2 x, int J, int R) {
  // reduce to sixteenths / odd radices; after unrolling J and R are constants
  J %= R;
  if (J == 0) return x;
  while ((J & 1) == 0 && (R & 1) == 0) { J >>= 1; R >>= 1; }     // lowest terms (folds after unrolling)
  if ((4 * J) % R == 0) {                 // multiples of a quarter turn
    int q = (4 * J) / R;                  // 1,2,3
    if (q == 2) return make_float2(-x.x, -x.y);
    bool minus_i = (q == 1) != INV;       // forward quarter turn = multiply by -j
    return minus_i ? make_float2(x.y, -x.x) : make_float2(-x.y, x.x);
  }
  if ((8 * J) % R == 0) {                 // odd eighths
    const float h = 0.70710678118654752440f;
    int e = (8 * J) / R;                  // 1,3,5,7
    if (INV) e = 8 - e;
    // exp(-j pi e / 4)
    switch (e) {
      case 1: return make_float2((x.x + x.y) * h, (x.y - x.x) * h);
      case 3: return make_float2((x.y - x.x) * h, -(x.x + x.y) * h);
      case 5: return make_float2(-(x.x + x.y) * h, (x.x - x.y) * h);
      default: return make_float2((x.x - x.y) * h, (x.x + x.y) * h);
    }
  }
  // general: literal cos/sin of 2 pi J / R (the switch folds after unrolling)
  float c = 1.0f, s = 0.0f;
  switch (R * 32 + J) {
    case 513: c = 0.92387953251128674f; s = 0.38268343236508978f; break;
    case 515: c = 0.38268343236508984f; s = 0.92387953251128674f; break;
    case 517: c = -0.38268343236508973f; s = 0.92387953251128674f; break;
    case 519: c = -0.92387953251128674f; s = 0.38268343236508989f; break;
    case 521: c = -0.92387953251128685f; s = -0.38268343236508967f; break;
    case 523: c = -0.38268343236509034f; s = -0.92387953251128652f; break;
    case 525: c = 0.38268343236509f; s = -0.92387953251128663f; break;
    case 527: c = 0.92387953251128652f; s = -0.38268343236509039f; break;
    case 97: c = -0.5f; s = 0.86602540378443871f; break;
    case 98: c = -0.5f; s = -0.86602540378443837f; break;
    case 161: c = 0.30901699437494745f; s = 0.95105651629515353f; break;
    case 162: c = -0.80901699437494734f; s = 0.58778525229247325f; break;
    case 163: c = -0.80901699437494756f; s = -0.58778525229247303f; break;
    case 164: c = 0.30901699437494723f; s = -0.95105651629515364f; break;
    case 225: c = 0.62348980185873359f; s = 0.7818314824680298f; break;
    case 226: c = -0.22252093395631434f; s = 0.97492791218182362f; break;
    case 227: c = -0.90096886790241903f; s = 0.43388373911755823f; break;
    case 228: c = -0.90096886790241915f; s = -0.43388373911755801f; break;
    case 229: c = -0.22252093395631459f; s = -0.97492791218182362f; break;
    case 230: c = 0.62348980185873337f; s = -0.78183148246802991f; break;
    case 1025: c = 0.98078528040323043f; s = 0.19509032201612825f; break;
    case 1027: c = 0.83146961230254524f; s = 0.55557023301960218f; break;
    case 1029: c = 0.55557023301960229f; s = 0.83146961230254524f; break;
    case 1031: c = 0.19509032201612833f; s = 0.98078528040323043f; break;
    case 1033: c = -0.19509032201612819f; s = 0.98078528040323043f; break;
    case 1035: c = -0.55557023301960196f; s = 0.83146961230254546f; break;
    case 1037: c = -0.83146961230254535f; s = 0.55557023301960218f; break;
    case 1039: c = -0.98078528040323043f; s = 0.19509032201612861f; break;
    case 1041: c = -0.98078528040323043f; s = -0.19509032201612836f; break;
    case 1043: c = -0.83146961230254546f; s = -0.55557023301960196f; break;
    case 1045: c = -0.55557023301960218f; s = -0.83146961230254524f; break;
    case 1047: c = -0.19509032201612866f; s = -0.98078528040323032f; break;
    case 1049: c = 0.1950903220161283f; s = -0.98078528040323043f; break;
    case 1051: c = 0.55557023301960184f; s = -0.83146961230254546f; break;
    case 1053: c = 0.83146961230254524f; s = -0.55557023301960218f; break;
    case 1055: c = 0.98078528040323032f; s = -0.19509032201612872f; break;
    default: break;
  }
  if (INV) s = -s;
  // x * (c - j s)
  return make_float2(fmaf(x.x, c, x.y * s), fmaf(x.y, c, -x.x * s));
}

// ---- in-register DFTs, natural order in and out ------------------------------
// Forward: X_k = sum_t x_t exp(-j 2 pi k t / R); INV uses the conjugate kernel
// (no 1/R scaling).
template <int R, bool INV> struct Dft;

template <bool INV> struct Dft<1, INV> {
  static __device__ __forceinline__ void run(float2 (&x)[1]) {}
};
template <bool INV> struct Dft<2, INV> {
  static __device__ __forceinline__ void run(float2 (&x)[2]) {
    float2 a = x[0], b = x[1];
    x[0] = cadd(a, b);
    x[1] = csub(a, b);
  }
};
template <bool INV> struct Dft<4, INV> {
  static __device__ __forceinline__ void run(float2 (&x)[4]) {
    float2 t0 = cadd(x[0], x[2]), t1 = csub(x[0], x[2]);
    float2 t2 = cadd(x[1], x[3]), t3 = csub(x[1], x[3]);
    x[0] = cadd(t0, t2);
    x[2] = csub(t0, t2);
    // forward: X1 = t1 - j t3, X3 = t1 + j t3
    float2 jt3 = make_float2(-t3.y, t3.x);
    if (!INV) { x[1] = csub(t1, jt3); x[3] = cadd(t1, jt3); }
    else      { x[1] = cadd(t1, jt3); x[3] = csub(t1, jt3); }
  }
};
// Cooley-Tukey step R = R1 * R2 on registers:
//   X[k1 + R1 k2] = sum_{n2} W_R^{n2 k1} [ sum_{n1} x[n1 R2 + n2] W_R1^{n1 k1} ] W_R2^{n2 k2}
template <int R1, int R2, bool INV>
__device__ __forceinline__ void dft_ct(float2 (&x)[R1 * R2]) {
  constexpr int R = R1 * R2;
  float2 a[R1][R2];
#pragma unroll
  for (int n2 = 0; n2 < R2; ++n2) {
    float2 t[R1];
#pragma unroll
    for (int n1 = 0; n1 < R1; ++n1) t[n1] = x[n1 * R2 + n2];
    Dft<R1, INV>::run(t);
#pragma unroll
    for (int k1 = 0; k1 < R1; ++k1) a[k1][n2] = mul_root<INV>(t[k1], n2 * k1, R);
  }
#pragma unroll
  for (int k1 = 0; k1 < R1; ++k1) {
    float2 u[R2];
#pragma unroll
    for (int n2 = 0; n2 < R2; ++n2) u[n2] = a[k1][n2];
    Dft<R2, INV>::run(u);
#pragma unroll
    for (int k2 = 0; k2 < R2; ++k2) x[k1 + R1 * k2] = u[k2];
  }
}
template <bool INV> struct Dft<8, INV> {
  static __device__ __forceinline__ void run(float2 (&x)[8]) { dft_ct<2, 4, INV>(x); }
};
template <bool INV> struct Dft<16, INV> {
  static __device__ __forceinline__ void run(float2 (&x)[16]) { dft_ct<4, 4, INV>(x); }
};
template <bool INV> struct Dft<32, INV> {
  static __device__ __forceinline__ void run(float2 (&x)[32]) { dft_ct<4, 8, INV>(x); }
};
// Odd radices: the defining sum with constant roots.
template <int R, bool INV>
__device__ __forceinline__ void dft_naive(float2 (&x)[R]) {
  float2 y[R];
#pragma unroll
  for (int k = 0; k < R; ++k) {
    float2 acc = x[0];
#pragma unroll
    for (int t = 1; t < R; ++t) acc = cadd(acc, mul_root<INV>(x[t], (k * t) % R, R));
    y[k] = acc;
  }
#pragma unroll
  for (int k = 0; k < R; ++k) x[k] = y[k];
}
template <bool INV> struct Dft<3, INV> {
  static __device__ __forceinline__ void run(float2 (&x)[3]) { dft_naive<3, INV>(x); }
};
template <bool INV> struct Dft<5, INV> {
  static __device__ __forceinline__ void run(float2 (&x)[5]) { dft_naive<5, INV>(x); }
};
template <bool INV> struct Dft<7, INV> {
  static __device__ __forceinline__ void run(float2 (&x)[7]) { dft_naive<7, INV>(x); }
};

// GELU with the exact error function.
__device__ __forceinline__ float gelu_erf(float x) { return 0.5f * x * (1.0f + erff(x * 0.70710678118654752440f)); }

#endif  // __CUDACC__
}  // namespace spectre
