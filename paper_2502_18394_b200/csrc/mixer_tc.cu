// Tensor-core spectral mixer for n = 8192, bf16 I/O (Sec. 3.2 steps 2 and 4).
//
// The length-8192 complex transform of a column pair z = a + jb (see mixer.cu for
// the pair packing) is factored 8192 = 2 * 64 * 64.  The radix-2 step runs on the
// ALUs while the rows are loaded (even / odd output bins become two independent
// 4096-point problems "e" and "o").  Each 64-point DFT stage of a 4096-point
// problem is a dense contraction on the 5th-generation tensor cores:
//
//     D[128 x 256] (fp32, TMEM) = F[128 x 128] (fp16, smem) * B[128 x 256] (fp16, smem)
//
// F is the 64-point DFT matrix in real form ([[C, S], [-S, C]], scaled by 1/8), its
// rows ordered so that Re and Im of one output bin sit 8 TMEM lanes apart, which is
// where a 16x256b TMEM load puts them in one thread.  B holds the 64 contracted
// samples (re, im interleaved along K) for 64 x 4 = 256 independent columns (the
// other digit x 4 column pairs).  Between stages the epilogue warps read D, apply
// the twiddle W_4096^{k1 t2} (or the gate, or the final radix-2 combine), round to
// fp16 and write the next stage's B operand in the canonical K-major layout.  The
// inverse transform is conj(FFT(conj(.))) so one F serves both directions.
//
// One CTA = one (batch, head, 4 column pairs); the "e" and "o" halves ping-pong:
// while the epilogue of one half runs on the ALUs the MMAs of the other half run on
// the tensor core.  Hand-offs are mbarriers; every wait is bounded and reports
// through a status word instead of hanging.
#include <cuda_fp16.h>

#include "common.cuh"

namespace spectre {

constexpr int kTcLbo = 144;                    // bytes between core matrices along K (128 + 16 pad)
constexpr int kTcSbo = 2320;                   // bytes between 8-column groups (16 * 144 + 16 pad)
constexpr int kTcBBytes = 32 * kTcSbo;         // one 256-column B operand
constexpr int kTcFBytes = 128 * 128 * 2;
constexpr int kTcGStride = 72;                 // gate table: entry (row, col) at row + 72 col (conflict-free reads)
constexpr int kTcGBytes = 64 * kTcGStride * 4; // per half, fp16 (re, im)
constexpr int kTcSmem = kTcFBytes + 2 * kTcBBytes + 2 * kTcGBytes + 64;
constexpr int kTcEpiWarps = 16;                // 4 per TMEM lane quadrant, one column quarter each
constexpr int kTcEpiThreads = 32 * kTcEpiWarps;
constexpr int kTcThreads = kTcEpiThreads + 32; // + 1 MMA-issuing warp
constexpr uint32_t kSpinLimit = 1u << 24;

// Optional phase stamps (SM clock), compiled in only for profiling builds.
#ifdef SPECTRE_TC_TIMING
__device__ long long g_tc_timing[1024][16];
#define TC_STAMP(slot) do { if (T == 0 && warp == 0 && blockIdx.x < 1024) g_tc_timing[blockIdx.x][slot] = clock64(); } while (0)
#else
#define TC_STAMP(slot) do { } while (0)
#endif

struct TcParams {
  const bf16* src;
  bf16* dst;
  int64_t s_sb, s_sl, s_sh, d_sb, d_sl, d_sh;
  const float2* g;        // [B*H][4097]
  const __half* F;        // 64-point DFT matrix, canonical smem layout
  const float2* tw;       // quarter-wave twiddle table (8192nds)
  int H, D, L, ntile;
  int* status;            // host-mapped status word (0 = fine)
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = (uint64_t)((saddr >> 4) & 0x3fff);
  d |= (uint64_t)((lbo >> 4) & 0x3fff) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3fff) << 32;
  d |= (uint64_t)1 << 46;                       // descriptor version for sm_100
  return d;                                     // no swizzle, K-major
}

// kind::f16, fp16 A and B (both K-major), fp32 accumulator, M = 128, N = 256
__device__ __forceinline__ uint32_t umma_idesc_128x256() {
  return (1u << 4) | ((256u >> 3) << 17) | ((128u >> 4) << 24);
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (ok) return true;
  }
  return false;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("{\n.reg .b64 st;\nmbarrier.arrive.shared::cta.b64 st, [%0];\n}" :: "r"(bar) : "memory");
}

__device__ __forceinline__ uint32_t pack_h2(float lo, float hi) {
  __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

// 16 lanes x 32 columns of fp32: thread T gets, per 8-column group x, rows T/4 (r[4x], r[4x+1])
// and T/4 + 8 (r[4x+2], r[4x+3]) at columns 8x + 2(T%4) + {0, 1}.
__device__ __forceinline__ void tmem_ld_16x256b_x4(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x4.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Byte offset of element (column nu, K index kappa) in a B operand.
__device__ __forceinline__ uint32_t b_off(int nu, int kappa) {
  return (uint32_t)((nu >> 3) * kTcSbo + (kappa >> 3) * kTcLbo + (nu & 7) * 16 + (kappa & 7) * 2);
}

// Hermitian extension of the half-spectrum gate (n = 8192).
__device__ __forceinline__ float2 gate8192(const float2* __restrict__ g, int k) {
  int kk = k <= 4096 ? k : 8192 - k;
  float2 v = __ldg(g + kk);
  if (kk != k) v.y = -v.y;
  if (k == 0 || k == 4096) v.y = 0.f;
  return v;
}

// Epilogue between two MMA stages of one half, for one warp: TMEM lane quadrant q, column
// quarter cq (64 of the 256 columns).  A thread owns rows (digit) 16 q' + T/4 for the two lane
// groups q' = 2q, 2q+1 and, per 8-column group, the column digit 2*group + p with the column
// pair c = 2cp, 2cp+1.  TMEM loads run one 32-column chunk ahead of the arithmetic.
//   MODE 1: twiddle W_4096^{row * col}, write transposed (row digit -> column index of B, col digit -> K)
//   MODE 2: gate (and conjugate for the inverse), write straight (col digit -> column index, row digit -> K)
template <int MODE>
__device__ __forceinline__ void epilogue_mid(uint32_t tmem_d, unsigned char* Bsm, int q, int cq, int T,
                                             const uint32_t* __restrict__ Gtab, const float2* __restrict__ tw) {
  const int i = T >> 2, p = (T >> 1) & 1, cp = T & 1;
  uint32_t r[2][16];
  const uint32_t taddr0 = tmem_d + ((uint32_t)(32 * q) << 16) + 64 * cq;
  tmem_ld_16x256b_x4(taddr0, r[0]);
  float2 w = make_float2(1.f, 0.f), wstep = w;
#pragma unroll
  for (int step = 0; step < 4; ++step) {                      // step = 2 j + chunk
    const int j = step >> 1, chunk = step & 1;
    const int row = 8 * (2 * q + j) + i;
    if (MODE == 1 && chunk == 0) {
      w = twiddle8192(tw, 2u * (unsigned)((row * (16 * cq + p)) & 4095));
      wstep = twiddle8192(tw, 4u * (unsigned)row);
    }
    tmem_ld_wait();
    if (step < 3) {
      const int nj = (step + 1) >> 1, nchunk = (step + 1) & 1;
      tmem_ld_16x256b_x4(taddr0 + ((uint32_t)(16 * nj) << 16) + 32 * nchunk, r[(step + 1) & 1]);
    }
    const uint32_t (&rr)[16] = r[step & 1];
    // byte offset of this thread's first element of the chunk in the next operand
    uint32_t base;
    if (MODE == 1) base = (uint32_t)((row >> 1) * kTcSbo + (4 * (row & 1) + 2 * cp) * 16 + (4 * cq + 2 * chunk) * kTcLbo + 4 * p);
    else base = (uint32_t)((8 * cq + 4 * chunk) * kTcSbo + (4 * p + 2 * cp) * 16 + (row >> 2) * kTcLbo + (row & 3) * 4);
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      float2 v0 = make_float2(__uint_as_float(rr[4 * x]), __uint_as_float(rr[4 * x + 2]));
      float2 v1 = make_float2(__uint_as_float(rr[4 * x + 1]), __uint_as_float(rr[4 * x + 3]));
      uint32_t off;
      if (MODE == 1) {
        v0 = cmul(v0, w);
        v1 = cmul(v1, w);
        w = cmul(w, wstep);
        off = base + (x >> 1) * kTcLbo + (x & 1) * 8;
      } else {
        const int col = 2 * (8 * cq + 4 * chunk + x) + p;
        const uint32_t gu = Gtab[row + kTcGStride * col];
        const float2 g = __half22float2(*reinterpret_cast<const __half2*>(&gu));
        v0 = cmul(v0, g);
        v1 = cmul(v1, g);
        v0.y = -v0.y;
        v1.y = -v1.y;
        off = base + x * kTcSbo;
      }
      *reinterpret_cast<uint32_t*>(Bsm + off) = pack_h2(v0.x, v0.y);
      *reinterpret_cast<uint32_t*>(Bsm + off + 16) = pack_h2(v1.x, v1.y);
    }
  }
}

__device__ __forceinline__ uint2 pack_bf16x4(float a, float b, float c, float d) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  uint2 r;
  r.x = *reinterpret_cast<unsigned*>(&lo);
  r.y = *reinterpret_cast<unsigned*>(&hi);
  return r;
}

__global__ void __launch_bounds__(kTcThreads, 1) mixer_tc8192_kernel(const TcParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* Fsm = smem;
  unsigned char* Bsm[2] = {smem + kTcFBytes, smem + kTcFBytes + kTcBBytes};
  uint32_t* Gsm[2] = {reinterpret_cast<uint32_t*>(smem + kTcFBytes + 2 * kTcBBytes),
                      reinterpret_cast<uint32_t*>(smem + kTcFBytes + 2 * kTcBBytes + kTcGBytes)};
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kTcFBytes + 2 * kTcBBytes + 2 * kTcGBytes);   // [0,1] B ready, [2,3] D ready
  __shared__ uint32_t tmem_slot;
  __shared__ float red[kTcEpiWarps];

  const int tid = threadIdx.x, warp = tid >> 5, T = tid & 31;
  const int tile = blockIdx.x % p.ntile, slab = blockIdx.x / p.ntile;
  const int b = slab / p.H, h = slab - b * p.H;
  const int col0 = tile * 8;
  const float2* g = p.g + (size_t)slab * 4097;

  TC_STAMP(0);
  if (warp == kTcEpiWarps) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&bars[0])), "r"(kTcEpiThreads));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&bars[1])), "r"(kTcEpiThreads));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&bars[2])), "r"(1));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&bars[3])), "r"(1));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // DFT matrix -> smem
  if (tid < kTcEpiThreads) {
    const uint4* Fg = reinterpret_cast<const uint4*>(p.F);
    for (int i = tid; i < kTcFBytes / 16; i += kTcEpiThreads) reinterpret_cast<uint4*>(Fsm)[i] = __ldg(Fg + i);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = tmem_slot;
  TC_STAMP(1);

  if (warp == kTcEpiWarps) {
    // ---- MMA issuer: 4 stages x 2 halves, 8 K-steps each ----
    const uint32_t idesc = umma_idesc_128x256();
    bool ok = true;
    for (int stage = 0; stage < 4 && ok; ++stage) {
      for (int half = 0; half < 2 && ok; ++half) {
        ok = mbar_wait(smem_u32(&bars[half]), stage & 1);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (T == 0) {
          const uint32_t a0 = smem_u32(Fsm), b0 = smem_u32(Bsm[half]);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            uint64_t da = umma_desc(a0 + ks * 256, 128, 2048);
            uint64_t db = umma_desc(b0 + ks * 2 * kTcLbo, kTcLbo, kTcSbo);
            uint32_t acc = ks > 0;
            asm volatile(
                "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                :: "r"(tmem + 256 * half), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
          }
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                       :: "r"(smem_u32(&bars[2 + half])) : "memory");
        }
        __syncwarp();
      }
    }
    if (!ok && T == 0) atomicExch(p.status, 1);
  } else {
    // ---- load: rows t and t + 4096, radix-2 step, fp16, stage-1 operand (K = t1, column = (t2, c)) ----
    {
      const bf16* src = p.src + b * p.s_sb + h * p.s_sh + col0;
      const int t1 = tid & 63, t2base = tid >> 6;          // 32 lanes = 32 consecutive t1: conflict-free stores
      constexpr int kIter = 64 / (kTcEpiThreads / 64);
      float2 w = twiddle8192(p.tw, (unsigned)(64 * t1 + t2base));
      const float2 wstep = twiddle8192(p.tw, (unsigned)(kTcEpiThreads / 64));
#pragma unroll 4
      for (int it = 0; it < kIter; ++it) {
        const int t2 = t2base + (kTcEpiThreads / 64) * it, t = 64 * t1 + t2;
        uint4 ra = make_uint4(0u, 0u, 0u, 0u), rb = ra;
        if (t < p.L) ra = __ldcg(reinterpret_cast<const uint4*>(src + (int64_t)t * p.s_sl));
        if (t + 4096 < p.L) rb = __ldcg(reinterpret_cast<const uint4*>(src + (int64_t)(t + 4096) * p.s_sl));
        const uint32_t ua[4] = {ra.x, ra.y, ra.z, ra.w}, ub[4] = {rb.x, rb.y, rb.z, rb.w};
        const uint32_t off = b_off(4 * t2, 2 * t1);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          float2 a = make_float2(__uint_as_float(ua[c] << 16), __uint_as_float(ua[c] & 0xffff0000u));
          float2 bb = make_float2(__uint_as_float(ub[c] << 16), __uint_as_float(ub[c] & 0xffff0000u));
          float2 e = cadd(a, bb), o = cmul(csub(a, bb), w);
          *reinterpret_cast<uint32_t*>(Bsm[0] + off + 16 * c) = pack_h2(e.x, e.y);
          *reinterpret_cast<uint32_t*>(Bsm[1] + off + 16 * c) = pack_h2(o.x, o.y);
        }
        w = cmul(w, wstep);
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    TC_STAMP(2);
    mbar_arrive(smem_u32(&bars[0]));
    mbar_arrive(smem_u32(&bars[1]));

    // ---- gate tables (while the first MMAs run): Hermitian extension, normalised by a bound on
    //      max |g| so that the gated spectrum stays in fp16 range; entry for bin 2 (col + 64 row) + parity
    float gmax = 0.f;
    constexpr int kGIter = 8192 / kTcEpiThreads;                 // table entries per thread
    float2 gv[kGIter];
#pragma unroll
    for (int i = 0; i < kGIter; ++i) gv[i] = gate8192(g, tid + i * kTcEpiThreads);   // all loads in flight
#pragma unroll
    for (int i = 0; i < kGIter; ++i) gmax = fmaxf(gmax, fmaxf(fabsf(gv[i].x), fabsf(gv[i].y)));
    for (int o = 16; o > 0; o >>= 1) gmax = fmaxf(gmax, __shfl_xor_sync(0xffffffffu, gmax, o));
    if (T == 0) red[warp] = gmax;
    asm volatile("bar.sync 1, %0;" :: "r"(kTcEpiThreads) : "memory");
    gmax = 0.f;
    for (int i = 0; i < kTcEpiWarps; ++i) gmax = fmaxf(gmax, red[i]);
    gmax *= 1.41421356f;
    const float ginv = gmax > 0.f ? 1.0f / gmax : 0.f;
#pragma unroll
    for (int i = 0; i < kGIter; ++i) {
      const int k = tid + i * kTcEpiThreads, m = k >> 1;
      Gsm[k & 1][(m >> 6) + kTcGStride * (m & 63)] = pack_h2(gv[i].x * ginv, gv[i].y * ginv);
    }
    asm volatile("bar.sync 1, %0;" :: "r"(kTcEpiThreads) : "memory");

    const int q = warp & 3, cq = warp >> 2;
    bool ok = true;
    // ---- stages 1..3: wait for D, transform, hand the next operand to the issuer ----
#pragma unroll 1
    for (int stage = 0; stage < 3 && ok; ++stage) {
#pragma unroll 1
      for (int half = 0; half < 2 && ok; ++half) {
        ok = mbar_wait(smem_u32(&bars[2 + half]), stage & 1);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t td = tmem + 256 * half;
        if (stage == 1) epilogue_mid<2>(td, Bsm[half], q, cq, T, Gsm[half], p.tw);
        else epilogue_mid<1>(td, Bsm[half], q, cq, T, Gsm[half], p.tw);
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        TC_STAMP(3 + 2 * stage + half);
        mbar_arrive(smem_u32(&bars[half]));
      }
    }
    // ---- final: y[t], y[t+4096] = (gmax/2) conj(D_e +- W_8192^t D_o), bf16 ----
    if (ok) ok = mbar_wait(smem_u32(&bars[2]), 1);
    if (ok) ok = mbar_wait(smem_u32(&bars[3]), 1);
    TC_STAMP(9);
    if (ok) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int i = T >> 2, pp = (T >> 1) & 1, cp = T & 1;
      const float gs = 0.5f * gmax;
      bf16* dst = p.dst + b * p.d_sb + h * p.d_sh + col0 + 4 * cp;
      const float2 wstep = twiddle8192(p.tw, 2u);
      const uint32_t taddr0 = tmem + ((uint32_t)(32 * q) << 16) + 64 * cq;
      uint32_t re[2][16], ro[2][16];
      tmem_ld_16x256b_x4(taddr0, re[0]);
      tmem_ld_16x256b_x4(taddr0 + 256, ro[0]);
      float2 w = make_float2(1.f, 0.f);
#pragma unroll
      for (int step = 0; step < 4; ++step) {
        const int j = step >> 1, chunk = step & 1;
        const int t1 = 8 * (2 * q + j) + i;
        if (chunk == 0) w = twiddle8192(p.tw, (unsigned)(64 * t1 + 16 * cq + pp));
        tmem_ld_wait();
        if (step < 3) {
          const uint32_t ta = taddr0 + ((uint32_t)(16 * ((step + 1) >> 1)) << 16) + 32 * ((step + 1) & 1);
          tmem_ld_16x256b_x4(ta, re[(step + 1) & 1]);
          tmem_ld_16x256b_x4(ta + 256, ro[(step + 1) & 1]);
        }
        const uint32_t (&xe)[16] = re[step & 1];
        const uint32_t (&xo)[16] = ro[step & 1];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const int t2 = 2 * (8 * cq + 4 * chunk + x) + pp, t = 64 * t1 + t2;
          float2 e0 = make_float2(__uint_as_float(xe[4 * x]), __uint_as_float(xe[4 * x + 2]));
          float2 e1 = make_float2(__uint_as_float(xe[4 * x + 1]), __uint_as_float(xe[4 * x + 3]));
          float2 o0 = cmul(make_float2(__uint_as_float(xo[4 * x]), __uint_as_float(xo[4 * x + 2])), w);
          float2 o1 = cmul(make_float2(__uint_as_float(xo[4 * x + 1]), __uint_as_float(xo[4 * x + 3])), w);
          w = cmul(w, wstep);
          if (t < p.L)
            *reinterpret_cast<uint2*>(dst + (int64_t)t * p.d_sl) =
                pack_bf16x4(gs * (e0.x + o0.x), -gs * (e0.y + o0.y), gs * (e1.x + o1.x), -gs * (e1.y + o1.y));
          if (t + 4096 < p.L)
            *reinterpret_cast<uint2*>(dst + (int64_t)(t + 4096) * p.d_sl) =
                pack_bf16x4(gs * (e0.x - o0.x), -gs * (e0.y - o0.y), gs * (e1.x - o1.x), -gs * (e1.y - o1.y));
        }
      }
    }
    TC_STAMP(10);
    if (!ok && T == 0) atomicExch(p.status, 1);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  TC_STAMP(11);
  if (warp == kTcEpiWarps) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(512));
  }
}

// 64-point DFT matrix in real form, scaled by 1/8, in the K-major core-matrix layout
// (8 rows x 16 bytes per core matrix, 128 bytes between K neighbours, 2048 between row groups).
// Row m = 16 g + 8 part + i is output bin 8 g + i, part 0 = Re, 1 = Im.
__global__ void build_dft64_kernel(__half* F) {
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= 128 * 128) return;
  int m = idx >> 7, kappa = idx & 127;
  int kd = 8 * (m >> 4) + (m & 7), part_out = (m >> 3) & 1;
  int t = kappa >> 1, part_in = kappa & 1;
  float s, c;
  sincospif(2.0f * (float)((kd * t) & 63) / 64.0f, &s, &c);
  // (a + jb)(c - js): Re = a c + b s, Im = -a s + b c
  float v = part_out == 0 ? (part_in == 0 ? c : s) : (part_in == 0 ? -s : c);
  size_t off = (size_t)(m >> 3) * 2048 + (size_t)(kappa >> 3) * 128 + (m & 7) * 16 + (kappa & 7) * 2;
  *reinterpret_cast<__half*>(reinterpret_cast<unsigned char*>(F) + off) = __float2half_rn(0.125f * v);
}

// (cos, sin)(2 pi r / 8192) for r = 0..2048
__global__ void build_tw8192_kernel(float2* tab) {
  int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r > 2048) return;
  float s, c;
  sincospif((float)r / 4096.0f, &s, &c);
  tab[r] = make_float2(c, s);
}

int build_tw8192(float2* tab, cudaStream_t st) {
  build_tw8192_kernel<<<9, 256, 0, st>>>(tab);
  SPECTRE_LAUNCH_OK("build_tw8192_kernel");
  return SPECTRE_OK;
}

int build_dft64(__half* F, cudaStream_t st) {
  build_dft64_kernel<<<64, 256, 0, st>>>(F);
  SPECTRE_LAUNCH_OK("build_dft64_kernel");
  return SPECTRE_OK;
}

int launch_mixer_tc8192(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, const float* g,
                        const spectre_act* y) {
  TcParams p = {};
  p.src = reinterpret_cast<const bf16*>(v->ptr);
  p.dst = reinterpret_cast<bf16*>(y->ptr);
  p.s_sb = v->stride_b; p.s_sl = v->stride_l; p.s_sh = v->stride_h;
  p.d_sb = y->stride_b; p.d_sl = y->stride_l; p.d_sh = y->stride_h;
  p.g = reinterpret_cast<const float2*>(g);
  p.F = reinterpret_cast<const __half*>(ctx->dft64);
  p.tw = reinterpret_cast<const float2*>(ctx->tw8192);
  p.H = v->H; p.D = v->D; p.L = v->L; p.ntile = v->D / 8;
  p.status = ctx->status_dev;
  SPECTRE_CUDA_OK(cudaFuncSetAttribute(mixer_tc8192_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmem));
  const unsigned grid = (unsigned)((size_t)v->B * v->H * p.ntile);
  mixer_tc8192_kernel<<<grid, kTcThreads, kTcSmem, st>>>(p);
  SPECTRE_LAUNCH_OK("mixer_tc8192_kernel");
  return SPECTRE_OK;
}


// =====================================================================================
// n = 196 (14 x 14 patch grids), bf16 I/O, D = 64: 196 = 4 * 49.
//
// t = 49 n1 + t', k = k1 + 4 kM.  The radix-4 DFT over n1 and the twiddle W_196^{k1 t'} run on
// the ALUs while whole 128-byte head rows are loaded; each 49-point DFT over t' is ONE tensor-core
// stage with the 49-point DFT matrix in real form (98 x 98, zero-padded to 128 x 112) as the A
// operand; the gate is applied to the accumulator, one more stage does the inverse 49-point DFT
// (conj trick), and the final epilogue does the inverse radix-4 and stores bf16 rows.
// A CTA takes 4 heads: columns (head, k1, pair) = 4 x 4 x 32 = 512 = the whole TMEM; the two
// 2-head halves ping-pong between tensor core and ALUs like the halves of the 8192 kernel.
// =====================================================================================
constexpr int k196Heads = 4;
constexpr int k196KSteps = 7;                 // K = 112 >= 98
constexpr int k196Smem = kTcFBytes + 2 * kTcBBytes + k196Heads * 256 * 4 + 64;

struct Tc196Params {
  const bf16* src;
  bf16* dst;
  int64_t s_sb, s_sl, s_sh, d_sb, d_sl, d_sh;
  const float2* g;        // [B*H][99]
  const __half* F;        // 49-point DFT matrix (real form, padded), canonical smem layout
  int H, L, nheads;       // nheads = B * H
  int* status;
};

__device__ __forceinline__ void tmem_ld_16x256b_x1(uint32_t taddr, uint32_t (&r)[4]) {
  asm volatile("tcgen05.ld.sync.aligned.16x256b.x1.b32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr));
}

__global__ void __launch_bounds__(kTcThreads, 1) mixer_tc196_kernel(const Tc196Params p) {
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* Fsm = smem;
  unsigned char* Bsm[2] = {smem + kTcFBytes, smem + kTcFBytes + kTcBBytes};
  uint32_t* Gsm = reinterpret_cast<uint32_t*>(smem + kTcFBytes + 2 * kTcBBytes);        // [4 heads][k1 * 64 + kM]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kTcFBytes + 2 * kTcBBytes + k196Heads * 256 * 4);
  __shared__ uint32_t tmem_slot;
  __shared__ float red[kTcEpiWarps];
  __shared__ float gmax_s[k196Heads];

  const int tid = threadIdx.x, warp = tid >> 5, T = tid & 31;
  const int head0 = blockIdx.x * k196Heads;
  TC_STAMP(0);

  if (warp == kTcEpiWarps) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&bars[0])), "r"(kTcEpiThreads));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&bars[1])), "r"(kTcEpiThreads));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&bars[2])), "r"(1));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&bars[3])), "r"(1));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < kTcEpiThreads) {
    const uint4* Fg = reinterpret_cast<const uint4*>(p.F);
    for (int i = tid; i < kTcFBytes / 16; i += kTcEpiThreads) reinterpret_cast<uint4*>(Fsm)[i] = __ldg(Fg + i);
    // zero the operands once: K rows 98..127 and the columns of absent heads must read as zero
    for (int i = tid; i < 2 * kTcBBytes / 16; i += kTcEpiThreads) reinterpret_cast<uint4*>(Bsm[0])[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = tmem_slot;
  TC_STAMP(1);

  if (warp == kTcEpiWarps) {
    // ---- MMA issuer: 2 stages x 2 halves, 7 K-steps each ----
    const uint32_t idesc = umma_idesc_128x256();
    bool ok = true;
    for (int stage = 0; stage < 2 && ok; ++stage) {
      for (int half = 0; half < 2 && ok; ++half) {
        ok = mbar_wait(smem_u32(&bars[half]), stage & 1);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (T == 0) {
          const uint32_t a0 = smem_u32(Fsm), b0 = smem_u32(Bsm[half]);
#pragma unroll
          for (int ks = 0; ks < k196KSteps; ++ks) {
            uint64_t da = umma_desc(a0 + ks * 256, 128, 2048);
            uint64_t db = umma_desc(b0 + ks * 2 * kTcLbo, kTcLbo, kTcSbo);
            uint32_t acc = ks > 0;
            asm volatile(
                "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                :: "r"(tmem + 256 * half), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
          }
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                       :: "r"(smem_u32(&bars[2 + half])) : "memory");
        }
        __syncwarp();
      }
    }
    if (!ok && T == 0) atomicExch(p.status, 1);
  } else {
    // ---- load: rows t' + 49 n1 of each head, radix-4 over n1, twiddle, fp16, operand (K = t', column = (head, k1, pair)) ----
    // a warp takes 4 consecutive t' x 8 chunks of 16 bytes (conflict-free operand stores); all of
    // a warp's rows (up to 4 items x 4 rows) are requested before the first one is used
    constexpr int kItems = (k196Heads * 13 + kTcEpiWarps - 1) / kTcEpiWarps;
    uint4 rr[kItems][4];
#pragma unroll
    for (int it = 0; it < kItems; ++it) {
      const int item = warp + it * kTcEpiWarps;
      const int hl = item / 13, tg = item - hl * 13;
      const int tp = 4 * tg + (T >> 3), hg = head0 + hl;
      const bool live = item < k196Heads * 13 && tp < 49 && hg < p.nheads;
      const int b = live ? hg / p.H : 0, h = live ? hg - b * p.H : 0;
      const bf16* src = p.src + b * p.s_sb + h * p.s_sh + 8 * (T & 7);
#pragma unroll
      for (int n1 = 0; n1 < 4; ++n1) {
        const int row = tp + 49 * n1;
        rr[it][n1] = (live && row < p.L) ? __ldcg(reinterpret_cast<const uint4*>(src + (int64_t)row * p.s_sl))
                                         : make_uint4(0u, 0u, 0u, 0u);
      }
    }
#pragma unroll
    for (int it = 0; it < kItems; ++it) {
      const int item = warp + it * kTcEpiWarps;
      const int hl = item / 13, tg = item - hl * 13;
      const int tp = 4 * tg + (T >> 3), chunk = T & 7, hg = head0 + hl;
      if (item >= k196Heads * 13 || tp >= 49 || hg >= p.nheads) continue;
      const float2 w1 = twiddle_fwd((unsigned)tp, 196u);
      const float2 w2 = cmul(w1, w1), w3 = cmul(w2, w1);
      unsigned char* Bh = Bsm[hl >> 1] + b_off((hl & 1) * 128 + 4 * chunk, 2 * tp);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float2 x[4];
#pragma unroll
        for (int n1 = 0; n1 < 4; ++n1) {
          const uint32_t u = j == 0 ? rr[it][n1].x : (j == 1 ? rr[it][n1].y : (j == 2 ? rr[it][n1].z : rr[it][n1].w));
          x[n1] = make_float2(0.5f * __uint_as_float(u << 16), 0.5f * __uint_as_float(u & 0xffff0000u));
        }
        Dft<4, false>::run(x);
        x[1] = cmul(x[1], w1);
        x[2] = cmul(x[2], w2);
        x[3] = cmul(x[3], w3);
        // column (head, k1, pair): k1 moves 32 columns = 4 groups of 8, j moves one row of 16 bytes
#pragma unroll
        for (int k1 = 0; k1 < 4; ++k1)
          *reinterpret_cast<uint32_t*>(Bh + 4 * k1 * kTcSbo + 16 * j) = pack_h2(x[k1].x, x[k1].y);
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    TC_STAMP(2);
    mbar_arrive(smem_u32(&bars[0]));
    mbar_arrive(smem_u32(&bars[1]));

    // ---- gate tables: head hl, entry k1 * 64 + kM holds G_ext[k1 + 4 kM] / gmax(head) as fp16 ----
    float2 gv[2];
    float gm[2];
#pragma unroll
    for (int it = 0; it < 2; ++it) {
      const int e = tid + it * kTcEpiThreads, hl = e >> 8, idx = e & 255, k1 = idx >> 6, kM = idx & 63;
      const int hg = head0 + hl;
      float2 v = make_float2(0.f, 0.f);
      if (kM < 49 && hg < p.nheads) {
        const int k = k1 + 4 * kM, kk = k <= 98 ? k : 196 - k;
        v = __ldg(p.g + (size_t)hg * 99 + kk);
        if (kk != k) v.y = -v.y;
        if (k == 0 || k == 98) v.y = 0.f;
      }
      gv[it] = v;
      float m = fmaxf(fabsf(v.x), fabsf(v.y));
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      gm[it] = m;
    }
    // warps 0-7 hold head 0 (it = 0) and head 2 (it = 1); warps 8-15 heads 1 and 3
    if (T == 0) red[warp] = gm[0];
    asm volatile("bar.sync 1, %0;" :: "r"(kTcEpiThreads) : "memory");
    if (tid < 2) { float m = 0.f; for (int i = 0; i < 8; ++i) m = fmaxf(m, red[8 * tid + i]); gmax_s[tid] = 1.41421356f * m; }
    asm volatile("bar.sync 1, %0;" :: "r"(kTcEpiThreads) : "memory");
    if (T == 0) red[warp] = gm[1];
    asm volatile("bar.sync 1, %0;" :: "r"(kTcEpiThreads) : "memory");
    if (tid < 2) { float m = 0.f; for (int i = 0; i < 8; ++i) m = fmaxf(m, red[8 * tid + i]); gmax_s[2 + tid] = 1.41421356f * m; }
    asm volatile("bar.sync 1, %0;" :: "r"(kTcEpiThreads) : "memory");
#pragma unroll
    for (int it = 0; it < 2; ++it) {
      const int e = tid + it * kTcEpiThreads, hl = e >> 8;
      const float gmx = gmax_s[hl], inv = gmx > 0.f ? 1.0f / gmx : 0.f;
      Gsm[e] = pack_h2(gv[it].x * inv, gv[it].y * inv);
    }
    asm volatile("bar.sync 1, %0;" :: "r"(kTcEpiThreads) : "memory");

    const int q = warp & 3, cq = warp >> 2;
    const int i = T >> 2, t4 = T & 3;
    bool ok = true;
    TC_STAMP(3);
    // ---- gate epilogue: rows kM, columns (head, k1, pair) unchanged; next operand has K = kM ----
#pragma unroll 1
    for (int half = 0; half < 2 && ok; ++half) {
      ok = mbar_wait(smem_u32(&bars[2 + half]), 0);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t taddr0 = tmem + 256 * half + ((uint32_t)(32 * q) << 16) + 64 * cq;
      const int hl = 2 * half + (cq >> 1);
      uint32_t r[2][16];
      tmem_ld_16x256b_x4(taddr0, r[0]);
#pragma unroll
      for (int step = 0; step < 4; ++step) {
        const int j = step >> 1, chunk = step & 1;
        const int kM = 8 * (2 * q + j) + i, k1 = 2 * (cq & 1) + chunk;
        tmem_ld_wait();
        if (step < 3) tmem_ld_16x256b_x4(taddr0 + ((uint32_t)(16 * ((step + 1) >> 1)) << 16) + 32 * ((step + 1) & 1), r[(step + 1) & 1]);
        const uint32_t (&rr)[16] = r[step & 1];
        const uint32_t gu = Gsm[hl * 256 + k1 * 64 + kM];
        const float2 g = __half22float2(*reinterpret_cast<const __half2*>(&gu));
        const uint32_t base = (uint32_t)((8 * cq + 4 * chunk) * kTcSbo + (2 * t4) * 16 + (kM >> 2) * kTcLbo + (kM & 3) * 4);
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          float2 v0 = cmul(make_float2(__uint_as_float(rr[4 * x]), __uint_as_float(rr[4 * x + 2])), g);
          float2 v1 = cmul(make_float2(__uint_as_float(rr[4 * x + 1]), __uint_as_float(rr[4 * x + 3])), g);
          *reinterpret_cast<uint32_t*>(Bsm[half] + base + x * kTcSbo) = pack_h2(v0.x, -v0.y);
          *reinterpret_cast<uint32_t*>(Bsm[half] + base + x * kTcSbo + 16) = pack_h2(v1.x, -v1.y);
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      TC_STAMP(4 + half);
      mbar_arrive(smem_u32(&bars[half]));
    }
    // ---- final: rows t', inverse radix-4 over k1 (columns 32 apart), bf16 rows t' + 49 n1 ----
#pragma unroll 1
    for (int half = 0; half < 2 && ok; ++half) {
      ok = mbar_wait(smem_u32(&bars[2 + half]), 1);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int hl = 2 * half + (cq >> 1), hg = head0 + hl;
      if (hg >= p.nheads) continue;
      const int b = hg / p.H, h = hg - b * p.H;
      const float gs = 0.5f * gmax_s[hl];
      bf16* dst = p.dst + b * p.d_sb + h * p.d_sh;
      const uint32_t tbase = tmem + 256 * half + ((uint32_t)(32 * q) << 16) + 128 * (cq >> 1) + 16 * (cq & 1);
      const int nstep = (16 * q >= 49) ? 0 : ((16 * q + 8 >= 49) ? 2 : 4);    // lane groups with valid rows (warp-uniform)
      uint32_t rk[2][4][4];
      if (nstep > 0) {
#pragma unroll
        for (int k1 = 0; k1 < 4; ++k1) tmem_ld_16x256b_x1(tbase + 32 * k1, rk[0][k1]);
      }
#pragma unroll
      for (int step = 0; step < 4; ++step) {                       // step = 2 j + g8; accumulator reads run one step ahead
        if (step < nstep) {
          const int j = step >> 1, g8 = step & 1;
          const int tp = 8 * (2 * q + j) + i;
          tmem_ld_wait();
          if (step + 1 < nstep) {
            const int nj = (step + 1) >> 1, ng = (step + 1) & 1;
#pragma unroll
            for (int k1 = 0; k1 < 4; ++k1)
              tmem_ld_16x256b_x1(tbase + ((uint32_t)(16 * nj) << 16) + 32 * k1 + 8 * ng, rk[(step + 1) & 1][k1]);
          }
          if (tp < 49) {
            const float2 w1 = twiddle_fwd((unsigned)tp, 196u);
            const float2 w2 = cmul(w1, w1), w3 = cmul(w2, w1);
            float2 y0[4], y1[4];
#pragma unroll
            for (int k1 = 0; k1 < 4; ++k1) {                         // conj of the accumulator = IDFT49 (conj trick)
              y0[k1] = make_float2(__uint_as_float(rk[step & 1][k1][0]), -__uint_as_float(rk[step & 1][k1][2]));
              y1[k1] = make_float2(__uint_as_float(rk[step & 1][k1][1]), -__uint_as_float(rk[step & 1][k1][3]));
            }
            y0[1] = cmulc(y0[1], w1); y0[2] = cmulc(y0[2], w2); y0[3] = cmulc(y0[3], w3);
            y1[1] = cmulc(y1[1], w1); y1[2] = cmulc(y1[2], w2); y1[3] = cmulc(y1[3], w3);
            Dft<4, true>::run(y0);
            Dft<4, true>::run(y1);
            const int col = 2 * (16 * (cq & 1) + 8 * g8 + 2 * t4);
#pragma unroll
            for (int n1 = 0; n1 < 4; ++n1) {
              const int row = tp + 49 * n1;
              if (row < p.L)
                __stcs(reinterpret_cast<uint2*>(dst + (int64_t)row * p.d_sl + col),
                       pack_bf16x4(gs * y0[n1].x, gs * y0[n1].y, gs * y1[n1].x, gs * y1[n1].y));
            }
          }
        }
      }
    }
    TC_STAMP(6);
    if (!ok && T == 0) atomicExch(p.status, 1);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == kTcEpiWarps) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(512));
  }
}

// 49-point DFT matrix in real form, scaled by 1/7, zero-padded to 128 x 128, same layout and row
// order as the 64-point matrix (row 16 g + 8 part + i is bin 8 g + i).
__global__ void build_dft49_kernel(__half* F) {
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= 128 * 128) return;
  int m = idx >> 7, kappa = idx & 127;
  int kd = 8 * (m >> 4) + (m & 7), part_out = (m >> 3) & 1;
  int t = kappa >> 1, part_in = kappa & 1;
  float v = 0.f;
  if (kd < 49 && t < 49) {
    float s, c;
    sincospif(2.0f * (float)((kd * t) % 49) / 49.0f, &s, &c);
    v = part_out == 0 ? (part_in == 0 ? c : s) : (part_in == 0 ? -s : c);
    v *= 0.14285714285714285f;
  }
  size_t off = (size_t)(m >> 3) * 2048 + (size_t)(kappa >> 3) * 128 + (m & 7) * 16 + (kappa & 7) * 2;
  *reinterpret_cast<__half*>(reinterpret_cast<unsigned char*>(F) + off) = __float2half_rn(v);
}

int build_dft49(__half* F, cudaStream_t st) {
  build_dft49_kernel<<<64, 256, 0, st>>>(F);
  SPECTRE_LAUNCH_OK("build_dft49_kernel");
  return SPECTRE_OK;
}

int launch_mixer_tc196(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, const float* g,
                       const spectre_act* y) {
  Tc196Params p = {};
  p.src = reinterpret_cast<const bf16*>(v->ptr);
  p.dst = reinterpret_cast<bf16*>(y->ptr);
  p.s_sb = v->stride_b; p.s_sl = v->stride_l; p.s_sh = v->stride_h;
  p.d_sb = y->stride_b; p.d_sl = y->stride_l; p.d_sh = y->stride_h;
  p.g = reinterpret_cast<const float2*>(g);
  p.F = reinterpret_cast<const __half*>(ctx->dft49);
  p.H = v->H; p.L = v->L; p.nheads = v->B * v->H;
  p.status = ctx->status_dev;
  SPECTRE_CUDA_OK(cudaFuncSetAttribute(mixer_tc196_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, k196Smem));
  const unsigned grid = (unsigned)((p.nheads + k196Heads - 1) / k196Heads);
  mixer_tc196_kernel<<<grid, kTcThreads, k196Smem, st>>>(p);
  SPECTRE_LAUNCH_OK("mixer_tc196_kernel");
  return SPECTRE_OK;
}

}  // namespace spectre
