// Tensor-core spectral mixer for n = 8192, bf16 or fp16 I/O (Sec. 3.2 steps 2 and 4), one kernel.
//
// The length-8192 complex transform of a column pair z = a + jb (see mixer.cu for the pair
// packing) is factored 8192 = 2 * 64 * 64.  The radix-2 step runs on the ALUs (even / odd output
// bins become two independent 4096-point problems "e" and "o").  Each 64-point DFT stage of a
// 4096-point problem is a dense contraction on the 5th-generation tensor cores:
//
//     D[128 x 256] (fp32, TMEM) = F[128 x 128] (fp16, smem) * B[128 x 256] (fp16, smem)
//
// F is the 64-point DFT matrix in real form ([[C, S], [-S, C]], scaled by 1/8), its rows ordered
// so that Re and Im of one output bin sit 8 TMEM lanes apart, which is where a 16x256b TMEM load
// puts them in one thread.  B holds the 64 contracted samples (re, im interleaved along K) for
// 64 x 4 = 256 independent columns (the other digit x 4 column pairs).  Between stages the
// epilogue warps read D, apply the twiddle W_4096^{k1 t2} (or the gate, or the final radix-2
// combine), round to fp16 and write the next stage's B operand.  The inverse transform is
// conj(FFT(conj(.))) so one F serves both directions.
//
// One CTA = one (batch, head, 4 column pairs) = a 16-byte piece of every one of the 8192 rows.
// Those pieces are moved by the TMA engine, not by the load/store units: a 5-D tensor map that
// splits the row index t = 64 t1 + t2 into its two digits drops 256 rows at a time into shared
// memory in exactly the order of a K-major operand (t2 and the pair index along the columns,
// t1 along K), so the radix-2 step converts bf16 to fp16 in place; the result rows are staged in
// shared memory with t1 running fastest (conflict-free from the accumulator layout) and written
// back through a second map whose digit order is swapped.  The gate tables are built while the
// rows are in flight.  The "e" and "o" halves ping-pong: while the epilogue of one half runs on
// the ALUs the MMAs of the other half run on the tensor core.  Hand-offs are mbarriers; every
// wait is bounded and reports through a status word instead of hanging.
#include <cuda.h>

#include <string>

#include "tc_stage.cuh"

namespace spectre {

constexpr int k8FBytes = 128 * 128 * 2;
constexpr int k8Smem = k8FBytes + 2 * k8BBytes + 2 * k8GBytes + 128;
constexpr int k8EpiWarps = 16;                   // 4 per TMEM lane quadrant, one column quarter each
constexpr int k8EpiThreads = 32 * k8EpiWarps;
constexpr int k8Threads = k8EpiThreads + 32;     // + 1 warp issuing copies and MMAs
static_assert(16 * k8Lbo1 <= k8BBytes && 16 * k8Lbo2 <= k8BBytes && k8Smem <= 232448, "shared memory layout");

struct Tc8kParams {
  const float2* g;        // [B*H][4097]
  const __half* F;        // 64-point DFT matrix, canonical smem layout
  const float2* tw;       // quarter-wave twiddle table (8192nds)
  const float2* tw64;     // stage twiddles W_4096^{row d} (even d) in epilogue order
  int H, ntile;
  int* status;            // host-mapped status word (0 = fine)
};

// Hermitian extension of the half-spectrum gate (n = 8192).
__device__ __forceinline__ float2 gate8192(const float2* __restrict__ g, int k) {
  int kk = k <= 4096 ? k : 8192 - k;
  float2 v = __ldg(g + kk);
  if (kk != k) v.y = -v.y;
  if (k == 0 || k == 4096) v.y = 0.f;
  return v;
}

// 256 rows x 16 bytes, global -> shared, through the digit-split map (t2 fastest in shared memory)
__device__ __forceinline__ void tma_load_rows(uint32_t dst, const CUtensorMap* tm, int col, int t1, int h, int b, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
      :: "r"(dst), "l"(tm), "r"(col), "r"(0), "r"(t1), "r"(h), "r"(b), "r"(bar) : "memory");
}
// 64 (t1) x 8 (t2) rows x 16 bytes, shared -> global, through the map with t1 fastest in shared memory
__device__ __forceinline__ void tma_store_rows(const CUtensorMap* tm, int col, int t1, int t2, int h, int b, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.5d.global.shared::cta.bulk_group [%0, {%1, %2, %3, %4, %5}], [%6];"
               :: "l"(tm), "r"(col), "r"(t1), "r"(t2), "r"(h), "r"(b), "r"(src) : "memory");
}

// four output values in the activation dtype (bf16 or fp16)
template <bool F16> __device__ __forceinline__ uint2 pack_io4(float a, float b, float c, float d) {
  return F16 ? make_uint2(pack_h2(a, b), pack_h2(c, d)) : pack_bf16x4(a, b, c, d);
}

template <bool F16>
__global__ void __launch_bounds__(k8Threads, 1) mixer_tc8192_kernel(const __grid_constant__ CUtensorMap tm_in,
                                                                    const __grid_constant__ CUtensorMap tm_out,
                                                                    const Tc8kParams p) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
  unsigned char* Fsm = smem;
  unsigned char* Bsm[2] = {smem + k8FBytes, smem + k8FBytes + k8BBytes};
  uint32_t* Gsm[2] = {reinterpret_cast<uint32_t*>(smem + k8FBytes + 2 * k8BBytes),
                      reinterpret_cast<uint32_t*>(smem + k8FBytes + 2 * k8BBytes + k8GBytes)};
  __shared__ __align__(8) uint64_t bars[8];    // [0,1] operand ready, [2,3] accumulator ready, [4,5] rows landed, [6] F landed
  __shared__ uint32_t tmem_slot;
  __shared__ float red[k8EpiWarps];

  const int tid = threadIdx.x, warp = tid >> 5, T = tid & 31;
  const int tile = blockIdx.x % p.ntile, slab = blockIdx.x / p.ntile;
  const int b = slab / p.H, h = slab - b * p.H;
  const int col0 = tile * 8;
  const float2* g = p.g + (size_t)slab * 4097;

  if (tid == 0) {
    mbar_init(smem_u32(&bars[0]), k8EpiThreads);
    mbar_init(smem_u32(&bars[1]), k8EpiThreads);
    for (int i = 2; i < 7; ++i) mbar_init(smem_u32(&bars[i]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == k8EpiWarps) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = tmem_slot;
  // Launched as a programmatic dependent of whatever precedes it in the stream: the set-up above may
  // run while that kernel finishes (if it triggers early, as the gate kernels do); nothing of V or g
  // is read before its writes are visible.
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (warp == k8EpiWarps) {
    bool ok = true;
    if (T == 0) {
      // ---- rows: two groups of 16 boxes (t1 = 4a..4a+3 and 64 + 4a..), then the DFT matrix ----
      for (int grp = 0; grp < 2; ++grp) {
        const uint32_t bar = smem_u32(&bars[4 + grp]);
        mbar_expect_tx(bar, 16 * 4096);
        for (int a = 8 * grp; a < 8 * grp + 8; ++a) {
          tma_load_rows(smem_u32(Bsm[0]) + 4096 * a, &tm_in, col0, 4 * a, h, b, bar);
          tma_load_rows(smem_u32(Bsm[1]) + 4096 * a, &tm_in, col0, 64 + 4 * a, h, b, bar);
        }
      }
      mbar_expect_tx(smem_u32(&bars[6]), k8FBytes);
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   :: "r"(smem_u32(Fsm)), "l"(p.F), "r"(k8FBytes), "r"(smem_u32(&bars[6])) : "memory");
    }
    __syncwarp();
    // ---- MMA issuer: 4 stages x 2 halves, 8 K-steps each ----
    const uint32_t idesc = umma_idesc_128x256();
    ok = mbar_wait(smem_u32(&bars[6]), 0);
    for (int stage = 0; stage < 4 && ok; ++stage) {
      const uint32_t lbo = stage == 0 ? k8Lbo0 : (stage == 1 ? k8Lbo1 : (stage == 2 ? k8Lbo2 : k8Lbo3));
      const uint32_t sbo = stage == 0 ? k8Sbo0 : (stage == 1 ? k8Sbo1 : (stage == 2 ? k8Sbo2 : k8Sbo3));
      for (int half = 0; half < 2 && ok; ++half) {
        ok = mbar_wait(smem_u32(&bars[half]), stage & 1);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (T == 0) {
          const uint32_t a0 = smem_u32(Fsm), b0 = smem_u32(Bsm[0]) + half * k8BBytes;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            uint64_t da = umma_desc(a0 + ks * 256, 128, 2048);
            uint64_t db = umma_desc(b0 + ks * 2 * lbo, lbo, sbo);
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
    if (!ok) {
      if (T == 0) report_timeout(p.status);
      // do not leave with copies into this CTA's shared memory still in flight (bounded again)
      mbar_wait(smem_u32(&bars[4]), 0);
      mbar_wait(smem_u32(&bars[5]), 0);
      mbar_wait(smem_u32(&bars[6]), 0);
    }
  } else {
    // ---- gate tables (while the rows are in flight): Hermitian extension, normalised by a bound
    //      on max |g| so that the gated spectrum stays in fp16 range; bin 2 (k1 + 64 k2) + parity ----
    float gmax = 0.f;
    constexpr int kGIter = 8192 / k8EpiThreads;                 // table entries per thread
    float2 gv[kGIter];
#pragma unroll
    for (int i = 0; i < kGIter; ++i) gv[i] = gate8192(g, tid + i * k8EpiThreads);   // all loads in flight
#pragma unroll
    for (int i = 0; i < kGIter; ++i) gmax = fmaxf(gmax, fmaxf(fabsf(gv[i].x), fabsf(gv[i].y)));
    for (int o = 16; o > 0; o >>= 1) gmax = fmaxf(gmax, __shfl_xor_sync(0xffffffffu, gmax, o));
    if (T == 0) red[warp] = gmax;
    asm volatile("bar.sync 1, %0;" :: "r"(k8EpiThreads) : "memory");
    gmax = 0.f;
    for (int i = 0; i < k8EpiWarps; ++i) gmax = fmaxf(gmax, red[i]);
    gmax *= 1.41421356f;
    const float ginv = gmax > 0.f ? 1.0f / gmax : 0.f;
#pragma unroll
    for (int i = 0; i < kGIter; ++i) {
      const int k = tid + i * k8EpiThreads, m = k >> 1;
      Gsm[0][(k & 1) * (k8GBytes / 4) + k8GStride * (m >> 6) + (m & 63)] = pack_h2(gv[i].x * ginv, gv[i].y * ginv);
    }
    asm volatile("bar.sync 1, %0;" :: "r"(k8EpiThreads) : "memory");

    // ---- radix-2 step in place: rows t (landed in Bsm[0]) and t + 4096 (Bsm[1]) -> e, o in fp16.
    //      A thread takes t1 = 4a..4a+3 at one t2: four 16-byte chunks (one row each, 4 pairs) in,
    //      four chunks (one pair each, 4 consecutive K) out, at the same addresses ----
    bool ok = true;
    {
      const int t2 = tid & 63;
      const float2 w64[4] = {make_float2(1.f, 0.f), make_float2(0.998795456f, -0.049067674f),
                             make_float2(0.995184727f, -0.098017140f), make_float2(0.989176510f, -0.146730474f)};
#pragma unroll 1
      for (int grp = 0; grp < 2 && ok; ++grp) {
        ok = mbar_wait(smem_u32(&bars[4 + grp]), 0);
        if (!ok) break;
        const int a = 8 * grp + (tid >> 6);
        unsigned char* p0 = Bsm[0] + 4096 * a + 16 * t2;
        unsigned char* p1 = Bsm[1] + 4096 * a + 16 * t2;
        uint4 ra[4], rb[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          ra[u] = *reinterpret_cast<const uint4*>(p0 + 1024 * u);
          rb[u] = *reinterpret_cast<const uint4*>(p1 + 1024 * u);
        }
        const float2 w0 = twiddle8192(p.tw, (unsigned)(256 * a + t2));
        float2 w[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) w[u] = cmul(w0, w64[u]);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t e[4], o[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const uint32_t ua = c == 0 ? ra[u].x : (c == 1 ? ra[u].y : (c == 2 ? ra[u].z : ra[u].w));
            const uint32_t ub = c == 0 ? rb[u].x : (c == 1 ? rb[u].y : (c == 2 ? rb[u].z : rb[u].w));
            const float2 va = F16 ? unpack_h2(ua) : unpack_bf2(ua), vb = F16 ? unpack_h2(ub) : unpack_bf2(ub);
            const float2 ve = cadd(va, vb), vo = cmul(csub(va, vb), w[u]);
            e[u] = pack_h2(ve.x, ve.y);
            o[u] = pack_h2(vo.x, vo.y);
          }
          *reinterpret_cast<uint4*>(p0 + 1024 * c) = make_uint4(e[0], e[1], e[2], e[3]);
          *reinterpret_cast<uint4*>(p1 + 1024 * c) = make_uint4(o[0], o[1], o[2], o[3]);
        }
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    mbar_arrive(smem_u32(&bars[0]));
    mbar_arrive(smem_u32(&bars[1]));

    const int q = warp & 3, cq = warp >> 2;
    // W_4096^{row} of this thread's two accumulator rows (8 (2q + j) + T / 4): the odd columns' stage twiddles
    const float2 wr0 = twiddle_fwd((unsigned)(16 * q + (T >> 2)), 4096u), wr1 = twiddle_fwd((unsigned)(16 * q + 8 + (T >> 2)), 4096u);
    // ---- stages 1..3: wait for D, transform, hand the next operand to the issuer ----
#pragma unroll 1
    for (int stage = 0; stage < 3 && ok; ++stage) {
#pragma unroll 1
      for (int half = 0; half < 2 && ok; ++half) {
        ok = mbar_wait(smem_u32(&bars[2 + half]), stage & 1);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t td = tmem + 256 * half;
        unsigned char* Bh = Bsm[0] + half * k8BBytes;
        if (stage == 0) epilogue_twiddle<k8Lbo1, k8Sbo1, true>(td, Bh, q, cq, T, p.tw64, wr0, wr1);
        else if (stage == 1) epilogue_gate(td, Bh, q, cq, T, Gsm[0] + half * (k8GBytes / 4));
        else epilogue_twiddle<k8Lbo3, k8Sbo3, false>(td, Bh, q, cq, T, p.tw64, wr0, wr1);
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive(smem_u32(&bars[half]));
      }
    }
    // ---- final: y[t], y[t+4096] = (gmax/2) conj(D_e +- W_8192^t D_o), t = 64 row + s1, staged as
    //      bf16 with the row digit fastest: box bi (s1 = 8 bi .. 8 bi + 7) at 8192 bi, row t at
    //      ((s1 & 7) * 64 + t1) * 16; each column quarter hands its boxes to the TMA engine ----
    if (ok) ok = mbar_wait(smem_u32(&bars[2]), 1);
    if (ok) ok = mbar_wait(smem_u32(&bars[3]), 1);
    if (ok) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int i = T >> 2, pp = (T >> 1) & 1, cp = T & 1;
      const float gs = 0.5f * gmax;
      const float2 wstep = twiddle8192(p.tw, 2u);
      const uint32_t taddr0 = tmem + ((uint32_t)(32 * q) << 16) + 64 * cq;
      uint32_t re[2][16], ro[2][16];
      bool bad = false;                                          // a non-finite result: the fp16 intermediates overflowed
      tmem_ld_16x256b_x4(taddr0, re[0]);
      tmem_ld_16x256b_x4(taddr0 + 256, ro[0]);
#pragma unroll
      for (int step = 0; step < 4; ++step) {                     // step = 2 chunk + j
        const int chunk = step >> 1, j = step & 1;
        const int t1 = 8 * (2 * q + j) + i;
        float2 w = twiddle8192(p.tw, (unsigned)(64 * t1 + 16 * cq + 8 * chunk + pp));
        tmem_ld_wait();
        if (step < 3) {
          const int nchunk = (step + 1) >> 1, nj = (step + 1) & 1;
          const uint32_t ta = taddr0 + ((uint32_t)(16 * nj) << 16) + 32 * nchunk;
          tmem_ld_16x256b_x4(ta, re[(step + 1) & 1]);
          tmem_ld_16x256b_x4(ta + 256, ro[(step + 1) & 1]);
        }
        const uint32_t (&xe)[16] = re[step & 1];
        const uint32_t (&xo)[16] = ro[step & 1];
        const uint32_t base = (uint32_t)((2 * cq + chunk) * 8192 + (pp * 64 + t1) * 16 + 8 * cp);
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const float2 e0 = make_float2(__uint_as_float(xe[4 * x]), __uint_as_float(xe[4 * x + 2]));
          const float2 e1 = make_float2(__uint_as_float(xe[4 * x + 1]), __uint_as_float(xe[4 * x + 3]));
          const float2 o0 = cmul(make_float2(__uint_as_float(xo[4 * x]), __uint_as_float(xo[4 * x + 2])), w);
          const float2 o1 = cmul(make_float2(__uint_as_float(xo[4 * x + 1]), __uint_as_float(xo[4 * x + 3])), w);
          if (x < 3) w = cmul(w, wstep);
          const uint2 ylo = pack_io4<F16>(gs * (e0.x + o0.x), -gs * (e0.y + o0.y), gs * (e1.x + o1.x), -gs * (e1.y + o1.y));
          const uint2 yhi = pack_io4<F16>(gs * (e0.x - o0.x), -gs * (e0.y - o0.y), gs * (e1.x - o1.x), -gs * (e1.y - o1.y));
          // an overflow anywhere in a column makes every row of it non-finite: one row per thread and pair is enough
          if (x == 0) bad |= nonfinite16x2<F16>(ylo.x) | nonfinite16x2<F16>(ylo.y);
          *reinterpret_cast<uint2*>(Bsm[0] + base + 2048 * x) = ylo;
          *reinterpret_cast<uint2*>(Bsm[1] + base + 2048 * x) = yhi;
        }
        if (j == 1) {
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          asm volatile("bar.sync %0, %1;" :: "r"(2 + cq), "r"(128) : "memory");
          if (q == 0 && T == 0) {
            const int bi = 2 * cq + chunk;
            tma_store_rows(&tm_out, col0, 0, 8 * bi, h, b, smem_u32(Bsm[0]) + 8192 * bi);
            tma_store_rows(&tm_out, col0, 64, 8 * bi, h, b, smem_u32(Bsm[1]) + 8192 * bi);
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          }
        }
      }
      if (q == 0 && T == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
      if (__any_sync(0xffffffffu, bad) && T == 0) report_range(p.status);
    }
    if (!ok && T == 0) report_timeout(p.status);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == k8EpiWarps) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(512));
  }
}

// ---- host side ---------------------------------------------------------------------------

// The tensor maps need 16-byte aligned bases and strides and whole 64-row blocks.
bool tc8192_supported(const spectre_act* v, const spectre_act* y) {
  auto ok = [](const spectre_act* a) {
    return (reinterpret_cast<uintptr_t>(a->ptr) & 15) == 0 && a->stride_l % 8 == 0 && a->stride_h % 8 == 0 &&
           a->stride_b % 8 == 0 && a->stride_l > 0 && a->stride_h > 0 && a->stride_b > 0;
  };
  return v->L % 64 == 0 && v->D % 8 == 0 && ok(v) && ok(y) && tensor_map_encoder() != nullptr;
}

// dims (column, row digit A, row digit B, head, batch); t1_fastest puts t1 (stride 64 rows) second.
static int make_row_map(CUtensorMap* tm, const spectre_act* a, bool t1_fastest, unsigned box1, unsigned box2) {
  const cuuint64_t sl = (cuuint64_t)a->stride_l * 2, sh = (cuuint64_t)a->stride_h * 2, sb = (cuuint64_t)a->stride_b * 2;
  cuuint64_t dims[5] = {(cuuint64_t)a->D, 64, (cuuint64_t)(a->L / 64), (cuuint64_t)a->H, (cuuint64_t)a->B};
  cuuint64_t strides[4] = {sl, 64 * sl, sh, sb};
  if (t1_fastest) {
    dims[1] = (cuuint64_t)(a->L / 64); dims[2] = 64;
    strides[0] = 64 * sl; strides[1] = sl;
  }
  cuuint32_t box[5] = {8, box1, box2, 1, 1};
  cuuint32_t es[5] = {1, 1, 1, 1, 1};
  CUresult r = tensor_map_encoder()(tm, a->dtype == SPECTRE_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, a->ptr, dims, strides, box, es,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                 CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(SPECTRE_ERR_CUDA, "cuTensorMapEncodeTiled failed (" + std::to_string((int)r) + ")");
  return SPECTRE_OK;
}

int launch_mixer_tc8192(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, const float* g,
                        const spectre_act* y) {
  CUtensorMap tm_in, tm_out;
  int rc = make_row_map(&tm_in, v, false, 64, 4);
  if (rc != SPECTRE_OK) return rc;
  rc = make_row_map(&tm_out, y, true, 64, 8);
  if (rc != SPECTRE_OK) return rc;
  Tc8kParams p = {};
  p.g = reinterpret_cast<const float2*>(g);
  p.F = reinterpret_cast<const __half*>(ctx->dft64);
  p.tw = reinterpret_cast<const float2*>(ctx->tw8192);
  p.tw64 = reinterpret_cast<const float2*>(ctx->tw64x64);
  p.H = v->H; p.ntile = v->D / 8;
  p.status = ctx->status_dev;
  const unsigned grid = (unsigned)((size_t)v->B * v->H * p.ntile);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(k8Threads);
  cfg.dynamicSmemBytes = k8Smem;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (v->dtype == SPECTRE_F16) {
    SPECTRE_CUDA_OK(cudaFuncSetAttribute(mixer_tc8192_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, k8Smem));
    SPECTRE_CUDA_OK(cudaLaunchKernelEx(&cfg, mixer_tc8192_kernel<true>, tm_in, tm_out, p));
  } else {
    SPECTRE_CUDA_OK(cudaFuncSetAttribute(mixer_tc8192_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, k8Smem));
    SPECTRE_CUDA_OK(cudaLaunchKernelEx(&cfg, mixer_tc8192_kernel<false>, tm_in, tm_out, p));
  }
  SPECTRE_LAUNCH_OK("mixer_tc8192_kernel");
  return SPECTRE_OK;
}

}  // namespace spectre
