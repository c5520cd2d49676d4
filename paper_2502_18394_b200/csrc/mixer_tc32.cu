// The radix-32 steps of the four-step split n = 32 * 4096 (Sec. 3.2 steps 2 and 4 at n = 131072) on
// the tensor cores, for bf16 or fp16 activations with d_head = 64.  They replace the transposing ALU
// kernels of mixer_tc4k.cu around the same core:
//
//   tc_in32_kernel   rows n1 * 4096 + t' of [B, L, H, D] are whole 128-byte lines.  A TMA box
//                    (64 columns, 1 t', 32 n1; 128-byte swizzle) lands them as an MN-major B operand
//                    with K = n1 and N = the 64 real columns, straight from HBM, no conversion.  One
//                    MMA does the real-input 32-point DFT over n1 for 8 values of t' at once:
//                    A (128 x 64) is block diagonal, two copies of [C; -S], so lanes 0-63 hold (k1,
//                    re / im) of four t' and lanes 64-127 of four others.  bf16 inputs force a bf16
//                    A (operand formats must match), so A = hi + lo and two passes accumulate.  The
//                    epilogue pairs the spectra of columns 2p, 2p + 1 (Z = A + jB, the pair packing of
//                    mixer.cu), applies W_n^{k1 t'} and writes fp16 into a shared-memory box from which
//                    one TMA store hands every unit (head, k1, 4 pairs) 32-byte runs of its operand image.
//                    After every 8th item the epilogue warps also write one gate image.
//   tc_out32_kernel  the units' results (already scaled and multiplied by conj W_n^{k1 t'} by the core)
//                    are whole 128-byte lines too (8 rows x 4 pairs of one unit): the box (128 bytes,
//                    1 tile, 32 k1) is the B operand with K = k1; A = two copies of [C; S] (fp16);
//                    lanes 0-63 serve tiles 0-3, lanes 64-127 tiles 4-7, so one MMA yields 8 rows t'
//                    x 32 n1 complete 128-byte output rows, staged (128-byte swizzle) and written by
//                    TMA stores.
//
// Both are persistent, one CTA per SM: a producer warp runs TMA loads one work item ahead and issues
// the MMAs, 16 epilogue warps drain the two accumulators of an item in turn.  Every wait is bounded
// and reports through the status word.
#include <cuda.h>

#include <string>

#include "tc_common.cuh"

namespace spectre {

constexpr int kXBox = 32 * 128;                   // one landed box: 32 rows of 128 bytes
constexpr int kXItemOp = 16 * kXBox;              // operands of one work item: 2 MMAs x 2 lane groups x 4 blocks
constexpr int kXMat = 128 * 64 * 2;               // one 128 x 64 matrix
constexpr int kXEpiWarps = 16, kXEpiThreads = 512;  // per TMEM lane quadrant: 2 column halves x 2 sixteen-lane halves
constexpr int kXInThreads = kXEpiThreads + 32;    // + producer warp
constexpr int kXOutThreads = kXEpiThreads + 32;
constexpr int kXInStage = 65536;                  // two store boxes of [tile (8)][k1 (32)][pair (4)][t2 (2)][4 t1], fp16 (re, im)
constexpr int kXInSmem = 2 * kXMat + 2 * kXItemOp + kXInStage + 160;
constexpr int kXOutSmem = kXMat + 2 * kXItemOp + 2 * 32768 + 128;
constexpr int kXImgBytes = 65536, kXGBytes = 16384, kXOutBytes = 65536;   // as in mixer_tc4k.cu
static_assert(kXInSmem <= 232448 && kXOutSmem <= 232448, "shared memory");

// ---- the four matrices ------------------------------------------------------------------------
// Row m of a matrix: lane group m / 64, then 16-lane blocks of 8 indices with part 0 in the lower 8
// lanes and part 1 in the upper 8 (where a 16x256b TMEM load puts both into one thread); column kk:
// group kk / 32, contracted index kk % 32; zero unless the groups agree.  K-major canonical layout.
__global__ void build_dft32_kernel(unsigned char* mats) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= 128 * 64) return;
  const int m = idx >> 6, kk = idx & 63;
  const int g = m >> 6, blk = (m >> 4) & 3, l = m & 15, a = 8 * blk + (l & 7), part = l >> 3;
  const int gk = kk >> 5, c = kk & 31;
  float s, co;
  sincospif((float)((a * c) & 31) / 16.0f, &s, &co);
  const float fwd = g == gk ? (part == 0 ? co : -s) : 0.f;      // [C; -S]: X[k1] = sum x (cos - j sin)
  const float inv = g == gk ? (part == 0 ? co : s) : 0.f;       // [C;  S]: W^{-k n} = cos + j sin
  const size_t off = (size_t)((m >> 3) * 1024 + (kk >> 3) * 128 + (m & 7) * 16 + (kk & 7) * 2);
  const __nv_bfloat16 hi = __float2bfloat16(fwd);
  *reinterpret_cast<__nv_bfloat16*>(mats + off) = hi;
  *reinterpret_cast<__nv_bfloat16*>(mats + kXMat + off) = __float2bfloat16(fwd - __bfloat162float(hi));
  *reinterpret_cast<__half*>(mats + 2 * kXMat + off) = __float2half(fwd);
  *reinterpret_cast<__half*>(mats + 3 * kXMat + off) = __float2half(inv);
}
int build_dft32(void* mats, cudaStream_t st) {
  build_dft32_kernel<<<32, 256, 0, st>>>(reinterpret_cast<unsigned char*>(mats));
  SPECTRE_LAUNCH_OK("build_dft32_kernel");
  return SPECTRE_OK;
}

// B operand landed by a 128-byte-swizzled TMA box: MN-major, 64 N elements (128 bytes) per K row, 8 K rows
// per 1024-byte atom; lbo = bytes between 64-element N blocks, sbo = bytes between 8-row K groups.
__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  return umma_desc(saddr, lbo, sbo) | ((uint64_t)2 << 61);
}
// kind::f16, A K-major, B MN-major, fp32 accumulator, M = 128, N = 256; fmt 0 = fp16, 1 = bf16 (both operands)
__device__ __forceinline__ uint32_t umma_idesc_x(uint32_t fmt) {
  return (1u << 4) | (fmt << 7) | (fmt << 10) | (1u << 16) | ((256u >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, int c2, int c3, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.4d.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
               :: "r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, int c2, int c3, int c4, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.5d.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
               :: "r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_store_5d(const CUtensorMap* tm, int c0, int c1, int c2, int c3, int c4, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.5d.global.shared::cta.bulk_group [%0, {%1, %2, %3, %4, %5}], [%6];"
               :: "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(src) : "memory");
}

// one item's MMAs for accumulator m: npass passes (matrix 0, then matrix 1 on top) x 4 K steps
__device__ __forceinline__ void issue_item_mmas(uint32_t tmem_d, uint32_t a_base, int npass, uint32_t op_m, uint32_t idesc) {
  for (int pass = 0; pass < npass; ++pass) {
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      const uint64_t da = umma_desc(a_base + pass * kXMat + ks * 256, 128, 1024);
      const uint64_t db = umma_desc_mn_sw128(op_m + (ks >> 1) * 4 * kXBox + (ks & 1) * 2048, kXBox, 1024);
      const uint32_t acc = (pass | ks) != 0;
      asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                   :: "r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
    }
  }
}

// =====================================================================================
// transpose-in, R = 32
// =====================================================================================
struct TcIn32Params {
  const unsigned char* mats;    // the context's four matrices
  const float2* twr;            // [32][128]: W_n^{64 k1 t1}, W_n^{k1 t2}
  unsigned char* ws_in;         // [unit][kXImgBytes]
  const float2* g;              // [B*H][K]
  unsigned char* gimg;          // [slab_local * 32 + k1][kXGBytes]
  float* gscale;                // [slab_local * 32 + k1]
  int H, slab0, cnt, n, K;
  float sc;                     // forward scale of the radix-32 step
  int* status;
};

// bins k = k1 + 32 kM, kM < 4096, of the Hermitian extension of one head's gate
__device__ __forceinline__ float2 gate_ext(const float2* __restrict__ g, int k, int n) {
  const int kk = (2 * k <= n) ? k : n - k;
  float2 v = __ldg(g + kk);
  if (kk != k) v.y = -v.y;
  if (k == 0 || 2 * k == n) v.y = 0.f;
  return v;
}

template <bool F16>
__global__ void __launch_bounds__(kXInThreads, 1) tc_in32_kernel(const __grid_constant__ CUtensorMap tm_in,
                                                                 const __grid_constant__ CUtensorMap tm_img, const TcIn32Params p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* Asm = smem;                                   // hi, lo (bf16) or the fp16 matrix
  unsigned char* Op = smem + 2 * kXMat;                        // two item slots
  uint32_t* Stg = reinterpret_cast<uint32_t*>(smem + 2 * kXMat + 2 * kXItemOp);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 2 * kXMat + 2 * kXItemOp + kXInStage);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 8);
  float* red = reinterpret_cast<float*>(bars + 9);             // 16 floats
  const int tid = threadIdx.x, warp = tid >> 5, T = tid & 31;
  const uint32_t barFull[2] = {smem_u32(&bars[0]), smem_u32(&bars[1])}, barFree[2] = {smem_u32(&bars[2]), smem_u32(&bars[3])};
  const uint32_t accFull[2] = {smem_u32(&bars[4]), smem_u32(&bars[5])}, accFree[2] = {smem_u32(&bars[6]), smem_u32(&bars[7])};

  if (tid == 0) {
    for (int s = 0; s < 2; ++s) { mbar_init(barFull[s], 1); mbar_init(barFree[s], 1); mbar_init(accFull[s], 1); mbar_init(accFree[s], kXEpiThreads); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kXEpiWarps) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  {
    const uint4* Ag = reinterpret_cast<const uint4*>(p.mats + (F16 ? 2 * kXMat : 0));
    for (int i = tid; i < (F16 ? 1 : 2) * kXMat / 16; i += kXInThreads) reinterpret_cast<uint4*>(Asm)[i] = __ldg(Ag + i);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *tmem_slot;
  asm volatile("griddepcontrol.wait;" ::: "memory");           // launched as a programmatic dependent
  const int nitems = p.cnt * 256;                               // (slab, 16 groups of 4 t1, 16 blocks of 4 t2): one head's images are written while L2 holds them
  bool ok = (smem_u32(smem) & 1023u) == 0;                      // the swizzled boxes need 1024-byte aligned slots

  if (warp == kXEpiWarps) {
    // ---- producer + MMA issuer ----
    const uint32_t idesc = umma_idesc_x(F16 ? 0u : 1u);
    auto fetch = [&](int item, int slot) {
      const int slab = p.slab0 + (item >> 8), a = (item >> 4) & 15, t2b = item & 15;
      const int b = slab / p.H, h = slab - b * p.H;
      mbar_expect_tx(barFull[slot], kXItemOp);
      for (int m = 0; m < 2; ++m)
        for (int gq = 0; gq < 2; ++gq)
          for (int u = 0; u < 4; ++u)
            tma_load_5d(smem_u32(Op) + slot * kXItemOp + ((m * 2 + gq) * 4 + u) * kXBox, &tm_in, 0,
                        64 * (4 * a + u) + 4 * t2b + 2 * m + gq, 0, h, b, barFull[slot]);
    };
    if (T == 0 && (int)blockIdx.x < nitems) fetch(blockIdx.x, 0);
    __syncwarp();
    int it = 0;
    for (int item = blockIdx.x; item < nitems && ok; item += gridDim.x, ++it) {
      const int slot = it & 1, next = item + gridDim.x;
      if (next < nitems) {                                      // the other slot: free once the MMAs of item it - 1 are done
        if (it >= 1) ok = mbar_wait(barFree[slot ^ 1], ((it - 1) >> 1) & 1);
        if (ok && T == 0) fetch(next, slot ^ 1);
        __syncwarp();
      }
      if (ok) ok = mbar_wait(barFull[slot], (it >> 1) & 1);
      for (int m = 0; m < 2 && ok; ++m) {
        if (it > 0) ok = mbar_wait(accFree[m], (it - 1) & 1);   // the epilogue has drained this accumulator
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (T == 0) {
          issue_item_mmas(tmem + 256 * m, smem_u32(Asm), F16 ? 1 : 2, smem_u32(Op) + slot * kXItemOp + m * 8 * kXBox, idesc);
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(accFull[m]) : "memory");
        }
        __syncwarp();
      }
      if (ok && T == 0)
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(barFree[slot]) : "memory");
      __syncwarp();
    }
    if (!ok) { mbar_wait(barFull[0], 0); mbar_wait(barFull[1], 0); }   // no copy into this CTA left in flight
  } else {
    // ---- epilogue warps: lane quadrant q = lane group q / 2, k1 = 16 (q % 2) + 8 j + i; column half wh ----
    const int q = warp & 3, wh = (warp >> 2) & 1, j = warp >> 3, i = T >> 2, tq = T & 3, gq = q >> 1;
    const int k1 = 16 * (q & 1) + 8 * j + i;
    int it = 0;
    for (int item = blockIdx.x; item < nitems && ok; item += gridDim.x, ++it) {
      const int slab_local = item >> 8, a = (item >> 4) & 15, t2b = item & 15;
      // One gate image with every 8th item (there are 8 items per image): its strided reads are issued
      // here and consumed after the item's epilogues, so their latency hides under them.
      const int sk = (int)blockIdx.x + (it >> 3) * (int)gridDim.x;
      const bool gate_item = (it & 7) == 0 && sk < p.cnt * 32;
      float2 gvv[8];
      if (gate_item) {
        const float2* g = p.g + (size_t)(p.slab0 + (sk >> 5)) * p.K;
#pragma unroll
        for (int t = 0; t < 8; ++t) gvv[t] = gate_ext(g, (sk & 31) + 32 * (tid + kXEpiThreads * t), p.n);
      }
      // sc W_n^{64 k1 (4a + u)} and W_n^{k1 t2} of this thread's two k1 and this item's rows
      float2 wA[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) { const float2 t = __ldg(p.twr + 128 * k1 + 4 * a + u); wA[u] = make_float2(t.x * p.sc, t.y * p.sc); }
#pragma unroll 1
      for (int m = 0; m < 2 && ok; ++m) {
        // the store that last read this box must be done with it
        if (tid == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        asm volatile("bar.sync 1, %0;" :: "r"(kXEpiThreads) : "memory");
        unsigned char* box = reinterpret_cast<unsigned char*>(Stg) + 32768 * m;   // [tile (8)][k1 (32)][pair c4 (4)][t2 (2)][4 t1 = 16 bytes]
        const float2 wB = __ldg(p.twr + 128 * k1 + 64 + 4 * t2b + 2 * m + gq);
        ok = mbar_wait(accFull[m], it & 1);
        if (ok) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t taddr0 = tmem + 256 * m + ((uint32_t)(32 * q + 16 * j) << 16) + 32 * wh;
          uint32_t r[2][16];
          tmem_ld_16x256b_x4(taddr0, r[0]);
          uint32_t chunk[4][4];                                   // [tile 4 wh + x][t1 = 4a + u]: one 16-byte piece of an operand image each
#pragma unroll
          for (int u = 0; u < 4; ++u) {                           // columns 64 u + 32 wh ..
            tmem_ld_wait();
            if (u < 3) tmem_ld_16x256b_x4(taddr0 + 64 * (u + 1), r[(u + 1) & 1]);
            const uint32_t (&rr)[16] = r[u & 1];
            const float2 w = cmul(wA[u], wB);
#pragma unroll
            for (int x = 0; x < 4; ++x) {                         // pair 16 wh + 4 x + tq: tile 4 wh + x, pair tq of the tile
              // spectra of the real columns 2p (A) and 2p + 1 (B): Z = A + jB
              const float2 z = make_float2(__uint_as_float(rr[4 * x]) - __uint_as_float(rr[4 * x + 3]),
                                           __uint_as_float(rr[4 * x + 2]) + __uint_as_float(rr[4 * x + 1]));
              const float2 v = cmul(z, w);
              chunk[x][u] = pack_h2(v.x, v.y);
            }
            if (u == 3) {
#pragma unroll
              for (int x = 0; x < 4; ++x)
                *reinterpret_cast<uint4*>(box + (((4 * wh + x) * 32 + k1) * 4 + tq) * 32 + 16 * gq) =
                    make_uint4(chunk[x][0], chunk[x][1], chunk[x][2], chunk[x][3]);
            }
          }
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          mbar_arrive(accFree[m]);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("bar.sync 1, %0;" :: "r"(kXEpiThreads) : "memory");
        if (tid == 0 && ok) {
          // every unit (k1, tile) of the head gets, per pair, two consecutive t2 = 32 bytes of its image
          asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%1, %2, %3, %4}], [%5];"
                       :: "l"(&tm_img), "r"(8 * (4 * t2b + 2 * m)), "r"(4 * a), "r"(32 * slab_local), "r"(0), "r"(smem_u32(box)) : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      }
      // ---- the gate image: per (head, k1) the 4096 gate values the core needs, normalised by a bound on
      //      their maximum, fp16, entry kM = kl + 64 k2 at 64 k2 + (kl ^ 8 (k2 % 4)) ----
      if (gate_item) {
        float mx = 0.f;
#pragma unroll
        for (int t = 0; t < 8; ++t) mx = fmaxf(mx, fmaxf(fabsf(gvv[t].x), fabsf(gvv[t].y)));
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        if (T == 0) red[warp] = mx;
        asm volatile("bar.sync 1, %0;" :: "r"(kXEpiThreads) : "memory");
        mx = 0.f;
        for (int w8 = 0; w8 < kXEpiWarps; ++w8) mx = fmaxf(mx, red[w8]);
        mx *= 1.41421356f;
        const float inv = mx > 0.f ? 1.0f / mx : 0.f;
        uint32_t* img = reinterpret_cast<uint32_t*>(p.gimg + (size_t)sk * kXGBytes);
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          const int idx = tid + kXEpiThreads * t, k2 = idx >> 6, kl = idx & 63;
          img[64 * k2 + (kl ^ (8 * (k2 & 3)))] = pack_h2(gvv[t].x * inv, gvv[t].y * inv);
        }
        if (tid == 0) p.gscale[sk] = mx;
        asm volatile("bar.sync 1, %0;" :: "r"(kXEpiThreads) : "memory");   // red[] may be rewritten
      }
    }
  }
  if (tid == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  if (!ok && T == 0) report_timeout(p.status);
  __syncwarp();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == kXEpiWarps) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(512));
  }
}

// =====================================================================================
// transpose-out, R = 32
// =====================================================================================
struct TcOut32Params {
  const unsigned char* mats;
  int H, slab0, cnt;
  int* status;
};

template <bool F16>
__global__ void __launch_bounds__(kXOutThreads, 1) tc_out32_kernel(const __grid_constant__ CUtensorMap tm_res,
                                                                  const __grid_constant__ CUtensorMap tm_out, const TcOut32Params p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* Op = smem;                                    // two item slots
  unsigned char* Stg = smem + 2 * kXItemOp;                    // two boxes of [t'l (8)][n1 (32)][128 bytes], swizzled
  unsigned char* Asm = smem + 2 * kXItemOp + 65536;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 2 * kXItemOp + 65536 + kXMat);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 8);
  const int tid = threadIdx.x, warp = tid >> 5, T = tid & 31;
  const uint32_t barFull[2] = {smem_u32(&bars[0]), smem_u32(&bars[1])}, barFree[2] = {smem_u32(&bars[2]), smem_u32(&bars[3])};
  const uint32_t accFull[2] = {smem_u32(&bars[4]), smem_u32(&bars[5])}, accFree[2] = {smem_u32(&bars[6]), smem_u32(&bars[7])};

  if (tid == 0) {
    for (int s = 0; s < 2; ++s) { mbar_init(barFull[s], 1); mbar_init(barFree[s], 1); mbar_init(accFull[s], 1); mbar_init(accFree[s], kXEpiThreads); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kXEpiWarps) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  {
    const uint4* Ag = reinterpret_cast<const uint4*>(p.mats + 3 * kXMat);
    for (int i = tid; i < kXMat / 16; i += kXOutThreads) reinterpret_cast<uint4*>(Asm)[i] = __ldg(Ag + i);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *tmem_slot;
  const int nitems = p.cnt * 256;                               // (16 consecutive row slots of every unit, slab)
  bool ok = (smem_u32(smem) & 1023u) == 0;                      // the swizzled boxes need 1024-byte aligned slots

  if (warp == kXEpiWarps) {
    // ---- producer + MMA issuer ----
    const uint32_t idesc = umma_idesc_x(0u);
    auto fetch = [&](int item, int slot) {
      const int slab_local = item % p.cnt, blk = item / p.cnt;
      mbar_expect_tx(barFull[slot], kXItemOp);
      for (int m = 0; m < 2; ++m)
        for (int gq = 0; gq < 2; ++gq)
          for (int jb = 0; jb < 4; ++jb)
            tma_load_4d(smem_u32(Op) + slot * kXItemOp + ((m * 2 + gq) * 4 + jb) * kXBox, &tm_res, 128 * blk + 64 * m,
                        4 * gq + jb, 0, slab_local, barFull[slot]);
    };
    if (T == 0 && (int)blockIdx.x < nitems) fetch(blockIdx.x, 0);
    __syncwarp();
    int it = 0;
    for (int item = blockIdx.x; item < nitems && ok; item += gridDim.x, ++it) {
      const int slot = it & 1, next = item + gridDim.x;
      if (next < nitems) {
        if (it >= 1) ok = mbar_wait(barFree[slot ^ 1], ((it - 1) >> 1) & 1);
        if (ok && T == 0) fetch(next, slot ^ 1);
        __syncwarp();
      }
      if (ok) ok = mbar_wait(barFull[slot], (it >> 1) & 1);
      for (int m = 0; m < 2 && ok; ++m) {
        if (it > 0) ok = mbar_wait(accFree[m], (it - 1) & 1);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (T == 0) {
          issue_item_mmas(tmem + 256 * m, smem_u32(Asm), 1, smem_u32(Op) + slot * kXItemOp + m * 8 * kXBox, idesc);
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(accFull[m]) : "memory");
        }
        __syncwarp();
      }
      if (ok && T == 0)
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(barFree[slot]) : "memory");
      __syncwarp();
    }
    if (!ok) { mbar_wait(barFull[0], 0); mbar_wait(barFull[1], 0); }
  } else {
    // ---- epilogue warps: lane quadrant q: tiles 4 (q / 2) .. + 3, n1 = 16 (q % 2) + 8 j + i; column half wh ----
    const int q = warp & 3, wh = (warp >> 2) & 1, j = warp >> 3, i = T >> 2, tq = T & 3, gq = q >> 1;
    const int n1 = 16 * (q & 1) + 8 * j + i;
    bool bad = false;                                            // a non-finite result: the fp16 intermediates overflowed
    int it = 0;
    for (int item = blockIdx.x; item < nitems && ok; item += gridDim.x, ++it) {
      const int slab = p.slab0 + item % p.cnt, blk = item / p.cnt;
      const int b = slab / p.H, h = slab - b * p.H;
      // row slots 16 blk .. + 15 of every unit: s1 / 4 = blk / 16, rows t' / 64 = 4 (blk % 16) + {0..3}, s1 % 4 = {0..3}
      const int k4 = blk >> 4, row0 = 4 * (blk & 15);
#pragma unroll 1
      for (int m = 0; m < 2 && ok; ++m) {
        // the stores that last read this box must be done with it
        if (tid == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        asm volatile("bar.sync 1, %0;" :: "r"(kXEpiThreads) : "memory");
        unsigned char* box = Stg + 32768 * m;
        ok = mbar_wait(accFull[m], it & 1);
        if (ok) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t taddr0 = tmem + 256 * m + ((uint32_t)(32 * q + 16 * j) << 16) + 32 * wh;
          uint32_t r[2][16];
          tmem_ld_16x256b_x4(taddr0, r[0]);
#pragma unroll
          for (int jb = 0; jb < 4; ++jb) {                      // block jb = tile 4 gq + jb
            tmem_ld_wait();
            if (jb < 3) tmem_ld_16x256b_x4(taddr0 + 64 * (jb + 1), r[(jb + 1) & 1]);
            const uint32_t (&rr)[16] = r[jb & 1];
            unsigned char* prow = box + n1 * 128 + (((4 * gq + jb) ^ (n1 & 7)) * 16) + 4 * tq;
#pragma unroll
            for (int x = 0; x < 4; ++x) {                       // row slot t'l = 4 wh + x of the box, pair tq
              // rows (n1, C) and (n1, S) applied to the columns (re, im): y = (C re - S im) + j (S re + C im)
              const float ya = __uint_as_float(rr[4 * x]) - __uint_as_float(rr[4 * x + 3]);
              const float yb = __uint_as_float(rr[4 * x + 2]) + __uint_as_float(rr[4 * x + 1]);
              const uint32_t yo = F16 ? pack_h2(ya, yb) : pack_bf2(ya, yb);
              if (x == 0) bad |= nonfinite16x2<F16>(yo);       // every row of an overflowed column is non-finite: one row is enough
              *reinterpret_cast<uint32_t*>(prow + (4 * wh + x) * 4096) = yo;
            }
          }
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          mbar_arrive(accFree[m]);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("bar.sync 1, %0;" :: "r"(kXEpiThreads) : "memory");
        if (tid == 0 && ok) {
          // box rows t'l = 0..3: t' = 64 (row0 + 2m) + 4 k4 + {0..3}; t'l = 4..7: the next t' / 64
          const int tp = 64 * (row0 + 2 * m) + 4 * k4;
          tma_store_5d(&tm_out, 0, 0, tp, h, b, smem_u32(box));
          tma_store_5d(&tm_out, 0, 0, tp + 64, h, b, smem_u32(box) + 16384);
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      }
    }
    if (tid == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (__any_sync(0xffffffffu, bad) && T == 0) report_range(p.status);
  }
  if (!ok && T == 0) report_timeout(p.status);
  __syncwarp();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == kXEpiWarps) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(512));
  }
}

// ---- host side ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn32)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                    const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn32 encode_fn32() {
  static EncodeTiledFn32 fn = [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      ptr = nullptr;
    return reinterpret_cast<EncodeTiledFn32>(ptr);
  }();
  return fn;
}

// Shapes the radix-32 tensor-core kernels take: n = 131072, 64 channels per head (one 128-byte line per
// row and head), whole 4096-row blocks, 16-byte aligned strides.
bool tc32_supported(const spectre_ctx* ctx, const spectre_act* v, const spectre_act* y, int n) {
  auto ok = [](const spectre_act* a) {
    return (reinterpret_cast<uintptr_t>(a->ptr) & 15) == 0 && a->stride_l % 8 == 0 && a->stride_h % 8 == 0 &&
           a->stride_b % 8 == 0 && a->stride_l > 0 && a->stride_h > 0 && a->stride_b > 0;
  };
  return n == 131072 && v->D == 64 && v->L % 4096 == 0 && ok(v) && ok(y) && ctx->dft32 != nullptr && ctx->tw_staged != nullptr &&
         encode_fn32() != nullptr;
}

// dims (column, A, B, head, batch) over [B, L, H, 64]: row = 4096 n1 + t'; n1_second puts n1 before t'
static int make_act_map(CUtensorMap* tm, const spectre_act* a, bool n1_second, unsigned box_n1, unsigned box_tp) {
  const cuuint64_t sl = (cuuint64_t)a->stride_l * 2, sh = (cuuint64_t)a->stride_h * 2, sb = (cuuint64_t)a->stride_b * 2;
  const cuuint64_t nb = (cuuint64_t)(a->L / 4096);
  cuuint64_t dims[5] = {64, 4096, nb, (cuuint64_t)a->H, (cuuint64_t)a->B};
  cuuint64_t strides[4] = {sl, 4096 * sl, sh, sb};
  cuuint32_t box[5] = {64, box_tp, box_n1, 1, 1};
  if (n1_second) {
    dims[1] = nb; dims[2] = 4096; strides[0] = 4096 * sl; strides[1] = sl;
    box[1] = box_n1; box[2] = box_tp;
  }
  cuuint32_t es[5] = {1, 1, 1, 1, 1};
  CUresult r = encode_fn32()(tm, a->dtype == SPECTRE_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, a->ptr,
                             dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(SPECTRE_ERR_CUDA, "cuTensorMapEncodeTiled failed (" + std::to_string((int)r) + ")");
  return SPECTRE_OK;
}

int launch_tc_in32(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, const float* g, int n, int slab0, int cnt,
                   unsigned char* ws_in, unsigned char* gimg, float* gscale, float sc) {
  CUtensorMap tm;
  int rc = make_act_map(&tm, v, false, 32, 1);
  if (rc != SPECTRE_OK) return rc;
  CUtensorMap tm_img;
  {
    // the operand images as fp16: (t2 x 4 t1 of one pair and K group: 1024 bytes; 4 a + c4; slab * 32 + k1; tile)
    cuuint64_t dims[4] = {512, 64, (cuuint64_t)cnt * 32, 8};
    cuuint64_t strides[3] = {1024, 8 * (cuuint64_t)kXImgBytes, (cuuint64_t)kXImgBytes};
    cuuint32_t box[4] = {16, 4, 32, 8};
    cuuint32_t es[4] = {1, 1, 1, 1};
    CUresult r = encode_fn32()(&tm_img, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, ws_in, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(SPECTRE_ERR_CUDA, "cuTensorMapEncodeTiled failed (" + std::to_string((int)r) + ")");
  }
  TcIn32Params p = {};
  p.mats = reinterpret_cast<const unsigned char*>(ctx->dft32);
  p.twr = reinterpret_cast<const float2*>(ctx->tw_staged) + 31 * 128;
  p.ws_in = ws_in; p.g = reinterpret_cast<const float2*>(g); p.gimg = gimg; p.gscale = gscale;
  p.H = v->H; p.slab0 = slab0; p.cnt = cnt; p.n = n; p.K = n / 2 + 1; p.sc = sc;
  p.status = ctx->status_dev;
  int grid = cnt * 256 < ctx->sm_count ? cnt * 256 : ctx->sm_count;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kXInThreads); cfg.dynamicSmemBytes = kXInSmem; cfg.stream = st;
  cfg.attrs = attr; cfg.numAttrs = 1;
  if (v->dtype == SPECTRE_F16) {
    SPECTRE_CUDA_OK(cudaFuncSetAttribute(tc_in32_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kXInSmem));
    SPECTRE_CUDA_OK(cudaLaunchKernelEx(&cfg, tc_in32_kernel<true>, tm, tm_img, p));
  } else {
    SPECTRE_CUDA_OK(cudaFuncSetAttribute(tc_in32_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kXInSmem));
    SPECTRE_CUDA_OK(cudaLaunchKernelEx(&cfg, tc_in32_kernel<false>, tm, tm_img, p));
  }
  SPECTRE_LAUNCH_OK("tc_in32_kernel");
  return SPECTRE_OK;
}

int launch_tc_out32(const spectre_ctx* ctx, cudaStream_t st, const unsigned char* ws_out, const spectre_act* y, int slab0, int cnt) {
  CUtensorMap tm_res, tm_out;
  int rc = make_act_map(&tm_out, y, true, 32, 4);
  if (rc != SPECTRE_OK) return rc;
  {
    // the units' results as fp16: (one unit, tile, k1, slab of the group)
    cuuint64_t dims[4] = {(cuuint64_t)kXOutBytes / 2, 8, 32, (cuuint64_t)cnt};
    cuuint64_t strides[3] = {(cuuint64_t)kXOutBytes, 8 * (cuuint64_t)kXOutBytes, 256 * (cuuint64_t)kXOutBytes};
    cuuint32_t box[4] = {64, 1, 32, 1};
    cuuint32_t es[4] = {1, 1, 1, 1};
    CUresult r = encode_fn32()(&tm_res, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<unsigned char*>(ws_out), dims, strides, box, es,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(SPECTRE_ERR_CUDA, "cuTensorMapEncodeTiled failed (" + std::to_string((int)r) + ")");
  }
  TcOut32Params p = {};
  p.mats = reinterpret_cast<const unsigned char*>(ctx->dft32);
  p.H = y->H; p.slab0 = slab0; p.cnt = cnt; p.status = ctx->status_dev;
  int grid = cnt * 256 < ctx->sm_count ? cnt * 256 : ctx->sm_count;
  if (y->dtype == SPECTRE_F16) {
    SPECTRE_CUDA_OK(cudaFuncSetAttribute(tc_out32_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kXOutSmem));
    tc_out32_kernel<true><<<grid, kXOutThreads, kXOutSmem, st>>>(tm_res, tm_out, p);
  } else {
    SPECTRE_CUDA_OK(cudaFuncSetAttribute(tc_out32_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kXOutSmem));
    tc_out32_kernel<false><<<grid, kXOutThreads, kXOutSmem, st>>>(tm_res, tm_out, p);
  }
  SPECTRE_LAUNCH_OK("tc_out32_kernel");
  return SPECTRE_OK;
}

}  // namespace spectre
