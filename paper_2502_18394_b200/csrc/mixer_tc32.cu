// The radix-R steps of the four-step split n = R * 4096 for R = 32 ... 2 (Sec. 3.2 steps 2 and 4 at
// n = 131072 ... 8192) on the tensor cores, for bf16 or fp16 activations with d_head = 64.  They
// replace the transposing ALU kernels of mixer_tc4k.cu around the same core.  Described for R = 32:
//
//   tc_in32_kernel   rows n1 * 4096 + t' of [B, L, H, D] are whole 128-byte lines.  A TMA box
//                    (64 columns, 32 n1, 2 t'; 128-byte swizzle) lands them as two MN-major B operands
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
// R < 32 uses the same MMA shape: the 32 contracted rows of a lane group are S = 32 / R independent
// sets of R rows (one TMA box of R rows x S sets lands them set by set), the matrices are block diagonal
// within a group as well (an R-point DFT per set), and a set stands for another t' (tc_in32: S times
// as many t2 per item, store runs of 32 S bytes) or another 128-byte piece of the units' results
// (tc_out32).
//
// Both are persistent, one CTA per SM, four roles joined by mbarriers: a load warp keeps up to three
// half items (32 KB of operands each) in flight through a ring of four slots, an MMA warp starts an
// accumulator as soon as its slot has landed and the accumulator is drained, 16 epilogue warps drain the
// two accumulators of an item in turn into two store boxes, a store warp hands each box to TMA stores.
// Every wait is bounded and reports through the status word.
#include <cuda.h>

#include <string>

#include "tc_common.cuh"

namespace spectre {

constexpr int kXBox = 32 * 128;                   // one landed box: 32 rows of 128 bytes
constexpr int kXItemOp = 16 * kXBox;              // operands of one work item: 2 accumulators x 2 lane groups x 4 blocks
constexpr int kXHalfOp = 8 * kXBox;               // one accumulator's operands: a slot of the four-deep load ring
constexpr int kXMat = 128 * 64 * 2;               // one 128 x 64 matrix
constexpr int kXEpiWarps = 16, kXEpiThreads = 512;  // per TMEM lane quadrant: 2 column halves x 2 sixteen-lane halves
constexpr int kXInThreads = kXEpiThreads + 96;    // + MMA warp + store warp + load warp
constexpr int kXOutThreads = kXEpiThreads + 96;
constexpr int kXInStage = 65536;                  // two store boxes of [tile (8)][k1 (32)][pair (4)][t2 (2)][4 t1], fp16 (re, im)
constexpr int kXInSmem = 2 * kXMat + 2 * kXItemOp + kXInStage + 256;
constexpr int kXOutSmem = kXMat + 2 * kXItemOp + 2 * 32768 + 192;
constexpr int kXImgBytes = 65536, kXGBytes = 16384, kXOutBytes = 65536;   // as in mixer_tc4k.cu
static_assert(kXInSmem <= 232448 && kXOutSmem <= 232448, "shared memory");

// ---- the matrices: four per radix R = 32, 16, 8, 4, 2 (in this order) -----------------------------
// Row m of a matrix: lane group m / 64, then 16-lane blocks of 8 indices with part 0 in the lower 8
// lanes and part 1 in the upper 8 (where a 16x256b TMEM load puts both into one thread); column kk:
// group kk / 32, contracted index kk % 32; zero unless the groups agree.  For R < 32 the 32 indices of
// a group are 32 / R independent sets of R (index = R set + k): an R-point DFT per set, zero across sets.
// K-major canonical layout.
__global__ void build_dft32_kernel(unsigned char* mats_all) {
  const int R = 32 >> blockIdx.y;
  unsigned char* mats = mats_all + (size_t)blockIdx.y * 4 * kXMat;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= 128 * 64) return;
  const int m = idx >> 6, kk = idx & 63;
  const int g = m >> 6, blk = (m >> 4) & 3, l = m & 15, a = 8 * blk + (l & 7), part = l >> 3;
  const int gk = kk >> 5, c = kk & 31;
  const bool on = g == gk && a / R == c / R;
  float s, co;
  sincospif((float)(((a % R) * (c % R)) % R) * 2.0f / (float)R, &s, &co);
  const float fwd = on ? (part == 0 ? co : -s) : 0.f;           // [C; -S]: X[k1] = sum x (cos - j sin)
  const float inv = on ? (part == 0 ? co : s) : 0.f;            // [C;  S]: W^{-k n} = cos + j sin
  const size_t off = (size_t)((m >> 3) * 1024 + (kk >> 3) * 128 + (m & 7) * 16 + (kk & 7) * 2);
  const __nv_bfloat16 hi = __float2bfloat16(fwd);
  *reinterpret_cast<__nv_bfloat16*>(mats + off) = hi;
  *reinterpret_cast<__nv_bfloat16*>(mats + kXMat + off) = __float2bfloat16(fwd - __bfloat162float(hi));
  *reinterpret_cast<__half*>(mats + 2 * kXMat + off) = __float2half(fwd);
  *reinterpret_cast<__half*>(mats + 3 * kXMat + off) = __float2half(inv);
}
int build_dft32(void* mats, cudaStream_t st) {
  build_dft32_kernel<<<dim3(32, 5), 256, 0, st>>>(reinterpret_cast<unsigned char*>(mats));
  SPECTRE_LAUNCH_OK("build_dft32_kernel");
  return SPECTRE_OK;
}

// kind::f16, A K-major, B MN-major, fp32 accumulator, M = 128, N = 256; fmt 0 = fp16, 1 = bf16 (both operands)
__device__ __forceinline__ uint32_t umma_idesc_x(uint32_t fmt) {
  return (1u << 4) | (fmt << 7) | (fmt << 10) | (1u << 16) | ((256u >> 3) << 17) | ((128u >> 4) << 24);
}
// one item's MMAs for accumulator m: npass passes (matrix 0, then matrix 1 on top) x 4 K steps
// op_m: the accumulator's first box; `grp` bytes between the boxes of the two lane groups, `lbo` bytes between
// the boxes of the four 64-column blocks
__device__ __forceinline__ void issue_item_mmas(uint32_t tmem_d, uint32_t a_base, int npass, uint32_t op_m, uint32_t grp, uint32_t lbo,
                                                uint32_t idesc) {
  for (int pass = 0; pass < npass; ++pass) {
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      const uint64_t da = umma_desc(a_base + pass * kXMat + ks * 256, 128, 1024);
      const uint64_t db = umma_desc_mn_sw128(op_m + (ks >> 1) * grp + (ks & 1) * 2048, lbo, 1024);
      const uint32_t acc = (pass | ks) != 0;
      asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                   :: "r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
    }
  }
}

// The 16 mbarriers of a CTA.  Operands travel through a ring of four half-item slots (one accumulator's
// operands each): the load warp fills a slot when its last MMAs are done, the MMA warp starts an
// accumulator when its slot is full and the epilogue has drained it, the epilogue warps fill a store box
// when its last TMA store has read it, and the store warp sends it off.  Three half items can be in
// flight while one is consumed: a single 64 KB item in flight per SM does not cover HBM latency.
struct XBars {
  uint32_t base;
  __device__ explicit XBars(uint32_t b) : base(b) {}
  __device__ uint32_t slotFull(int s) const { return base + 8u * s; }          // TMA bytes landed (count 1 + tx)
  __device__ uint32_t slotFree(int s) const { return base + 32u + 8u * s; }    // its MMAs committed
  __device__ uint32_t accFull(int m) const { return base + 64u + 8u * m; }     // accumulator complete
  __device__ uint32_t accFree(int m) const { return base + 80u + 8u * m; }     // every epilogue thread has read it
  __device__ uint32_t boxFull(int m) const { return base + 96u + 8u * m; }     // every epilogue warp has written its part
  __device__ uint32_t boxFree(int m) const { return base + 112u + 8u * m; }    // the store has read the box
  __device__ void init() const {
    for (int s = 0; s < 4; ++s) { mbar_init(slotFull(s), 1); mbar_init(slotFree(s), 1); }
    for (int m = 0; m < 2; ++m) {
      mbar_init(accFull(m), 1); mbar_init(accFree(m), kXEpiThreads); mbar_init(boxFull(m), kXEpiWarps); mbar_init(boxFree(m), 1);
    }
  }
};

// MMA warp: half item hseq = 2 it + m takes ring slot hseq % 4 and accumulator m
template <typename Issue>
__device__ __forceinline__ bool mma_warp_loop(const XBars& bar, int nitems, int T, bool ok, Issue issue) {
  int hseq = 0, it = 0;
  for (int item = blockIdx.x; item < nitems && ok; item += gridDim.x, ++it) {
    for (int m = 0; m < 2 && ok; ++m, ++hseq) {
      const int slot = hseq & 3;
      ok = mbar_wait(bar.slotFull(slot), (hseq >> 2) & 1);
      if (ok && it > 0) ok = mbar_wait(bar.accFree(m), (it - 1) & 1);   // the epilogue has drained this accumulator
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (T == 0) {
        issue(m, slot);
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar.accFull(m)) : "memory");
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar.slotFree(slot)) : "memory");
      }
      __syncwarp();
    }
  }
  return ok;
}

// load warp: fills the ring up to three half items ahead of the MMAs
template <typename Fetch>
__device__ __forceinline__ bool load_warp_loop(const XBars& bar, int nitems, int T, bool ok, Fetch fetch) {
  int hseq = 0;
  for (int item = blockIdx.x; item < nitems && ok; item += gridDim.x) {
    for (int m = 0; m < 2 && ok; ++m) {
      const int slot = hseq & 3;
      if (hseq >= 4) ok = mbar_wait(bar.slotFree(slot), ((hseq >> 2) - 1) & 1);
      if (!ok) break;
      if (T == 0) { mbar_expect_tx(bar.slotFull(slot), kXHalfOp); fetch(item, m, slot); }
      __syncwarp();
      ++hseq;
    }
  }
  if (!ok)                                                      // leave no copy into this CTA in flight
    for (int back = 1; back <= 4 && back <= hseq; ++back) mbar_wait(bar.slotFull((hseq - back) & 3), ((hseq - back) >> 2) & 1);
  return ok;
}

// =====================================================================================
// transpose-in, R = 32
// =====================================================================================
struct TcIn32Params {
  const unsigned char* mats;    // the context's four matrices
  const float2* twr;            // [32][128]: W_n^{64 k1 t1}, W_n^{k1 t2}
  unsigned char* ws_in;         // [unit][kXImgBytes]
  const float2* g;              // [B*H][K]
  unsigned char* gimg;          // [slab_local * R + k1][kXGBytes]
  float* gscale;                // [slab_local * R + k1]
  int H, slab0, cnt, n, K;
  float sc;                     // forward scale of the radix-R step
  int* status;
};

// bins k = k1 + R kM, kM < 4096, of the Hermitian extension of one head's gate
__device__ __forceinline__ float2 gate_ext(const float2* __restrict__ g, int k, int n) {
  const int kk = (2 * k <= n) ? k : n - k;
  float2 v = __ldg(g + kk);
  if (kk != k) v.y = -v.y;
  if (k == 0 || 2 * k == n) v.y = 0.f;
  return v;
}

// R = 32 ... 2 (n = 4096 R).  The 32 contracted rows of a lane group hold S = 32 / R sets of R rows n1:
// set s of lane group gq is row t' = 64 (4 a + u) + t2 with t2 = 4 S t2b + 2 S m + S gq + s (one TMA box of
// R n1 x S t' lands a lane group's 32 rows set by set), so an accumulator m covers 2 S consecutive t2 and a
// store box row (tile, k1, pair) is a run of 32 S bytes (at most 256: R = 2 stores two boxes of 128).
template <bool F16, int R>
__global__ void __launch_bounds__(kXInThreads, 1) tc_in32_kernel(const __grid_constant__ CUtensorMap tm_in,
                                                                 const __grid_constant__ CUtensorMap tm_img, const TcIn32Params p) {
  constexpr int S = 32 / R, T2B = 16 / S;                      // sets per lane group; t2 blocks (of 4 S) per unit row
  static_assert(R == 32 || R == 16 || R == 8 || R == 4 || R == 2, "radix");
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* Asm = smem;                                   // hi, lo (bf16) or the fp16 matrix
  unsigned char* Op = smem + 2 * kXMat;                        // ring of four half-item slots
  uint32_t* Stg = reinterpret_cast<uint32_t*>(smem + 2 * kXMat + 2 * kXItemOp);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 2 * kXMat + 2 * kXItemOp + kXInStage);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
  float* red = reinterpret_cast<float*>(bars + 17);            // 16 floats
  const int tid = threadIdx.x, warp = tid >> 5, T = tid & 31;
  const XBars bar(smem_u32(bars));

  if (tid == 0) {
    bar.init();
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
  const int nitems = p.cnt * 16 * T2B;                          // (slab, 16 groups of 4 t1, blocks of 4 S t2): one head's images are written while L2 holds them
  bool ok = (smem_u32(smem) & 1023u) == 0;                      // the swizzled boxes need 1024-byte aligned slots

  if (warp == kXEpiWarps) {
    // ---- MMA warp ----
    const uint32_t idesc = umma_idesc_x(F16 ? 0u : 1u);
    ok = mma_warp_loop(bar, nitems, T, ok, [&](int m, int slot) {
      issue_item_mmas(tmem + 256 * m, smem_u32(Asm), F16 ? 1 : 2, smem_u32(Op) + slot * kXHalfOp, kXBox, 2 * kXBox, idesc);
    });
  } else if (warp == kXEpiWarps + 2) {
    // ---- load warp: R = 32: per u one box of the rows of both lane groups (t' and t' + 1), all 32 n1 of each;
    //      R < 32: per (u, lane group) one box of S consecutive t' x R rows n1 ----
    ok = load_warp_loop(bar, nitems, T, ok, [&](int item, int m, int slot) {
      const int slab = p.slab0 + item / (16 * T2B), a = (item / T2B) & 15, t2b = item % T2B;
      const int b = slab / p.H, h = slab - b * p.H;
      for (int u = 0; u < 4; ++u) {
        const int tp = 64 * (4 * a + u) + 4 * S * t2b + 2 * S * m;
        if (S == 1) {
          tma_load_5d(smem_u32(Op) + slot * kXHalfOp + u * 2 * kXBox, &tm_in, 0, 0, tp, h, b, bar.slotFull(slot));
        } else {
          for (int gq = 0; gq < 2; ++gq)
            tma_load_5d(smem_u32(Op) + slot * kXHalfOp + (u * 2 + gq) * kXBox, &tm_in, 0, 0, tp + S * gq, h, b, bar.slotFull(slot));
        }
      }
    });
  } else if (warp == kXEpiWarps + 1) {
    // ---- store warp: hands each filled box to one TMA store, frees it once the copy has read it ----
    int it = 0;
    for (int item = blockIdx.x; item < nitems && ok; item += gridDim.x, ++it) {
      const int slab_local = item / (16 * T2B), a = (item / T2B) & 15, t2b = item % T2B;
      for (int m = 0; m < 2 && ok; ++m) {
        ok = mbar_wait(bar.boxFull(m), it & 1);
        if (ok && T == 0) {
          // every unit (k1, tile) of the head gets, per pair, 2 S consecutive t2 = 32 S bytes of its image
          asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%1, %2, %3, %4}], [%5];"
                       :: "l"(&tm_img), "r"(8 * (4 * S * t2b + 2 * S * m)), "r"(4 * a), "r"(R * slab_local), "r"(0),
                          "r"(smem_u32(Stg) + 32768 * m) : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          mbar_arrive(bar.boxFree(m));
        }
        __syncwarp();
      }
    }
    if (T == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  } else {
    // ---- epilogue warps: lane quadrant q = lane group q / 2, index 16 (q % 2) + 8 j + i = R set + k1; column half wh ----
    const int q = warp & 3, wh = (warp >> 2) & 1, j = warp >> 3, i = T >> 2, tq = T & 3, gq = q >> 1;
    const int set = (16 * (q & 1) + 8 * j + i) / R, k1 = (16 * (q & 1) + 8 * j + i) % R;
    // twiddles of an item's rows, fetched one item ahead: W_n^{64 k1 (4a + u)} and W_n^{k1 t2}
    float2 nA[4], nB0, nB1;
    auto fetch_tw = [&](int item) {
      const int a = (item / T2B) & 15, t2b = item % T2B;
#pragma unroll
      for (int u = 0; u < 4; ++u) nA[u] = __ldg(p.twr + 128 * k1 + 4 * a + u);
      nB0 = __ldg(p.twr + 128 * k1 + 64 + 4 * S * t2b + S * gq + set);
      nB1 = __ldg(p.twr + 128 * k1 + 64 + 4 * S * t2b + 2 * S + S * gq + set);
    };
    if ((int)blockIdx.x < nitems) fetch_tw(blockIdx.x);
    int it = 0;
    for (int item = blockIdx.x; item < nitems && ok; item += gridDim.x, ++it) {
      // One gate image with every 8th item (there are 8 items per image): its strided reads are issued
      // here and consumed after the item's epilogues, so their latency hides under them.
      const int sk = (int)blockIdx.x + (it >> 3) * (int)gridDim.x;
      const bool gate_item = (it & 7) == 0 && sk < p.cnt * R;
      float2 gvv[8];
      if (gate_item) {
        const float2* g = p.g + (size_t)(p.slab0 + sk / R) * p.K;
#pragma unroll
        for (int t = 0; t < 8; ++t) gvv[t] = gate_ext(g, sk % R + R * (tid + kXEpiThreads * t), p.n);
      }
      // sc W_n^{64 k1 (4a + u)} and W_n^{k1 t2} of this thread's k1 and this item's rows
      float2 wA[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) wA[u] = make_float2(nA[u].x * p.sc, nA[u].y * p.sc);
      const float2 wB0 = nB0, wB1 = nB1;
      if (item + (int)gridDim.x < nitems) fetch_tw(item + gridDim.x);
#pragma unroll 1
      for (int m = 0; m < 2 && ok; ++m) {
        unsigned char* box = reinterpret_cast<unsigned char*>(Stg) + 32768 * m;   // [tile (8)][k1 (R)][pair c4 (4)][t2 (2 S)][4 t1 = 16 bytes]
        const float2 wB = m ? wB1 : wB0;
        if (it > 0) ok = mbar_wait(bar.boxFree(m), (it - 1) & 1);   // the store that last read this box is done with it
        if (ok) ok = mbar_wait(bar.accFull(m), it & 1);
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
                *reinterpret_cast<uint4*>(box + (((4 * wh + x) * R + k1) * 4 + tq) * (32 * S) +
                                          16 * (S == 1 ? (gq ^ (k1 & 1)) : S * gq + set)) =        // R = 32: 32-byte swizzle of the box
                    make_uint4(chunk[x][0], chunk[x][1], chunk[x][2], chunk[x][3]);
            }
          }
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          mbar_arrive(bar.accFree(m));
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (T == 0) mbar_arrive(bar.boxFull(m));
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

// R = 32 ... 2.  A unit's result is 512 pieces of 128 bytes (8 row slots x 4 pairs; piece e2 holds rows
// t' / 64 = 2 (e2 % 32) + {0, 1}, s1 / 4 = e2 / 32, s1 % 4 = 0..3).  The 32 contracted rows of a lane group
// hold S = 32 / R sets of R rows k1: set s of accumulator m is piece e2 = 2 S blk + S m + s (one TMA box of
// R k1 x S pieces per lane group and tile), so an item covers 16 S values of t' and R output rows n1 for each.
template <bool F16, int R>
__global__ void __launch_bounds__(kXOutThreads, 1) tc_out32_kernel(const __grid_constant__ CUtensorMap tm_res,
                                                                  const __grid_constant__ CUtensorMap tm_out, const TcOut32Params p) {
  constexpr int S = 32 / R;
  static_assert(R == 32 || R == 16 || R == 8 || R == 4 || R == 2, "radix");
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* Op = smem;                                    // ring of four half-item slots
  unsigned char* Stg = smem + 2 * kXItemOp;                    // two boxes of [set (S)][t'l (8)][n1 (R)][128 bytes], swizzled
  unsigned char* Asm = smem + 2 * kXItemOp + 65536;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 2 * kXItemOp + 65536 + kXMat);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
  const int tid = threadIdx.x, warp = tid >> 5, T = tid & 31;
  const XBars bar(smem_u32(bars));

  if (tid == 0) {
    bar.init();
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
  const int nitems = p.cnt * (256 / S);                         // (S blocks of 16 consecutive row slots of every unit, slab)
  bool ok = (smem_u32(smem) & 1023u) == 0;                      // the swizzled boxes need 1024-byte aligned slots

  if (warp == kXEpiWarps) {
    // ---- MMA warp ----
    const uint32_t idesc = umma_idesc_x(0u);
    ok = mma_warp_loop(bar, nitems, T, ok, [&](int m, int slot) {
      issue_item_mmas(tmem + 256 * m, smem_u32(Asm), 1, smem_u32(Op) + slot * kXHalfOp, 4 * kXBox, kXBox, idesc);
    });
  } else if (warp == kXEpiWarps + 2) {
    // ---- load warp: per lane group and tile one box of S pieces x R k1 ----
    ok = load_warp_loop(bar, nitems, T, ok, [&](int item, int m, int slot) {
      const int slab_local = item % p.cnt, blk = item / p.cnt;
      for (int gq = 0; gq < 2; ++gq)
        for (int jb = 0; jb < 4; ++jb)
          tma_load_5d(smem_u32(Op) + slot * kXHalfOp + (gq * 4 + jb) * kXBox, &tm_res, 0, 0, 2 * S * blk + S * m, 4 * gq + jb, slab_local,
                      bar.slotFull(slot));
    });
  } else if (warp == kXEpiWarps + 1) {
    // ---- store warp: two TMA stores per filled box, the box is free once they have read it ----
    int it = 0;
    for (int item = blockIdx.x; item < nitems && ok; item += gridDim.x, ++it) {
      const int slab = p.slab0 + item % p.cnt, blk = item / p.cnt;
      const int b = slab / p.H, h = slab - b * p.H;
      for (int m = 0; m < 2 && ok; ++m) {
        ok = mbar_wait(bar.boxFull(m), it & 1);
        if (ok && T == 0) {
          for (int s = 0; s < S; ++s) {
            // box rows t'l = 0..3: t' = 64 row + 4 k4 + {0..3}; t'l = 4..7: the next t' / 64
            const int e2 = 2 * S * blk + S * m + s, k4 = e2 >> 5, row = 2 * (e2 & 31);
            const int tp = 64 * row + 4 * k4;
            const uint32_t src = smem_u32(Stg) + 32768 * m + s * (8 * R * 128);
            tma_store_5d(&tm_out, 0, 0, tp, h, b, src);
            tma_store_5d(&tm_out, 0, 0, tp + 64, h, b, src + 4 * R * 128);
          }
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          mbar_arrive(bar.boxFree(m));
        }
        __syncwarp();
      }
    }
    if (T == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  } else {
    // ---- epilogue warps: lane quadrant q: tiles 4 (q / 2) .. + 3, index 16 (q % 2) + 8 j + i = R set + n1; column half wh ----
    const int q = warp & 3, wh = (warp >> 2) & 1, j = warp >> 3, i = T >> 2, tq = T & 3, gq = q >> 1;
    const int set = (16 * (q & 1) + 8 * j + i) / R, n1 = (16 * (q & 1) + 8 * j + i) % R;
    bool bad = false;                                            // a non-finite result: the fp16 intermediates overflowed
    int it = 0;
    for (int item = blockIdx.x; item < nitems && ok; item += gridDim.x, ++it) {
#pragma unroll 1
      for (int m = 0; m < 2 && ok; ++m) {
        unsigned char* box = Stg + 32768 * m;
        if (it > 0) ok = mbar_wait(bar.boxFree(m), (it - 1) & 1);   // the stores that last read this box are done with it
        if (ok) ok = mbar_wait(bar.accFull(m), it & 1);
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
            unsigned char* pcol = box + (set * 8 * R + n1) * 128 + 4 * tq;          // + t'l R rows, + the swizzled 16-byte chunk
#pragma unroll
            for (int x = 0; x < 4; ++x) {                       // row slot t'l = 4 wh + x of the box, pair tq
              // rows (n1, C) and (n1, S) applied to the columns (re, im): y = (C re - S im) + j (S re + C im)
              const float ya = __uint_as_float(rr[4 * x]) - __uint_as_float(rr[4 * x + 3]);
              const float yb = __uint_as_float(rr[4 * x + 2]) + __uint_as_float(rr[4 * x + 1]);
              const uint32_t yo = F16 ? pack_h2(ya, yb) : pack_bf2(ya, yb);
              if (x == 0) bad |= nonfinite16x2<F16>(yo);       // every row of an overflowed column is non-finite: one row is enough
              const int srow = (4 * wh + x) * R + n1;                      // row of the set's block: the swizzle key is row % 8
              *reinterpret_cast<uint32_t*>(pcol + (4 * wh + x) * (R * 128) + (((4 * gq + jb) ^ (srow & 7)) * 16)) = yo;
            }
          }
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          mbar_arrive(bar.accFree(m));
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (T == 0) mbar_arrive(bar.boxFull(m));
        }
      }
    }
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
// Shapes the tensor-core transpose kernels take: n = 4096 R with R = 32, 16 or 8, 64 channels per head (one
// 128-byte line per row and head), whole 4096-row blocks, 16-byte aligned strides.
bool tc32_supported(const spectre_ctx* ctx, const spectre_act* v, const spectre_act* y, int n) {
  auto ok = [](const spectre_act* a) {
    return (reinterpret_cast<uintptr_t>(a->ptr) & 15) == 0 && a->stride_l % 8 == 0 && a->stride_h % 8 == 0 &&
           a->stride_b % 8 == 0 && a->stride_l > 0 && a->stride_h > 0 && a->stride_b > 0;
  };
  return n >= 8192 && n <= 131072 && (n & (n - 1)) == 0 && v->D == 64 && v->L % 4096 == 0 && ok(v) && ok(y) && ctx->dft32 != nullptr &&
         ctx->tw_staged != nullptr && tensor_map_encoder() != nullptr;
}

// dims (column, n1, t', head, batch) over [B, L, H, 64]: row = 4096 n1 + t'
static int make_act_map(CUtensorMap* tm, const spectre_act* a, unsigned box_n1, unsigned box_tp) {
  const cuuint64_t sl = (cuuint64_t)a->stride_l * 2, sh = (cuuint64_t)a->stride_h * 2, sb = (cuuint64_t)a->stride_b * 2;
  const cuuint64_t nb = (cuuint64_t)(a->L / 4096);
  cuuint64_t dims[5] = {64, nb, 4096, (cuuint64_t)a->H, (cuuint64_t)a->B};
  cuuint64_t strides[4] = {4096 * sl, sl, sh, sb};
  cuuint32_t box[5] = {64, box_n1, box_tp, 1, 1};
  cuuint32_t es[5] = {1, 1, 1, 1, 1};
  CUresult r = tensor_map_encoder()(tm, a->dtype == SPECTRE_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, a->ptr,
                             dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(SPECTRE_ERR_CUDA, "cuTensorMapEncodeTiled failed (" + std::to_string((int)r) + ")");
  return SPECTRE_OK;
}

static int radix_index(int R) { return R == 32 ? 0 : (R == 16 ? 1 : (R == 8 ? 2 : (R == 4 ? 3 : 4))); }   // order of the matrix sets in the context

template <int R>
static int launch_tc_in_r(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, const float* g, int n, int slab0, int cnt,
                          unsigned char* ws_in, unsigned char* gimg, float* gscale, float sc) {
  constexpr int S = 32 / R;
  CUtensorMap tm;
  int rc = make_act_map(&tm, v, R, S == 1 ? 2 : S);
  if (rc != SPECTRE_OK) return rc;
  CUtensorMap tm_img;
  {
    // the operand images as fp16: (t2 x 4 t1 of one pair and K group: 1024 bytes; 4 a + c4; slab * R + k1; tile)
    cuuint64_t dims[4] = {512, 64, (cuuint64_t)cnt * R, 8};
    cuuint64_t strides[3] = {1024, 8 * (cuuint64_t)kXImgBytes, (cuuint64_t)kXImgBytes};
    cuuint32_t box[4] = {16 * S, 4, R, 8};
    cuuint32_t es[4] = {1, 1, 1, 1};
    CUresult r = tensor_map_encoder()(&tm_img, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, ws_in, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                               S == 1 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(SPECTRE_ERR_CUDA, "cuTensorMapEncodeTiled failed (" + std::to_string((int)r) + ")");
  }
  TcIn32Params p = {};
  p.mats = reinterpret_cast<const unsigned char*>(ctx->dft32) + (size_t)radix_index(R) * 4 * kXMat;
  p.twr = reinterpret_cast<const float2*>(ctx->tw_staged) + (size_t)(R - 1) * 128;
  p.ws_in = ws_in; p.g = reinterpret_cast<const float2*>(g); p.gimg = gimg; p.gscale = gscale;
  p.H = v->H; p.slab0 = slab0; p.cnt = cnt; p.n = n; p.K = n / 2 + 1; p.sc = sc;
  p.status = ctx->status_dev;
  const int nitems = cnt * (256 / S);
  int grid = nitems < ctx->sm_count ? nitems : ctx->sm_count;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kXInThreads); cfg.dynamicSmemBytes = kXInSmem; cfg.stream = st;
  cfg.attrs = attr; cfg.numAttrs = 1;
  if (v->dtype == SPECTRE_F16) {
    SPECTRE_CUDA_OK(cudaFuncSetAttribute(tc_in32_kernel<true, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, kXInSmem));
    SPECTRE_CUDA_OK(cudaLaunchKernelEx(&cfg, tc_in32_kernel<true, R>, tm, tm_img, p));
  } else {
    SPECTRE_CUDA_OK(cudaFuncSetAttribute(tc_in32_kernel<false, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, kXInSmem));
    SPECTRE_CUDA_OK(cudaLaunchKernelEx(&cfg, tc_in32_kernel<false, R>, tm, tm_img, p));
  }
  SPECTRE_LAUNCH_OK("tc_in32_kernel");
  return SPECTRE_OK;
}

int launch_tc_in32(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, const float* g, int n, int slab0, int cnt,
                   unsigned char* ws_in, unsigned char* gimg, float* gscale, float sc) {
  switch (n / 4096) {
    case 32: return launch_tc_in_r<32>(ctx, st, v, g, n, slab0, cnt, ws_in, gimg, gscale, sc);
    case 16: return launch_tc_in_r<16>(ctx, st, v, g, n, slab0, cnt, ws_in, gimg, gscale, sc);
    case 8: return launch_tc_in_r<8>(ctx, st, v, g, n, slab0, cnt, ws_in, gimg, gscale, sc);
    case 4: return launch_tc_in_r<4>(ctx, st, v, g, n, slab0, cnt, ws_in, gimg, gscale, sc);
    case 2: return launch_tc_in_r<2>(ctx, st, v, g, n, slab0, cnt, ws_in, gimg, gscale, sc);
    default: return fail(SPECTRE_ERR_UNSUPPORTED, "radix not supported by the tensor-core transpose kernels");
  }
}

template <int R>
static int launch_tc_out_r(const spectre_ctx* ctx, cudaStream_t st, const unsigned char* ws_out, const spectre_act* y, int slab0, int cnt) {
  constexpr int S = 32 / R;
  CUtensorMap tm_res, tm_out;
  int rc = make_act_map(&tm_out, y, R, 4);
  if (rc != SPECTRE_OK) return rc;
  {
    // the units' results as fp16: (128-byte piece, k1, piece index within the unit, tile, slab of the group)
    cuuint64_t dims[5] = {64, R, 512, 8, (cuuint64_t)cnt};
    cuuint64_t strides[4] = {8 * (cuuint64_t)kXOutBytes, 128, (cuuint64_t)kXOutBytes, 8 * R * (cuuint64_t)kXOutBytes};
    cuuint32_t box[5] = {64, R, S, 1, 1};
    cuuint32_t es[5] = {1, 1, 1, 1, 1};
    CUresult r = tensor_map_encoder()(&tm_res, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 5, const_cast<unsigned char*>(ws_out), dims, strides, box, es,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(SPECTRE_ERR_CUDA, "cuTensorMapEncodeTiled failed (" + std::to_string((int)r) + ")");
  }
  TcOut32Params p = {};
  p.mats = reinterpret_cast<const unsigned char*>(ctx->dft32) + (size_t)radix_index(R) * 4 * kXMat;
  p.H = y->H; p.slab0 = slab0; p.cnt = cnt; p.status = ctx->status_dev;
  const int nitems = cnt * (256 / S);
  int grid = nitems < ctx->sm_count ? nitems : ctx->sm_count;
  if (y->dtype == SPECTRE_F16) {
    SPECTRE_CUDA_OK(cudaFuncSetAttribute(tc_out32_kernel<true, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, kXOutSmem));
    tc_out32_kernel<true, R><<<grid, kXOutThreads, kXOutSmem, st>>>(tm_res, tm_out, p);
  } else {
    SPECTRE_CUDA_OK(cudaFuncSetAttribute(tc_out32_kernel<false, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, kXOutSmem));
    tc_out32_kernel<false, R><<<grid, kXOutThreads, kXOutSmem, st>>>(tm_res, tm_out, p);
  }
  SPECTRE_LAUNCH_OK("tc_out32_kernel");
  return SPECTRE_OK;
}

int launch_tc_out32(const spectre_ctx* ctx, cudaStream_t st, const unsigned char* ws_out, const spectre_act* y, int n, int slab0, int cnt) {
  switch (n / 4096) {
    case 32: return launch_tc_out_r<32>(ctx, st, ws_out, y, slab0, cnt);
    case 16: return launch_tc_out_r<16>(ctx, st, ws_out, y, slab0, cnt);
    case 8: return launch_tc_out_r<8>(ctx, st, ws_out, y, slab0, cnt);
    case 4: return launch_tc_out_r<4>(ctx, st, ws_out, y, slab0, cnt);
    case 2: return launch_tc_out_r<2>(ctx, st, ws_out, y, slab0, cnt);
    default: return fail(SPECTRE_ERR_UNSUPPORTED, "radix not supported by the tensor-core transpose kernels");
  }
}

}  // namespace spectre
