// Tensor-core spectral mixer for n = 4096 * R, R in {1, 2, 4, 8, 16, 32}, bf16 or fp16 I/O
// (Sec. 3.2 steps 2 and 4; covers n = 4096 ... 131072).
//
// Four-step split n = R * 4096 with t = n1 * 4096 + t', k = k1 + R * kM:
//
//   tc_in_kernel    reads whole 128-byte rows of [B, L, H, D] (coalesced), does the radix-R
//                   DFT over n1 and the twiddle W_n^{k1 t'} on the ALUs, rounds to fp16 and
//                   writes, for every unit (head, k1, 4 column pairs), the first tensor-core
//                   operand as an image of its shared-memory layout (transposed through
//                   shared memory so that the workspace writes are whole lines too)
//   (gate images)   per (head, k1): the 4096 gate values the unit needs (Hermitian extension,
//                   normalised by their maximum, fp16) in the order the core reads them; written by
//                   the first CTAs of the tc_in_kernel launch
//   tc_core_kernel  persistent, one CTA per SM, units taken in pairs: 16 epilogue warps alternate
//                   between the two units while a producer warp fetches the operand images with
//                   bulk async copies and issues the MMAs (64-point DFT matrix as the A operand,
//                   see mixer_tc.cu for the formulation), so one unit's epilogue on the ALUs
//                   overlaps the other unit's stage on the tensor core; 4 x [MMA -> epilogue] per
//                   unit.  Result: the unit's 4096 x 4 complex outputs in fp16, tile-major
//   tc_out_kernel   inverse radix-R over k1 with conj twiddles, 1/n and gate scale, bf16,
//                   transposed through shared memory into whole-row stores
//
// Heads are processed in groups sized by the workspace (operand images + unit results + gate
// images per head); larger groups measured faster than groups small enough to stay in L2.
#include <cuda_fp16.h>

#include "tc_stage.cuh"

namespace spectre {

// ---- shared with mixer_tc.cu (same conventions) ------------------------------------
constexpr int k4Lbo = 4096, k4Sbo = 128;         // every operand image of the core is dense: 4096 bytes between K groups, 128 between 8-column groups
constexpr int k4BBytes = 16 * k4Lbo;             // one 256-column operand buffer
constexpr int k4ImgBytes = k4BBytes;             // stage-0 operand image in the workspace (columns 64 c + t2, K = t1)
constexpr int k4FBytes = 128 * 128 * 2;
constexpr int k4GBytes = 4096 * 4;               // gate table: bin kM = k1 + 64 k2 at 64 k2 + (k1 ^ 8 (k2 % 4)), fp16 (re, im)
constexpr int k4OutBytes = 4096 * 4 * 4;         // unit result: [unit_row_slot(t')][4 pairs] half2
constexpr int k4EpiWarps = 8;                    // 2 per TMEM lane quadrant, one column half each
constexpr int k4EpiThreads = 32 * k4EpiWarps;
constexpr int k4CoreThreads = k4EpiThreads + 32;    // + producer / MMA-issuing warp
constexpr int k4CoreSmem = k4FBytes + k4BBytes + k4GBytes + 64;
static_assert(2 * (k4CoreSmem + 1024) <= 233472, "two core CTAs per SM");

// XOR skew of the low five bits of a staged word's index: the 8 tiles x 4 pairs a warp writes at once
// land in 32 different banks
__device__ __forceinline__ int stage_skew(int tile, int c4) { return (tile & 7) | (c4 << 3); }

// forward-scale of the radix-R step (keeps fp16 magnitudes near the input's)
__host__ __device__ constexpr float in_scale(int R) {
  return R <= 2 ? 1.0f : (R <= 8 ? 0.5f : (R == 16 ? 0.25f : 0.125f));
}

// Twiddles of the four-step split for every supported R: row R - 1 + k1 (k1 < R) holds W_n^{64 k1 t1} for
// t1 < 64 and then W_n^{k1 t2} for t2 < 64, n = 4096 R (angles reduced in integers).
__global__ void build_tw_staged_kernel(float2* tab) {
  const int row = blockIdx.x, e = threadIdx.x;                 // 63 rows x 128 entries
  int R = 1;
  while (2 * R - 1 <= row) R *= 2;
  const int k1 = row - (R - 1);
  const unsigned n = 4096u * (unsigned)R;
  const unsigned m = e < 64 ? (64u * (unsigned)k1 * (unsigned)e) % n : ((unsigned)k1 * (unsigned)(e - 64)) % n;
  tab[row * 128 + e] = twiddle_fwd(m, n);
}
int build_tw_staged(float2* tab, cudaStream_t st) {
  build_tw_staged_kernel<<<63, 128, 0, st>>>(tab);
  SPECTRE_LAUNCH_OK("build_tw_staged_kernel");
  return SPECTRE_OK;
}

// =====================================================================================
// gate images: per (head, k1) the 4096 gate values the unit needs (Hermitian extension, normalised
// by their maximum, fp16) in the order the core reads them.  Runs as the first CTAs of the
// transpose-in launch (it depends on the gate only, the other CTAs on the activations only), so its
// strided reads fill the gaps of that kernel instead of standing alone in the stream.
// =====================================================================================
struct TcGateParams {
  const float2* g;          // [B*H][K]
  unsigned char* gimg;      // [slab_local * R + k1][k4GBytes]
  float* gscale;            // [slab_local * R + k1]
  int n, K, R, slab0;
};

// vals: 4096 float2 of shared memory
__device__ __forceinline__ void tc_gate_body(const TcGateParams& p, int sk, float2* vals) {
  __shared__ float red[8];
  const int slab_local = sk / p.R, k1 = sk - slab_local * p.R;
  const float2* g = p.g + (size_t)(p.slab0 + slab_local) * p.K;
  float m = 0.f;
  float2 gv[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) {                                 // 16 strided loads in flight per thread
    const int k = k1 + p.R * (threadIdx.x + 256 * i);
    const int kk = (2 * k <= p.n) ? k : p.n - k;
    float2 v = __ldg(g + kk);
    if (kk != k) v.y = -v.y;
    if (k == 0 || 2 * k == p.n) v.y = 0.f;
    gv[i] = v;
  }
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    vals[threadIdx.x + 256 * i] = gv[i];
    m = fmaxf(m, fmaxf(fabsf(gv[i].x), fabsf(gv[i].y)));
  }
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  m = 0.f;
  for (int i = 0; i < 8; ++i) m = fmaxf(m, red[i]);
  m *= 1.41421356f;
  const float inv = m > 0.f ? 1.0f / m : 0.f;
  if (threadIdx.x == 0) p.gscale[sk] = m;
  uint32_t* img = reinterpret_cast<uint32_t*>(p.gimg + (size_t)sk * k4GBytes);
  for (int idx = threadIdx.x; idx < 4096; idx += 256) {
    const int k2 = idx >> 6, k1 = idx & 63;                            // kM = k1 + 64 k2
    const float2 gv2 = vals[idx];
    img[64 * k2 + (k1 ^ (8 * (k2 & 3)))] = pack_h2(gv2.x * inv, gv2.y * inv);
  }
}

// =====================================================================================
// transpose-in
// =====================================================================================
struct TcInParams {
  const bf16* src;
  int64_t s_sb, s_sl, s_sh;
  unsigned char* ws_in;       // [unit][k4ImgBytes]
  int H, D, L, n, ntile, slab0;
};

// CTA = (slab, group of 4 consecutive t1, block of NT2 values of t2); t' = 64 t1 + t2.
// A warp takes one (t1, t2) at a time with lane = column pair; staging holds, for every
// (k1, tile), the core matrices (8 operand columns x 16 bytes) of this CTA's slice.
// The first ngate CTAs write the gate images (tc_gate_body) instead.
template <int R, bool F16>
__global__ void __launch_bounds__(256, 3) tc_in_kernel(const TcInParams p, const TcGateParams gp, int ngate) {
  constexpr int NT2 = (R <= 2) ? 64 : 128 / R;
  constexpr int UNR = R <= 2 ? 4 : (R <= 8 ? 2 : 1);          // row sets in flight per warp
  extern __shared__ __align__(128) uint32_t stage[];          // [R][ntile][4 pairs][NT2][4 t1] words (skewed); >= 32 KB
  asm volatile("griddepcontrol.wait;" ::: "memory");          // launched as a programmatic dependent
  if ((int)blockIdx.x < ngate) {
    tc_gate_body(gp, (int)blockIdx.x, reinterpret_cast<float2*>(stage));
    return;
  }
  const int t2blocks = 64 / NT2;
  int u = (int)blockIdx.x - ngate;
  const int t2b = u % t2blocks;  u /= t2blocks;
  const int t1g = u % 16;  u /= 16;
  const int slab_local = u, slab = p.slab0 + u;
  const int b = slab / p.H, h = slab - b * p.H;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int npair = p.D / 2;
  const bf16* src = p.src + b * p.s_sb + h * p.s_sh;
  const float sc = in_scale(R);
  // W_n^{t'} of this CTA's 4 NT2 values of t', once (index = row set)
  __shared__ float2 tws[4 * NT2];
  for (int rs = threadIdx.x; rs < 4 * NT2; rs += 256)
    tws[rs] = twiddle_fwd((unsigned)(64 * (4 * t1g + (rs & 3)) + t2b * NT2 + (rs >> 2)), (unsigned)p.n);
  __syncthreads();

  for (int cb = 0; cb < npair; cb += 32) {                     // column blocks of 32 pairs (D = 64: one)
    const int c = cb + lane;
    const bool live = c < npair;
    const int tile = c >> 2, c4 = c & 3;
#pragma unroll UNR
    for (int rs = warp; rs < 4 * NT2; rs += 8) {
      const int t1m = rs & 3, t2l = rs >> 2;
      const int tp = 64 * (4 * t1g + t1m) + t2b * NT2 + t2l;
      // rows n1 * 4096 + t' are a constant stride apart; rows >= L read as zero
      const uint32_t* pl = reinterpret_cast<const uint32_t*>(src + (int64_t)tp * p.s_sl + 2 * c);
      const int64_t lstride = 2048 * p.s_sl;                     // 4096 rows, in 32-bit words
      const int nvalid = live ? (p.L - tp + 4095) >> 12 : 0;     // number of n1 with a row below L
      float2 x[R];
#pragma unroll
      for (int n1 = 0; n1 < R; ++n1) {
        const uint32_t v = n1 < nvalid ? __ldg(pl + n1 * lstride) : 0u;
        x[n1] = F16 ? unpack_h2(v) : make_float2(__uint_as_float(v << 16), __uint_as_float(v & 0xffff0000u));
      }
      Dft<R, false>::run(x);
      const float2 w1 = tws[rs];
      if (live) {
        // word of the unit's slice [c4][t2][t1 % 4], XOR-skewed in its low five bits
        const int wl = ((c4 * NT2 + t2l) * 4 + t1m) ^ stage_skew(tile, c4);
        uint32_t* ps = stage + tile * (16 * NT2) + wl;
        const int sstride = p.ntile * (16 * NT2);                  // words between consecutive k1
        float2 w = make_float2(sc, 0.f);                          // sc * W_n^{k1 t'}
#pragma unroll
        for (int k1 = 0; k1 < R; ++k1) {
          const float2 v = cmul(x[k1], w);
          ps[k1 * sstride] = pack_h2(v.x, v.y);
          w = cmul(w, w1);
        }
      }
    }
  }
  __syncthreads();
  // copy out: per (k1, tile) unit and pair c4 the CTA holds NT2 consecutive t2 x 4 t1 = NT2 16-byte
  // chunks, contiguous in the unit's image (column 64 c4 + t2, K group t1g).  The skew permutes the
  // words inside a chunk (low two bits) and the chunks among their neighbours (next three bits).
  unsigned char* img0 = p.ws_in + (size_t)slab_local * R * p.ntile * k4ImgBytes + (size_t)t1g * k8Lbo0 +
                        (size_t)(t2b * NT2) * 16;
  const bool pow2 = (p.ntile & (p.ntile - 1)) == 0;
  const int nchunk = R * p.ntile * 4 * NT2;
  for (int idx = threadIdx.x; idx < nchunk; idx += 256) {
    const int lc = idx & (4 * NT2 - 1), ut = idx / (4 * NT2);        // logical chunk c4 * NT2 + t2l; ut = k1 * ntile + tile
    const int c4 = lc / NT2, t2l = lc - c4 * NT2;
    const int tile = pow2 ? (ut & (p.ntile - 1)) : (ut % p.ntile);
    const int sk = stage_skew(tile, c4);
    const uint4 v = *reinterpret_cast<const uint4*>(stage + ut * (16 * NT2) + ((lc ^ (sk >> 2)) << 2));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint4 o;
    o.x = w[0 ^ (sk & 3)]; o.y = w[1 ^ (sk & 3)]; o.z = w[2 ^ (sk & 3)]; o.w = w[3 ^ (sk & 3)];
    *reinterpret_cast<uint4*>(img0 + (size_t)ut * k4ImgBytes + c4 * 1024 + t2l * 16) = o;
  }
}

// =====================================================================================
// core: 4096-point units on the tensor cores
// =====================================================================================
struct TcCoreParams {
  const unsigned char* ws_in;
  const unsigned char* gimg;
  unsigned char* ws_out;
  const __half* F;
  const float2* tw64;       // stage twiddles W_4096^{row d} (even d) in epilogue order
  const float2* twr;        // [R][128]: W_n^{64 k1 t1}, W_n^{k1 t2} (the rows of this R in the context's table)
  const float* gscale;      // [slab_local * R + k1] gate scale of the unit's (head, k1)
  float out_scale;          // 1 / (R * forward scale of the radix-R step)
  int nunits, ntile, R;
  int* status;
  int first_stage;          // 0: whole units.  2: the images are third-stage operands (gated spectra, see
                            // tc_spec_in_kernel): only the two inverse stages run, no gate table is read
};

// Where row t' of a unit's result lies, in 16-byte units (the four pairs of a row stay together): rows
// are ordered (s1 / 4, t' / 64, s1 % 4) with s1 = t' % 64, the order in which the core's last epilogue
// holds them (8 lanes = 8 values of t' / 64, 4 lanes = 4 values of s1 % 4), so one of its store
// instructions writes 512 contiguous bytes.
__host__ __device__ __forceinline__ int unit_row_slot(int tp) {
  const int row = tp >> 6, s1 = tp & 63;
  return ((s1 >> 2) * 64 + row) * 4 + (s1 & 3);
}

// Last epilogue of a unit for one warp (TMEM lane quadrant q, column half ch): the accumulator has rows
// s2 and columns 16 (s1 / 4) + 8 (c / 2) + 2 (s1 % 4) + c % 2 (tc_stage.cuh, COLS = 2): D = the inverse
// stages' conj(FFT(conj(.))) of the unit at t' = 64 row + s1, all four pairs of two values of s1 per
// 32-column chunk in one thread.  What leaves is ready for the inverse radix-R step over k1:
// conj(D W_n^{k1 t'}) times the gate scale and 1 / (R s_in), as half2 [unit_row_slot(t')][pair], one
// 16-byte store per row.  tw = this k1's 128 table entries.  TMEM loads run one chunk ahead.
__device__ __forceinline__ void core_store(uint32_t tmem_d, unsigned char* out, int q, int ch, int T,
                                           const float2* __restrict__ tw, float gsc) {
  const int i = T >> 2, tq = T & 3;
  float2 fa[2], fb[8];
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const float2 t = __ldg(tw + 8 * (2 * q + j) + i);
    fa[j] = make_float2(t.x * gsc, t.y * gsc);
  }
#pragma unroll
  for (int k = 0; k < 8; ++k) fb[k] = __ldg(tw + 64 + 4 * (8 * ch + k) + tq);   // s1 = 4 (8 ch + k) + tq
  uint32_t r[2][16];
  const uint32_t taddr0 = tmem_d + ((uint32_t)(32 * q) << 16) + 128 * ch;
  tmem_ld_16x256b_x4(taddr0, r[0]);
#pragma unroll
  for (int step = 0; step < 8; ++step) {                        // step = 2 cc + j: columns 128 ch + 32 cc .. + 31
    const int cc = step >> 1, j = step & 1;
    const int row = 8 * (2 * q + j) + i;
    tmem_ld_wait();
    if (step < 7) {
      const int ns = step + 1;
      tmem_ld_16x256b_x4(taddr0 + ((uint32_t)(16 * (ns & 1)) << 16) + 32 * (ns >> 1), r[ns & 1]);
    }
    const uint32_t (&rr)[16] = r[step & 1];
#pragma unroll
    for (int s = 0; s < 2; ++s) {                               // s1 / 4 = 8 ch + 2 cc + s; 8-column groups 2 s, 2 s + 1 = pairs 0-1, 2-3
      // conj(D w) = D conj-multiplied: (re, -im) of D w, with the sign folded into the second factor
      const float2 w = cmul(fa[j], fb[2 * cc + s]);
      const uint64_t WX = pk2(w.x, w.x), WYn = pk2(-w.y, -w.y);
      uint2 o[2];
#pragma unroll
      for (int e2 = 0; e2 < 2; ++e2) {                          // pairs 2 e2, 2 e2 + 1: 8-column group 2 s + e2
        const int b0 = 4 * (2 * s + e2);
        const uint64_t RE = pk2u(rr[b0], rr[b0 + 1]), IM = pk2u(rr[b0 + 2], rr[b0 + 3]);
        // D w = (re w.x - im w.y) + j (re w.y + im w.x); stored: (real, -imag)
        const uint64_t X = fma2(IM, WYn, mul2(RE, WX));
        const uint64_t Yn = sub2(mul2(RE, WYn), mul2(IM, WX));
        float x0, x1, y0, y1;
        upk2(X, x0, x1);
        upk2(Yn, y0, y1);
        o[e2] = make_uint2(pack_h2(x0, y0), pack_h2(x1, y1));
      }
      const int k = 8 * ch + 2 * cc + s;                        // s1 / 4
      *reinterpret_cast<uint4*>(out + (size_t)((k * 64 + row) * 4 + tq) * 16) = make_uint4(o[0].x, o[0].y, o[1].x, o[1].y);
    }
  }
}

// Persistent, two CTAs per SM (112 KB of shared memory, 256 TMEM columns, 8 epilogue warps + 1 warp that
// fetches and issues).  A CTA works through a contiguous range of units, one at a time: operand image
// (64 KB, one bulk copy) and, when the (head, k1) changes, the gate table (16 KB) -> 4 x [MMA -> epilogue]
// in place on one operand buffer -> result to the workspace.  The next unit's image is fetched as soon
// as the last MMAs of the current one have read the buffer, under the last epilogue.  One CTA's MMAs and
// copies run under the other CTA's epilogues.  (Splitting a unit into two 128-column halves that
// ping-pong inside the CTA measured slower: an MMA of N = 128 re-reads the DFT matrix per half and the
// stage becomes bound by shared-memory reads.)
//   barL  operand image (+ gate table) landed (transaction count)       1 phase per unit
//   barD  the stage's MMAs completed                                     4 phases per unit
//   barB  all epilogue threads done with the stage: next operand written (stages 0-2) or the
//         accumulator drained (stage 3)                                  4 phases per unit
// Operand images (tc_stage.cuh): stages 0-2 have columns 64 c + digit, the last operand has columns
// 16 (s1 / 4) + 8 (c / 2) + 2 (s1 % 4) + c % 2.
__global__ void __launch_bounds__(k4CoreThreads, 2) tc_core_kernel(const TcCoreParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* Fsm = smem;
  unsigned char* Bsm = smem + k4FBytes;
  uint32_t* Gsm = reinterpret_cast<uint32_t*>(smem + k4FBytes + k4BBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + k4FBytes + k4BBytes + k4GBytes);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 6);
  const int tid = threadIdx.x, warp = tid >> 5, T = tid & 31;
  const uint32_t barL = smem_u32(&bars[0]);
  const uint32_t barD = smem_u32(&bars[1]), barB = smem_u32(&bars[2]);

  if (warp == k4EpiWarps) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(tmem_slot)), "r"(256));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  if (tid == 0) {
    mbar_init(barL, 1);
    mbar_init(barD, 1);
    mbar_init(barB, k4EpiThreads);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < k4EpiThreads) {
    const uint4* Fg = reinterpret_cast<const uint4*>(p.F);
    for (int i = tid; i < k4FBytes / 16; i += k4EpiThreads) reinterpret_cast<uint4*>(Fsm)[i] = __ldg(Fg + i);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *tmem_slot;
  // this CTA's units: a contiguous range, so that consecutive units mostly share the gate table
  const int per = (p.nunits + (int)gridDim.x - 1) / (int)gridDim.x;
  const int u0 = (int)blockIdx.x * per, u1 = min(p.nunits, u0 + per);
  bool ok = true;

  if (warp == k4EpiWarps) {
    // ---- producer + MMA issuer ----
    const uint32_t idesc = umma_idesc_128x256();
    auto fetch = [&](int unit) {
      const bool new_gate = p.first_stage == 0 && (unit == u0 || unit / p.ntile != (unit - 1) / p.ntile);
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(barL), "r"(k4ImgBytes + (new_gate ? k4GBytes : 0)) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   :: "r"(smem_u32(Bsm)), "l"(p.ws_in + (size_t)unit * k4ImgBytes), "r"(k4ImgBytes), "r"(barL) : "memory");
      if (new_gate)
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     :: "r"(smem_u32(Gsm)), "l"(p.gimg + (size_t)(unit / p.ntile) * k4GBytes), "r"(k4GBytes), "r"(barL) : "memory");
    };
    if (T == 0 && u0 < u1) fetch(u0);
    __syncwarp();
    for (int unit = u0, it = 0; unit < u1 && ok; ++unit, ++it) {
      for (int stage = p.first_stage; stage < 4 && ok; ++stage) {
        if (stage == p.first_stage) {
          ok = mbar_wait(barL, it & 1);                         // operand landed
          if (ok && it > 0) ok = mbar_wait(barB, 1);            // previous result has left TMEM
        } else {
          ok = mbar_wait(barB, (stage - 1) & 1);
        }
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (T == 0) {
          const uint32_t a0 = smem_u32(Fsm), b0 = smem_u32(Bsm);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint64_t da = umma_desc(a0 + ks * 256, 128, 2048);
            const uint64_t db = umma_desc(b0 + ks * 2 * k4Lbo, k4Lbo, k4Sbo);
            const uint32_t acc = ks > 0;
            asm volatile(
                "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                :: "r"(tmem), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
          }
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(barD) : "memory");
        }
        __syncwarp();
      }
      // the operand buffer is free once the last MMAs completed: fetch the next unit under the last epilogues
      if (ok && unit + 1 < u1) {
        ok = mbar_wait(barD, 1);
        if (ok && T == 0) fetch(unit + 1);
        __syncwarp();
      }
    }
    if (!ok) mbar_wait(barL, 0);                                // do not leave with a copy into this CTA still in flight
  } else {
    // ---- epilogue warps: quadrant q, the two 64-column quarters of column half wh ----
    const int q = warp & 3, wh = warp >> 2;
    // W_4096^{row} of this thread's two accumulator rows (8 (2q + j) + T / 4): odd columns' stage twiddles
    const float2* twh = p.tw64;
    const float2 wr0 = twiddle_fwd((unsigned)(16 * q + (T >> 2)), 4096u), wr1 = twiddle_fwd((unsigned)(16 * q + 8 + (T >> 2)), 4096u);
    for (int unit = u0; unit < u1 && ok; ++unit) {
#pragma unroll 1
      for (int stage = p.first_stage; stage < 4 && ok; ++stage) {
        ok = mbar_wait(barD, stage & 1);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (stage == 3) {
          const int gi = unit / p.ntile;                         // slab_local * R + k1
          core_store(tmem, p.ws_out + (size_t)unit * k4OutBytes, q, wh, T, p.twr + 128 * (gi % p.R),
                     __ldg(p.gscale + gi) * p.out_scale);
        } else {
          if (stage == 0) epilogue_twiddle2<k4Lbo, k4Sbo, 1>(tmem, Bsm, q, 2 * wh, T, twh, wr0, wr1);
          else if (stage == 2) epilogue_twiddle2<k4Lbo, k4Sbo, 2>(tmem, Bsm, q, 2 * wh, T, twh, wr0, wr1);
          else {
#pragma unroll 1
            for (int cc = 0; cc < 2; ++cc) epilogue_gate_t<k4Lbo, k4Sbo, 64, true>(tmem, Bsm, q, 2 * wh + cc, T, Gsm);
          }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive(barB);
      }
    }
  }
  if (!ok && T == 0) report_timeout(p.status);
  __syncwarp();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == k4EpiWarps) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(256));
  }
}

// =====================================================================================
// transpose-out
// =====================================================================================
struct TcOutParams {
  const unsigned char* ws_out;   // [unit][unit_row_slot(t')][4] half2
  bf16* dst;
  int64_t d_sb, d_sl, d_sh;
  int H, D, L, n, ntile, slab0;
  int* status;
};

// CTA = (slab, block of NT consecutive t'); rows n1 * 4096 + t' for all n1 are produced.  The units'
// results arrive ready for the inverse radix-R step (conjugated, scaled, times conj(W_n^{k1 t'})).
template <int R, bool F16>
__global__ void __launch_bounds__(256, 3) tc_out_kernel(const TcOutParams p) {
  constexpr int NT = 512 / R;
  extern __shared__ __align__(128) uint32_t stage[];            // [R][NT][D/2 words]
  const int nblk = 4096 / NT;
  const int tb = blockIdx.x % nblk, slab_local = blockIdx.x / nblk, slab = p.slab0 + slab_local;
  const int b = slab / p.H, h = slab - b * p.H;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t8 = lane >> 2, c4 = lane & 3;
  const int npair = p.D / 2;
  const int skew_mask = (p.ntile & (p.ntile - 1)) == 0 ? min(p.ntile, 8) - 1 : 0;   // XOR stays inside the row

  // phase 1: a warp takes (tile, 8 consecutive t'); lane = (t' % 8, pair within the tile)
  const int nitems = p.ntile * (NT / 8);
  bool bad = false;                                             // a non-finite result: the fp16 intermediates overflowed
  const uint32_t* wsl = reinterpret_cast<const uint32_t*>(p.ws_out + (size_t)slab_local * R * p.ntile * k4OutBytes);
  const int ustride = p.ntile * (k4OutBytes / 4);               // words between consecutive k1 (same tile)
  // the 4-byte loads of UN items (R each) are issued before the first butterfly: short radices alone leave
  // too few bytes in flight per SM
  constexpr int UN = R >= 16 ? 1 : (R == 8 ? 2 : 4);
  for (int item0 = warp; item0 < nitems; item0 += 8 * UN) {
    uint32_t raw[UN][R];
#pragma unroll
    for (int u = 0; u < UN; ++u) {
      const int item = item0 + 8 * u;
      if (item < nitems) {
        const int tile = item % p.ntile, tl = (item / p.ntile) * 8 + t8;
        const uint32_t* pu = wsl + tile * (k4OutBytes / 4) + unit_row_slot(tb * NT + tl) * 4 + c4;
#pragma unroll
        for (int k1 = 0; k1 < R; ++k1) raw[u][k1] = __ldg(pu + k1 * ustride);   // scaled and twiddled by the core
      }
    }
#pragma unroll
    for (int u = 0; u < UN; ++u) {
      const int item = item0 + 8 * u;
      if (item >= nitems) break;
      const int tile = item % p.ntile, tl = (item / p.ntile) * 8 + t8;
      float2 x[R];
#pragma unroll
      for (int k1 = 0; k1 < R; ++k1) x[k1] = unpack_h2(raw[u][k1]);
      Dft<R, true>::run(x);
      const int word = (tile * 4 + c4) ^ ((tl & skew_mask) << 2);   // skew: the 8 rows of a warp hit 8 bank groups
      uint32_t* ps = stage + tl * npair + word;
#pragma unroll
      for (int n1 = 0; n1 < R; ++n1) {
        const uint32_t o = F16 ? pack_h2(x[n1].x, x[n1].y) : pack_bf2(x[n1].x, x[n1].y);
        if (n1 == 0) bad |= nonfinite16x2<F16>(o);              // every row of an overflowed column is non-finite: one row is enough
        ps[n1 * NT * npair] = o;
      }
    }
  }
  if (__any_sync(0xffffffffu, bad) && lane == 0) report_range(p.status);
  __syncthreads();
  // phase 2: whole rows
  bf16* dst = p.dst + b * p.d_sb + h * p.d_sh;
  const int cpr = npair / 4;                                    // 16-byte chunks per row
  for (int idx = threadIdx.x; idx < R * NT * cpr; idx += 256) {
    const int r = idx / cpr, q16 = idx - r * cpr;
    const int n1 = r / NT, tl = r & (NT - 1);                   // NT is a power of two
    const int row = n1 * 4096 + tb * NT + tl;
    if (row >= p.L) continue;
    const uint4 v = *reinterpret_cast<const uint4*>(stage + r * npair + ((q16 ^ (tl & skew_mask)) << 2));
    *reinterpret_cast<uint4*>(dst + (int64_t)row * p.d_sl + 8 * q16) = v;
  }
}

// =====================================================================================
// host
// =====================================================================================
// =====================================================================================
// whole-window read-out from cached half spectra (Sec. 3.3.2 step (e)): the inverse half of the path.
// tc_spec_in_kernel writes, per unit (head, k1, tile), what the core's gate epilogue would have left:
// the operand of the third stage, conj(s Z_k g_k / m) as fp16 with columns 64 c + kA and K = kB, bin
// k = k1 + R (kA + 64 kB), Z = the pair's full-spectrum value from the two half spectra (Hermitian
// completion, real DC / Nyquist products), s = the forward scale the transforms would have applied
// (in_scale(R) / 64) and m = sqrt(2) max |g| of the head, which the core's last epilogue undoes.
// =====================================================================================
struct TcSpecParams {
  const float2* spec;       // [B*H][K][D] half spectra, fp32
  const float2* g;          // [B*H][K]
  unsigned char* ws_in;     // [unit][k4ImgBytes]
  float* gscale;            // [slab_local * R + k1]
  int n, K, R, D, ntile, slab0;
  float sc;
};

// one CTA per head of the group: m for all its R units
__global__ void __launch_bounds__(256) tc_gate_amax_kernel(const TcSpecParams p) {
  __shared__ float red[8];
  const float2* g = p.g + (size_t)(p.slab0 + blockIdx.x) * p.K;
  float m = 0.f;
  for (int k = threadIdx.x; k < p.K; k += 256) {
    const float2 v = __ldg(g + k);
    m = fmaxf(m, fmaxf(fabsf(v.x), fabsf(v.y)));
  }
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  m = 0.f;
  for (int i = 0; i < 8; ++i) m = fmaxf(m, red[i]);
  if ((int)threadIdx.x < p.R) p.gscale[blockIdx.x * p.R + threadIdx.x] = m * 1.41421356f;
}

// CTA = (head, k1, K group j): the 256 bins kA < 64, kB = 4 j .. 4 j + 3 of the unit row.  A warp takes
// the four bins kB of one kA at a time, two kA per round (8 rows of 512 bytes in flight; lane = column pair:
// two float2).  With A, B the pair's half-spectrum values, the value to store is conj(Z) with
//   Z = g (A + jB) for a bin of the lower half, Z = conj(g) (conj(A) + j conj(B)) for a mirrored one
// (one complex product per bin; at DC and Nyquist only the real parts of gA and gB survive, App. B).  The
// four fp16 results of a (pair, kA) go into the staging array [pair][kA][kB % 4] as one 16-byte store (pair
// stride 260 words: no bank conflicts); the CTA then writes each tile's 4096 contiguous bytes of K group j.
constexpr int kSpecPitch = 260;

// The bins of a CTA lie on one side of the Nyquist bin: k = k1 + R kA + (n / 64) kB with kB = 4 j + u, so
// j < 8 means k < n/2 and j >= 8 means k > n/2, except for the two real bins k = 0 (j = 0) and k = n/2 (j = 8)
// of the first unit row, which the caller patches.  MIRROR is therefore a property of the CTA.
template <bool MIRROR>
__device__ __forceinline__ void spec_in_bins(const TcSpecParams& p, const float4* __restrict__ spec, const float2* __restrict__ g,
                                             uint32_t* spec_stage, int j, int k1, int warp, int l, bool live, float s) {
  const unsigned rowq = (unsigned)(p.D / 2);                    // float4 per bin row
  const int kbase = k1 + p.R * (warp + 256 * j), r8 = 8 * p.R, r64 = 64 * p.R;
#pragma unroll 1
  for (int it = 0; it < 8; it += 2) {
    float4 ab[2][4];
    float2 gk[2][4];
#pragma unroll
    for (int a = 0; a < 2; ++a) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int k = kbase + (it + a) * r8 + u * r64;
        const unsigned kk = (unsigned)(MIRROR ? p.n - k : k);
        ab[a][u] = __ldg(spec + kk * rowq);
        gk[a][u] = __ldg(g + kk);
      }
    }
#pragma unroll
    for (int a = 0; a < 2; ++a) {
      uint32_t h[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float4 v = ab[a][u];
        const float2 gs = cscale(gk[a][u], s);
        // conj(Z): conj(g) conj(A + jB) below the Nyquist bin, g conj(conj A + j conj B) above it
        const float2 cz = MIRROR ? cmul(gs, make_float2(v.x + v.w, v.y - v.z))
                                 : cmul(make_float2(gs.x, -gs.y), make_float2(v.x - v.w, -(v.y + v.z)));
        h[u] = pack_h2(cz.x, cz.y);
      }
      if (live) *reinterpret_cast<uint4*>(spec_stage + l * kSpecPitch + 4 * (warp + 8 * (it + a))) = make_uint4(h[0], h[1], h[2], h[3]);
    }
  }
}

__global__ void __launch_bounds__(256, 3) tc_spec_in_kernel(const TcSpecParams p) {
  extern __shared__ __align__(16) uint32_t spec_stage[];        // [D / 2][kSpecPitch]
  const int tid = threadIdx.x, warp = tid >> 5, l = tid & 31;
  const int j = blockIdx.x & 15, sk = blockIdx.x >> 4;
  const int slab_local = sk / p.R, k1 = sk - slab_local * p.R, slab = p.slab0 + slab_local;
  const int npair = p.D / 2;
  const bool live = l < npair;
  const float m = p.gscale[sk];
  const float s = m > 0.f ? p.sc / m : 0.f;
  const float4* spec = reinterpret_cast<const float4*>(p.spec + (size_t)slab * p.K * p.D) + (live ? l : 0);
  const float2* g = p.g + (size_t)slab * p.K;
  if (j >= 8) spec_in_bins<true>(p, spec, g, spec_stage, j, k1, warp, l, live, s);
  else spec_in_bins<false>(p, spec, g, spec_stage, j, k1, warp, l, live, s);
  if (k1 == 0 && warp == 0 && (j == 0 || j == 8) && live) {
    // the real bins k = 0 and k = n/2 (kA = 0, first kB of the group): only Re(gA) and Re(gB) survive (App. B)
    const unsigned kk = j == 0 ? 0u : (unsigned)(p.n / 2);
    const float4 v = __ldg(spec + kk * (unsigned)(p.D / 2));
    const float2 gs = cscale(__ldg(g + kk), s);
    spec_stage[l * kSpecPitch] = pack_h2(gs.x * v.x - gs.y * v.y, -(gs.x * v.z - gs.y * v.w));
  }
  __syncthreads();
  for (int e = tid; e < p.ntile * 256; e += 256) {
    const int tile = e >> 8, pc = e & 255;                      // pc = 64 c + kA
    const uint4 v = *reinterpret_cast<const uint4*>(spec_stage + (4 * tile + (pc >> 6)) * kSpecPitch + 4 * (pc & 63));
    *reinterpret_cast<uint4*>(p.ws_in + (size_t)(sk * p.ntile + tile) * k4ImgBytes + j * 4096 + pc * 16) = v;
  }
}

static size_t tc4k_slab_bytes(int R, int D) {
  const int ntile = D / 8;
  return (size_t)R * ntile * (k4ImgBytes + k4OutBytes) + (size_t)R * k4GBytes + 256;
}

bool tc4k_supported(int n, int D) {
  if (n < 4096 || n > 131072 || (n & (n - 1))) return false;
  return D % 8 == 0 && D <= 128;
}

// Workspace for `group` heads: operand images, unit results, gate images, gate scales.
size_t tc4k_workspace_bytes(const spectre_ctx* ctx, int n, int D, int nslab) {
  const int R = n / 4096;
  size_t per = tc4k_slab_bytes(R, D);
  // heads per group: measured on B200, larger groups win (fewer, fuller launches) although the
  // intermediates then no longer stay in L2; the preferred workspace is capped at 1.25 GiB
  size_t budget = (size_t)1280 << 20;
  size_t g = budget / per;
  if (g < 1) g = 1;
  if (g > (size_t)nslab) g = nslab;
  return g * per;
}

// mixer_tc32.cu: the radix-32 steps on the tensor cores (n = 131072, d_head = 64)
bool tc32_supported(const spectre_ctx* ctx, const spectre_act* v, const spectre_act* y, int n);
int launch_tc_in32(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, const float* g, int n, int slab0, int cnt,
                   unsigned char* ws_in, unsigned char* gimg, float* gscale, float sc);
int launch_tc_out32(const spectre_ctx* ctx, cudaStream_t st, const unsigned char* ws_out, const spectre_act* y, int n, int slab0, int cnt);

template <int R, bool F16>
static int tc4k_group(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, const float* g,
                      const spectre_act* y, int n, int slab0, int cnt, unsigned char* ws) {
  const int D = v->D, ntile = D / 8;
  const size_t nunits = (size_t)cnt * R * ntile;
  unsigned char* ws_in = ws;
  unsigned char* ws_out = ws_in + nunits * k4ImgBytes;
  unsigned char* gimg = ws_out + nunits * k4OutBytes;
  float* gscale = reinterpret_cast<float*>(gimg + (size_t)cnt * R * k4GBytes);

  const bool tc32 = R >= 2 && tc32_supported(ctx, v, y, n);       // radix-32 ... 2 steps on the tensor cores
  TcGateParams gp = {reinterpret_cast<const float2*>(g), gimg, gscale, n, n / 2 + 1, R, slab0};

  if (tc32) {
    int rc = launch_tc_in32(ctx, st, v, g, n, slab0, cnt, ws_in, gimg, gscale, in_scale(R));
    if (rc != SPECTRE_OK) return rc;
  } else {
  constexpr int NT2 = (R <= 2) ? 64 : 128 / R;
  TcInParams ip = {reinterpret_cast<const bf16*>(v->ptr), v->stride_b, v->stride_l, v->stride_h, ws_in,
                   v->H, D, v->L, n, ntile, slab0};
  size_t smem_in = (size_t)R * ntile * (NT2 / 2) * 128;
  if (smem_in < 4096 * sizeof(float2)) smem_in = 4096 * sizeof(float2);       // the gate CTAs' staging
  if (smem_in > 48 * 1024)
    SPECTRE_CUDA_OK(cudaFuncSetAttribute(tc_in_kernel<R, F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_in));
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(cnt * R + cnt * 16 * (64 / NT2)));
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = smem_in;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  SPECTRE_CUDA_OK(cudaLaunchKernelEx(&cfg, tc_in_kernel<R, F16>, ip, gp, cnt * R));
  SPECTRE_LAUNCH_OK("tc_in_kernel");
  }

  TcCoreParams cp = {ws_in, gimg, ws_out, reinterpret_cast<const __half*>(ctx->dft64),
                     reinterpret_cast<const float2*>(ctx->tw64x64),
                     reinterpret_cast<const float2*>(ctx->tw_staged) + (size_t)(R - 1) * 128, gscale,
                     1.0f / ((float)R * in_scale(R)), (int)nunits, ntile, R, ctx->status_dev, 0};
  SPECTRE_CUDA_OK(cudaFuncSetAttribute(tc_core_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, k4CoreSmem));
  int grid = 2 * ctx->sm_count;                     // two resident CTAs per SM, a contiguous range of units each
  if ((size_t)grid > nunits) grid = (int)nunits;
  tc_core_kernel<<<grid, k4CoreThreads, k4CoreSmem, st>>>(cp);
  SPECTRE_LAUNCH_OK("tc_core_kernel");

  if (tc32) return launch_tc_out32(ctx, st, ws_out, y, n, slab0, cnt);
  constexpr int NT = 512 / R;
  TcOutParams op = {ws_out, reinterpret_cast<bf16*>(y->ptr), y->stride_b, y->stride_l, y->stride_h,
                    y->H, D, y->L, n, ntile, slab0, ctx->status_dev};
  const size_t smem_out = (size_t)R * NT * (D / 2) * 4;
  if (smem_out > 48 * 1024)
    SPECTRE_CUDA_OK(cudaFuncSetAttribute(tc_out_kernel<R, F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_out));
  tc_out_kernel<R, F16><<<cnt * (4096 / NT), 256, smem_out, st>>>(op);
  SPECTRE_LAUNCH_OK("tc_out_kernel");
  return SPECTRE_OK;
}

int launch_mixer_tc4k(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, const float* g,
                      const spectre_act* y, int n, void* ws, size_t ws_bytes) {
  const int R = n / 4096, nslab = v->B * v->H;
  const size_t per = tc4k_slab_bytes(R, v->D);
  int group = (int)(ws_bytes / per);
  const int pref = (int)(tc4k_workspace_bytes(ctx, n, v->D, nslab) / per);
  if (group > pref) group = pref;
  if (group < 1) return fail(SPECTRE_ERR_WORKSPACE, "mixer workspace smaller than one (batch, head) slab");
  group = (nslab + (nslab + group - 1) / group - 1) / ((nslab + group - 1) / group);     // equal groups, no small remainder
  unsigned char* w = reinterpret_cast<unsigned char*>(ws);
  for (int s0 = 0; s0 < nslab; s0 += group) {
    const int cnt = nslab - s0 < group ? nslab - s0 : group;
    int rc;
    const bool f16 = v->dtype == SPECTRE_F16;              // 16-bit activations: bf16 or fp16 (same kernels, other unpack / pack)
#define SPECTRE_TC4K_GROUP(RR) (f16 ? tc4k_group<RR, true>(ctx, st, v, g, y, n, s0, cnt, w) : tc4k_group<RR, false>(ctx, st, v, g, y, n, s0, cnt, w))
    switch (R) {
      case 1: rc = SPECTRE_TC4K_GROUP(1); break;
      case 2: rc = SPECTRE_TC4K_GROUP(2); break;
      case 4: rc = SPECTRE_TC4K_GROUP(4); break;
      case 8: rc = SPECTRE_TC4K_GROUP(8); break;
      case 16: rc = SPECTRE_TC4K_GROUP(16); break;
      case 32: rc = SPECTRE_TC4K_GROUP(32); break;
      default: return fail(SPECTRE_ERR_UNSUPPORTED, "transform length not supported by the tensor-core path");
    }
#undef SPECTRE_TC4K_GROUP
    if (rc != SPECTRE_OK) return rc;
  }
  return SPECTRE_OK;
}

size_t tc4k_min_workspace(int n, int D) { return tc4k_slab_bytes(n / 4096, D); }

// ---- whole-window read-out: cached half spectra -> gated operand images -> inverse stages -> rows ----
bool tc4k_readout_supported(const spectre_ctx* ctx, const spectre_act* y, int n) {
  return (y->dtype == SPECTRE_BF16 || y->dtype == SPECTRE_F16) && ctx->dft64 != nullptr && ctx->tw_staged != nullptr &&
         tc4k_supported(n, y->D) && y->D <= 64;
}
// preferred workspace: groups of heads worth up to 1.25 GiB, as for the mixer (c4 read-out: 1.80 ms at 160 MB,
// 1.64 at 320 MB, 1.54 at 640 MB, 1.50 at 1.25 GiB, 1.48 ms with all 256 heads in one group)
size_t tc4k_readout_workspace_bytes(int n, int D, int nslab) {
  const size_t per = tc4k_slab_bytes(n / 4096, D);
  size_t g = ((size_t)1280 << 20) / per;
  if (g < 1) g = 1;
  if (g > (size_t)nslab) g = nslab;
  return g * per;
}

template <int R, bool F16>
static int tc4k_readout_group(const spectre_ctx* ctx, cudaStream_t st, const float* spec, const float* g, const spectre_act* y,
                              int n, int slab0, int cnt, unsigned char* ws) {
  const int D = y->D, ntile = D / 8;
  const size_t nunits = (size_t)cnt * R * ntile;
  unsigned char* ws_in = ws;
  unsigned char* ws_out = ws_in + nunits * k4ImgBytes;
  unsigned char* gimg = ws_out + nunits * k4OutBytes;          // unused here: the gate is already in the images
  float* gscale = reinterpret_cast<float*>(gimg + (size_t)cnt * R * k4GBytes);

  TcSpecParams sp = {reinterpret_cast<const float2*>(spec), reinterpret_cast<const float2*>(g), ws_in, gscale,
                     n, n / 2 + 1, R, D, ntile, slab0, in_scale(R) / 64.0f};
  tc_gate_amax_kernel<<<cnt, 256, 0, st>>>(sp);
  SPECTRE_LAUNCH_OK("tc_gate_amax_kernel");
  const size_t smem_spec = (size_t)(D / 2) * kSpecPitch * 4;
  tc_spec_in_kernel<<<cnt * R * 16, 256, smem_spec, st>>>(sp);
  SPECTRE_LAUNCH_OK("tc_spec_in_kernel");

  TcCoreParams cp = {ws_in, gimg, ws_out, reinterpret_cast<const __half*>(ctx->dft64),
                     reinterpret_cast<const float2*>(ctx->tw64x64),
                     reinterpret_cast<const float2*>(ctx->tw_staged) + (size_t)(R - 1) * 128, gscale,
                     1.0f / ((float)R * in_scale(R)), (int)nunits, ntile, R, ctx->status_dev, 2};
  SPECTRE_CUDA_OK(cudaFuncSetAttribute(tc_core_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, k4CoreSmem));
  int grid = 2 * ctx->sm_count;
  if ((size_t)grid > nunits) grid = (int)nunits;
  tc_core_kernel<<<grid, k4CoreThreads, k4CoreSmem, st>>>(cp);
  SPECTRE_LAUNCH_OK("tc_core_kernel");

  if (R >= 2 && tc32_supported(ctx, y, y, n)) return launch_tc_out32(ctx, st, ws_out, y, n, slab0, cnt);
  constexpr int NT = 512 / R;
  TcOutParams op = {ws_out, reinterpret_cast<bf16*>(y->ptr), y->stride_b, y->stride_l, y->stride_h,
                    y->H, D, y->L, n, ntile, slab0, ctx->status_dev};
  const size_t smem_out = (size_t)R * NT * (D / 2) * 4;
  if (smem_out > 48 * 1024)
    SPECTRE_CUDA_OK(cudaFuncSetAttribute(tc_out_kernel<R, F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_out));
  tc_out_kernel<R, F16><<<cnt * (4096 / NT), 256, smem_out, st>>>(op);
  SPECTRE_LAUNCH_OK("tc_out_kernel");
  return SPECTRE_OK;
}

int launch_readout_tc4k(const spectre_ctx* ctx, cudaStream_t st, const float* spec, const float* g, const spectre_act* y, int n,
                        void* ws, size_t ws_bytes) {
  const int R = n / 4096, nslab = y->B * y->H;
  const size_t per = tc4k_slab_bytes(R, y->D);
  int group = (int)(ws_bytes / per);
  const int pref = (int)(tc4k_readout_workspace_bytes(n, y->D, nslab) / per);
  if (group > pref) group = pref;
  if (group < 1) return fail(SPECTRE_ERR_WORKSPACE, "read-out workspace smaller than one (batch, head) slab");
  group = (nslab + (nslab + group - 1) / group - 1) / ((nslab + group - 1) / group);     // equal groups, no small remainder
  unsigned char* w = reinterpret_cast<unsigned char*>(ws);
  const bool f16 = y->dtype == SPECTRE_F16;
  for (int s0 = 0; s0 < nslab; s0 += group) {
    const int cnt = nslab - s0 < group ? nslab - s0 : group;
    int rc;
#define SPECTRE_TC4K_READOUT(RR) (f16 ? tc4k_readout_group<RR, true>(ctx, st, spec, g, y, n, s0, cnt, w) : tc4k_readout_group<RR, false>(ctx, st, spec, g, y, n, s0, cnt, w))
    switch (R) {
      case 1: rc = SPECTRE_TC4K_READOUT(1); break;
      case 2: rc = SPECTRE_TC4K_READOUT(2); break;
      case 4: rc = SPECTRE_TC4K_READOUT(4); break;
      case 8: rc = SPECTRE_TC4K_READOUT(8); break;
      case 16: rc = SPECTRE_TC4K_READOUT(16); break;
      case 32: rc = SPECTRE_TC4K_READOUT(32); break;
      default: return fail(SPECTRE_ERR_UNSUPPORTED, "transform length not supported by the tensor-core path");
    }
#undef SPECTRE_TC4K_READOUT
    if (rc != SPECTRE_OK) return rc;
  }
  return SPECTRE_OK;
}

}  // namespace spectre
