// Tensor-core kernels shared by the blocked-DFT mixers: the DFT-matrix and twiddle-table builders
// (owned by the context) and the n = 196 mixer.  The n = 8192 mixer lives in mixer_tc8k.cu, the
// multi-kernel path for longer transforms in mixer_tc4k.cu.
#include "tc_common.cuh"

namespace spectre {

constexpr int kTcLbo = 144;                    // bytes between core matrices along K (128 + 16 pad)
constexpr int kTcSbo = 2320;                   // bytes between 8-column groups (16 * 144 + 16 pad)
constexpr int kTcBBytes = 32 * kTcSbo;         // one 256-column B operand
constexpr int kTcFBytes = 128 * 128 * 2;
// Byte offset of element (column nu, K index kappa) in a B operand.
__device__ __forceinline__ uint32_t b_off(int nu, int kappa) {
  return (uint32_t)((nu >> 3) * kTcSbo + (kappa >> 3) * kTcLbo + (nu & 7) * 16 + (kappa & 7) * 2);
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

// Twiddles between the two 64-point stages of a 4096-point transform, in the order the epilogue
// threads use them: entry ((((q 2 + j) 2 + chunk) 4 + x) 32 + lane) holds W_4096^{row d} for
// row = 8 (2q + j) + lane / 4 and the even column d = 32 chunk + 8 x + 2 (lane % 4).
__global__ void build_tw64x64_kernel(float2* tab) {
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= 2048) return;
  int lane = idx & 31, x = (idx >> 5) & 3, chunk = (idx >> 7) & 1, j = (idx >> 8) & 1, q = idx >> 9;
  int row = 8 * (2 * q + j) + (lane >> 2), d = 32 * chunk + 8 * x + 2 * (lane & 3);
  float s0, c0;
  sincospif((float)((row * d) & 4095) / 2048.0f, &s0, &c0);
  tab[idx] = make_float2(c0, -s0);
}

int build_tw64x64(float2* tab, cudaStream_t st) {
  build_tw64x64_kernel<<<8, 256, 0, st>>>(tab);
  SPECTRE_LAUNCH_OK("build_tw64x64_kernel");
  return SPECTRE_OK;
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

// =====================================================================================
// n = 196 (14 x 14 patch grids), bf16 or fp16 I/O, D = 64: 196 = 4 * 49.
//
// t = 49 n1 + t', k = k1 + 4 kM.  The radix-4 DFT over n1 and the twiddle W_196^{k1 t'} run on
// the ALUs while whole 128-byte head rows are loaded; each 49-point DFT over t' is ONE tensor-core
// stage with the 49-point DFT matrix in real form (98 x 98, zero-padded to 128 x 112) as the A
// operand; the gate is applied to the accumulator, one more stage does the inverse 49-point DFT
// (conj trick), and the final epilogue does the inverse radix-4 and stores bf16 rows.
// A work item is 2 heads (the same head index of two batch entries): columns (head, k1, pair) =
// 2 x 4 x 32 = 256 TMEM columns and one operand buffer, so two CTAs share an SM and one's loads run
// under the other's arithmetic; a CTA loops over its work items (persistent grid).  The kernel is
// written for NH = 2 or 4 heads per item (4: two halves that ping-pong between tensor core and ALUs
// like the halves of the 8192 kernel, one CTA per SM); 2 measured faster and is what is launched.
// =====================================================================================
constexpr int k196Heads = 2;                  // heads per CTA the launcher uses: two CTAs per SM (4 per CTA measured slower)
constexpr int k196KSteps = 7;                 // K = 112 >= 98
constexpr int k196WHidden = 256;              // widest level-gate MLP the fused refinement handles
constexpr int k196StageRow = 160;             // bytes per staged output row (128 + pad against bank conflicts)
constexpr int k196_smem(int NH) { return kTcFBytes + (NH / 2) * kTcBBytes + NH * 256 * 4 + 64 + NH * 3 * 64 * 4; }
static_assert(2 * 196 * k196StageRow <= kTcBBytes, "staged rows of two heads fit one operand buffer");

struct Tc196Params {
  const bf16* src;
  bf16* dst;
  int64_t s_sb, s_sl, s_sh, d_sb, d_sl, d_sh;
  const float2* g;        // [B*H][99]
  const __half* F;        // 49-point DFT matrix (real form, padded), canonical smem layout
  int H, L, B;
  int* status;
  // wavelet refinement fused into the store (Sec. 3.5), J = 0: off
  int J;
  const float* level_gates;       // [B,H,J+1,64]
  const int* skip;                // [B] or NULL: non-zero = no refinement for this batch entry
};

// Level gates of the refinement (Sec. 3.5 step b): s = GELU(q_bar Ww1 + bw1) Ww2 + bw2, [B,H,NG] with
// NG = (J + 1) 64.  A CTA takes kLgBatch batch entries of one head index, so each weight is fetched
// once per kLgBatch entries.  Hidden layer: an item is one hidden unit x a quarter of the 64 inputs
// (partial sums meet in shared memory); output layer: a thread owns one output.  The first item's
// weights and the first 32 rows of W2 are requested together at the start; three CTAs fit an SM, so
// the grid of a ViT-sized batch is resident at once.  The mixer kernel launched next may start while this one runs.
constexpr int kLgBatch = 8;
struct LevelGateParams {
  const float* qbar; const void* Ww1; const float* bw1; const void* Ww2; const float* bw2;
  size_t hs_w1, hs_b1, hs_w2, hs_b2;     // per-head strides in elements (0: shared across heads)
  float* out;
  int B, H, hidden, NG;
};

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(bf16 x) { return __bfloat162float(x); }

template <typename WT>
__global__ void __launch_bounds__(256, 3) level_gates_kernel(const LevelGateParams p) {
  __shared__ __align__(16) float qs[kLgBatch][64];
  extern __shared__ float part_raw[];                        // [4][kLgBatch][hidden]: hidden-layer partial sums per input quarter
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int tid = threadIdx.x, h = blockIdx.x, b0 = blockIdx.y * kLgBatch;
  const WT* W1 = reinterpret_cast<const WT*>(p.Ww1) + h * p.hs_w1;
  const WT* W2 = reinterpret_cast<const WT*>(p.Ww2) + h * p.hs_w2;
  const int nitems = 4 * p.hidden;
  float qv[2];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int e = tid + 256 * i, b = b0 + (e >> 6);
    qv[i] = b < p.B ? p.qbar[((size_t)b * p.H + h) * 64 + (e & 63)] : 0.f;
  }
  WT w1[16], w2[32];
  {
    const int it = min(tid, nitems - 1), jj = it % p.hidden, cq = it / p.hidden;
#pragma unroll
    for (int c = 0; c < 16; ++c) w1[c] = W1[(size_t)(16 * cq + c) * p.hidden + jj];
  }
  const int ii = min(tid, p.NG - 1);
#pragma unroll
  for (int u = 0; u < 32; ++u) w2[u] = W2[(size_t)min(u, p.hidden - 1) * p.NG + ii];
#pragma unroll
  for (int i = 0; i < 2; ++i) qs[(tid + 256 * i) >> 6][(tid + 256 * i) & 63] = qv[i];
  __syncthreads();
  for (int it = tid; it < nitems; it += 256) {
    const int jj = it % p.hidden, cq = it / p.hidden;
    if (it != tid) {
#pragma unroll
      for (int c = 0; c < 16; ++c) w1[c] = W1[(size_t)(16 * cq + c) * p.hidden + jj];
    }
    float acc[kLgBatch];
#pragma unroll
    for (int e = 0; e < kLgBatch; ++e) acc[e] = 0.f;
#pragma unroll
    for (int c4 = 0; c4 < 4; ++c4) {
#pragma unroll
      for (int e = 0; e < kLgBatch; ++e) {
        const float4 q4 = *reinterpret_cast<const float4*>(&qs[e][16 * cq + 4 * c4]);
        acc[e] = fmaf(q4.x, to_float(w1[4 * c4]), acc[e]);
        acc[e] = fmaf(q4.y, to_float(w1[4 * c4 + 1]), acc[e]);
        acc[e] = fmaf(q4.z, to_float(w1[4 * c4 + 2]), acc[e]);
        acc[e] = fmaf(q4.w, to_float(w1[4 * c4 + 3]), acc[e]);
      }
    }
#pragma unroll
    for (int e = 0; e < kLgBatch; ++e) part_raw[(cq * kLgBatch + e) * p.hidden + jj] = acc[e];
  }
  __syncthreads();
  for (int i = tid; i < kLgBatch * p.hidden; i += 256) {       // u = GELU(sum of the quarters + bias), kept in part[0]
    const int e = i / p.hidden, jj = i - e * p.hidden;
    const int st = kLgBatch * p.hidden;
    part_raw[i] = gelu_erf(p.bw1[h * p.hs_b1 + jj] + ((part_raw[i] + part_raw[st + i]) + (part_raw[2 * st + i] + part_raw[3 * st + i])));
  }
  __syncthreads();
  if (tid < p.NG) {
    float acc[kLgBatch];
    const float b2 = p.bw2[h * p.hs_b2 + ii];
#pragma unroll
    for (int e = 0; e < kLgBatch; ++e) acc[e] = b2;
    for (int j0 = 0; j0 < p.hidden; j0 += 32) {
      if (j0 > 0) {
#pragma unroll
        for (int u = 0; u < 32; ++u) w2[u] = W2[(size_t)min(j0 + u, p.hidden - 1) * p.NG + ii];
      }
#pragma unroll
      for (int u = 0; u < 32; ++u) {
        if (j0 + u < p.hidden) {
          const float wv = to_float(w2[u]);
#pragma unroll
          for (int e = 0; e < kLgBatch; ++e) acc[e] = fmaf(part_raw[e * p.hidden + j0 + u], wv, acc[e]);
        }
      }
    }
#pragma unroll
    for (int e = 0; e < kLgBatch; ++e)
      if (b0 + e < p.B) p.out[((size_t)(b0 + e) * p.H + h) * p.NG + ii] = acc[e];
  }
}

// NH heads per CTA (2 or 4): NH / 2 operand buffers and accumulators of 256 columns, 4 NH epilogue
// warps + the issuing warp.  With NH = 2 two CTAs share an SM, so one CTA's loads and weight fetches
// run under the other's arithmetic.
template <int NH, int J, bool F16>
__global__ void __launch_bounds__(128 * NH + 32, NH == 2 ? 2 : 1) mixer_tc196_kernel(const Tc196Params p) {
  constexpr int NHALF = NH / 2, EW = 4 * NH, ET = 32 * EW;        // halves, epilogue warps and threads
  constexpr int HPI = NH / 2;                                     // heads per gate-table pass
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* Fsm = smem;
  unsigned char* Bsm[2] = {smem + kTcFBytes, smem + kTcFBytes + (NHALF - 1) * kTcBBytes};
  uint32_t* Gsm = reinterpret_cast<uint32_t*>(smem + kTcFBytes + NHALF * kTcBBytes);        // [NH heads][k1 * 64 + kM]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kTcFBytes + NHALF * kTcBBytes + NH * 256 * 4);
  float* wsg = reinterpret_cast<float*>(smem + kTcFBytes + NHALF * kTcBBytes + NH * 256 * 4 + 64);  // [NH][3][64] holds 1 + s
  __shared__ uint32_t tmem_slot;
  __shared__ float red[2 * EW];
  __shared__ float gmax_s[NH];

  __shared__ int abort_s;
  __shared__ float2 tw_s[3 * 49];                    // W_196^{m t'}, m = 1, 2, 3

  const int tid = threadIdx.x, warp = tid >> 5, T = tid & 31;
  const int nwork = p.H * ((p.B + NH - 1) / NH);     // work items: NH batch entries of one head index

  if (warp == EW) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&tmem_slot)), "r"(256 * NHALF));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  if (tid < 49) {
    const float2 w1 = twiddle_fwd((unsigned)tid, 196u);
    const float2 w2 = cmul(w1, w1);
    tw_s[3 * tid] = w1;
    tw_s[3 * tid + 1] = w2;
    tw_s[3 * tid + 2] = cmul(w2, w1);
  }
  if (tid == 0) {
    abort_s = 0;
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&bars[0])), "r"(ET));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&bars[1])), "r"(ET));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&bars[2])), "r"(1));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&bars[3])), "r"(1));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < ET) {
    const uint4* Fg = reinterpret_cast<const uint4*>(p.F);
    for (int i = tid; i < kTcFBytes / 16; i += ET) reinterpret_cast<uint4*>(Fsm)[i] = __ldg(Fg + i);
    // zero the operands once: K rows 98..127 and the columns of absent heads must read as zero
    for (int i = tid; i < NHALF * kTcBBytes / 16; i += ET) reinterpret_cast<uint4*>(Bsm[0])[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = tmem_slot;

  if (warp == EW) {
    // ---- MMA issuer: per work item 2 stages x NH / 2 halves, 7 K-steps each ----
    const uint32_t idesc = umma_idesc_128x256();
    bool ok = true;
    for (int work = blockIdx.x; work < nwork && ok; work += gridDim.x)
    for (int stage = 0; stage < 2 && ok; ++stage) {
      for (int half = 0; half < NHALF && ok; ++half) {
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
    if (!ok && T == 0) report_timeout(p.status);
  } else {
    // The CTA keeps its DFT matrix, accumulators and barriers over all its work items: the barriers
    // complete two phases per item, so every item sees the same parities.
    bool ok = true;
    bool bad = false;                                 // a non-finite result: the fp16 intermediates overflowed
#pragma unroll 1
    for (int work = blockIdx.x; work < nwork; work += gridDim.x) {
    // the item's heads are batch entries bg NH .. bg NH + NH - 1 of ONE head index hh: they share the
    // level-gate weights, and neighbouring items read neighbouring 128-byte pieces of the same rows
    const int hh = work % p.H, bg = work / p.H;
    // per-thread indices re-derived from an opaque copy, so that the compiler keeps the item's index
    // arithmetic and twiddles inside the loop instead of carrying them in registers across items
    int tid_item = threadIdx.x;
    asm volatile("" : "+r"(tid_item));
    const int tid = tid_item, warp = tid >> 5, T = tid & 31;
    if (J > 0 && work != (int)blockIdx.x) {
      // the staged rows of the previous item covered K rows 98..111, which the MMA reads as zero padding:
      // clear them again (bytes 4..15 of slot 12's rows, all of slot 13; the loads below write the rest)
#pragma unroll
      for (int half = 0; half < NHALF; ++half) {
        for (int idx = tid; idx < 32 * 8; idx += ET) {               // (group of 8 columns, column)
          unsigned char* z = Bsm[half] + (idx >> 3) * kTcSbo + 12 * kTcLbo + (idx & 7) * 16;
          *reinterpret_cast<uint32_t*>(z + 4) = 0u;
          *reinterpret_cast<uint2*>(z + 8) = make_uint2(0u, 0u);
          *reinterpret_cast<uint4*>(z + kTcLbo) = make_uint4(0u, 0u, 0u, 0u);
        }
      }
    }
    // ---- load: rows t' + 49 n1 of each head, radix-4 over n1, twiddle, fp16, operand (K = t', column = (head, k1, pair)) ----
    // a warp takes 4 consecutive t' x 8 chunks of 16 bytes (conflict-free operand stores); all of
    // a warp's rows (up to 4 items x 4 rows) are requested before the first one is used
    constexpr int kItems = (NH * 13 + EW - 1) / EW;
    uint4 rr[kItems][4];
#pragma unroll
    for (int it = 0; it < kItems; ++it) {
      const int item = warp + it * EW;
      const int hl = item / 13, tg = item - hl * 13;
      const int tp = 4 * tg + (T >> 3), b = bg * NH + hl;
      const bool live = item < NH * 13 && tp < 49 && b < p.B;
      const bf16* src = p.src + (live ? b : 0) * p.s_sb + hh * p.s_sh + 8 * (T & 7);
#pragma unroll
      for (int n1 = 0; n1 < 4; ++n1) {
        const int row = tp + 49 * n1;
        rr[it][n1] = (live && row < p.L) ? __ldcg(reinterpret_cast<const uint4*>(src + (int64_t)row * p.s_sl))
                                         : make_uint4(0u, 0u, 0u, 0u);
      }
    }
#pragma unroll
    for (int it = 0; it < kItems; ++it) {
      const int item = warp + it * EW;
      const int hl = item / 13, tg = item - hl * 13;
      const int tp = 4 * tg + (T >> 3), chunk = T & 7;
      if (item >= NH * 13 || tp >= 49 || bg * NH + hl >= p.B) continue;
      const float2 w1 = tw_s[3 * tp], w2 = tw_s[3 * tp + 1], w3 = tw_s[3 * tp + 2];
      unsigned char* Bh = Bsm[hl >> 1] + b_off((hl & 1) * 128 + 4 * chunk, 2 * tp);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float2 x[4];
#pragma unroll
        for (int n1 = 0; n1 < 4; ++n1) {
          const uint32_t u = j == 0 ? rr[it][n1].x : (j == 1 ? rr[it][n1].y : (j == 2 ? rr[it][n1].z : rr[it][n1].w));
          const float2 xv = F16 ? unpack_h2(u) : make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
          x[n1] = make_float2(0.5f * xv.x, 0.5f * xv.y);
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
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");     // the previous item's accumulator reads are done
    mbar_arrive(smem_u32(&bars[0]));
    if (NHALF == 2) mbar_arrive(smem_u32(&bars[1]));

    // ---- level gates of the refinement (Sec. 3.5 step b), [B,H,J+1,64]: requested here, used after the gate
    //      tables.  They may come from the kernel launched just before this one (programmatic dependent
    //      launch): griddepcontrol.wait returns once that grid's writes are visible ----
    constexpr int NG = (J + 1) * 64;
    float2 lgv = make_float2(0.f, 0.f);
    const int lg_hl = tid / (NG / 2), lg_i = 2 * (tid % (NG / 2));
    if (J > 0) {
      asm volatile("griddepcontrol.wait;" ::: "memory");
      if (lg_hl < NH && bg * NH + lg_hl < p.B)
        lgv = *reinterpret_cast<const float2*>(p.level_gates + ((size_t)(bg * NH + lg_hl) * p.H + hh) * NG + lg_i);
    }

    // ---- gate tables: head hl, entry k1 * 64 + kM holds G_ext[k1 + 4 kM] / gmax(head) as fp16 ----
    float2 gv[2];
    float gm[2];
#pragma unroll
    for (int it = 0; it < 2; ++it) {
      const int e = tid + it * ET, hl = e >> 8, idx = e & 255, k1 = idx >> 6, kM = idx & 63;
      const int b = bg * NH + hl;
      float2 v = make_float2(0.f, 0.f);
      if (kM < 49 && b < p.B) {
        const int k = k1 + 4 * kM, kk = k <= 98 ? k : 196 - k;
        v = __ldg(p.g + ((size_t)b * p.H + hh) * 99 + kk);
        if (kk != k) v.y = -v.y;
        if (k == 0 || k == 98) v.y = 0.f;
      }
      gv[it] = v;
      float m = fmaxf(fabsf(v.x), fabsf(v.y));
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      gm[it] = m;
    }
    // 8 consecutive warps hold one head per pass: pass `it` covers heads HPI * it .. HPI * it + HPI - 1
    if (T == 0) { red[warp] = gm[0]; red[EW + warp] = gm[1]; }
    asm volatile("bar.sync 1, %0;" :: "r"(ET) : "memory");
    if (tid < NH) {                                   // head tid = HPI * it + w: warps 8 w .. 8 w + 7 of pass it
      const int it = tid / HPI, w8 = tid - it * HPI;
      float m = 0.f;
      for (int i = 0; i < 8; ++i) m = fmaxf(m, red[it * EW + 8 * w8 + i]);
      gmax_s[tid] = 1.41421356f * m;
    }
    asm volatile("bar.sync 1, %0;" :: "r"(ET) : "memory");
#pragma unroll
    for (int it = 0; it < 2; ++it) {
      const int e = tid + it * ET, hl = e >> 8;
      const float gmx = gmax_s[hl], inv = gmx > 0.f ? 1.0f / gmx : 0.f;
      Gsm[e] = pack_h2(gv[it].x * inv, gv[it].y * inv);
    }
    if (J > 0 && lg_hl < NH) {
      wsg[lg_hl * 192 + lg_i] = 1.0f + lgv.x;
      wsg[lg_hl * 192 + lg_i + 1] = 1.0f + lgv.y;
    }
    asm volatile("bar.sync 1, %0;" :: "r"(ET) : "memory");

    // a warp owns TMEM lanes 32 q .. 32 q + 31; per unit it takes 64 columns: with 4 heads unit = half and
    // the column quarter is fixed, with 2 heads the one half's quarters 2 (warp >> 2) + unit
    const int q = warp & 3;
    const int i = T >> 2, t4 = T & 3;
    // ---- gate epilogue: rows kM, columns (head, k1, pair) unchanged; next operand has K = kM ----
#pragma unroll 1
    for (int unit = 0; unit < 2 && ok; ++unit) {
      const int half = NH == 4 ? unit : 0, cq = NH == 4 ? (warp >> 2) : 2 * (warp >> 2) + unit;
      if (NH == 4 || unit == 0) {
        ok = mbar_wait(smem_u32(&bars[2 + half]), 0);
        if (!ok) break;
      }
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
      if (NH == 4 || unit == 1) mbar_arrive(smem_u32(&bars[half]));
    }
    // ---- final: rows t', inverse radix-4 over k1 (columns 32 apart), bf16 rows t' + 49 n1 ----
#pragma unroll 1
    for (int unit = 0; unit < 2 && ok; ++unit) {
      const int half = NH == 4 ? unit : 0, cq = NH == 4 ? (warp >> 2) : 2 * (warp >> 2) + unit;
      if (NH == 4 || unit == 0) {
        ok = mbar_wait(smem_u32(&bars[2 + half]), 1);
        if (!ok) break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int hl = 2 * half + (cq >> 1), b = bg * NH + hl, h = hh;
      if (b >= p.B) continue;
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
            const float2 w1 = tw_s[3 * tp], w2 = tw_s[3 * tp + 1], w3 = tw_s[3 * tp + 2];
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
              const uint2 out = F16 ? make_uint2(pack_h2(gs * y0[n1].x, gs * y0[n1].y), pack_h2(gs * y1[n1].x, gs * y1[n1].y))
                                    : pack_bf16x4(gs * y0[n1].x, gs * y0[n1].y, gs * y1[n1].x, gs * y1[n1].y);
              // an overflow anywhere in a column makes every row of it non-finite: one row per thread is enough
              if (n1 == 0) bad |= nonfinite16x2<F16>(out.x) | nonfinite16x2<F16>(out.y);
              if (J > 0) *reinterpret_cast<uint2*>(Bsm[half] + ((hl & 1) * 196 + row) * k196StageRow + 2 * col) = out;
              else if (row < p.L) __stcs(reinterpret_cast<uint2*>(dst + (int64_t)row * p.d_sl + col), out);
            }
          }
        }
      }
    }
    if (J > 0) {
      // ---- wavelet refinement on the staged bf16 rows (Sec. 3.5): Haar over aligned blocks of 2^J
      //      tokens, bands scaled by 1 + s, synthesis; a thread takes 8 channels of one block and
      //      writes whole 16-byte pieces, 8 lanes per 128-byte row ----
      asm volatile("bar.sync 1, %0;" :: "r"(ET) : "memory");
      if (ok) {
        constexpr int S = 1 << J;
        const float r2 = 0.70710678118654752440f;
        const int nblk = p.L / S;
        for (int item = tid; item < NH * nblk * 8; item += ET) {
          const int cch = item & 7, blk = (item >> 3) % nblk, hl = item / (8 * nblk), b = bg * NH + hl, h = hh;
          if (b >= p.B) continue;
          const unsigned char* st = Bsm[hl >> 1] + ((hl & 1) * 196 + blk * S) * k196StageRow + 16 * cch;
          if (p.skip && p.skip[b]) {                             // skipped batch entry: the mixer output as it is
            bf16* dst0 = p.dst + b * p.d_sb + h * p.d_sh + 8 * cch;
#pragma unroll
            for (int r = 0; r < S; ++r)
              __stcs(reinterpret_cast<uint4*>(dst0 + (int64_t)(blk * S + r) * p.d_sl), *reinterpret_cast<const uint4*>(st + r * k196StageRow));
            continue;
          }
          float x[S][8];
#pragma unroll
          for (int r = 0; r < S; ++r) {
            const uint4 u4 = *reinterpret_cast<const uint4*>(st + r * k196StageRow);
            const uint32_t w4[4] = {u4.x, u4.y, u4.z, u4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float2 xv = F16 ? unpack_h2(w4[e]) : make_float2(__uint_as_float(w4[e] << 16), __uint_as_float(w4[e] & 0xffff0000u));
              x[r][2 * e] = xv.x;
              x[r][2 * e + 1] = xv.y;
            }
          }
          // analysis in place: after level l, slot i 2^l holds a_l and slot i 2^l + 2^(l-1) holds d_l
#pragma unroll
          for (int l = 1; l <= J; ++l) {
            const int span = 1 << l, hs = span >> 1;
#pragma unroll
            for (int i0 = 0; i0 < S; i0 += span)
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const float a = x[i0][e], d = x[i0 + hs][e];
                x[i0][e] = (a + d) * r2;
                x[i0 + hs][e] = (a - d) * r2;
              }
          }
          // slot 0 is a_J, slot r > 0 is d_l with l = ctz(r) + 1; gate order a_J, d_J, ..., d_1
          const float* sg = wsg + hl * 192 + 8 * cch;
#pragma unroll
          for (int r = 0; r < S; ++r) {
            const int lev = r == 0 ? 0 : 1 + (J - (__ffs(r)));
#pragma unroll
            for (int e = 0; e < 8; ++e) x[r][e] *= sg[lev * 64 + e];
          }
#pragma unroll
          for (int l = J; l >= 1; --l) {
            const int span = 1 << l, hs = span >> 1;
#pragma unroll
            for (int i0 = 0; i0 < S; i0 += span)
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const float a = x[i0][e], d = x[i0 + hs][e];
                x[i0][e] = (a + d) * r2;
                x[i0 + hs][e] = (a - d) * r2;
              }
          }
          bf16* dst = p.dst + b * p.d_sb + h * p.d_sh + 8 * cch;
#pragma unroll
          for (int r = 0; r < S; ++r) {
            uint4 o;
            if (F16) {
              o.x = pack_h2(x[r][0], x[r][1]); o.y = pack_h2(x[r][2], x[r][3]);
              o.z = pack_h2(x[r][4], x[r][5]); o.w = pack_h2(x[r][6], x[r][7]);
            } else {
              o.x = pack_bf2(x[r][0], x[r][1]); o.y = pack_bf2(x[r][2], x[r][3]);
              o.z = pack_bf2(x[r][4], x[r][5]); o.w = pack_bf2(x[r][6], x[r][7]);
            }
            __stcs(reinterpret_cast<uint4*>(dst + (int64_t)(blk * S + r) * p.d_sl), o);
          }
        }
      }
    }
    // end of the item: the staged rows and level gates are free again; a wait that ran out ends the loop for all
    if (!ok) abort_s = 1;
    asm volatile("bar.sync 1, %0;" :: "r"(ET) : "memory");
    if (abort_s) break;
    }
    if (!ok && T == 0) report_timeout(p.status);
    if (__any_sync(0xffffffffu, bad) && T == 0) report_range(p.status);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == EW) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(256 * NHALF));
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

// The refinement can ride in the store phase when the block length divides 196 (J <= 2) and the
// level-gate MLP fits the kernel's scratch.
bool tc196_fuses_wavelet(const spectre_wavelet* w) {
  return w && (w->levels == 1 || w->levels == 2) &&
         (w->level_gates || (w->hidden >= 1 && w->hidden <= k196WHidden));
}

size_t tc196_level_gate_bytes(int B, int H) { return (size_t)B * H * 3 * 64 * sizeof(float); }

// level_gate_scratch: tc196_level_gate_bytes(B, H) bytes, needed when wrm carries the MLP weights
int launch_mixer_tc196(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, const float* g,
                       const spectre_act* y, const spectre_wavelet* wrm, float* level_gate_scratch) {
  Tc196Params p = {};
  p.src = reinterpret_cast<const bf16*>(v->ptr);
  p.dst = reinterpret_cast<bf16*>(y->ptr);
  p.s_sb = v->stride_b; p.s_sl = v->stride_l; p.s_sh = v->stride_h;
  p.d_sb = y->stride_b; p.d_sl = y->stride_l; p.d_sh = y->stride_h;
  p.g = reinterpret_cast<const float2*>(g);
  p.F = reinterpret_cast<const __half*>(ctx->dft49);
  p.H = v->H; p.L = v->L; p.B = v->B;
  p.status = ctx->status_dev;
  bool dependent = false;            // the mixer kernel follows a kernel of ours whose output it reads
  if (wrm) {
    const int J = wrm->levels;
    p.J = J;
    p.skip = wrm->skip;
    p.level_gates = wrm->level_gates;
    if (!wrm->level_gates) {
      LevelGateParams lp = {};
      const int hid = wrm->hidden;
      const size_t one = wrm->shared_across_heads ? 0 : 1;
      lp.qbar = wrm->qbar; lp.Ww1 = wrm->Ww1; lp.bw1 = wrm->bw1; lp.Ww2 = wrm->Ww2; lp.bw2 = wrm->bw2;
      lp.hs_w1 = one * (size_t)64 * hid; lp.hs_b1 = one * hid;
      lp.hs_w2 = one * (size_t)hid * (J + 1) * 64; lp.hs_b2 = one * (size_t)(J + 1) * 64;
      lp.out = level_gate_scratch;
      lp.B = v->B; lp.H = v->H; lp.hidden = hid; lp.NG = (J + 1) * 64;
      const dim3 lgrid((unsigned)v->H, (unsigned)((v->B + kLgBatch - 1) / kLgBatch));
      const size_t lsmem = (size_t)4 * kLgBatch * hid * sizeof(float);       // <= 32 KB
      if (wrm->wdtype == SPECTRE_BF16) level_gates_kernel<bf16><<<lgrid, 256, lsmem, st>>>(lp);
      else level_gates_kernel<float><<<lgrid, 256, lsmem, st>>>(lp);
      SPECTRE_LAUNCH_OK("level_gates_kernel");
      p.level_gates = level_gate_scratch;
      dependent = true;
    }
  }
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  const unsigned nwork = (unsigned)(p.H * ((p.B + k196Heads - 1) / k196Heads)), slots = 2u * (unsigned)ctx->sm_count;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(nwork < slots ? nwork : slots);        // persistent: two CTAs per SM
  cfg.blockDim = dim3(128 * k196Heads + 32);
  cfg.dynamicSmemBytes = k196_smem(k196Heads);
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = dependent ? 1 : 0;
#define SPECTRE_TC196_LAUNCH(JJ, FH)                                                                              \
  do {                                                                                                            \
    SPECTRE_CUDA_OK(cudaFuncSetAttribute(mixer_tc196_kernel<k196Heads, JJ, FH>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                         k196_smem(k196Heads)));                                                  \
    SPECTRE_CUDA_OK(cudaLaunchKernelEx(&cfg, mixer_tc196_kernel<k196Heads, JJ, FH>, p));                          \
  } while (0)
  const bool f16 = v->dtype == SPECTRE_F16;
  if (p.J == 2) { if (f16) SPECTRE_TC196_LAUNCH(2, true); else SPECTRE_TC196_LAUNCH(2, false); }
  else if (p.J == 1) { if (f16) SPECTRE_TC196_LAUNCH(1, true); else SPECTRE_TC196_LAUNCH(1, false); }
  else { if (f16) SPECTRE_TC196_LAUNCH(0, true); else SPECTRE_TC196_LAUNCH(0, false); }
#undef SPECTRE_TC196_LAUNCH
  SPECTRE_LAUNCH_OK("mixer_tc196_kernel");
  return SPECTRE_OK;
}

}  // namespace spectre
