// Token projections (Sec. 3.2 step 1, Eq. 2): Q = X W^(q), V = X W^(v) per head, d = 64, bf16,
// on the 5th-generation tensor cores, with the pooled query sum of step 3a as a by-product.
//
// One CTA = 128 tokens of one (batch, head):
//     D[128 tokens x 128 outputs] (fp32, TMEM) = A[128 x 64] (X tile, bf16) * B[64 x 128] ([W^(q) | W^(v)], bf16)
// Both operands sit in shared memory in the K-major core-matrix layout without swizzle (8 rows x
// 16 bytes per core matrix).  The X tile is read as whole 128-byte head rows (8 lanes per row);
// the weights come from a copy transposed once per call to [head][output][input].  Four warps
// read the accumulator (a thread gets two tokens x two adjacent outputs per 8-column group),
// round to bf16 into a staging tile, and add up the fp32 accumulators of the Q half over the
// tile's tokens (shuffles, shared memory, one atomic per output and CTA); then the whole CTA
// writes Q and V rows as 16-byte pieces, 8 lanes per 128-byte row.
#include "tc_common.cuh"

namespace spectre {

constexpr int kPjTok = 128;                      // tokens per CTA
constexpr int kPjLbo = 2064;                     // K-group stride: 16 row groups x 128 + 16 (stores of a row spread over all banks)
constexpr int kPjSbo = 128;                      // 8-row group stride
constexpr int kPjOpBytes = 8 * kPjLbo;           // one 128 x 64 operand
constexpr int kPjStagePitch = 272;               // staged output row: 128 outputs x 2 bytes + 16 (conflict-free 4-byte stores)
constexpr int kPjSmem = 2 * kPjOpBytes + kPjTok * kPjStagePitch + 128;
constexpr int kPjThreads = 256;

struct ProjParams {
  const bf16* x; bf16* q; bf16* v;
  int64_t x_sb, x_sl, x_sh, q_sb, q_sl, q_sh, v_sb, v_sl, v_sh;
  const bf16* wt;          // [H][128 outputs (q then v)][64 inputs]
  float* sum_q;            // [B,H,64] or NULL
  int H, L, tiles;         // tiles per (batch, head)
  int* status;
};

template <typename WT> __device__ __forceinline__ float pj_wload(const WT* p);
template <> __device__ __forceinline__ float pj_wload<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float pj_wload<bf16>(const bf16* p) { return __bfloat162float(*p); }

// [H][d_in][d_out] (x @ W) for q and v  ->  wt[H][2 * 64][64] bf16 (output-major)
template <typename WT>
__global__ void __launch_bounds__(256) proj_weights_kernel(const WT* __restrict__ Wq, const WT* __restrict__ Wv,
                                                           bf16* __restrict__ wt, int H) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= H * 128 * 64) return;
  const int i = idx & 63, o = (idx >> 6) & 127, h = idx >> 13;
  const WT* W = o < 64 ? Wq : Wv;
  const float w = pj_wload<WT>(W + ((size_t)h * 64 + i) * 64 + (o & 63));
  wt[idx] = __float2bfloat16_rn(w);
}

__global__ void __launch_bounds__(kPjThreads, 3) project_qv_kernel(const ProjParams p) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
  unsigned char* Asm = smem;                         // X tile
  unsigned char* Bsm = smem + kPjOpBytes;            // weights
  unsigned char* stage = smem + 2 * kPjOpBytes;      // [128 tokens][272 bytes]
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t tmem_slot;
  __shared__ float qsum[4][64];

  const int tid = threadIdx.x, warp = tid >> 5, T = tid & 31;
  const int tile = blockIdx.x % p.tiles, slab = blockIdx.x / p.tiles;
  const int b = slab / p.H, h = slab - b * p.H;
  const int t0 = tile * kPjTok;

  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&tmem_slot)), "r"(128));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  if (tid == 0) {
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // operands: 128 rows x 8 chunks of 16 bytes each; chunk (row r, K-group kg) -> (r/8) SBO + kg LBO + (r%8) 16
  {
    const bf16* xs = p.x + b * p.x_sb + h * p.x_sh;
    const bf16* ws = p.wt + (size_t)h * 128 * 64;
#pragma unroll
    for (int it = 0; it < (kPjTok * 8) / kPjThreads; ++it) {
      const int idx = tid + it * kPjThreads, r = idx >> 3, kg = idx & 7;
      const uint32_t off = (uint32_t)((r >> 3) * kPjSbo + kg * kPjLbo + (r & 7) * 16);
      uint4 xv = make_uint4(0u, 0u, 0u, 0u);
      if (t0 + r < p.L) xv = __ldcg(reinterpret_cast<const uint4*>(xs + (int64_t)(t0 + r) * p.x_sl + 8 * kg));
      const uint4 wv = __ldg(reinterpret_cast<const uint4*>(ws + r * 64 + 8 * kg));
      *reinterpret_cast<uint4*>(Asm + off) = xv;
      *reinterpret_cast<uint4*>(Bsm + off) = wv;
    }
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = tmem_slot;

  if (warp == 4 && T == 0) {
    // kind::f16 with bf16 operands (both K-major), fp32 accumulator, M = 128, N = 128; K = 64 in 4 steps
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      const uint64_t da = umma_desc(smem_u32(Asm) + ks * 2 * kPjLbo, kPjLbo, kPjSbo);
      const uint64_t db = umma_desc(smem_u32(Bsm) + ks * 2 * kPjLbo, kPjLbo, kPjSbo);
      const uint32_t acc = ks > 0;
      asm volatile(
          "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
          :: "r"(tmem), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
    }
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(smem_u32(&bar)) : "memory");
  }

  bool ok = true;
  if (warp < 4) {
    // ---- accumulator -> bf16 staging, Q column sums ----
    ok = mbar_wait(smem_u32(&bar), 0);
    if (ok) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int i = T >> 2, tq = T & 3;
      float cs[2][4][2];                                 // [chunk][x][e]: sums over this thread's tokens, Q half only
#pragma unroll
      for (int c = 0; c < 2; ++c)
#pragma unroll
        for (int x = 0; x < 4; ++x) cs[c][x][0] = cs[c][x][1] = 0.f;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int tokA = 32 * warp + 16 * j + i, tokB = tokA + 8;
#pragma unroll
        for (int chunk = 0; chunk < 4; ++chunk) {
          uint32_t r[16];
          tmem_ld_16x256b_x4(tmem + ((uint32_t)(32 * warp + 16 * j) << 16) + 32 * chunk, r);
          tmem_ld_wait();
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            const int col = 32 * chunk + 8 * x + 2 * tq;
            const float a0 = __uint_as_float(r[4 * x]), a1 = __uint_as_float(r[4 * x + 1]);
            const float b0 = __uint_as_float(r[4 * x + 2]), b1 = __uint_as_float(r[4 * x + 3]);
            *reinterpret_cast<uint32_t*>(stage + tokA * kPjStagePitch + 2 * col) = pack_bf2(a0, a1);
            *reinterpret_cast<uint32_t*>(stage + tokB * kPjStagePitch + 2 * col) = pack_bf2(b0, b1);
            if (chunk < 2) {                             // rows beyond L were loaded as zeros and add nothing
              cs[chunk][x][0] += a0 + b0;
              cs[chunk][x][1] += a1 + b1;
            }
          }
        }
      }
      if (p.sum_q) {
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              float s = cs[c][x][e];
              s += __shfl_xor_sync(0xffffffffu, s, 4);
              s += __shfl_xor_sync(0xffffffffu, s, 8);
              s += __shfl_xor_sync(0xffffffffu, s, 16);
              if (i == 0) qsum[warp][32 * c + 8 * x + 2 * tq + e] = s;
            }
      }
    }
    if (!ok && T == 0) report_timeout(p.status);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  // ---- whole rows out: 128 tokens x 16 pieces of 16 bytes (8 of Q, 8 of V) ----
  {
    bf16* qd = p.q + b * p.q_sb + h * p.q_sh;
    bf16* vd = p.v + b * p.v_sb + h * p.v_sh;
#pragma unroll
    for (int it = 0; it < (kPjTok * 16) / kPjThreads; ++it) {
      const int idx = tid + it * kPjThreads, pc = idx & 7, isv = (idx >> 3) & 1, r = idx >> 4;
      if (t0 + r < p.L) {
        const uint4 val = *reinterpret_cast<const uint4*>(stage + r * kPjStagePitch + isv * 128 + pc * 16);
        bf16* dst = isv ? vd + (int64_t)(t0 + r) * p.v_sl : qd + (int64_t)(t0 + r) * p.q_sl;
        __stcs(reinterpret_cast<uint4*>(dst + 8 * pc), val);
      }
    }
    if (p.sum_q && tid < 64) atomicAdd(p.sum_q + (size_t)slab * 64 + tid, qsum[0][tid] + qsum[1][tid] + qsum[2][tid] + qsum[3][tid]);
  }
  if (warp == 4) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(128));
  }
}

}  // namespace spectre

using namespace spectre;

extern "C" size_t spectre_project_workspace_bytes(const spectre_ctx* ctx, int32_t H, int32_t D) {
  (void)ctx;
  if (H < 1 || D != 64) return 0;
  return (size_t)H * 128 * 64 * sizeof(bf16);
}

extern "C" int spectre_project_qv(spectre_ctx* ctx, void* stream, const spectre_act* x, const void* Wq, const void* Wv,
                                  int32_t wdtype, const spectre_act* q, const spectre_act* v, float* sum_q, void* workspace,
                                  size_t workspace_bytes) {
  if (!ctx) return fail(SPECTRE_ERR_INVALID_ARG, "ctx is NULL");
  int rc = check_act(x, "x");
  if (rc != SPECTRE_OK) return rc;
  rc = check_act(q, "q");
  if (rc != SPECTRE_OK) return rc;
  rc = check_act(v, "v");
  if (rc != SPECTRE_OK) return rc;
  if (!Wq || !Wv) return fail(SPECTRE_ERR_INVALID_ARG, "a weight pointer is NULL");
  if (wdtype != SPECTRE_F32 && wdtype != SPECTRE_BF16) return fail(SPECTRE_ERR_INVALID_ARG, "unknown weight dtype");
  for (const spectre_act* a : {q, v})
    if (a->B != x->B || a->L != x->L || a->H != x->H || a->D != x->D || a->dtype != x->dtype)
      return fail(SPECTRE_ERR_INVALID_ARG, "q / v differ from x in shape or dtype");
  if (x->dtype != SPECTRE_BF16 || x->D != 64)
    return fail(SPECTRE_ERR_UNSUPPORTED, "the projection kernel takes bf16 activations with D = 64");
  if (q->ptr == x->ptr || v->ptr == x->ptr || q->ptr == v->ptr) return fail(SPECTRE_ERR_INVALID_ARG, "x, q and v must be distinct");
  const size_t need = (size_t)x->H * 128 * 64 * sizeof(bf16);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 15)) return fail(SPECTRE_ERR_WORKSPACE, "workspace is NULL or not 16-byte aligned");
  if (workspace_bytes < need) return fail(SPECTRE_ERR_WORKSPACE, "projection workspace too small");
  const int tiles = (x->L + kPjTok - 1) / kPjTok;
  if ((size_t)x->B * x->H * tiles > (size_t)0x7fffffff) return fail(SPECTRE_ERR_UNSUPPORTED, "too many tiles");
  SPECTRE_CUDA_OK(cudaSetDevice(ctx->device));
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  bf16* wt = reinterpret_cast<bf16*>(workspace);
  const unsigned wblocks = (unsigned)((x->H * 128 * 64 + 255) / 256);
  if (wdtype == SPECTRE_BF16)
    proj_weights_kernel<bf16><<<wblocks, 256, 0, st>>>(reinterpret_cast<const bf16*>(Wq), reinterpret_cast<const bf16*>(Wv), wt, x->H);
  else
    proj_weights_kernel<float><<<wblocks, 256, 0, st>>>(reinterpret_cast<const float*>(Wq), reinterpret_cast<const float*>(Wv), wt, x->H);
  SPECTRE_LAUNCH_OK("proj_weights_kernel");
  if (sum_q) SPECTRE_CUDA_OK(cudaMemsetAsync(sum_q, 0, (size_t)x->B * x->H * 64 * sizeof(float), st));
  ProjParams p = {};
  p.x = reinterpret_cast<const bf16*>(x->ptr); p.q = reinterpret_cast<bf16*>(q->ptr); p.v = reinterpret_cast<bf16*>(v->ptr);
  p.x_sb = x->stride_b; p.x_sl = x->stride_l; p.x_sh = x->stride_h;
  p.q_sb = q->stride_b; p.q_sl = q->stride_l; p.q_sh = q->stride_h;
  p.v_sb = v->stride_b; p.v_sl = v->stride_l; p.v_sh = v->stride_h;
  p.wt = wt; p.sum_q = sum_q; p.H = x->H; p.L = x->L; p.tiles = tiles; p.status = ctx->status_dev;
  SPECTRE_CUDA_OK(cudaFuncSetAttribute(project_qv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPjSmem));
  project_qv_kernel<<<(unsigned)((size_t)x->B * x->H * tiles), kPjThreads, kPjSmem, st>>>(p);
  SPECTRE_LAUNCH_OK("project_qv_kernel");
  return SPECTRE_OK;
}
