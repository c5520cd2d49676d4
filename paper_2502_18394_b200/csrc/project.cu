// Token projections (Sec. 3.2 step 1, Eq. 2): Q = X W^(q), V = X W^(v) per head, d = 64, bf16,
// on the 5th-generation tensor cores, with the pooled query sum of step 3a as a by-product.
//
// Per tile of 128 tokens of one (batch, head):
//     D[128 tokens x 128 outputs] (fp32, TMEM) = A[128 x 64] (X tile, bf16) * B[64 x 128] ([W^(q) | W^(v)], bf16)
// A is the X tile as a 128-byte-swizzled TMA box lands it (K-major: a row is one token's 64 channels);
// B, the weights, sits in shared memory in the K-major core-matrix layout without swizzle (8 rows x 16
// bytes per core matrix), copied from a transposed copy made once per call ([head][output][input]).
// The kernel is persistent (see project_qv_persistent_kernel).
#include <string>

#include "tc_common.cuh"

namespace spectre {

constexpr int kPjTok = 128;                      // tokens per tile
constexpr int kPjLbo = 2064;                     // K-group stride: 16 row groups x 128 + 16 (stores of a row spread over all banks)
constexpr int kPjSbo = 128;                      // 8-row group stride
constexpr int kPjOpBytes = 8 * kPjLbo;           // one 128 x 64 operand

template <typename WT> __device__ __forceinline__ float pj_wload(const WT* p);
template <> __device__ __forceinline__ float pj_wload<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float pj_wload<bf16>(const bf16* p) { return __bfloat162float(*p); }

// [H][d_in][d_out] (x @ W) for q and v  ->  wt[H][2 * 64][64] bf16 (output-major)
template <typename WT>
__global__ void __launch_bounds__(256) proj_weights_kernel(const WT* __restrict__ Wq, const WT* __restrict__ Wv,
                                                           bf16* __restrict__ wt, int H, float* __restrict__ sum_q, size_t nsum) {
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < nsum) sum_q[idx] = 0.f;             // the projection kernel adds its token sums into these (no memset node in the stream)
  if (idx >= (size_t)H * 128 * 64) return;
  const int i = idx & 63, o = (idx >> 6) & 127, h = idx >> 13;
  const WT* W = o < 64 ? Wq : Wv;
  const float w = pj_wload<WT>(W + ((size_t)h * 64 + i) * 64 + (o & 63));
  wt[idx] = __float2bfloat16_rn(w);
}

// =====================================================================================
// Persistent, one CTA per SM: whole [128 tokens x 64] tiles arrive as 128-byte-swizzled TMA boxes (the
// A operand as it lands, K-major), and leave as two such boxes (Q and V) through TMA stores.  Roles joined by mbarriers: a load warp
// keeps a ring of four X tiles full, an MMA warp issues the four K steps of a tile into one of two
// accumulators (and reloads the weights when its range of tiles crosses into another head), 8 epilogue
// warps (lane quadrant x Q / V half) round the accumulator to bf16 into one of two staging buffers and
// keep the Q column sums in registers until the (batch, head) changes, a store warp hands the staging
// buffers to TMA.  A CTA takes a contiguous range of tiles.  Every wait is bounded.
// =====================================================================================
constexpr int kPpRing = 4;                                   // X tiles in flight
constexpr int kPpTile = kPjTok * 128;                         // one [128 x 64] bf16 tile
constexpr int kPpEpiWarps = 8, kPpEpiThreads = 256;
constexpr int kPpThreads = kPpEpiThreads + 96;                // + MMA warp + load warp + store warp
constexpr int kPpSmem = kPpRing * kPpTile + 2 * 2 * kPpTile + kPjOpBytes + 256 + 1024;

struct ProjPersistParams {
  const bf16* wt;          // [H][128 outputs (q then v)][64 inputs]
  float* sum_q;            // [B,H,64] or NULL
  int H, tiles, nitems;    // tiles per (batch, head); items = B * H * tiles
  int* status;
};

__global__ void __launch_bounds__(kPpThreads, 1) project_qv_persistent_kernel(const __grid_constant__ CUtensorMap tm_x,
                                                                             const __grid_constant__ CUtensorMap tm_q,
                                                                             const __grid_constant__ CUtensorMap tm_v,
                                                                             const ProjPersistParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* Xs = smem;                                   // ring of X tiles (swizzled)
  unsigned char* Stg = smem + kPpRing * kPpTile;              // two buffers of [Q tile | V tile] (swizzled)
  unsigned char* Bsm = Stg + 4 * kPpTile;                     // weights, K-major without swizzle
  uint64_t* bars = reinterpret_cast<uint64_t*>(Bsm + kPjOpBytes);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 17);
  const int tid = threadIdx.x, warp = tid >> 5, T = tid & 31;
  const uint32_t bar0 = smem_u32(bars);
  auto xFull = [&](int s) { return bar0 + 8u * s; };
  auto xFree = [&](int s) { return bar0 + 32u + 8u * s; };
  auto accFull = [&](int a) { return bar0 + 64u + 8u * a; };
  auto accFree = [&](int a) { return bar0 + 80u + 8u * a; };
  auto stgFull = [&](int b) { return bar0 + 96u + 8u * b; };
  auto stgFree = [&](int b) { return bar0 + 112u + 8u * b; };
  const uint32_t wDone = bar0 + 128u;                         // all MMAs issued so far have read the weights

  if (tid == 0) {
    for (int s = 0; s < kPpRing; ++s) { mbar_init(xFull(s), 1); mbar_init(xFree(s), 1); }
    for (int a = 0; a < 2; ++a) {
      mbar_init(accFull(a), 1); mbar_init(accFree(a), kPpEpiThreads); mbar_init(stgFull(a), kPpEpiWarps); mbar_init(stgFree(a), 1);
    }
    mbar_init(wDone, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kPpEpiWarps) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(tmem_slot)), "r"(256));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *tmem_slot;
  const int per = (p.nitems + (int)gridDim.x - 1) / (int)gridDim.x;
  const int i0 = (int)blockIdx.x * per, i1 = min(p.nitems, i0 + per);
  bool ok = true;

  if (warp == kPpEpiWarps + 2) {
    // ---- load warp ----
    for (int item = i0, k = 0; item < i1 && ok; ++item, ++k) {
      const int slot = k % kPpRing;
      if (k >= kPpRing) ok = mbar_wait(xFree(slot), ((k / kPpRing) - 1) & 1);
      if (!ok) break;
      if (T == 0) {
        const int slab = item / p.tiles, tile = item - slab * p.tiles, b = slab / p.H, h = slab - b * p.H;
        mbar_expect_tx(xFull(slot), kPpTile);
        tma_load_4d(smem_u32(Xs) + slot * kPpTile, &tm_x, 0, tile * kPjTok, h, b, xFull(slot));
      }
      __syncwarp();
    }
    if (!ok) {                                                // leave no copy into this CTA in flight
      const int issued = min(i1 - i0, kPpRing);
      for (int s = 0; s < issued; ++s) mbar_wait(xFull(s), 0);
    }
  } else if (warp == kPpEpiWarps) {
    // ---- MMA warp (and the weights) ----
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
    int cur_h = -1, wphase = 0;
    for (int item = i0, k = 0; item < i1 && ok; ++item, ++k) {
      const int slab = item / p.tiles, h = slab % p.H, slot = k % kPpRing, a = k & 1;
      if (h != cur_h) {
        if (k > 0) {                                          // the MMAs issued so far still read the old weights
          if (T == 0) asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(wDone) : "memory");
          __syncwarp();
          ok = mbar_wait(wDone, wphase);
          wphase ^= 1;
          if (!ok) break;
        }
        const bf16* ws = p.wt + (size_t)h * 128 * 64;
        for (int idx = T; idx < 128 * 8; idx += 32) {
          const int r = idx >> 3, kg = idx & 7;
          *reinterpret_cast<uint4*>(Bsm + (r >> 3) * kPjSbo + kg * kPjLbo + (r & 7) * 16) = __ldg(reinterpret_cast<const uint4*>(ws + r * 64 + 8 * kg));
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        cur_h = h;
      }
      ok = mbar_wait(xFull(slot), (k / kPpRing) & 1);
      if (ok && k >= 2) ok = mbar_wait(accFree(a), ((k >> 1) - 1) & 1);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (T == 0) {
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          const uint64_t da = umma_desc_k_sw128(smem_u32(Xs) + slot * kPpTile + ks * 32, 1024);
          const uint64_t db = umma_desc(smem_u32(Bsm) + ks * 2 * kPjLbo, kPjLbo, kPjSbo);
          const uint32_t acc = ks > 0;
          asm volatile(
              "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
              :: "r"(tmem + 128 * a), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(accFull(a)) : "memory");
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(xFree(slot)) : "memory");
      }
      __syncwarp();
    }
  } else if (warp == kPpEpiWarps + 1) {
    // ---- store warp ----
    for (int item = i0, k = 0; item < i1 && ok; ++item, ++k) {
      const int bsel = k & 1;
      ok = mbar_wait(stgFull(bsel), (k >> 1) & 1);
      if (ok && T == 0) {
        const int slab = item / p.tiles, tile = item - slab * p.tiles, b = slab / p.H, h = slab - b * p.H;
        const uint32_t src = smem_u32(Stg) + bsel * 2 * kPpTile;
        tma_store_4d(&tm_q, 0, tile * kPjTok, h, b, src);     // rows beyond L fall outside the map and are not written
        tma_store_4d(&tm_v, 0, tile * kPjTok, h, b, src + kPpTile);
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        mbar_arrive(stgFree(bsel));
      }
      __syncwarp();
    }
    if (T == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  } else {
    // ---- epilogue warps: lane quadrant q, half 0 = the Q columns, 1 = the V columns ----
    const int q = warp & 3, half = warp >> 2, i = T >> 2, tq = T & 3;
    float cs[2][4][2];                                        // Q column sums over this thread's tokens of the current (batch, head)
#pragma unroll
    for (int c = 0; c < 2; ++c)
#pragma unroll
      for (int x = 0; x < 4; ++x) cs[c][x][0] = cs[c][x][1] = 0.f;
    auto flush = [&](int slab) {
#pragma unroll
      for (int c = 0; c < 2; ++c)
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            float sv = cs[c][x][e];
            sv += __shfl_xor_sync(0xffffffffu, sv, 4);
            sv += __shfl_xor_sync(0xffffffffu, sv, 8);
            sv += __shfl_xor_sync(0xffffffffu, sv, 16);
            if (i == 0) atomicAdd(p.sum_q + (size_t)slab * 64 + 32 * c + 8 * x + 2 * tq + e, sv);
            cs[c][x][e] = 0.f;
          }
    };
    int cur_slab = -1;
    for (int item = i0, k = 0; item < i1 && ok; ++item, ++k) {
      const int slab = item / p.tiles, a = k & 1;
      if (half == 0 && p.sum_q && slab != cur_slab) {
        if (cur_slab >= 0) flush(cur_slab);
        cur_slab = slab;
      }
      unsigned char* stg = Stg + a * 2 * kPpTile + half * kPpTile;
      if (k >= 2) ok = mbar_wait(stgFree(a), ((k >> 1) - 1) & 1);
      if (ok) ok = mbar_wait(accFull(a), (k >> 1) & 1);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      // the thread's four accumulator pieces (two 16-lane halves x two 32-column chunks) are requested together
      uint32_t r4[2][2][16];
#pragma unroll
      for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int chunk = 0; chunk < 2; ++chunk)
          tmem_ld_16x256b_x4(tmem + 128 * a + ((uint32_t)(32 * q + 16 * j) << 16) + 64 * half + 32 * chunk, r4[j][chunk]);
      tmem_ld_wait();
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive(accFree(a));                                  // the accumulator is in registers: the next MMAs may overwrite it
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int tokA = 32 * q + 16 * j + i, tokB = tokA + 8;
#pragma unroll
        for (int chunk = 0; chunk < 2; ++chunk) {
          const uint32_t (&r)[16] = r4[j][chunk];
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            const float a0 = __uint_as_float(r[4 * x]), a1 = __uint_as_float(r[4 * x + 1]);
            const float b0 = __uint_as_float(r[4 * x + 2]), b1 = __uint_as_float(r[4 * x + 3]);
            const int c16 = 4 * chunk + x;                    // 16-byte piece of the 128-byte row
            *reinterpret_cast<uint32_t*>(stg + tokA * 128 + ((c16 ^ (tokA & 7)) << 4) + 4 * tq) = pack_bf2(a0, a1);
            *reinterpret_cast<uint32_t*>(stg + tokB * 128 + ((c16 ^ (tokB & 7)) << 4) + 4 * tq) = pack_bf2(b0, b1);
            if (half == 0) {                                  // rows beyond L were read as zeros and add nothing
              cs[chunk][x][0] += a0 + b0;
              cs[chunk][x][1] += a1 + b1;
            }
          }
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (T == 0) mbar_arrive(stgFull(a));
    }
    if (half == 0 && p.sum_q && cur_slab >= 0) flush(cur_slab);
  }
  if (!ok && T == 0) report_timeout(p.status);
  __syncwarp();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == kPpEpiWarps) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(256));
  }
}

// tiles of [128 tokens x 64 channels] of [B, L, H, 64]: dims (channel, token, head, batch)
static int make_tile_map(CUtensorMap* tm, const spectre_act* a) {
  cuuint64_t dims[4] = {64, (cuuint64_t)a->L, (cuuint64_t)a->H, (cuuint64_t)a->B};
  cuuint64_t strides[3] = {(cuuint64_t)a->stride_l * 2, (cuuint64_t)a->stride_h * 2, (cuuint64_t)a->stride_b * 2};
  cuuint32_t box[4] = {64, kPjTok, 1, 1};
  cuuint32_t es[4] = {1, 1, 1, 1};
  CUresult r = tensor_map_encoder()(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, a->ptr, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(SPECTRE_ERR_CUDA, "cuTensorMapEncodeTiled failed (" + std::to_string((int)r) + ")");
  return SPECTRE_OK;
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
  const size_t nsum = sum_q ? (size_t)x->B * x->H * 64 : 0, nw = (size_t)x->H * 128 * 64;
  const unsigned wblocks = (unsigned)(((nsum > nw ? nsum : nw) + 255) / 256);
  if (wdtype == SPECTRE_BF16)
    proj_weights_kernel<bf16><<<wblocks, 256, 0, st>>>(reinterpret_cast<const bf16*>(Wq), reinterpret_cast<const bf16*>(Wv), wt, x->H,
                                                       sum_q, nsum);
  else
    proj_weights_kernel<float><<<wblocks, 256, 0, st>>>(reinterpret_cast<const float*>(Wq), reinterpret_cast<const float*>(Wv), wt, x->H,
                                                        sum_q, nsum);
  SPECTRE_LAUNCH_OK("proj_weights_kernel");
  if (tensor_map_encoder() == nullptr) return fail(SPECTRE_ERR_UNSUPPORTED, "the driver does not provide cuTensorMapEncodeTiled");
  CUtensorMap tm_x, tm_q, tm_v;
  rc = make_tile_map(&tm_x, x);
  if (rc == SPECTRE_OK) rc = make_tile_map(&tm_q, q);
  if (rc == SPECTRE_OK) rc = make_tile_map(&tm_v, v);
  if (rc != SPECTRE_OK) return rc;
  ProjPersistParams pp = {wt, sum_q, x->H, tiles, (int)((size_t)x->B * x->H * tiles), ctx->status_dev};
  SPECTRE_CUDA_OK(cudaFuncSetAttribute(project_qv_persistent_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPpSmem));
  const int grid = pp.nitems < ctx->sm_count ? pp.nitems : ctx->sm_count;
  project_qv_persistent_kernel<<<grid, kPpThreads, kPpSmem, st>>>(tm_x, tm_q, tm_v, pp);
  SPECTRE_LAUNCH_OK("project_qv_persistent_kernel");
  return SPECTRE_OK;
}
