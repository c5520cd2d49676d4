// Spectral mixer kernels: Y = R_n^{-1}( diag(g) R_n(V) )  (Sec. 3.2 steps 2 and 4).
//
// Formulation.  Two adjacent real columns a, b of a head are carried as ONE
// complex sequence z = a + jb.  With G the Hermitian extension of the half
// spectrum gate g (G_k = g_k for k <= n/2, conj(g_{n-k}) above, Im G_0 =
// Im G_{n/2} = 0), ifft_n(G * fft_n(z)) = irfft(g * rfft a) + j irfft(g * rfft b),
// so a head is D/2 complex transforms with no real/complex split or merge.
//
// The forward transform is decimation-in-frequency (natural order in,
// digit-reversed order out), the gate is applied in digit-reversed order, and
// the inverse is the mirrored decimation-in-time network, so no reordering pass
// exists.  A tile is 8 complex pairs (16 real columns) of one (batch, head).
//
//   onchip kernel   whole transform of a tile in shared memory; optionally a
//                   cluster of C CTAs splits the sequence and exchanges one
//                   radix-C stage through distributed shared memory.
//   strided kernels the outer factor N1 of a four-step transform n = N1 * M for
//                   n beyond the on-chip range, with the twiddles fused.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

#include <cstdlib>
#include <cstring>

namespace spectre {

int launch_mixer_tc8192(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, const float* g,
                        const spectre_act* y);   // mixer_tc.cu
bool tc8192_supported(const spectre_act* v, const spectre_act* y);                     // mixer_tc8k.cu
int launch_mixer_tc196(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, const float* g,
                       const spectre_act* y, const spectre_wavelet* wrm, float* level_gate_scratch);
bool tc196_fuses_wavelet(const spectre_wavelet* w);
size_t tc196_level_gate_bytes(int B, int H);

bool tc4k_supported(int n, int D);                                                     // mixer_tc4k.cu
size_t tc4k_workspace_bytes(const spectre_ctx* ctx, int n, int D, int nslab);
size_t tc4k_min_workspace(int n, int D);
bool tc4k_readout_supported(const spectre_ctx* ctx, const spectre_act* y, int n);
size_t tc4k_readout_workspace_bytes(int n, int D, int nslab);
int launch_readout_tc4k(const spectre_ctx* ctx, cudaStream_t st, const float* spec, const float* g, const spectre_act* y, int n,
                        void* ws, size_t ws_bytes);
int launch_mixer_tc4k(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, const float* g,
                      const spectre_act* y, int n, void* ws, size_t ws_bytes);

// Path choice for bf16 transforms.  SPECTRE_FORCE_PATH = alu | fused | staged overrides it (tests):
//   alu     fp32 butterflies only
//   fused   the single-kernel tensor-core mixer (n = 8192 only)
//   staged  transpose-in / tensor-core units / transpose-out (n = 4096 ... 131072, needs workspace)
enum { kPathAuto = 0, kPathAlu = 1, kPathFused = 2, kPathStaged = 3 };
static int forced_path() {
  const char* e = std::getenv("SPECTRE_FORCE_PATH");
  if (!e) return kPathAuto;
  if (std::strcmp(e, "alu") == 0) return kPathAlu;
  if (std::strcmp(e, "fused") == 0) return kPathFused;
  if (std::strcmp(e, "staged") == 0) return kPathStaged;
  return kPathAuto;
}

constexpr int kMaxStages = 8;
constexpr int kLocalMax = 2048;      // rows of a tile one CTA keeps in shared memory

struct OnchipParams {
  const void* src;       // real [B,L,H,D] tensor (src_ws = 0)
  void* dst;             // real [B,L,H,D] tensor (dst_ws = 0)
  float2* ws;            // complex workspace [slab_local][N1][M][D/2]
  const float2* g;       // gate [B*H][K]
  const float2* spec;    // half spectra [B*H][K][D] (mode 2)
  int64_t s_sb, s_sl, s_sh;
  int64_t d_sb, d_sl, d_sh;
  int H, D, L;
  int n, K;              // full transform length, bins
  int M, Mloc, C;        // this kernel's transform: M = C * Mloc
  int N1;                // outer factor of the four-step split (1 = none)
  int slab0;             // first (b*H + h) slab handled by this launch
  int ntile;             // 16-column tiles per slab
  int nstage;
  int radix[kMaxStages];
  int prefix[kMaxStages];   // prefix[i] = radix[0] * ... * radix[i-1]
  int mode;              // 0: forward, gate, inverse   1: forward only -> spectrum in ws
                         // 2: inverse only, from the gated half spectra in `spec`
  int src_ws, dst_ws;
  int decim;             // src_ws = 0 only: element j of sequence k1 is token N1 j + k1 (decimated input)
  int direct;            // C = 1, 2048 rows, 512 threads: the tile is fetched in one round of 16-byte loads
  void* ring;            // direct only: dense [B][n][H][D] copy of the (zero-padded) input written while loading, or NULL
  const float2* twq;     // (cos, sin)(2 pi r / 8192), r = 0..2048 (quarter wave): source of the twiddles of the fixed plan
  float scale;           // 1/n, folded into the gate
};

struct TileCoord {
  int rank, tile, k1, slab_local, b, h;
};

__device__ __forceinline__ TileCoord tile_coord(const OnchipParams& p) {
  TileCoord t;
  int u = blockIdx.x;
  t.rank = u % p.C;  u /= p.C;
  t.tile = u % p.ntile;  u /= p.ntile;
  t.k1 = u % p.N1;  u /= p.N1;
  t.slab_local = u;
  int slab = p.slab0 + u;
  t.b = slab / p.H;
  t.h = slab - t.b * p.H;
  return t;
}

// Element j of the length-M sequence, pair group pg (4 real columns / 2 pairs).
template <typename T>
__device__ __forceinline__ float4 load_elem(const OnchipParams& p, const TileCoord& tc, int j, int pg) {
  int col = tc.tile * 16 + pg * 4;
  if (col >= p.D) return make_float4(0.f, 0.f, 0.f, 0.f);
  if (p.src_ws) {
    size_t row = ((size_t)tc.slab_local * p.N1 + tc.k1) * p.M + j;
    return *reinterpret_cast<const float4*>(p.ws + row * (p.D / 2) + col / 2);
  }
  const int t = p.decim ? j * p.N1 + tc.k1 : j;
  if (t >= p.L) return make_float4(0.f, 0.f, 0.f, 0.f);
  const T* ptr = reinterpret_cast<const T*>(p.src) + tc.b * p.s_sb + (int64_t)t * p.s_sl + tc.h * p.s_sh + col;
  return io<T>::load4(ptr);
}

template <typename T>
__device__ __forceinline__ void store_elem(const OnchipParams& p, const TileCoord& tc, int j, int pg, float4 v) {
  int col = tc.tile * 16 + pg * 4;
  if (col >= p.D) return;
  if (p.dst_ws) {
    size_t row = ((size_t)tc.slab_local * p.N1 + tc.k1) * p.M + j;
    *reinterpret_cast<float4*>(p.ws + row * (p.D / 2) + col / 2) = v;
    return;
  }
  if (j >= p.L) return;
  T* ptr = reinterpret_cast<T*>(p.dst) + tc.b * p.d_sb + (int64_t)j * p.d_sl + tc.h * p.d_sh + col;
  io<T>::store4(ptr, v);
}

// Hermitian extension of the half-spectrum gate at full-spectrum index k.
__device__ __forceinline__ float2 gate_at(const float2* __restrict__ g, int k, int n) {
  int kk = (2 * k <= n) ? k : n - k;
  float2 v = __ldg(g + kk);
  if (kk != k) v.y = -v.y;
  if (k == 0 || 2 * k == n) v.y = 0.f;
  return v;
}

// One radix-R stage on block size S of the tile in shared memory.
//   forward (decimation in frequency): y_q'[m] = W_S^{m q'} sum_q x[m + q S/R] W_R^{q q'}
//   inverse (decimation in time):      x[m + q S/R] = sum_q' conj(W_R^{q q'}) conj(W_S^{m q'}) y_q'[m]
// COMPACT: tw holds only this stage's factors, W_S^{m q} at [q * (S/R) + m], so that the lanes of a warp
// (consecutive m) read consecutive words; the strided reads of the full table collide on a few banks when
// S is small.
template <int R, bool INV, bool COMPACT = false>
__device__ __forceinline__ void stage(float4* sm, const float2* tw, int Mloc, int S) {
  const int sub = S / R;
  const int step = Mloc / S;
  const int nwork = (Mloc / R) * 4;
  for (int w = threadIdx.x; w < nwork; w += blockDim.x) {
    int pg = w & 3, bf = w >> 2;
    int blk = bf / sub, m = bf - blk * sub;
    float4* base = sm + ((size_t)(blk * S + m) * 4 + pg);
    float2 xa[R], xb[R];
#pragma unroll
    for (int q = 0; q < R; ++q) {
      float4 v = base[(size_t)q * sub * 4];
      xa[q] = make_float2(v.x, v.y);
      xb[q] = make_float2(v.z, v.w);
    }
    if (INV) {
#pragma unroll
      for (int q = 1; q < R; ++q) {
        float2 t = COMPACT ? tw[q * sub + m] : tw[m * q * step];
        xa[q] = cmulc(xa[q], t);
        xb[q] = cmulc(xb[q], t);
      }
    }
    Dft<R, INV>::run(xa);
    Dft<R, INV>::run(xb);
    if (!INV) {
#pragma unroll
      for (int q = 1; q < R; ++q) {
        float2 t = COMPACT ? tw[q * sub + m] : tw[m * q * step];
        xa[q] = cmul(xa[q], t);
        xb[q] = cmul(xb[q], t);
      }
    }
#pragma unroll
    for (int q = 0; q < R; ++q) base[(size_t)q * sub * 4] = make_float4(xa[q].x, xa[q].y, xb[q].x, xb[q].y);
  }
}

template <bool INV>
__device__ __forceinline__ void run_stage(int R, float4* sm, const float2* tw, int Mloc, int S) {
  switch (R) {
    case 16: stage<16, INV>(sm, tw, Mloc, S); break;
    case 8: stage<8, INV>(sm, tw, Mloc, S); break;
    case 4: stage<4, INV>(sm, tw, Mloc, S); break;
    case 2: stage<2, INV>(sm, tw, Mloc, S); break;
    case 7: stage<7, INV>(sm, tw, Mloc, S); break;
    case 5: stage<5, INV>(sm, tw, Mloc, S); break;
    case 3: stage<3, INV>(sm, tw, Mloc, S); break;
    default: break;
  }
}

// Last forward stage (block size = radix, no twiddles) fused with the gate and,
// in mode 0, the first inverse stage.  Local position blk*R + q' holds local
// frequency kl = rev(blk) + (Mloc/R) q'.  Mode 2 starts here: the values come from
// the gated half spectra instead of the forward stages.
// FIX: the plan is known at compile time (Mloc = 2048 as 16 x 16 x 8), so the index arithmetic of the
// stages is shifts and masks instead of divisions by run-time values.
constexpr int kFixMloc = 2048;
template <typename T, int R, bool FIX>
__device__ __forceinline__ void middle(const OnchipParams& p, const TileCoord& tc, float4* sm) {
  const int Mloc = FIX ? kFixMloc : p.Mloc;
  const int nwork = (Mloc / R) * 4;
  const int nst = p.nstage;
  const int slab = p.slab0 + tc.slab_local;
  const float2* g = p.g + (size_t)slab * p.K;
  for (int w = threadIdx.x; w < nwork; w += blockDim.x) {
    int pg = w & 3, blk = w >> 2;
    float4* base = sm + ((size_t)blk * R * 4 + pg);
    float2 xa[R], xb[R];
    if (p.mode != 2) {
#pragma unroll
      for (int q = 0; q < R; ++q) {
        float4 v = base[q * 4];
        xa[q] = make_float2(v.x, v.y);
        xb[q] = make_float2(v.z, v.w);
      }
      Dft<R, false>::run(xa);
      Dft<R, false>::run(xb);
    }
    int rev = 0, tmp = blk;
    if (FIX) {
      rev = ((blk & 15) << 4) | (blk >> 4);          // blk < 256: two radix-16 digits swapped
    } else {
      for (int i = nst - 2; i >= 0; --i) {
        int d = tmp % p.radix[i];
        tmp /= p.radix[i];
        rev += d * p.prefix[i];
      }
    }
    const int kstep = Mloc / R;
#pragma unroll
    for (int q = 0; q < R; ++q) {
      int kl = rev + kstep * q;
      int kM = tc.rank + p.C * kl;
      if (p.mode == 0) {
        int k = tc.k1 + p.N1 * kM;
        float2 G = cscale(gate_at(g, k, p.n), p.scale);
        xa[q] = cmul(xa[q], G);
        xb[q] = cmul(xb[q], G);
      } else if (p.mode == 1) {
        store_elem<T>(p, tc, kM, pg, make_float4(xa[q].x, xa[q].y, xb[q].x, xb[q].y));
      } else {
        const int k = tc.k1 + p.N1 * kM, kk = (2 * k <= p.n) ? k : p.n - k;
        const int col = tc.tile * 16 + pg * 4;
        xa[q] = xb[q] = make_float2(0.f, 0.f);
        if (col < p.D) {
          const float2* row = p.spec + ((size_t)slab * p.K + kk) * p.D + col;
          const float2 gk = cscale(__ldg(g + kk), p.scale);
          xa[q] = pair_from_half(gk, *reinterpret_cast<const float4*>(row), k, kk, p.n);
          xb[q] = pair_from_half(gk, *reinterpret_cast<const float4*>(row + 2), k, kk, p.n);
        }
      }
    }
    if (p.mode != 1) {
      Dft<R, true>::run(xa);
      Dft<R, true>::run(xb);
#pragma unroll
      for (int q = 0; q < R; ++q) base[q * 4] = make_float4(xa[q].x, xa[q].y, xb[q].x, xb[q].y);
    }
  }
}

template <typename T>
__device__ __forceinline__ void run_middle(int R, const OnchipParams& p, const TileCoord& tc, float4* sm) {
  switch (R) {
    case 16: middle<T, 16, false>(p, tc, sm); break;
    case 8: middle<T, 8, false>(p, tc, sm); break;
    case 4: middle<T, 4, false>(p, tc, sm); break;
    case 2: middle<T, 2, false>(p, tc, sm); break;
    case 7: middle<T, 7, false>(p, tc, sm); break;
    case 5: middle<T, 5, false>(p, tc, sm); break;
    case 3: middle<T, 3, false>(p, tc, sm); break;
    default: middle<T, 1, false>(p, tc, sm); break;
  }
}

// Radix-C stage across the CTAs of a cluster.  CTA `rank` computes the
// butterflies of rows m in [rank*Mloc/C, (rank+1)*Mloc/C): forward reads
// x[m + q Mloc] from global memory and writes y_q'[m] into CTA q' (remote
// shared memory); inverse reads y_q'[m] from CTA q' and writes x[m + q Mloc].
template <typename T, int C, bool INV>
__device__ __forceinline__ void cross_stage(const OnchipParams& p, const TileCoord& tc, float4* sm,
                                            cg::cluster_group& cluster) {
  const int per = p.Mloc / C;
  const int nwork = per * 4;
  float4* remote[C];
#pragma unroll
  for (int q = 0; q < C; ++q) remote[q] = cluster.map_shared_rank(sm, q);
  // forward: the global loads of two work items are issued before either is used
  constexpr int UN = INV ? 1 : 2;
  for (int w0 = threadIdx.x; w0 < nwork; w0 += UN * blockDim.x) {
    float4 vin[UN][C];
#pragma unroll
    for (int u = 0; u < UN; ++u) {
      const int w = w0 + u * blockDim.x;
      if (w < nwork) {
        const int pg = w & 3, m = tc.rank * per + (w >> 2);
#pragma unroll
        for (int q = 0; q < C; ++q) vin[u][q] = INV ? remote[q][(size_t)m * 4 + pg] : load_elem<T>(p, tc, m + q * p.Mloc, pg);
      }
    }
#pragma unroll
    for (int u = 0; u < UN; ++u) {
      const int w = w0 + u * blockDim.x;
      if (w >= nwork) break;
      const int pg = w & 3, m = tc.rank * per + (w >> 2);
      float2 xa[C], xb[C];
      float2 w1 = twiddle_fwd((unsigned)m, (unsigned)p.M);
      float2 wq[C];
      wq[0] = make_float2(1.f, 0.f);
#pragma unroll
      for (int q = 1; q < C; ++q) wq[q] = (q == 1) ? w1 : cmul(wq[q / 2], wq[q - q / 2]);
#pragma unroll
      for (int q = 0; q < C; ++q) {
        const float4 v = vin[u][q];
        xa[q] = make_float2(v.x, v.y);
        xb[q] = make_float2(v.z, v.w);
        if (INV && q > 0) {
          xa[q] = cmulc(xa[q], wq[q]);
          xb[q] = cmulc(xb[q], wq[q]);
        }
      }
      Dft<C, INV>::run(xa);
      Dft<C, INV>::run(xb);
#pragma unroll
      for (int q = 0; q < C; ++q) {
        if (!INV && q > 0) {
          xa[q] = cmul(xa[q], wq[q]);
          xb[q] = cmul(xb[q], wq[q]);
        }
        float4 v = make_float4(xa[q].x, xa[q].y, xb[q].x, xb[q].y);
        if (INV) store_elem<T>(p, tc, m + q * p.Mloc, pg, v);
        else remote[q][(size_t)m * 4 + pg] = v;
      }
    }
  }
}

// 16 bytes of a row as float4 groups of 4 columns: one group for fp32, two for the 16-bit types
template <typename T> struct RowPiece;
template <> struct RowPiece<float> {
  static constexpr int kGroups = 1;
  static __device__ __forceinline__ float4 group(const uint4& r, int) {
    return make_float4(__uint_as_float(r.x), __uint_as_float(r.y), __uint_as_float(r.z), __uint_as_float(r.w));
  }
};
template <> struct RowPiece<bf16> {
  static constexpr int kGroups = 2;
  static __device__ __forceinline__ float4 group(const uint4& r, int g) {
    const unsigned lo = g ? r.z : r.x, hi = g ? r.w : r.y;
    return make_float4(__uint_as_float(lo << 16), __uint_as_float(lo & 0xffff0000u), __uint_as_float(hi << 16),
                       __uint_as_float(hi & 0xffff0000u));
  }
};
template <> struct RowPiece<f16> {
  static constexpr int kGroups = 2;
  static __device__ __forceinline__ float4 group(const uint4& r, int g) {
    const unsigned lo = g ? r.z : r.x, hi = g ? r.w : r.y;
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&lo));
    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&hi));
    return make_float4(a.x, a.y, b.x, b.y);
  }
};

// Input of a single-CTA transform of 2048 rows, 512 threads: the tile's 16 columns of a row are 4 / G
// 16-byte pieces, exactly kPieces per thread, fetched in one round with all loads in flight: fetch() issues
// them (first thing in the kernel, so their latency runs under the set-up), place() converts them into the
// shared-memory tile, ring() stores the raw pieces into a dense copy of the input, if one is wanted.
template <typename T>
struct TileRows {
  static constexpr int G = RowPiece<T>::kGroups;
  static constexpr int kPieces = 16 / G;
  static constexpr int kPerRow = 4 / G;              // pieces of a row that belong to the tile
  uint4 v[kPieces];

  static __device__ __forceinline__ int token(const OnchipParams& p, const TileCoord& tc, int i) {
    const int j = i / kPerRow;
    return p.decim ? j * p.N1 + tc.k1 : j;
  }
  __device__ __forceinline__ void fetch(const OnchipParams& p, const TileCoord& tc) {
    const T* src = reinterpret_cast<const T*>(p.src) + tc.b * p.s_sb + tc.h * p.s_sh + tc.tile * 16;
#pragma unroll
    for (int u = 0; u < kPieces; ++u) {
      const int i = threadIdx.x + u * blockDim.x;
      const int t = token(p, tc, i), col = 4 * G * (i % kPerRow);
      v[u] = make_uint4(0u, 0u, 0u, 0u);
      if (i < p.Mloc * kPerRow && t < p.L && tc.tile * 16 + col < p.D)
        v[u] = __ldcs(reinterpret_cast<const uint4*>(src + (int64_t)t * p.s_sl + col));
    }
  }
  __device__ __forceinline__ void place(const OnchipParams& p, float4* sm) const {
#pragma unroll
    for (int u = 0; u < kPieces; ++u) {
      const int i = threadIdx.x + u * blockDim.x;
      if (i < p.Mloc * kPerRow) {
#pragma unroll
        for (int g = 0; g < G; ++g) sm[(size_t)(i / kPerRow) * 4 + (i % kPerRow) * G + g] = RowPiece<T>::group(v[u], g);
      }
    }
  }
  __device__ __forceinline__ void ring(const OnchipParams& p, const TileCoord& tc) const {
    T* dst = reinterpret_cast<T*>(p.ring) + ((size_t)tc.b * p.n * p.H + tc.h) * p.D + tc.tile * 16;
#pragma unroll
    for (int u = 0; u < kPieces; ++u) {
      const int i = threadIdx.x + u * blockDim.x;
      const int col = 4 * G * (i % kPerRow);
      if (i < p.Mloc * kPerRow && tc.tile * 16 + col < p.D)
        __stcs(reinterpret_cast<uint4*>(dst + (size_t)token(p, tc, i) * p.H * p.D + col), v[u]);
    }
  }
};

template <typename T, int C, bool FIX>
__global__ void __launch_bounds__(512, 1) onchip_kernel(const OnchipParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int Mloc = FIX ? kFixMloc : p.Mloc;
  float4* sm = reinterpret_cast<float4*>(smem_raw);                       // [Mloc][4] (8 complex pairs per row)
  float2* tw = reinterpret_cast<float2*>(smem_raw + (size_t)Mloc * 64);    // [Mloc] exp(-j 2 pi i / Mloc)
  float2* tw128 = tw + Mloc;                                               // FIX: [16][8] W_128^{m q}, the second stage's factors
  const TileCoord tc = tile_coord(p);
  const bool direct = C == 1 && p.direct && p.mode != 2;
  TileRows<T> rows;
  if (direct) rows.fetch(p, tc);

  if (FIX) {
    // W_2048^i = exp(-j(quadrant pi/2 + 2 pi 4 (i % 512) / 8192)) from the quarter-wave table: one load serves
    // the four quadrants; 512 threads
    auto rot = [](float2 cs, int qd) {
      return qd == 0 ? make_float2(cs.x, -cs.y) : qd == 1 ? make_float2(-cs.y, -cs.x)
           : qd == 2 ? make_float2(-cs.x, cs.y) : make_float2(cs.y, cs.x);
    };
    const float2 cs = __ldg(p.twq + 4 * (threadIdx.x & 511));
    float2 cs2 = make_float2(1.f, 0.f);
    const int i2 = 16 * (threadIdx.x >> 3) * (threadIdx.x & 7);          // threads 0..127: q = tid / 8, m = tid % 8
    if (threadIdx.x < 128) cs2 = __ldg(p.twq + 4 * (i2 & 511));
    for (int i = threadIdx.x; i < Mloc; i += blockDim.x) tw[i] = rot(cs, i >> 9);
    if (threadIdx.x < 128) tw128[threadIdx.x] = rot(cs2, i2 >> 9);
  } else {
    for (int i = threadIdx.x; i < Mloc; i += blockDim.x) tw[i] = twiddle_fwd((unsigned)i, (unsigned)Mloc);
  }

  int S = Mloc;
  if (p.mode == 2) {
    if (FIX) S = 8;
    else for (int s = 0; s + 1 < p.nstage; ++s) S /= p.radix[s];   // where the forward stages would have left off
  } else {
    if (direct) {
      rows.place(p, sm);
      if (p.ring) rows.ring(p, tc);
      __syncthreads();
    } else if (C == 1) {
      // four elements per thread and round, their loads issued together
      for (int i0 = threadIdx.x; i0 < Mloc * 4; i0 += 4 * blockDim.x) {
        float4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int i = i0 + u * blockDim.x;
          if (i < Mloc * 4) v[u] = load_elem<T>(p, tc, i >> 2, i & 3);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int i = i0 + u * blockDim.x;
          if (i < Mloc * 4) sm[i] = v[u];
        }
      }
      __syncthreads();
    } else {
      cg::cluster_group cluster = cg::this_cluster();
      cluster.sync();                       // every CTA of the cluster is resident before remote writes
      cross_stage<T, C, false>(p, tc, sm, cluster);
      cluster.sync();
    }
    // forward stages (all but the last), the fused middle, inverse stages mirrored
    if (FIX) {
      stage<16, false>(sm, tw, kFixMloc, 2048);
      __syncthreads();
      stage<16, false, true>(sm, tw128, kFixMloc, 128);
      __syncthreads();
    } else {
      for (int s = 0; s + 1 < p.nstage; ++s) {
        run_stage<false>(p.radix[s], sm, tw, Mloc, S);
        S /= p.radix[s];
        __syncthreads();
      }
    }
  }
  if (FIX) middle<T, 8, true>(p, tc, sm);
  else run_middle<T>(p.nstage > 0 ? p.radix[p.nstage - 1] : 1, p, tc, sm);
  if (p.mode == 1) return;                // forward only: spectrum already written
  __syncthreads();
  if (FIX) {
    stage<16, true, true>(sm, tw128, kFixMloc, 128);
    __syncthreads();
    stage<16, true>(sm, tw, kFixMloc, 2048);
    __syncthreads();
  } else {
    for (int s = p.nstage - 2; s >= 0; --s) {
      S *= p.radix[s];
      run_stage<true>(p.radix[s], sm, tw, Mloc, S);
      __syncthreads();
    }
  }

  if (C == 1) {
    for (int i = threadIdx.x; i < Mloc * 4; i += blockDim.x) store_elem<T>(p, tc, i >> 2, i & 3, sm[i]);
  } else {
    cg::cluster_group cluster = cg::this_cluster();
    cluster.sync();
    cross_stage<T, C, true>(p, tc, sm, cluster);
    cluster.sync();                       // no CTA exits while a peer still reads its shared memory
  }
}

// ---- four-step outer factor -------------------------------------------------
// n = N1 * M, t = n1 M + n2, k = k1 + N1 k2.  Forward: for each n2 an N1-point
// DFT over n1, times W_n^{n2 k1}, stored at ws[k1][n2].  Inverse: the mirror.
struct StridedParams {
  const void* src;
  void* dst;
  float2* ws;
  int64_t s_sb, s_sl, s_sh;
  int64_t d_sb, d_sl, d_sh;
  int H, D, L, n, M, slab0, nslab;
};

template <typename T, int N1, bool INV>
__global__ void __launch_bounds__(256) strided_kernel(const StridedParams p) {
  const int npg = p.D / 4;
  const size_t total = (size_t)p.nslab * p.M * npg;
  size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  int pg = (int)(idx % npg);
  size_t r = idx / npg;
  int n2 = (int)(r % p.M);
  int slab_local = (int)(r / p.M);
  int slab = p.slab0 + slab_local;
  int b = slab / p.H, h = slab - b * p.H;
  const int col = pg * 4;

  float2 w1 = twiddle_fwd((unsigned)n2, (unsigned)p.n);
  float2 wq[N1];
  wq[0] = make_float2(1.f, 0.f);
#pragma unroll
  for (int q = 1; q < N1; ++q) wq[q] = (q == 1) ? w1 : cmul(wq[q / 2], wq[q - q / 2]);

  float2 xa[N1], xb[N1];
  if (!INV) {
    const T* src = reinterpret_cast<const T*>(p.src) + b * p.s_sb + h * p.s_sh + col;
#pragma unroll
    for (int n1 = 0; n1 < N1; ++n1) {
      int t = n1 * p.M + n2;
      float4 v = (t < p.L) ? io<T>::load4(src + (int64_t)t * p.s_sl) : make_float4(0.f, 0.f, 0.f, 0.f);
      xa[n1] = make_float2(v.x, v.y);
      xb[n1] = make_float2(v.z, v.w);
    }
  } else {
#pragma unroll
    for (int k1 = 0; k1 < N1; ++k1) {
      size_t row = ((size_t)slab_local * N1 + k1) * p.M + n2;
      float4 v = *reinterpret_cast<const float4*>(p.ws + row * (p.D / 2) + col / 2);
      xa[k1] = make_float2(v.x, v.y);
      xb[k1] = make_float2(v.z, v.w);
      if (k1 > 0) {
        xa[k1] = cmulc(xa[k1], wq[k1]);
        xb[k1] = cmulc(xb[k1], wq[k1]);
      }
    }
  }
  Dft<N1, INV>::run(xa);
  Dft<N1, INV>::run(xb);
  if (!INV) {
#pragma unroll
    for (int k1 = 0; k1 < N1; ++k1) {
      if (k1 > 0) {
        xa[k1] = cmul(xa[k1], wq[k1]);
        xb[k1] = cmul(xb[k1], wq[k1]);
      }
      size_t row = ((size_t)slab_local * N1 + k1) * p.M + n2;
      *reinterpret_cast<float4*>(p.ws + row * (p.D / 2) + col / 2) = make_float4(xa[k1].x, xa[k1].y, xb[k1].x, xb[k1].y);
    }
  } else {
    T* dst = reinterpret_cast<T*>(p.dst) + b * p.d_sb + h * p.d_sh + col;
#pragma unroll
    for (int n1 = 0; n1 < N1; ++n1) {
      int t = n1 * p.M + n2;
      if (t < p.L) io<T>::store4(dst + (int64_t)t * p.d_sl, make_float4(xa[n1].x, xa[n1].y, xb[n1].x, xb[n1].y));
    }
  }
}

// ---- host side ----------------------------------------------------------------
struct TransformPlan {
  int n, M, Mloc, C, N1;
  int nstage, radix[kMaxStages], prefix[kMaxStages];
  int threads;
  size_t smem;
};

// Chooses the decomposition for transform length n; false if unsupported.
static bool make_plan(const spectre_ctx* ctx, int n, TransformPlan* pl) {
  pl->n = n;
  pl->N1 = 1;
  pl->C = 1;
  if (n < 1) return false;
  int M = n;
  if (n > kLocalMax) {
    if (!is_pow2(n) || n > (1 << 17) || !ctx->cluster_ok) return false;
    if (n <= 4 * kLocalMax) {
      pl->C = n / kLocalMax;
    } else {
      pl->C = 4;
      pl->N1 = n / (4 * kLocalMax);
      M = 4 * kLocalMax;
    }
  }
  pl->M = M;
  pl->Mloc = M / pl->C;
  pl->nstage = radix_plan(pl->Mloc, pl->radix);
  if (pl->nstage < 0) return false;
  int pre = 1;
  for (int i = 0; i < pl->nstage; ++i) { pl->prefix[i] = pre; pre *= pl->radix[i]; }
  int want = pl->Mloc * 4 / 8;
  int thr = (want + 31) / 32 * 32;
  pl->threads = thr < 64 ? 64 : (thr > 512 ? 512 : thr);
  pl->smem = (size_t)pl->Mloc * 64 + (size_t)pl->Mloc * 8 + 128 * sizeof(float2);
  return pl->smem <= (size_t)ctx->max_smem_optin;
}

template <typename T, int C, bool FIX>
static int launch_onchip_cf(const OnchipParams& p, const TransformPlan& pl, int nslab, cudaStream_t st) {
  auto kern = onchip_kernel<T, C, FIX>;
  if (pl.smem > 48 * 1024)
    SPECTRE_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((size_t)nslab * pl.N1 * p.ntile * C), 1, 1);
  cfg.blockDim = dim3(pl.threads, 1, 1);
  cfg.dynamicSmemBytes = pl.smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (C > 1) ? 1 : 0;
  SPECTRE_CUDA_OK(cudaLaunchKernelEx(&cfg, kern, p));
  return SPECTRE_OK;
}

template <typename T, int C>
static int launch_onchip_c(const OnchipParams& p, const TransformPlan& pl, int nslab, cudaStream_t st) {
  const bool fix = pl.Mloc == kFixMloc && pl.nstage == 3 && pl.radix[0] == 16 && pl.radix[1] == 16 && pl.radix[2] == 8;
  return fix ? launch_onchip_cf<T, C, true>(p, pl, nslab, st) : launch_onchip_cf<T, C, false>(p, pl, nslab, st);
}

template <typename T>
static int launch_onchip(const OnchipParams& p, const TransformPlan& pl, int nslab, cudaStream_t st) {
  switch (pl.C) {
    case 1: return launch_onchip_c<T, 1>(p, pl, nslab, st);
    case 2: return launch_onchip_c<T, 2>(p, pl, nslab, st);
    case 4: return launch_onchip_c<T, 4>(p, pl, nslab, st);
    default: return fail(SPECTRE_ERR_UNSUPPORTED, "cluster size not supported");
  }
}

template <typename T, bool INV>
static int launch_strided(const StridedParams& p, int N1, cudaStream_t st) {
  size_t total = (size_t)p.nslab * p.M * (p.D / 4);
  unsigned blocks = (unsigned)((total + 255) / 256);
  switch (N1) {
    case 2: strided_kernel<T, 2, INV><<<blocks, 256, 0, st>>>(p); break;
    case 4: strided_kernel<T, 4, INV><<<blocks, 256, 0, st>>>(p); break;
    case 8: strided_kernel<T, 8, INV><<<blocks, 256, 0, st>>>(p); break;
    case 16: strided_kernel<T, 16, INV><<<blocks, 256, 0, st>>>(p); break;
    default: return fail(SPECTRE_ERR_UNSUPPORTED, "outer factor not supported");
  }
  SPECTRE_LAUNCH_OK("strided_kernel");
  return SPECTRE_OK;
}

static void fill_common(const spectre_ctx* ctx, OnchipParams& p, const TransformPlan& pl, int H, int D, int L) {
  p.twq = reinterpret_cast<const float2*>(ctx->tw8192);
  p.H = H; p.D = D; p.L = L;
  p.n = pl.n; p.K = pl.n / 2 + 1;
  p.M = pl.M; p.Mloc = pl.Mloc; p.C = pl.C; p.N1 = pl.N1;
  p.ntile = (D + 15) / 16;
  p.nstage = pl.nstage;
  for (int i = 0; i < kMaxStages; ++i) { p.radix[i] = i < pl.nstage ? pl.radix[i] : 1; p.prefix[i] = i < pl.nstage ? pl.prefix[i] : 1; }
  p.scale = 1.0f / (float)pl.n;
}

static size_t slab_ws_bytes(int n, int D) { return (size_t)n * (D / 2) * sizeof(float2); }

// Number of (batch, head) slabs whose four-step intermediates are processed per
// group of launches: few enough that the group's workspace stays L2-resident.
static int preferred_group(const spectre_ctx* ctx, int n, int D, int nslab_total) {
  size_t per = slab_ws_bytes(n, D);
  size_t budget = ctx->l2_bytes / 2;
  int g = (int)(budget / per);
  if (g < 1) g = 1;
  if (g > nslab_total) g = nslab_total;
  return g;
}

template <typename T>
static int mixer_typed(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, const float* g,
                       const spectre_act* y, const TransformPlan& pl, void* ws, size_t ws_bytes) {
  const int nslab = v->B * v->H;
  OnchipParams p = {};
  fill_common(ctx, p, pl, v->H, v->D, v->L);
  p.src = v->ptr; p.dst = y->ptr;
  p.s_sb = v->stride_b; p.s_sl = v->stride_l; p.s_sh = v->stride_h;
  p.d_sb = y->stride_b; p.d_sl = y->stride_l; p.d_sh = y->stride_h;
  p.g = reinterpret_cast<const float2*>(g);
  p.mode = 0;
  if (pl.N1 == 1) {
    p.slab0 = 0; p.src_ws = 0; p.dst_ws = 0; p.ws = nullptr;
    return launch_onchip<T>(p, pl, nslab, st);
  }
  const size_t per = slab_ws_bytes(pl.n, v->D);
  int group = (int)(ws_bytes / per);
  int pref = preferred_group(ctx, pl.n, v->D, nslab);
  if (group > pref) group = pref;
  if (group < 1) return fail(SPECTRE_ERR_WORKSPACE, "mixer workspace smaller than one (batch, head) slab");
  StridedParams sp = {};
  sp.src = v->ptr; sp.dst = y->ptr; sp.ws = reinterpret_cast<float2*>(ws);
  sp.s_sb = v->stride_b; sp.s_sl = v->stride_l; sp.s_sh = v->stride_h;
  sp.d_sb = y->stride_b; sp.d_sl = y->stride_l; sp.d_sh = y->stride_h;
  sp.H = v->H; sp.D = v->D; sp.L = v->L; sp.n = pl.n; sp.M = pl.M;
  p.ws = sp.ws; p.src_ws = 1; p.dst_ws = 1;
  for (int s0 = 0; s0 < nslab; s0 += group) {
    int cnt = nslab - s0 < group ? nslab - s0 : group;
    sp.slab0 = s0; sp.nslab = cnt;
    p.slab0 = s0;
    int rc = launch_strided<T, false>(sp, pl.N1, st);
    if (rc != SPECTRE_OK) return rc;
    rc = launch_onchip<T>(p, pl, cnt, st);
    if (rc != SPECTRE_OK) return rc;
    rc = launch_strided<T, true>(sp, pl.N1, st);
    if (rc != SPECTRE_OK) return rc;
  }
  return SPECTRE_OK;
}

// Forward transforms of the decimated sequences (used by the cache prefill and the gate gradient): with n = N1 M and token
// t = N1 n2 + n1, ws[slab_local][n1][k2][D/2] = sum_n2 z[N1 n2 + n1] W_M^{n2 k2}, read straight from the
// activations.  The radix-N1 step over n1 (bin k2 + M k1 = sum_n1 W_N1^{n1 k1} W_n^{n1 k2} ws[n1][k2]) is
// left to the caller, which can fuse it with what follows.  N1 = 1: the spectrum itself.  With `ring`
// (dense [B][n][H][D], the activations' dtype) the pass also writes the zero-padded input there when its
// load path can; *ring_done tells the caller whether it did.
int forward_decimated(const spectre_ctx* ctx, cudaStream_t st, const spectre_act* v, int n, int slab0, int cnt,
                      float2* ws, int* N1_out, int* M_out, void* ring, int* ring_done) {
  TransformPlan pl;
  if (!make_plan(ctx, n, &pl)) return fail(SPECTRE_ERR_UNSUPPORTED, "transform length not supported");
  // Up to 16 sequences of kLocalMax tokens: single-CTA transforms, no exchange between CTAs.
  const bool direct = n > kLocalMax && n <= 16 * kLocalMax && v->D % 8 == 0;
  if (direct) {
    TransformPlan one;
    if (!make_plan(ctx, kLocalMax, &one)) return fail(SPECTRE_ERR_UNSUPPORTED, "transform length not supported");
    pl = one;
    pl.n = n;
    pl.N1 = n / kLocalMax;
  }
  *N1_out = pl.N1; *M_out = pl.M;
  OnchipParams p = {};
  fill_common(ctx, p, pl, v->H, v->D, v->L);
  p.src = v->ptr;
  p.s_sb = v->stride_b; p.s_sl = v->stride_l; p.s_sh = v->stride_h;
  p.ws = ws; p.mode = 1; p.dst_ws = 1; p.slab0 = slab0;
  p.src_ws = 0; p.decim = pl.N1 > 1; p.direct = direct;
  p.ring = direct ? ring : nullptr;
  *ring_done = direct && ring != nullptr;
  SPECTRE_IO_DISPATCH(v->dtype, return launch_onchip<T>(p, pl, cnt, st));
}

// Inverse transform only (read-out of the Prefix-FFT cache): y = R_n^{-1}(diag(g) spec) for all
// slabs, spec = half spectra [B*H][K][D].  Same kernels as the mixer, entered after the gate.
template <typename T>
static int inverse_typed(const spectre_ctx* ctx, cudaStream_t st, const float2* spec, const float* g, const spectre_act* y,
                         const TransformPlan& pl, void* ws, size_t ws_bytes) {
  const int nslab = y->B * y->H;
  OnchipParams p = {};
  fill_common(ctx, p, pl, y->H, y->D, y->L);
  p.dst = y->ptr;
  p.d_sb = y->stride_b; p.d_sl = y->stride_l; p.d_sh = y->stride_h;
  p.g = reinterpret_cast<const float2*>(g);
  p.spec = spec;
  p.mode = 2;
  if (pl.N1 == 1) {
    p.slab0 = 0; p.dst_ws = 0; p.ws = nullptr;
    return launch_onchip<T>(p, pl, nslab, st);
  }
  const size_t per = slab_ws_bytes(pl.n, y->D);
  int group = (int)(ws_bytes / per);
  int pref = preferred_group(ctx, pl.n, y->D, nslab);
  if (group > pref) group = pref;
  if (group < 1) return fail(SPECTRE_ERR_WORKSPACE, "read-out workspace smaller than one (batch, head) slab");
  StridedParams sp = {};
  sp.dst = y->ptr; sp.ws = reinterpret_cast<float2*>(ws);
  sp.d_sb = y->stride_b; sp.d_sl = y->stride_l; sp.d_sh = y->stride_h;
  sp.H = y->H; sp.D = y->D; sp.L = y->L; sp.n = pl.n; sp.M = pl.M;
  p.ws = sp.ws; p.dst_ws = 1;
  for (int s0 = 0; s0 < nslab; s0 += group) {
    int cnt = nslab - s0 < group ? nslab - s0 : group;
    sp.slab0 = s0; sp.nslab = cnt;
    p.slab0 = s0;
    int rc = launch_onchip<T>(p, pl, cnt, st);
    if (rc != SPECTRE_OK) return rc;
    rc = launch_strided<T, true>(sp, pl.N1, st);
    if (rc != SPECTRE_OK) return rc;
  }
  return SPECTRE_OK;
}

// Enough for either route of inverse_from_spectrum (the output dtype is not known here)
size_t inverse_workspace_bytes(const spectre_ctx* ctx, int n, int D, int nslab) {
  TransformPlan pl;
  if (!make_plan(ctx, n, &pl)) return 0;
  size_t a = pl.N1 == 1 ? 0 : (size_t)preferred_group(ctx, n, D, nslab) * slab_ws_bytes(n, D);
  if (ctx->dft64 && tc4k_supported(n, D) && D <= 64 && forced_path() != kPathAlu) {
    const size_t b = tc4k_readout_workspace_bytes(n, D, nslab);
    if (b > a) a = b;
  }
  return a;
}

int inverse_from_spectrum(const spectre_ctx* ctx, cudaStream_t st, const float* spec, const float* g, const spectre_act* y,
                          int n, void* ws, size_t ws_bytes) {
  TransformPlan pl;
  if (!make_plan(ctx, n, &pl)) return fail(SPECTRE_ERR_UNSUPPORTED, "transform length not supported");
  if (pl.N1 > 1) {
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 15)) return fail(SPECTRE_ERR_WORKSPACE, "workspace is NULL or not 16-byte aligned");
  }
  // 16-bit outputs of a staged length: gated operand images from the spectra, then the inverse half of the
  // tensor-core path (the fp16 intermediates meet the 16-bit output bound; fp32 outputs stay on the fp32 kernels)
  if (forced_path() != kPathAlu && tc4k_readout_supported(ctx, y, n) && ws && !(reinterpret_cast<uintptr_t>(ws) & 15) &&
      ws_bytes >= tc4k_min_workspace(n, y->D))
    return launch_readout_tc4k(ctx, st, spec, g, y, n, ws, ws_bytes);
  const float2* sp = reinterpret_cast<const float2*>(spec);
  SPECTRE_IO_DISPATCH(y->dtype, return inverse_typed<T>(ctx, st, sp, g, y, pl, ws, ws_bytes));
}

bool transform_supported(const spectre_ctx* ctx, int n) {
  TransformPlan pl;
  return make_plan(ctx, n, &pl);
}

size_t transform_slab_bytes(int n, int D) { return slab_ws_bytes(n, D); }

}  // namespace spectre

using namespace spectre;

extern "C" size_t spectre_mixer_workspace_bytes(const spectre_ctx* ctx, int32_t B, int32_t L, int32_t H, int32_t D,
                                                int32_t n_fft, int32_t dtype) {
  (void)L;
  TransformPlan pl;
  if (!ctx || B < 1 || H < 1 || D < 8 || !make_plan(ctx, n_fft, &pl)) return 0;
  const int force = forced_path();
  if ((dtype == SPECTRE_BF16 || dtype == SPECTRE_F16) && ctx->dft64 && tc4k_supported(n_fft, D) && force != kPathAlu && force != kPathFused &&
      (n_fft != 8192 || force == kPathStaged))               // n = 8192 defaults to the single-kernel path
    return tc4k_workspace_bytes(ctx, n_fft, D, B * H);
  if ((dtype == SPECTRE_BF16 || dtype == SPECTRE_F16) && n_fft == 196 && D == 64 && ctx->dft49 && force != kPathAlu)
    return tc196_level_gate_bytes(B, H);                     // level gates of a fused refinement
  if (pl.N1 == 1) return 0;
  return (size_t)preferred_group(ctx, n_fft, D, B * H) * slab_ws_bytes(n_fft, D);
}

extern "C" int spectre_mixer_forward(spectre_ctx* ctx, void* stream, const spectre_act* v, const float* g,
                                     const spectre_act* y, int32_t n_fft, const spectre_wavelet* wrm,
                                     void* workspace, size_t workspace_bytes) {
  if (!ctx) return fail(SPECTRE_ERR_INVALID_ARG, "ctx is NULL");
  int rc = check_act(v, "v");
  if (rc != SPECTRE_OK) return rc;
  rc = check_act(y, "y");
  if (rc != SPECTRE_OK) return rc;
  if (!g || (reinterpret_cast<uintptr_t>(g) & 7)) return fail(SPECTRE_ERR_INVALID_ARG, "g is NULL or not 8-byte aligned");
  if (v->B != y->B || v->L != y->L || v->H != y->H || v->D != y->D || v->dtype != y->dtype)
    return fail(SPECTRE_ERR_INVALID_ARG, "v and y differ in shape or dtype");
  if (n_fft < v->L) return fail(SPECTRE_ERR_INVALID_ARG, "n_fft smaller than L");
  TransformPlan pl;
  if (!make_plan(ctx, n_fft, &pl)) return fail(SPECTRE_ERR_UNSUPPORTED, "n_fft outside the supported set");
  const int force = forced_path();
  const bool tc_ok = (v->dtype == SPECTRE_BF16 || v->dtype == SPECTRE_F16) && ctx->dft64 != nullptr && force != kPathAlu;
  const bool ws_ok = workspace && !(reinterpret_cast<uintptr_t>(workspace) & 15);
  const bool tc196 = tc_ok && n_fft == 196 && v->D == 64 && ctx->dft49 != nullptr;
  const bool fused = tc_ok && n_fft == 8192 && force != kPathStaged && tc8192_supported(v, y);
  const bool staged = !fused && tc_ok && force != kPathFused && tc4k_supported(n_fft, v->D) && ws_ok &&
                      workspace_bytes >= tc4k_min_workspace(n_fft, v->D);
  if (!staged && !fused && pl.N1 > 1) {
    if (!ws_ok) return fail(SPECTRE_ERR_WORKSPACE, "workspace is NULL or not 16-byte aligned");
    if (workspace_bytes < slab_ws_bytes(n_fft, v->D))
      return fail(SPECTRE_ERR_WORKSPACE, "mixer workspace smaller than one (batch, head) slab");
  }
  if (staged || pl.N1 > 1) {
    // any overlap of the two views' byte extents counts, not only equal base pointers
    auto extent = [](const spectre_act* a, const char** lo, const char** hi) {
      const int64_t es = io_elem_bytes(a->dtype);
      const int64_t last = (a->B - 1) * a->stride_b + (a->L - 1) * a->stride_l + (a->H - 1) * a->stride_h + a->D;
      *lo = reinterpret_cast<const char*>(a->ptr);
      *hi = *lo + last * es;
    };
    const char *vl, *vh, *yl, *yh;
    extent(v, &vl, &vh);
    extent(y, &yl, &yh);
    if (vl < yh && yl < vh) return fail(SPECTRE_ERR_INVALID_ARG, "y may not overlap v on the multi-pass path");
  }
  if (wrm) {
    if (wrm->levels < 1 || wrm->levels > 10 || (v->L % (1 << wrm->levels)) != 0)
      return fail(SPECTRE_ERR_INVALID_ARG, "wavelet levels: 2^J must divide L");
  }
  SPECTRE_CUDA_OK(cudaSetDevice(ctx->device));
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (staged || fused || tc196) {
    // n = 196: the refinement rides in the kernel's store phase when it can
    // (level gates given, 8-byte aligned; or the MLP's weights and room for its output in the workspace)
    const bool fuse_wrm = tc196 && wrm && tc196_fuses_wavelet(wrm) &&
                          (wrm->level_gates ? !(reinterpret_cast<uintptr_t>(wrm->level_gates) & 7)
                                            : (wrm->qbar && wrm->Ww1 && wrm->bw1 && wrm->Ww2 && wrm->bw2 &&
                                               (wrm->wdtype == SPECTRE_F32 || wrm->wdtype == SPECTRE_BF16) && ws_ok &&
                                               workspace_bytes >= tc196_level_gate_bytes(v->B, v->H)));
    rc = tc196 ? launch_mixer_tc196(ctx, st, v, g, y, fuse_wrm ? wrm : nullptr, reinterpret_cast<float*>(workspace))
               : (staged ? launch_mixer_tc4k(ctx, st, v, g, y, n_fft, workspace, workspace_bytes)
                         : launch_mixer_tc8192(ctx, st, v, g, y));
    if (rc != SPECTRE_OK) return rc;
    if (wrm && !fuse_wrm) return spectre_wavelet_refine(ctx, stream, y, y, wrm);
    return SPECTRE_OK;
  }
  SPECTRE_IO_DISPATCH(v->dtype, rc = mixer_typed<T>(ctx, st, v, g, y, pl, workspace, workspace_bytes));
  if (rc != SPECTRE_OK) return rc;
  if (wrm) return spectre_wavelet_refine(ctx, stream, y, y, wrm);
  return SPECTRE_OK;
}
