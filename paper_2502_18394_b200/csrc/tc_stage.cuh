// The 64 x 64 stages of a 4096-point transform on the tensor cores, shared by the n = 8192 kernel
// (two such problems per tile) and the core kernel of the longer transforms (one per unit): operand
// strides per stage and the epilogues between the stages.  Conventions as in mixer_tc8k.cu: the
// accumulator of a stage has the new digit along its rows and, along its columns, the column pair c
// and the digit that is contracted next.
#pragma once
#include "tc_common.cuh"

namespace spectre {

// Operand strides (bytes) per stage: LBO between core matrices along K, SBO between 8-column
// groups.  Stage 0 is the TMA landing image (dense).  The others are chosen so that the stores
// of the epilogue that writes them spread over all 32 banks.
constexpr int k8Lbo0 = 4096, k8Sbo0 = 128;       // columns 64 c + t2, K = t1
constexpr int k8Lbo1 = 4160, k8Sbo1 = 128;       // columns 64 c + k1, K = t2
constexpr int k8Lbo2 = 4112, k8Sbo2 = 128;       // columns 64 c + k1, K = k2
constexpr int k8Lbo3 = 144, k8Sbo3 = 2336;       // columns 4 s1 + c,  K = k1
constexpr int k8BBytes = 32 * k8Sbo3;            // largest of the four images (74752)
constexpr int k8GStride = 72;                    // gate table: entry (k1, k2) at 72 k2 + k1
constexpr int k8GBytes = 64 * k8GStride * 4;     // per half, fp16 (re, im)

// Epilogue after a stage whose accumulator has columns 64 c + d (d = the digit still to be
// contracted), for one warp: TMEM lane quadrant q, pair c.  A thread owns rows (new digit)
// 16 q' + T/4 for the two lane groups q' = 2q, 2q+1 and the columns d = 32 chunk + 8 x + 2 (T%4)
// + {0, 1}.  It multiplies by W_4096^{row d}: the even column's factor comes from a table laid out in
// this thread order (one 8-byte load per x; 16 KiB in all, which stays in the 28 KB of L1 that 228 KB of
// shared memory leave: a table with both columns' factors does not, and its reads were L2 traffic of
// the size of the operands), the odd column's is that times W_4096^{row} (wr0, wr1: the thread's two
// rows).  The two products of an x run as packed fp32 pairs; the transposed operand (row -> column index,
// d -> K) leaves as one 8-byte store per x.  TMEM loads run one 32-column chunk ahead.
//   COLS: order of the output columns.  1: 64 c + row.  0: 4 row + c.  2: 16 (row / 4) + 8 (c / 2) +
//   2 (row % 4) + c % 2, which keeps the four rows a half-warp writes at once in four different
//   16-byte slots of a core matrix even when LBO and SBO are multiples of 128 (dense images), and
//   leaves all four pairs of a row in one thread of the epilogue that reads the next accumulator.
template <int LBO, int SBO, int COLS>
__device__ __forceinline__ void epilogue_twiddle(uint32_t tmem_d, unsigned char* Bout, int q, int c, int T,
                                                 const float2* __restrict__ tw, float2 wr0, float2 wr1) {
  const int i = T >> 2, tq = T & 3;
  uint32_t r[2][16];
  const uint32_t taddr0 = tmem_d + ((uint32_t)(32 * q) << 16) + 64 * c;
  tmem_ld_16x256b_x4(taddr0, r[0]);
  tw += q * 512 + T;
#pragma unroll
  for (int step = 0; step < 4; ++step) {                      // step = 2 j + chunk
    const int j = step >> 1, chunk = step & 1;
    const int row = 8 * (2 * q + j) + i;
    float2 w[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) w[x] = __ldg(tw + (4 * step + x) * 32);
    tmem_ld_wait();
    if (step < 3) {
      const int nj = (step + 1) >> 1, nchunk = (step + 1) & 1;
      tmem_ld_16x256b_x4(taddr0 + ((uint32_t)(16 * nj) << 16) + 32 * nchunk, r[(step + 1) & 1]);
    }
    const uint32_t (&rr)[16] = r[step & 1];
    const uint32_t colpart = COLS == 1 ? (uint32_t)((8 * c + (row >> 3)) * SBO + (row & 7) * 16)
                           : COLS == 0 ? (uint32_t)((row >> 1) * SBO + (4 * (row & 1) + c) * 16)
                                       : (uint32_t)((2 * (row >> 2) + (c >> 1)) * SBO + (2 * (row & 3) + (c & 1)) * 16);
    const uint32_t base = colpart + (uint32_t)((8 * chunk + (tq >> 1)) * LBO + 8 * (tq & 1));
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const float2 w1 = cmul(w[x], j ? wr1 : wr0);
      *reinterpret_cast<uint2*>(Bout + base + 2 * x * LBO) =
          cmul2_pack_h2(pk2u(rr[4 * x], rr[4 * x + 1]), pk2u(rr[4 * x + 2], rr[4 * x + 3]), pk2(w[x].x, w1.x), pk2(w[x].y, w1.y));
    }
  }
}

// The same for the two pairs c0 and c0 + 1 of one warp: the twiddles depend on (row, d) only, so each
// table entry is fetched once and used for both pairs.  The eight (step, pair) accumulator chunks are
// walked in the order (step, pair) with the TMEM loads one chunk ahead.
template <int LBO, int SBO, int COLS>
__device__ __forceinline__ void epilogue_twiddle2(uint32_t tmem_d, unsigned char* Bout, int q, int c0, int T,
                                                  const float2* __restrict__ tw, float2 wr0, float2 wr1) {
  const int i = T >> 2, tq = T & 3;
  uint32_t r[2][16];
  const uint32_t taddr0 = tmem_d + ((uint32_t)(32 * q) << 16) + 64 * c0;
  tmem_ld_16x256b_x4(taddr0, r[0]);
  tw += q * 512 + T;
  float2 w[4];
#pragma unroll
  for (int s8 = 0; s8 < 8; ++s8) {                            // s8 = 2 step + cc, step = 2 j + chunk
    const int step = s8 >> 1, cc = s8 & 1, c = c0 + cc;
    const int j = step >> 1, chunk = step & 1;
    const int row = 8 * (2 * q + j) + i;
    if (cc == 0) {
#pragma unroll
      for (int x = 0; x < 4; ++x) w[x] = __ldg(tw + (4 * step + x) * 32);
    }
    tmem_ld_wait();
    if (s8 < 7) {
      const int ns = (s8 + 1) >> 1, ncc = (s8 + 1) & 1;
      tmem_ld_16x256b_x4(taddr0 + ((uint32_t)(16 * (ns >> 1)) << 16) + 32 * (ns & 1) + 64 * ncc, r[(s8 + 1) & 1]);
    }
    const uint32_t (&rr)[16] = r[s8 & 1];
    const uint32_t colpart = COLS == 1 ? (uint32_t)((8 * c + (row >> 3)) * SBO + (row & 7) * 16)
                           : COLS == 0 ? (uint32_t)((row >> 1) * SBO + (4 * (row & 1) + c) * 16)
                                       : (uint32_t)((2 * (row >> 2) + (c >> 1)) * SBO + (2 * (row & 3) + (c & 1)) * 16);
    const uint32_t base = colpart + (uint32_t)((8 * chunk + (tq >> 1)) * LBO + 8 * (tq & 1));
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const float2 w1 = cmul(w[x], j ? wr1 : wr0);
      *reinterpret_cast<uint2*>(Bout + base + 2 * x * LBO) =
          cmul2_pack_h2(pk2u(rr[4 * x], rr[4 * x + 1]), pk2u(rr[4 * x + 2], rr[4 * x + 3]), pk2(w[x].x, w1.x), pk2(w[x].y, w1.y));
    }
  }
}

// Epilogue after the second forward stage: rows k2, columns 64 c + k1; bin 2 (k1 + 64 k2) + parity
// of the half.  Gate, conjugate (for the inverse by the conj trick) and write the operand with
// the same columns and K = k2.  GXOR: the table is dense (64 entries per k2) with k1 XOR 8 (k2 % 4)
// as the column, which spreads the four rows of a half-warp over the banks without padding;
// otherwise entry (k1, k2) sits at GSTRIDE k2 + k1.
template <int LBO, int SBO, int GSTRIDE, bool GXOR>
__device__ __forceinline__ void epilogue_gate_t(uint32_t tmem_d, unsigned char* Bout, int q, int c, int T,
                                                const uint32_t* __restrict__ Gtab) {
  const int i = T >> 2, tq = T & 3;
  uint32_t r[2][16];
  const uint32_t taddr0 = tmem_d + ((uint32_t)(32 * q) << 16) + 64 * c;
  tmem_ld_16x256b_x4(taddr0, r[0]);
#pragma unroll
  for (int step = 0; step < 4; ++step) {
    const int j = step >> 1, chunk = step & 1;
    const int row = 8 * (2 * q + j) + i;
    tmem_ld_wait();
    if (step < 3) {
      const int nj = (step + 1) >> 1, nchunk = (step + 1) & 1;
      tmem_ld_16x256b_x4(taddr0 + ((uint32_t)(16 * nj) << 16) + 32 * nchunk, r[(step + 1) & 1]);
    }
    const uint32_t (&rr)[16] = r[step & 1];
    const uint32_t base = (uint32_t)((8 * c + 4 * chunk) * SBO + (2 * tq) * 16 + (row >> 2) * LBO + (row & 3) * 4);
    const uint32_t* grow = Gtab + GSTRIDE * row + 32 * chunk + 2 * tq;
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const uint2 gp = *reinterpret_cast<const uint2*>(grow + 8 * (GXOR ? (x ^ (row & 3)) : x));
      const float2 v0 = cmul(make_float2(__uint_as_float(rr[4 * x]), __uint_as_float(rr[4 * x + 2])), unpack_h2(gp.x));
      const float2 v1 = cmul(make_float2(__uint_as_float(rr[4 * x + 1]), __uint_as_float(rr[4 * x + 3])), unpack_h2(gp.y));
      *reinterpret_cast<uint32_t*>(Bout + base + x * SBO) = pack_h2(v0.x, -v0.y);
      *reinterpret_cast<uint32_t*>(Bout + base + x * SBO + 16) = pack_h2(v1.x, -v1.y);
    }
  }
}
__device__ __forceinline__ void epilogue_gate(uint32_t tmem_d, unsigned char* Bout, int q, int c, int T,
                                              const uint32_t* __restrict__ Gtab) {
  epilogue_gate_t<k8Lbo2, k8Sbo2, k8GStride, false>(tmem_d, Bout, q, c, T, Gtab);
}

}  // namespace spectre
