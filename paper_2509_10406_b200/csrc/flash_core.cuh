// FFMA tile primitives for the exact-attention kernels: 64 x 64 score tiles, 256 threads laid
// out 16 x 16, each thread owning a 4 x 4 patch of a score tile and, for D-wide results,
// 4 rows x the columns {tx*4 + 64*k}.  Operand tiles live in shared memory in the input
// element type; probabilities in fp32.
#pragma once
#include "common.cuh"

namespace muse {

constexpr int kTile = 64;          // rows and columns of a score tile
constexpr int kFlashThreads = 256;
constexpr int kLDP = kTile + 4;    // leading dimension of the fp32 probability tile

template <class T> struct Pad { static constexpr int v = 16 / sizeof(T); };

// acc[r][c] = sum_d A[ty*4+r][d] * B[tx*4+c][d]
template <class T, int D>
__device__ __forceinline__ void mm_nt(const T* __restrict__ A, const T* __restrict__ B, float acc[4][4], int ty, int tx) {
  constexpr int LD = D + Pad<T>::v;
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;
#pragma unroll 4
  for (int d = 0; d < D; d += 4) {
    float4 a[4], b[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) a[r] = ld4(A + (ty * 4 + r) * LD + d);
#pragma unroll
    for (int c = 0; c < 4; ++c) b[c] = ld4(B + (tx * 4 + c) * LD + d);
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        acc[r][c] = fmaf(a[r].x, b[c].x, acc[r][c]); acc[r][c] = fmaf(a[r].y, b[c].y, acc[r][c]);
        acc[r][c] = fmaf(a[r].z, b[c].z, acc[r][c]); acc[r][c] = fmaf(a[r].w, b[c].w, acc[r][c]);
      }
  }
}

// acc[r][k][c] += sum_j P[ty*4+r][j] * B[j][tx*4 + 64k + c]     (P fp32 [64][kLDP])
template <class T, int D>
__device__ __forceinline__ void mm_pn(const float* __restrict__ P, const T* __restrict__ B, float acc[4][D / 64][4], int ty, int tx) {
  constexpr int LD = D + Pad<T>::v;
#pragma unroll 2
  for (int j = 0; j < kTile; j += 4) {
    float4 p[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) p[r] = ld4(P + (ty * 4 + r) * kLDP + j);
#pragma unroll
    for (int jj = 0; jj < 4; ++jj)
#pragma unroll
      for (int k = 0; k < D / 64; ++k) {
        float4 b = ld4(B + (j + jj) * LD + tx * 4 + 64 * k);
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          float pv = jj == 0 ? p[r].x : jj == 1 ? p[r].y : jj == 2 ? p[r].z : p[r].w;
          acc[r][k][0] = fmaf(pv, b.x, acc[r][k][0]); acc[r][k][1] = fmaf(pv, b.y, acc[r][k][1]);
          acc[r][k][2] = fmaf(pv, b.z, acc[r][k][2]); acc[r][k][3] = fmaf(pv, b.w, acc[r][k][3]);
        }
      }
  }
}

// acc[jj][k][c] += sum_r P[r][ty*4+jj] * B[r][tx*4 + 64k + c]   (P transposed on the fly)
template <class T, int D>
__device__ __forceinline__ void mm_tn(const float* __restrict__ P, const T* __restrict__ B, float acc[4][D / 64][4], int ty, int tx) {
  constexpr int LD = D + Pad<T>::v;
#pragma unroll 4
  for (int r = 0; r < kTile; ++r) {
    float4 p = ld4(P + r * kLDP + ty * 4);
#pragma unroll
    for (int k = 0; k < D / 64; ++k) {
      float4 b = ld4(B + r * LD + tx * 4 + 64 * k);
      acc[0][k][0] = fmaf(p.x, b.x, acc[0][k][0]); acc[0][k][1] = fmaf(p.x, b.y, acc[0][k][1]);
      acc[0][k][2] = fmaf(p.x, b.z, acc[0][k][2]); acc[0][k][3] = fmaf(p.x, b.w, acc[0][k][3]);
      acc[1][k][0] = fmaf(p.y, b.x, acc[1][k][0]); acc[1][k][1] = fmaf(p.y, b.y, acc[1][k][1]);
      acc[1][k][2] = fmaf(p.y, b.z, acc[1][k][2]); acc[1][k][3] = fmaf(p.y, b.w, acc[1][k][3]);
      acc[2][k][0] = fmaf(p.z, b.x, acc[2][k][0]); acc[2][k][1] = fmaf(p.z, b.y, acc[2][k][1]);
      acc[2][k][2] = fmaf(p.z, b.z, acc[2][k][2]); acc[2][k][3] = fmaf(p.z, b.w, acc[2][k][3]);
      acc[3][k][0] = fmaf(p.w, b.x, acc[3][k][0]); acc[3][k][1] = fmaf(p.w, b.y, acc[3][k][1]);
      acc[3][k][2] = fmaf(p.w, b.z, acc[3][k][2]); acc[3][k][3] = fmaf(p.w, b.w, acc[3][k][3]);
    }
  }
}

// Copy `n` rows of D elements (row r from src + row_index(r) * D) into a [64][D+pad] tile,
// zero-filling rows n..63.
template <class T, int D, class RowFn>
__device__ __forceinline__ void load_tile(T* __restrict__ dst, const T* __restrict__ src, int n, RowFn row_index, int tid) {
  constexpr int LD = D + Pad<T>::v;
  constexpr int VPR = D * sizeof(T) / 16;
  for (int e = tid; e < kTile * VPR; e += kFlashThreads) {
    int r = e / VPR, v = e % VPR;
    uint4 x = make_uint4(0u, 0u, 0u, 0u);
    if (r < n) x = reinterpret_cast<const uint4*>(src + (size_t)row_index(r) * D)[v];
    reinterpret_cast<uint4*>(dst + r * LD)[v] = x;
  }
}

template <class T, int D> constexpr size_t tile_bytes() { return (size_t)kTile * (D + Pad<T>::v) * sizeof(T); }
constexpr size_t ptile_bytes() { return (size_t)kTile * kLDP * sizeof(float); }

// max / sum over the 16 threads (tx) that share a row: lanes of one half-warp.
__device__ __forceinline__ float row_max16(float v) {
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float row_sum16(float v) {
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// One online-softmax step over a 64 x 64 score tile held in registers (already scaled, masked
// entries = -inf): updates the running max / sum, rescales the output accumulator and writes
// the probabilities to shared memory.
template <int D>
__device__ __forceinline__ void online_softmax_step(float sc[4][4], float m_run[4], float l_run[4],
                                                    float o[4][D / 64][4], float* __restrict__ Ps, int ty, int tx) {
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    float mx = fmaxf(fmaxf(sc[r][0], sc[r][1]), fmaxf(sc[r][2], sc[r][3]));
    mx = row_max16(mx);
    const float mn = fmaxf(m_run[r], mx);
    const float base = mn == -INFINITY ? 0.f : mn;           // all masked so far: keep zeros
    const float scale = expf(m_run[r] - base);                 // exp(-inf) = 0
    float p[4], ps = 0.f;
#pragma unroll
    for (int c = 0; c < 4; ++c) { p[c] = expf(sc[r][c] - base); ps += p[c]; }
    ps = row_sum16(ps);
    l_run[r] = l_run[r] * scale + ps;
    m_run[r] = mn;
#pragma unroll
    for (int k = 0; k < D / 64; ++k)
#pragma unroll
      for (int c = 0; c < 4; ++c) o[r][k][c] *= scale;
    st4(Ps + (ty * 4 + r) * kLDP + tx * 4, make_float4(p[0], p[1], p[2], p[3]));
  }
}

}  // namespace muse
