// k-means assignment on the tensor cores (bf16 inputs): argmin_c |c|^2 - 2 x.c with the dot
// products from tcgen05 MMAs.  The centres are fp32; they enter the MMA as a bf16 hi + lo pair
// (two accumulating products), which keeps ~16 mantissa bits so that the discrete assignment
// agrees with an fp64 evaluation except at genuine near-ties (Appendix "Balanced Assignment":
// the |x|^2 term cancels between centres).  One CTA = 128 points; the distance rows are scanned
// straight out of tensor memory while the next centre tile is being multiplied.
#include <cuda.h>
#include "common.cuh"
#include "tc05.cuh"

namespace muse {

typedef __nv_bfloat16 bf16;
constexpr int kAtRows = 128, kAtCols = 128;

// fp32 centres -> bf16 hi and lo planes
__global__ void k_split_centres(const float* __restrict__ c, long long n, bf16* __restrict__ hi, bf16* __restrict__ lo) {
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= n) return;
  const float x = c[e];
  const bf16 h = __float2bfloat16_rn(x);
  hi[e] = h;
  lo[e] = __float2bfloat16_rn(x - __bfloat162float(h));
}

// Warp roles: warps 0-7 read the distance rows out of tensor memory (two warpgroups, 64 columns each),
// warp 8 feeds the centre tiles by TMA through a ring, warp 9 issues the MMAs into two alternating
// accumulator buffers, so that the arg-min sweep of one centre tile overlaps the products of the next.
constexpr int kAtThreads = 320, kAtEpi = 256;

struct AtBars { uint64_t full[4], empty[4], tfull[2], tempty[2], xbar; };

template <int D, bool DIST>     // DIST: also write the matrix |c|^2 - 2 x.c (the balanced assignment's second step reads it)
__global__ void __launch_bounds__(kAtThreads, 1)
k_assign_tc(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_hi, const __grid_constant__ CUtensorMap tm_lo,
            int N, int C, int ns, const float* __restrict__ cnorm, int32_t* __restrict__ assign, float* __restrict__ dist_out,
            int* __restrict__ status) {
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ AtBars bars;
  __shared__ uint32_t tbase_s;
  __shared__ float best_s[kAtRows];
  __shared__ int idx_s[kAtRows];
  constexpr int kX = kAtRows * D * 2, kC = kAtCols * D * 2, kStage = 2 * kC;     // stage = hi tile | lo tile
  unsigned char* sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);
  unsigned char* Xs = sm;
  unsigned char* ring = sm + kX;
  float* cn = reinterpret_cast<float*>(ring + ns * kStage);                      // |c|^2 of every centre of this problem
  const int tid = threadIdx.x, warp = tid >> 5, prob = blockIdx.y, row0 = blockIdx.x * kAtRows;
  const int NT = (C + kAtCols - 1) / kAtCols;
  if (warp == 0) tc::tmem_alloc(&tbase_s, 2 * kAtCols);
  if (tid == 0) {
    for (int s = 0; s < 4; ++s) { tc::mbar_init(&bars.full[s], 1); tc::mbar_init(&bars.empty[s], 1); }
    for (int b = 0; b < 2; ++b) { tc::mbar_init(&bars.tfull[b], 1); tc::mbar_init(&bars.tempty[b], kAtEpi); }
    tc::mbar_init(&bars.xbar, 1);
    tc::mbar_init_fence();
  }
  for (int c = tid; c < NT * kAtCols; c += kAtThreads) cn[c] = c < C ? cnorm[(size_t)prob * C + c] : INFINITY;
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tbase = tbase_s;
  bool ok = true;

  if (warp == 8) {
    if (tid == 8 * 32) {                                   // ---- producer
      tc::mbar_expect_tx(&bars.xbar, kX);
      for (int g = 0; g < D / 64; ++g) tc::tma_load_2d(Xs + g * kAtRows * 128, &tm_x, 64 * g, prob * N + row0, &bars.xbar);
      for (int t = 0, s = 0, ph = 0; t < NT && ok; ++t) {                // (stage and phase by increments: no division per tile)
        if (!tc::mbar_wait(&bars.empty[s], ph ^ 1)) { ok = false; break; }
        tc::mbar_expect_tx(&bars.full[s], kStage);
        unsigned char* st = ring + s * kStage;
        for (int g = 0; g < D / 64; ++g) {
          tc::tma_load_2d(st + g * kAtCols * 128, &tm_hi, 64 * g, prob * C + t * kAtCols, &bars.full[s]);
          tc::tma_load_2d(st + kC + g * kAtCols * 128, &tm_lo, 64 * g, prob * C + t * kAtCols, &bars.full[s]);
        }
        if (++s == ns) { s = 0; ph ^= 1; }
      }
    }
  } else if (warp == 9) {
    if (tid == 9 * 32) {                                   // ---- MMA issuer
      const uint32_t idesc = tc::idesc_bf16(kAtRows, kAtCols, 0, 0);
      const uint64_t dx0 = tc::smem_desc_sw128(tc::smem_u32(Xs), 16, 1024), dr0 = tc::smem_desc_sw128(tc::smem_u32(ring), 16, 1024);
      if (!tc::mbar_wait(&bars.xbar, 0)) ok = false;
      for (int t = 0, s = 0, ph = 0; t < NT && ok; ++t) {
        const int b = t & 1;
        if (!tc::mbar_wait(&bars.tempty[b], ((t >> 1) & 1) ^ 1)) { ok = false; break; }
        if (!tc::mbar_wait(&bars.full[s], ph)) { ok = false; break; }
        tc::fence_after_sync();
        const uint64_t dh = tc::desc_step(dr0, (uint32_t)s * kStage), dl = tc::desc_step(dh, kC);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc::mma_bf16_ss(tbase + b * kAtCols, tc::desc_step(dx0, (ks / 4) * kAtRows * 128 + (ks % 4) * 32),
                          tc::desc_step(dh, (ks / 4) * kAtCols * 128 + (ks % 4) * 32), idesc, ks > 0);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc::mma_bf16_ss(tbase + b * kAtCols, tc::desc_step(dx0, (ks / 4) * kAtRows * 128 + (ks % 4) * 32),
                          tc::desc_step(dl, (ks / 4) * kAtCols * 128 + (ks % 4) * 32), idesc, 1);
        tc::mma_commit(&bars.empty[s]);                    // the centre tiles may be overwritten ...
        tc::mma_commit(&bars.tfull[b]);                    // ... and the distances read
        if (++s == ns) { s = 0; ph ^= 1; }
      }
    }
  } else {
    // ---- arg-min sweep: thread = (point row, half of the 128 columns of a tile)
    const int row = tid & 127, wg = tid >> 7;
    const uint32_t tlane = tbase + ((uint32_t)((warp & 3) * 32) << 16);
    float best = INFINITY;
    int bidx = 0x7fffffff;
    for (int t = 0; t < NT && ok; ++t) {
      const int b = t & 1;
      if (!tc::mbar_wait(&bars.tfull[b], (t >> 1) & 1)) { ok = false; break; }
      tc::fence_after_sync();
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        float v[32];
        tc::tmem_ld32(tlane + b * kAtCols + wg * 64 + 32 * q, v);
        const int c0 = t * kAtCols + wg * 64 + 32 * q;
#pragma unroll
        for (int k = 0; k < 32; ++k) {
          const float dist = fmaf(-2.f, v[k], cn[c0 + k]);
          if (dist < best) { best = dist; bidx = c0 + k; }     // ascending index: ties keep the lower
        }
        if (DIST && row0 + row < N) {                            // optional output: the whole matrix |c|^2 - 2 x.c
#pragma unroll
          for (int k = 0; k < 32; ++k) v[k] = fmaf(-2.f, v[k], cn[c0 + k]);
          float* dr = dist_out + ((size_t)prob * N + row0 + row) * C + c0;
          if (c0 + 32 <= C && (C & 3) == 0) {
#pragma unroll
            for (int k = 0; k < 32; k += 4) *reinterpret_cast<float4*>(dr + k) = make_float4(v[k], v[k + 1], v[k + 2], v[k + 3]);
          } else {
#pragma unroll
            for (int k = 0; k < 32; ++k) if (c0 + k < C) dr[k] = v[k];
          }
        }
      }
      tc::fence_before_sync();
      tc::mbar_arrive(&bars.tempty[b]);
    }
    // the two column halves of a row meet: lower distance wins, the lower index on a tie
    if (wg == 1) { best_s[row] = best; idx_s[row] = bidx; }
    tc::named_bar_sync(1, kAtEpi);
    if (wg == 0 && ok) {
      const float ob = best_s[row];
      const int oi = idx_s[row];
      if (ob < best || (ob == best && oi < bidx)) bidx = oi;
      // a row of NaN or infinities never compares below the running minimum: it goes to cluster 0
      if (row0 + row < N) assign[(size_t)prob * N + row0 + row] = (unsigned)bidx < (unsigned)C ? bidx : 0;
    }
  }
  if (!ok) report_status(status, 6);
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tbase, 2 * kAtCols);
}

int make_tmap_bf16_rows(void* out_map, const void* base, uint64_t rows, uint32_t cols, uint32_t box_rows);

int assign_tc(const void* X, int problems, int N, int D, int C, const float* centres, const float* cnorm, void* chi,
              void* clo, int32_t* assign, float* dist_out, int* status, cudaStream_t st) {
  const long long n = (long long)problems * C * D;
  prof_mark("k_split_centres", st);
  k_split_centres<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(centres, n, (bf16*)chi, (bf16*)clo);
  MUSE_LAUNCH_OK();
  CUtensorMap tx, thi, tlo;
  int rc = make_tmap_bf16_rows(&tx, X, (uint64_t)problems * N, (uint32_t)D, kAtRows);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&thi, chi, (uint64_t)problems * C, (uint32_t)D, kAtCols);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&tlo, clo, (uint64_t)problems * C, (uint32_t)D, kAtCols);
  if (rc != MUSE_OK) return rc;
  const int NT = (C + kAtCols - 1) / kAtCols;
  const int ns = D == 128 ? 2 : 4;                          // ring stages of 64 KB / 32 KB
  const size_t smem = (size_t)kAtRows * D * 2 + (size_t)ns * 2 * kAtCols * D * 2 + (size_t)NT * kAtCols * 4 + 1024;
  dim3 grid(cdiv(N, kAtRows), problems);
  prof_mark("k_assign_tc", st);
#define MUSE_AT_LAUNCH(DD, DI)                                                                                             \
  {                                                                                                                        \
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_assign_tc<DD, DI>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));      \
    k_assign_tc<DD, DI><<<grid, kAtThreads, smem, st>>>(tx, thi, tlo, N, C, ns, cnorm, assign, dist_out, status);        \
  }
  if (D == 128) { if (dist_out) MUSE_AT_LAUNCH(128, true) else MUSE_AT_LAUNCH(128, false) }
  else { if (dist_out) MUSE_AT_LAUNCH(64, true) else MUSE_AT_LAUNCH(64, false) }
#undef MUSE_AT_LAUNCH
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

}  // namespace muse
