// Pre-merge of the dipole matrices on the tensor cores (bf16 mode):
//   Cbar[(head, plane)][i][x] = sum_j P[(head, plane)][i][j] * Cov[(kv head, plane)][j][x],  x over D*D
// (Appendix "Error Analysis", the merged covariance of the "Dipole Correction" paragraph.)
// One CTA computes a [256 query clusters] x [128 columns] tile: both 128-row halves share every
// covariance tile, so the covariances (the large operand) are read from HBM once when Cq <= 256.
// P tiles [128 i][64 j] (K-major A) and covariance tiles [64 j][128 x] (MN-major B) arrive by TMA
// in a ring; one thread issues loads and tcgen05 MMAs, accumulators live in TMEM
// (2 halves x 128 columns), four warps read them back and store bf16 rows.
#include <cuda.h>
#include "common.cuh"
#include "tc05.cuh"

namespace muse {

typedef __nv_bfloat16 bf16;
int make_tmap_bf16_rows(void* out_map, const void* base, uint64_t rows, uint32_t cols, uint32_t box_rows);

constexpr int kDmN = 128, kDmK = 64, kDmStages = 3;
constexpr int kDmA = 128 * kDmK * 2;                 // 16 KB: one 128-row half of the P tile
constexpr int kDmB = kDmK * kDmN * 2;                // 16 KB: covariance tile (two 64-column groups)
constexpr int kDmStage = 2 * kDmA + kDmB;            // 48 KB
constexpr int kDmCols = 256;                         // TMEM columns: half 0 at 0, half 1 at 128

struct DmBars { uint64_t full[kDmStages], empty[kDmStages], done; };

template <class OT>
__global__ void __launch_bounds__(128)
k_dipole_merge_tc(Dims dm, const __grid_constant__ CUtensorMap tm_p, const __grid_constant__ CUtensorMap tm_cov,
                  OT* __restrict__ cbar, int* __restrict__ status) {
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ DmBars bars;
  __shared__ uint32_t tbase_s;
  unsigned char* sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);
  const int tid = threadIdx.x, warp = tid >> 5;
  const int DD = dm.D * dm.D;
  const int x0 = blockIdx.x * kDmN, i0 = blockIdx.y * 256;
  const int pp = blockIdx.z, pq = pp / dm.SB, pl = pp % dm.SB;
  const int pk = dm.dipole == 2 ? pq : (pq / dm.Hq) * dm.Hkv + dm.hm.g[pq % dm.Hq];   // head that owns the covariances
  const int halves = dm.Cq - i0 > 128 ? 2 : 1;
  const int rowA = pp * dm.Cq + i0;                              // first P row of this tile
  const int rowB = (pk * dm.SB + pl) * dm.Ck;                    // first covariance row of this (kv head, plane)
  const int KT = dm.Ck / kDmK;

  if (warp == 0) tc::tmem_alloc(&tbase_s, kDmCols);
  if (tid == 0) {
    for (int s = 0; s < kDmStages; ++s) { tc::mbar_init(&bars.full[s], 1); tc::mbar_init(&bars.empty[s], 1); }
    tc::mbar_init(&bars.done, 1);
    tc::mbar_init_fence();
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tbase = tbase_s;
  bool ok = true;

  if (tid == 0) {
    const uint32_t idesc = tc::idesc_bf16(128, kDmN, 0, 1);
    uint32_t use[kDmStages];
    for (int s = 0; s < kDmStages; ++s) use[s] = 0;
    const int look = kDmStages - 1;
    for (int t = 0; t < KT + look && ok; ++t) {
      if (t < KT) {
        const int s = t % kDmStages;
        if (!tc::mbar_wait(&bars.empty[s], (use[s] & 1) ^ 1)) { ok = false; break; }
        unsigned char* st = sm + s * kDmStage;
        tc::mbar_expect_tx(&bars.full[s], halves * kDmA + kDmB);
        tc::tma_load_2d(st, &tm_p, t * kDmK, rowA, &bars.full[s]);
        if (halves == 2) tc::tma_load_2d(st + kDmA, &tm_p, t * kDmK, rowA + 128, &bars.full[s]);
        tc::tma_load_2d(st + 2 * kDmA, &tm_cov, x0, rowB + t * kDmK, &bars.full[s]);
        tc::tma_load_2d(st + 2 * kDmA + kDmK * 128, &tm_cov, x0 + 64, rowB + t * kDmK, &bars.full[s]);
      }
      const int u = t - look;
      if (u >= 0) {
        const int s = u % kDmStages;
        if (!tc::mbar_wait(&bars.full[s], use[s] & 1)) { ok = false; break; }
        tc::fence_after_sync();
        const uint32_t a0 = tc::smem_u32(sm + s * kDmStage), b0 = a0 + 2 * kDmA;
        for (int hf = 0; hf < halves; ++hf) {
#pragma unroll
          for (int ks = 0; ks < kDmK / 16; ++ks)
            tc::mma_bf16_ss(tbase + hf * kDmN, tc::smem_desc_sw128(a0 + hf * kDmA + ks * 32, 16, 1024),
                            tc::smem_desc_sw128(b0 + ks * 16 * 128, kDmK * 128, 1024), idesc, u > 0 || ks > 0);
        }
        tc::mma_commit(&bars.empty[s]);
        use[s]++;
      }
    }
    tc::mma_commit(&bars.done);
  }
  __syncwarp();
  if (!tc::mbar_wait(&bars.done, 0)) ok = false;
  tc::fence_after_sync();
  // epilogue: thread = accumulator row (query cluster); all threads run the TMEM loads
  for (int hf = 0; hf < halves; ++hf) {
    const int i = i0 + hf * 128 + tid;
    OT* out = cbar + ((size_t)pp * dm.Cq + i) * DD + x0;
#pragma unroll
    for (int q = 0; q < kDmN / 32; ++q) {
      float v[32];
      tc::tmem_ld32(tbase + ((uint32_t)(warp * 32) << 16) + hf * kDmN + 32 * q, v);
      if (ok && i < dm.Cq && sizeof(OT) == 4) {
#pragma unroll
        for (int c = 0; c < 32; c += 4)
          *reinterpret_cast<float4*>((float*)out + 32 * q + c) = make_float4(v[c], v[c + 1], v[c + 2], v[c + 3]);
      } else if (ok && i < dm.Cq) {
#pragma unroll
        for (int c = 0; c < 32; c += 8) {
          __nv_bfloat162 w0 = __floats2bfloat162_rn(v[c], v[c + 1]), w1 = __floats2bfloat162_rn(v[c + 2], v[c + 3]);
          __nv_bfloat162 w2 = __floats2bfloat162_rn(v[c + 4], v[c + 5]), w3 = __floats2bfloat162_rn(v[c + 6], v[c + 7]);
          *reinterpret_cast<uint4*>((bf16*)out + 32 * q + c) = make_uint4(*reinterpret_cast<uint32_t*>(&w0), *reinterpret_cast<uint32_t*>(&w1),
                                                                    *reinterpret_cast<uint32_t*>(&w2), *reinterpret_cast<uint32_t*>(&w3));
        }
      }
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tbase, kDmCols);
  if (!ok && tid == 0) report_status(status, 7);
}

bool dipole_merge_tc_supported(const Dims& d, int dtype) {
  // row coordinates of the tensor maps are 32-bit
  const long long rows_p = (long long)d.B * d.Hq * d.SB * d.Cq, rows_c = (long long)d.B * (d.dipole == 2 ? d.Hq : d.Hkv) * d.SB * d.Ck;
  return dtype == MUSE_BF16 && d.Ck % kDmK == 0 && (d.D * d.D) % kDmN == 0 && rows_p < (1ll << 31) && rows_c < (1ll << 31);
}

int dipole_merge_tc(const Dims& d, const void* P, const void* cov, void* cbar, int out_f32, int* status, cudaStream_t st) {
  CUtensorMap tp, tcv;
  int rc = make_tmap_bf16_rows(&tp, P, (uint64_t)d.B * d.Hq * d.SB * d.Cq, d.Ck, 128);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&tcv, cov, (uint64_t)d.B * (d.dipole == 2 ? d.Hq : d.Hkv) * d.SB * d.Ck, d.D * d.D, kDmK);
  if (rc != MUSE_OK) return rc;
  const size_t smem = (size_t)kDmStages * kDmStage + 1024;
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_dipole_merge_tc<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_dipole_merge_tc<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  prof_mark("k_dipole_merge_tc", st);
  const dim3 grid(d.D * d.D / kDmN, cdiv(d.Cq, 256), d.B * d.Hq * d.SB);
  if (out_f32) k_dipole_merge_tc<float><<<grid, 128, smem, st>>>(d, tp, tcv, (float*)cbar, status);
  else k_dipole_merge_tc<bf16><<<grid, 128, smem, st>>>(d, tp, tcv, (bf16*)cbar, status);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

}  // namespace muse
