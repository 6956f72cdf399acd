// The two dense contractions of the dipole correction's backward pass on the tensor cores (bf16 mode):
//   dCov[(head, plane)][j][x] += sum_i P[(head, plane)][i][j] * dCbar[(head, plane)][i][x]        x over D*D
//   dP[(head, plane)][i][j]   += sum_x dCbar[(head, plane)][i][x] * Cov[(cov head, plane)][j][x] + dZsum[i]
// (Appendix "Error Analysis", "Dipole Correction": the transposes of the pre-merge Cbar = P Cov.)  dCbar is converted to
// bf16 once for both.  Same structure as the pre-merge kernel: TMA ring of 128-byte-swizzled tiles, one thread issuing
// loads and tcgen05 MMAs, fp32 accumulators in TMEM, four warps reading them back; every wait is bounded.
//   k_dipole_dcov_tc: A = P^T (MN-major: the tile arrives as [64 i][128 j]), B = dCbar (MN-major, [64 i][128 x]),
//                     CTA tile 128 j x 128 x, K = C_q in steps of 64; read-modify-write of the fp32 dCov rows.
//   k_dipole_dpw_tc:  A = dCbar, B = Cov (both K-major, [128 rows][64 x]), CTA tile 128 i x 128 j, K = D*D in steps of 64.
#include <cuda.h>
#include "common.cuh"
#include "tc05.cuh"

namespace muse {

typedef __nv_bfloat16 bf16;
int make_tmap_bf16_rows(void* out_map, const void* base, uint64_t rows, uint32_t cols, uint32_t box_rows);

constexpr int kDbK = 64, kDbStages = 4;
constexpr int kDbTile = 128 * kDbK * 2;             // 16 KB: one operand tile of a stage
constexpr int kDbStage = 2 * kDbTile;               // 32 KB
constexpr int kDbCols = 128;                        // TMEM columns

struct DbBars { uint64_t full[kDbStages], empty[kDbStages], done; };

__global__ void k_to_bf16(const float* __restrict__ src, size_t n4, bf16* __restrict__ dst) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= n4) return;
  const float4 v = reinterpret_cast<const float4*>(src)[e];
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  reinterpret_cast<uint2*>(dst)[e] = make_uint2(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b));
}

// MODE 0: dCov (both operands MN-major), MODE 1: dP (both K-major).
template <int MODE>
__global__ void __launch_bounds__(128)
k_dipole_bwd_gemm_tc(Dims dm, const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                     const float* __restrict__ dzs, float* __restrict__ out, int accumulate, const int32_t* __restrict__ goff,
                     int* __restrict__ status) {
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ DbBars bars;
  __shared__ uint32_t tbase_s;
  unsigned char* sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);
  const int tid = threadIdx.x, warp = tid >> 5;
  const int DD = dm.D * dm.D;
  const int pp = blockIdx.z, pq = pp / dm.SB, pl = pp % dm.SB;
  const int pk = dm.dipole == 2 ? pq : (pq / dm.Hq) * dm.Hkv + dm.hm.g[pq % dm.Hq];   // head that owns the covariances
  // MODE 0: rows of the output = key clusters j, columns = x;  MODE 1: rows = query clusters i, columns = key clusters j
  const int n0 = blockIdx.x * 128, m0 = blockIdx.y * 128;
  const int KT = MODE == 0 ? dm.Cq / kDbK : DD / kDbK;

  if (warp == 0) tc::tmem_alloc(&tbase_s, kDbCols);
  if (tid == 0) {
    for (int s = 0; s < kDbStages; ++s) { tc::mbar_init(&bars.full[s], 1); tc::mbar_init(&bars.empty[s], 1); }
    tc::mbar_init(&bars.done, 1);
    tc::mbar_init_fence();
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tbase = tbase_s;
  bool ok = true;

  if (tid == 0) {
    const uint32_t idesc = MODE == 0 ? tc::idesc_bf16(128, 128, 1, 1) : tc::idesc_bf16(128, 128, 0, 0);
    uint32_t use[kDbStages];
    for (int s = 0; s < kDbStages; ++s) use[s] = 0;
    const int look = kDbStages - 1;
    for (int t = 0; t < KT + look && ok; ++t) {
      if (t < KT) {
        const int s = t % kDbStages;
        if (!tc::mbar_wait(&bars.empty[s], (use[s] & 1) ^ 1)) { ok = false; break; }
        unsigned char* st = sm + s * kDbStage;
        tc::mbar_expect_tx(&bars.full[s], kDbStage);
        if (MODE == 0) {
          const int row = pp * dm.Cq + t * kDbK;                 // 64 query clusters of this (head, plane)
          tc::tma_load_2d(st, &tm_a, m0, row, &bars.full[s]);                          // P[i][j0 .. j0+63]
          tc::tma_load_2d(st + kDbK * 128, &tm_a, m0 + 64, row, &bars.full[s]);
          tc::tma_load_2d(st + kDbTile, &tm_b, n0, row, &bars.full[s]);                // dCbar[i][x0 .. x0+63]
          tc::tma_load_2d(st + kDbTile + kDbK * 128, &tm_b, n0 + 64, row, &bars.full[s]);
        } else {
          tc::tma_load_2d(st, &tm_a, t * kDbK, pp * dm.Cq + m0, &bars.full[s]);        // dCbar[i0 .. +127][x chunk]
          tc::tma_load_2d(st + kDbTile, &tm_b, t * kDbK, (pk * dm.SB + pl) * dm.Ck + n0, &bars.full[s]);   // Cov[j0 .. +127][x chunk]
        }
      }
      const int u = t - look;
      if (u >= 0) {
        const int s = u % kDbStages;
        if (!tc::mbar_wait(&bars.full[s], use[s] & 1)) { ok = false; break; }
        tc::fence_after_sync();
        const uint32_t a0 = tc::smem_u32(sm + s * kDbStage), b0 = a0 + kDbTile;
#pragma unroll
        for (int ks = 0; ks < kDbK / 16; ++ks) {
          if (MODE == 0)
            tc::mma_bf16_ss(tbase, tc::smem_desc_sw128(a0 + ks * 16 * 128, kDbK * 128, 1024),
                            tc::smem_desc_sw128(b0 + ks * 16 * 128, kDbK * 128, 1024), idesc, u > 0 || ks > 0);
          else
            tc::mma_bf16_ss(tbase, tc::smem_desc_sw128(a0 + ks * 32, 16, 1024), tc::smem_desc_sw128(b0 + ks * 32, 16, 1024), idesc,
                            u > 0 || ks > 0);
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
  // epilogue: thread = accumulator row; all threads run the TMEM loads
  const int r = m0 + tid;
  const int rows = MODE == 0 ? dm.Ck : dm.Cq, cols = MODE == 0 ? DD : dm.Ck;
  float* orow = out + ((size_t)pp * rows + r) * cols + n0;
  const float add = MODE == 1 && r < rows ? dzs[(size_t)pp * dm.Cq + r] : 0.f;
  if (MODE == 0 && goff != nullptr && r < rows) {
    // dCov rows of clusters that no query retrieved in this plane were left unwritten by the per-pair kernel: overwrite
    const int32_t* go = goff + (size_t)pq * (dm.SB * dm.Ck + 1) + (size_t)r * dm.SB + pl;
    accumulate = go[1] > go[0] ? 1 : 0;
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    float v[32];
    tc::tmem_ld32(tbase + ((uint32_t)(warp * 32) << 16) + 32 * q, v);
    if (ok && r < rows) {
#pragma unroll
      for (int c = 0; c < 32; c += 4) {
        const int col = n0 + 32 * q + c;
        if (col + 3 < cols) {
          float4 o = accumulate ? *reinterpret_cast<float4*>(orow + 32 * q + c) : make_float4(0.f, 0.f, 0.f, 0.f);
          o.x += v[c] + add; o.y += v[c + 1] + add; o.z += v[c + 2] + add; o.w += v[c + 3] + add;
          *reinterpret_cast<float4*>(orow + 32 * q + c) = o;
        } else {
          for (int e = 0; e < 4; ++e)
            if (col + e < cols) orow[32 * q + c + e] = (accumulate ? orow[32 * q + c + e] : 0.f) + v[c + e] + add;
        }
      }
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tbase, kDbCols);
  if (!ok && tid == 0) report_status(status, MUSE_STATUS_SUMM_BWD_TIMEOUT);
}

bool dipole_bwd_tc_supported(const Dims& d, int dtype) {
  const long long rows_p = (long long)d.B * d.Hq * d.SB * d.Cq, rows_c = (long long)d.B * (d.dipole == 2 ? d.Hq : d.Hkv) * d.SB * d.Ck;
  // P^T tiles hold 64 query clusters of ONE (head, plane); row strides of the tensor maps are multiples of 16 bytes;
  // fp32 output rows are read and written as float4
  return dtype == MUSE_BF16 && d.Cq % kDbK == 0 && d.Ck % 8 == 0 && rows_p < (1ll << 31) && rows_c < (1ll << 31);
}

// dcbar_bf: scratch for the bf16 copy of dCbar ([B*Hq*SB*Cq][D*D]).
// goff != NULL (m > 0): the rows of dCov whose (cluster, plane) group of the inverse index has pairs already hold the retrieved
// clusters' (negative) share and are added to; every other row is overwritten.
int dipole_bwd_tc(const Dims& d, const void* P, const void* cov, const float* dcbar, void* dcbar_bf, const float* dzs, float* dcov,
                  float* dpw, int with_dpw, const int32_t* goff, int* status, cudaStream_t st) {
  const int DD = d.D * d.D;
  const uint64_t rows_p = (uint64_t)d.B * d.Hq * d.SB * d.Cq, rows_c = (uint64_t)d.B * (d.dipole == 2 ? d.Hq : d.Hkv) * d.SB * d.Ck;
  const size_t n4 = rows_p * DD / 4;
  prof_mark("k_to_bf16", st);
  k_to_bf16<<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(dcbar, n4, (bf16*)dcbar_bf);
  MUSE_LAUNCH_OK();
  CUtensorMap tp64, tg64, tg128, tc128;
  int rc = make_tmap_bf16_rows(&tp64, P, rows_p, d.Ck, kDbK);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&tg64, dcbar_bf, rows_p, DD, kDbK);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&tg128, dcbar_bf, rows_p, DD, 128);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&tc128, cov, rows_c, DD, 128);
  if (rc != MUSE_OK) return rc;
  const size_t smem = (size_t)kDbStages * kDbStage + 1024;
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_dipole_bwd_gemm_tc<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_dipole_bwd_gemm_tc<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  prof_mark("k_dipole_dcov_tc", st);
  k_dipole_bwd_gemm_tc<0><<<dim3(DD / 128, cdiv(d.Ck, 128), d.B * d.Hq * d.SB), 128, smem, st>>>(d, tp64, tg64, nullptr, dcov, 0, goff, status);
  MUSE_LAUNCH_OK();
  if (with_dpw) {
    prof_mark("k_dipole_dpw_tc", st);
    k_dipole_bwd_gemm_tc<1><<<dim3(cdiv(d.Ck, 128), cdiv(d.Cq, 128), d.B * d.Hq * d.SB), 128, smem, st>>>(d, tg128, tc128, dzs, dpw, 1, nullptr, status);
    MUSE_LAUNCH_OK();
  }
  return MUSE_OK;
}

}  // namespace muse
