// Far-field forward on the tensor cores (bf16 mode, D = 128, Ck a multiple of 128, Ck <= 1024).
// One CTA per (query cluster i, plane, head) segment; its ~32 queries share the Ck accumulated
// summaries of (i, plane).  The summaries sit on the MMA M side (128 clusters per tile, one TMEM
// lane each) and the queries on the N side (32 columns), so no tensor work is wasted on the
// short segment:
//   A  scores^T[j][r] = (kappa_hi[j] + kappa_lo[j]) . q[r]   two accumulating MMAs per tile,
//      kappa tiles streamed by TMA through a 2-stage ring;  score = sigma * that + beta[j] (Eq. 6)
//   B  TMEM -> shared memory transposed to [r][j] fp32
//   C  per query (one warp each): top-m selection, far-set softmax, P written as a bf16 operand
//   D  out^T[d][r] = sum_j nu[j][d] P[r][j]      nu tiles (MN-major A operand) streamed by TMA
//   E  TMEM -> o_far (thread = d, coalesced over d for each query)
#include <cuda.h>
#include "common.cuh"
#include "tc05.cuh"

namespace muse {

typedef __nv_bfloat16 bf16;
int make_tmap_bf16_rows(void* out_map, const void* base, uint64_t rows, uint32_t cols, uint32_t box_rows);

constexpr int kFD = 128, kFJ = 128, kFR = 32;       // head dim, clusters per tile, queries per pass
constexpr int kTileBytes = kFJ * kFD * 2;           // 32 KB: one [128][128] bf16 operand tile
constexpr int kR1 = 0, kR1Bytes = 2 * kTileBytes;   // ring of kappa tiles, later the P operand
constexpr int kR2 = kR1 + kR1Bytes;                 // scores [32][Ck] fp32, later ring of nu tiles
constexpr int kFarTcCols = 512;

struct FarBars { uint64_t fullA[2], emptyA[2], fullD[4], emptyD[4], done; };

__global__ void __launch_bounds__(128)
k_far_fwd_tc(Dims dm, const __grid_constant__ CUtensorMap tm_khi, const __grid_constant__ CUtensorMap tm_klo,
             const __grid_constant__ CUtensorMap tm_nu, const bf16* __restrict__ Q, const int32_t* __restrict__ off_q,
             const int32_t* __restrict__ perm_q, const float* __restrict__ mu, const float* __restrict__ beta,
             const int32_t* __restrict__ sel_in, int32_t* __restrict__ sel_out, float* __restrict__ o_far,
             float* __restrict__ lse_far, int r2_bytes, int nsD, int* __restrict__ status) {
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ FarBars bars;
  __shared__ uint32_t tbase_s;
  __shared__ int32_t rows[kFR];
  __shared__ float rinv[kFR];
  __shared__ int32_t selq[kMaxM];
  const int i = blockIdx.x, pl = blockIdx.y, pq = blockIdx.z;
  const int blk = dm.causal ? pl + 1 : 0, Ck = dm.Ck, NJ = Ck / kFJ, m = dm.m;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int32_t* oq = off_q + (size_t)pq * (dm.S * dm.Cq + 1) + (size_t)blk * dm.Cq + i;
  const int p0 = oq[0], p1 = oq[1];
  if (p0 >= p1) return;
  unsigned char* sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);
  unsigned char* R1 = sm + kR1;
  float* sc = reinterpret_cast<float*>(sm + kR2);
  unsigned char* Qs = sm + kR2 + r2_bytes;
  const size_t ent0 = (((size_t)pq * dm.SB + pl) * dm.Cq + i) * Ck;
  const float* mup = mu + ent0;
  const float* bep = beta + ent0;
  const bf16* Qp = Q + (size_t)pq * dm.N * kFD;
  const int32_t* pm = perm_q + (size_t)pq * dm.N;

  if (warp == 0) tc::tmem_alloc(&tbase_s, kFarTcCols);
  if (tid == 0) {
    for (int s = 0; s < 2; ++s) { tc::mbar_init(&bars.fullA[s], 1); tc::mbar_init(&bars.emptyA[s], 1); }
    for (int s = 0; s < 4; ++s) { tc::mbar_init(&bars.fullD[s], 1); tc::mbar_init(&bars.emptyD[s], 1); }
    tc::mbar_init(&bars.done, 1);
    tc::mbar_init_fence();
  }
  if (dm.sel_mode == MUSE_SEL_PER_QCLUSTER && sel_in == nullptr && m > 0 && warp == 1) {
    // one selection per segment: rank clusters by accumulated log-mass alone
    float* tmp = sc;
    for (int j = lane; j < Ck; j += 32) tmp[j] = mup[j];
    __syncwarp();
    for (int k = 0; k < m; ++k) {
      float bv = -INFINITY; int bi = 0x7fffffff;
      for (int j = lane; j < Ck; j += 32) { float v = tmp[j]; if (v > bv) { bv = v; bi = j; } }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        float ov = __shfl_xor_sync(0xffffffffu, bv, o); int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
      }
      if (lane == 0) selq[k] = bv == -INFINITY ? -1 : bi;
      if (bv != -INFINITY && (bi & 31) == lane) tmp[bi] = -INFINITY;
      __syncwarp();
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tbase = tbase_s;
  uint32_t useA[2] = {0, 0}, useD[4] = {0, 0, 0, 0}, done_ph = 0;    // barrier phase counters (thread 0 / all)
  bool ok = true;

  for (int r0 = p0; r0 < p1 && ok; r0 += kFR) {
    const int n = min(kFR, p1 - r0);
    if (tid < kFR) rows[tid] = tid < n ? pm[r0 + tid] : -1;
    // query rows -> K-major swizzled tile [32][128] bf16 (2 blocks of [32][128 B])
    for (int e = tid; e < kFR * (kFD / 8); e += 128) {
      const int r = e >> 4, ck = e & 15, kb = ck >> 3, c = ck & 7;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (r < n) v = reinterpret_cast<const uint4*>(Qp + (size_t)pm[r0 + r] * kFD)[ck];
      *reinterpret_cast<uint4*>(Qs + kb * kFR * 128 + tc::sw128_off(r, c)) = v;
    }
    tc::fence_async_smem();
    tc::fence_before_sync();
    __syncthreads();
    // ---- A: scores^T for all clusters, kappa_hi / kappa_lo tiles through a 2-stage TMA ring ----
    if (tid == 0) {
      tc::fence_after_sync();
      const uint32_t idesc = tc::idesc_bf16(kFJ, kFR, 0, 0);
      const uint32_t qa = tc::smem_u32(Qs);
      const int T = 2 * NJ;
      for (int t = 0; t <= T && ok; ++t) {
        if (t < T) {
          const int s = t & 1;
          if (!tc::mbar_wait(&bars.emptyA[s], (useA[s] & 1) ^ 1)) { ok = false; break; }
          tc::mbar_expect_tx(&bars.fullA[s], kTileBytes);
          const void* map = (t & 1) ? (const void*)&tm_klo : (const void*)&tm_khi;
          const int row = (int)(ent0 + (size_t)(t >> 1) * kFJ);
          tc::tma_load_2d(R1 + s * kTileBytes, map, 0, row, &bars.fullA[s]);
          tc::tma_load_2d(R1 + s * kTileBytes + kFJ * 128, map, 64, row, &bars.fullA[s]);
        }
        if (t >= 1) {
          const int u = t - 1, s = u & 1;
          if (!tc::mbar_wait(&bars.fullA[s], useA[s] & 1)) { ok = false; break; }
          tc::fence_after_sync();
          const uint32_t a0 = tc::smem_u32(R1 + s * kTileBytes);
#pragma unroll
          for (int ks = 0; ks < kFD / 16; ++ks)
            tc::mma_bf16_ss(tbase + (u >> 1) * kFR, tc::smem_desc_sw128(a0 + (ks / 4) * kFJ * 128 + (ks % 4) * 32, 16, 1024),
                            tc::smem_desc_sw128(qa + (ks / 4) * kFR * 128 + (ks % 4) * 32, 16, 1024), idesc, (u & 1) || ks > 0);
          tc::mma_commit(&bars.emptyA[s]);
          useA[s]++;
        }
      }
      tc::mma_commit(&bars.done);
    }
    if (!tc::mbar_wait(&bars.done, done_ph)) ok = false;
    done_ph ^= 1;
    tc::fence_after_sync();
    // ---- B: TMEM -> sc[r][j]
    for (int jt = 0; jt < NJ; ++jt) {
      float v[32];
      tc::tmem_ld32(tbase + ((uint32_t)(warp * 32) << 16) + jt * kFR, v);
      const int j = jt * kFJ + tid;
      const float b = bep[j];
#pragma unroll
      for (int r = 0; r < kFR; ++r) sc[r * Ck + j] = b == -INFINITY ? -INFINITY : fmaf(v[r], dm.sigma, b);
    }
    tc::fence_before_sync();
    __syncthreads();
    // ---- C: selection + softmax of the far set; P (bf16) -> R1 as a K-major operand [32][Ck]
    for (int r = warp; r < kFR; r += 4) {
      float* s = sc + r * Ck;
      float sum = 0.f, mx = -INFINITY;
      if (r < n) {
        const int t = rows[r];
        int32_t* so = sel_out + ((size_t)pq * dm.N + t) * m;
        if (sel_in != nullptr) {
          const int32_t* si = sel_in + ((size_t)pq * dm.N + t) * m;
          for (int k = lane; k < m; k += 32) { int c = si[k]; so[k] = c; if (c >= 0 && c < Ck) s[c] = -INFINITY; }
        } else if (dm.sel_mode == MUSE_SEL_PER_QCLUSTER) {
          for (int k = lane; k < m; k += 32) { int c = selq[k]; so[k] = c; if (c >= 0) s[c] = -INFINITY; }
        } else {
          float lv = -INFINITY; int li = 0x7fffffff;
          for (int j = lane; j < Ck; j += 32) { float v = s[j]; if (v > lv) { lv = v; li = j; } }
          for (int k = 0; k < m; ++k) {
            float bv = lv; int bi = li;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
              float ov = __shfl_xor_sync(0xffffffffu, bv, o); int oi = __shfl_xor_sync(0xffffffffu, bi, o);
              if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
            }
            const bool any = bv != -INFINITY;
            if (lane == 0) so[k] = any ? bi : -1;
            if (any && (bi & 31) == lane) {
              s[bi] = -INFINITY;
              lv = -INFINITY; li = 0x7fffffff;
              for (int j = lane; j < Ck; j += 32) { float v = s[j]; if (v > lv) { lv = v; li = j; } }
            }
          }
        }
        __syncwarp();
        for (int j = lane; j < Ck; j += 32) mx = fmaxf(mx, s[j]);
        mx = warp_max(mx);
      }
      // probabilities, 8 consecutive clusters (one 16-byte chunk) per lane and step
      for (int q = lane; q < Ck / 8; q += 32) {
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          float p0_ = 0.f, p1_ = 0.f;
          if (mx != -INFINITY) { p0_ = __expf(s[q * 8 + 2 * k] - mx); p1_ = __expf(s[q * 8 + 2 * k + 1] - mx); }
          __nv_bfloat162 b = __floats2bfloat162_rn(p0_, p1_);
          sum += __low2float(b) + __high2float(b);
          w[k] = *reinterpret_cast<uint32_t*>(&b);
        }
        *reinterpret_cast<uint4*>(R1 + (q >> 3) * (kFR * 128) + tc::sw128_off(r, q & 7)) = make_uint4(w[0], w[1], w[2], w[3]);
      }
      sum = warp_sum(sum);
      if (lane == 0) {
        rinv[r] = sum > 0.f ? 1.f / sum : 0.f;
        if (r < n) lse_far[(size_t)pq * dm.N + rows[r]] = sum > 0.f ? mx + logf(sum) : -INFINITY;
      }
    }
    tc::fence_async_smem();
    tc::fence_before_sync();
    __syncthreads();
    // ---- D: out^T = nu^T P^T, nu tiles through an nsD-stage TMA ring in the score region;
    //         loads run nsD - 1 tiles ahead of the MMAs
    if (tid == 0 && ok) {
      tc::fence_after_sync();
      const uint32_t idesc = tc::idesc_bf16(kFD, kFR, 1, 0);
      const uint32_t pa = tc::smem_u32(R1);
      unsigned char* ring = sm + kR2;
      const int look = nsD - 1;
      for (int t = 0; t < NJ + look && ok; ++t) {
        if (t < NJ) {
          const int s = t % nsD;
          if (!tc::mbar_wait(&bars.emptyD[s], (useD[s] & 1) ^ 1)) { ok = false; break; }
          tc::mbar_expect_tx(&bars.fullD[s], kTileBytes);
          const int row = (int)(ent0 + (size_t)t * kFJ);
          tc::tma_load_2d(ring + s * kTileBytes, &tm_nu, 0, row, &bars.fullD[s]);
          tc::tma_load_2d(ring + s * kTileBytes + kFJ * 128, &tm_nu, 64, row, &bars.fullD[s]);
        }
        const int u = t - look;
        if (u >= 0) {
          const int s = u % nsD;
          if (!tc::mbar_wait(&bars.fullD[s], useD[s] & 1)) { ok = false; break; }
          tc::fence_after_sync();
          const uint32_t a0 = tc::smem_u32(ring + s * kTileBytes);
#pragma unroll
          for (int ks = 0; ks < kFJ / 16; ++ks)
            tc::mma_bf16_ss(tbase + 256, tc::smem_desc_sw128(a0 + ks * 16 * 128, kFJ * 128, 1024),
                            tc::smem_desc_sw128(pa + (2 * u + ks / 4) * (kFR * 128) + (ks % 4) * 32, 16, 1024), idesc,
                            u > 0 || ks > 0);
          tc::mma_commit(&bars.emptyD[s]);
          useD[s]++;
        }
      }
      tc::mma_commit(&bars.done);
    }
    if (!tc::mbar_wait(&bars.done, done_ph)) ok = false;
    done_ph ^= 1;
    tc::fence_after_sync();
    // ---- E: thread = output dim d
    {
      float v[32];
      tc::tmem_ld32(tbase + ((uint32_t)(warp * 32) << 16) + 256, v);
      if (ok) {
#pragma unroll
        for (int r = 0; r < kFR; ++r)
          if (r < n) o_far[((size_t)pq * dm.N + rows[r]) * kFD + tid] = v[r] * rinv[r];
      }
    }
    tc::fence_before_sync();
    __syncthreads();
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tbase, kFarTcCols);
  if (!ok && tid == 0) atomicExch(status, 3);
}

bool far_fwd_tc_supported(const Dims& d, int dtype) {
  return dtype == MUSE_BF16 && d.D == kFD && d.Ck % kFJ == 0 && d.Ck <= 1024 && d.Ck >= kFJ;
}

int far_fwd_tc(const Dims& d, const SummPtrs& sp, const void* Q, const int32_t* off_q, const int32_t* perm_q,
               const int32_t* sel_in, int32_t* sel_out, float* o_far, float* lse_far, int* status, cudaStream_t st) {
  const uint64_t ent = (uint64_t)d.B * d.Hq * d.SB * d.Cq * d.Ck;
  CUtensorMap khi, klo, nu;
  int rc = make_tmap_bf16_rows(&khi, sp.khi, ent, kFD, kFJ);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&klo, sp.klo, ent, kFD, kFJ);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&nu, sp.nu, ent, kFD, kFJ);
  if (rc != MUSE_OK) return rc;
  const int sc_bytes = kFR * d.Ck * 4;
  int nsD = sc_bytes / kTileBytes;
  nsD = nsD < 2 ? 2 : nsD > 4 ? 4 : nsD;
  const int r2_bytes = sc_bytes > nsD * kTileBytes ? sc_bytes : nsD * kTileBytes;
  const size_t smem = (size_t)kR1Bytes + r2_bytes + kFR * kFD * 2 + 1024;
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_far_fwd_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  prof_mark("k_far_fwd_tc", st);
  k_far_fwd_tc<<<dim3(d.Cq, d.SB, d.B * d.Hq), 128, smem, st>>>(d, khi, klo, nu, (const bf16*)Q, off_q, perm_q, sp.mu, sp.beta,
                                                               sel_in, sel_out, o_far, lse_far, r2_bytes, nsD, status);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

}  // namespace muse
