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

constexpr int kFarTcThreads = 512;      // 16 warps: the per-query selection (phase C) is the long pole

__global__ void __launch_bounds__(kFarTcThreads, 1)
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
#ifdef MUSE_PHASE_CLOCKS
    long long ck0 = clock64(), ck1 = 0, ck2 = 0, ck3 = 0, ck4 = 0;
#endif
    if (tid < kFR) rows[tid] = tid < n ? pm[r0 + tid] : -1;
    // query rows -> K-major swizzled tile [32][128] bf16 (2 blocks of [32][128 B])
    for (int e = tid; e < kFR * (kFD / 8); e += kFarTcThreads) {
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
    __syncwarp();     // lanes 1..31 of warp 0 park here instead of spinning beside the issuing lane
    if (!tc::mbar_wait(&bars.done, done_ph)) ok = false;
    done_ph ^= 1;
    tc::fence_after_sync();
#ifdef MUSE_PHASE_CLOCKS
    ck1 = clock64();
#endif
    // ---- B: TMEM -> sc[r][j]
    float bq[2];                                        // beta of this thread's clusters, loaded ahead of the TMEM reads
#pragma unroll
    for (int k = 0; k < 2; ++k) { const int jt = (warp >> 2) + 4 * k; bq[k] = jt < NJ ? bep[jt * kFJ + (tid & 127)] : 0.f; }
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int jt = (warp >> 2) + 4 * k;
      if (jt >= NJ) break;
      float v[32];
      tc::tmem_ld32(tbase + ((uint32_t)((warp & 3) * 32) << 16) + jt * kFR, v);
      const int j = jt * kFJ + (tid & 127);
      const float b = bq[k];
#pragma unroll
      for (int r = 0; r < kFR; ++r) sc[r * Ck + j] = b == -INFINITY ? -INFINITY : fmaf(v[r], dm.sigma, b);
    }
    tc::fence_before_sync();
    __syncthreads();
#ifdef MUSE_PHASE_CLOCKS
    ck2 = clock64();
#endif
    // ---- C: selection + softmax of the far set; P (bf16) -> R1 as a K-major operand [32][Ck]
    for (int r = warp; r < kFR; r += kFarTcThreads / 32) {
      float* s = sc + r * Ck;
      float sum = 0.f, mx = -INFINITY;
#ifdef MUSE_PHASE_CLOCKS
      long long cc0 = clock64(), cc1 = 0, cc2 = 0;
#endif
      if (r < n) {
        const int t = rows[r];
        int32_t* so = sel_out + ((size_t)pq * dm.N + t) * m;
        if (sel_in != nullptr) {
          const int32_t* si = sel_in + ((size_t)pq * dm.N + t) * m;
          for (int k = lane; k < m; k += 32) { int c = si[k]; so[k] = c; if (c >= 0 && c < Ck) s[c] = -INFINITY; }
        } else if (dm.sel_mode == MUSE_SEL_PER_QCLUSTER) {
          for (int k = lane; k < m; k += 32) { int c = selq[k]; so[k] = c; if (c >= 0) s[c] = -INFINITY; }
        } else if (m > 0) {
          // Top-m by bisection on an order-preserving integer key of the score: find the key T
          // of the m-th largest with warp ballots (no serial arg-max rounds), take everything
          // above T and, among ties at T, the lowest cluster indices.
          const int NK = Ck >> 5;                       // scores per lane (<= 32)
          uint32_t key[32];
#pragma unroll
          for (int k = 0; k < 32; ++k) {
            const uint32_t b = __float_as_uint(k < NK ? s[lane + 32 * k] : -INFINITY);
            key[k] = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
          }
          const uint32_t kFinite = 0x00800000u;         // smallest key above key(-inf) = 0x007fffff
          auto count_ge = [&](uint32_t thr) {          // lane-local count, then one warp reduction
            int c = 0;
#pragma unroll
            for (int k = 0; k < 32; ++k) c += key[k] >= thr ? 1 : 0;
            return (int)__reduce_add_sync(0xffffffffu, (unsigned)c);
          };
          uint32_t T = kFinite;
          if (count_ge(kFinite) > m) {
            // the leading bits shared by the largest and the smallest finite key need no search
            uint32_t kmx = 0u, kmn = 0xffffffffu;
#pragma unroll
            for (int k = 0; k < 32; ++k) { kmx = max(kmx, key[k]); kmn = min(kmn, key[k] >= kFinite ? key[k] : 0xffffffffu); }
            const uint32_t lane_max = kmx;
            kmx = __reduce_max_sync(0xffffffffu, kmx);
            kmn = __reduce_min_sync(0xffffffffu, kmn);
            if (m <= 32) {
              // the m-th largest of the 32 lane maxima bounds the m-th largest score from below:
              // a cheap one-value-per-lane bisection that shortens the search interval
              uint32_t lb = 0;
              for (int bit = 31; bit >= 0; --bit) {
                const uint32_t cand = lb | (1u << bit);
                if (__popc(__ballot_sync(0xffffffffu, lane_max >= cand)) >= m) lb = cand;
              }
              kmn = max(kmn, lb);
            }
            const int shared = __clz((int)(kmx ^ kmn));            // 32 if the interval is a single key
            T = shared >= 32 ? kmx : (kmx & ~(0xffffffffu >> shared));
            for (int bit = 31 - shared; bit >= 0; --bit) {
              const uint32_t cand = T | (1u << bit);
              const int c = count_ge(cand);
              if (c >= m) { T = cand; if (c == m) break; }
            }
          }
          const int need = m - count_ge(T + 1);         // ties at T to take (all of them if T == kFinite)
          const uint32_t lt = (1u << lane) - 1u;
          int base = 0, ties_seen = 0;
#pragma unroll
          for (int k = 0; k < 32; ++k) {
            if (k < NK) {
              const bool tie = key[k] == T && T != kFinite ? true : false;
              const bool gt = T == kFinite ? key[k] >= T : key[k] > T;
              const uint32_t mt = __ballot_sync(0xffffffffu, tie);
              const bool take = gt || (tie && ties_seen + __popc(mt & lt) < need);
              ties_seen += __popc(mt);
              const uint32_t ms = __ballot_sync(0xffffffffu, take);
              if (take) { so[base + __popc(ms & lt)] = lane + 32 * k; s[lane + 32 * k] = -INFINITY; }
              base += __popc(ms);
            }
          }
          for (int k = base + lane; k < m; k += 32) so[k] = -1;
        }
        __syncwarp();
        for (int j = lane; j < Ck; j += 32) mx = fmaxf(mx, s[j]);
        mx = warp_max(mx);
      }
#ifdef MUSE_PHASE_CLOCKS
      cc1 = clock64();
#endif
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
#ifdef MUSE_PHASE_CLOCKS
      cc2 = clock64();
      if (tid == 0 && blockIdx.x == 5 && blockIdx.y == 3 && blockIdx.z == 0 && r0 == p0 && r == 0) { status[13] = (int)(cc1 - cc0); status[14] = (int)(cc2 - cc1); }
#endif
      sum = warp_sum(sum);
      if (lane == 0) {
        rinv[r] = sum > 0.f ? 1.f / sum : 0.f;
        if (r < n) lse_far[(size_t)pq * dm.N + rows[r]] = sum > 0.f ? mx + logf(sum) : -INFINITY;
      }
    }
    tc::fence_async_smem();
    tc::fence_before_sync();
    __syncthreads();
#ifdef MUSE_PHASE_CLOCKS
    ck3 = clock64();
#endif
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
    __syncwarp();
    if (!tc::mbar_wait(&bars.done, done_ph)) ok = false;
    done_ph ^= 1;
    tc::fence_after_sync();
#ifdef MUSE_PHASE_CLOCKS
    ck4 = clock64();
    if (tid == 0 && blockIdx.x == 5 && blockIdx.y == 3 && blockIdx.z == 0 && r0 == p0) {
      status[8] = (int)(ck1 - ck0); status[9] = (int)(ck2 - ck1); status[10] = (int)(ck3 - ck2); status[11] = (int)(ck4 - ck3);
      status[12] = n;
    }
#endif
    // ---- E: thread = output dim d
    if (warp < 4) {
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
  k_far_fwd_tc<<<dim3(d.Cq, d.SB, d.B * d.Hq), kFarTcThreads, smem, st>>>(d, khi, klo, nu, (const bf16*)Q, off_q, perm_q, sp.mu, sp.beta,
                                                               sel_in, sel_out, o_far, lse_far, r2_bytes, nsD, status);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

}  // namespace muse
