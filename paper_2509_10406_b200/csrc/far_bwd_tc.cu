// Far-field backward on the tensor cores (bf16 mode, D = 64 or 128, Ck a multiple of 128, <= 2048).
// One CTA per (query cluster i, plane, head) segment.  Clusters sit on the MMA M side (128 per
// tile, one TMEM lane each), the segment's queries on the N side (64 per sweep; a longer segment
// takes further sweeps that add to the stored gradients).  Per cluster tile, with L the merged log-sum-exp and delta = dO.O:
//   S^T   = (kappa_hi + kappa_lo) Q^T,  dPnu^T = nu dO^T                      (tcgen05, TMA-fed tiles)
//   p     = exp(sigma S + beta - L) on the far set,  g = p (dPnu - delta)      (one thread per cluster)
//   dnu  += p dO,   dkappa_raw += (sigma g) Q,   dq^T += kappa^T (sigma g)     (tcgen05; the G tile carries sigma)
//   dkappa = dkappa_raw - sigma (sum_r g) qbar_i
//   dS = sum_r g - dkappa.kappa - dnu.nu = sum_r g (1 + mu - score) - sum_r p dPnu   (no row dot products)
// dkappa and dnu are stored as bf16 rows for the key-side pass, dS as fp32.
#include <cuda.h>
#include "common.cuh"
#include "tc05.cuh"


namespace muse {

typedef __nv_bfloat16 bf16;
int make_tmap_bf16_rows(void* out_map, const void* base, uint64_t rows, uint32_t cols, uint32_t box_rows);
int make_tmap_bf16_nd(void* out_map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                      const uint32_t* box);

namespace fb {
constexpr int TJ = 128, NR = 64, NP = 1;
constexpr int THREADS = 288, CW = 256, ISSUER = 256;   // warps 0-7 do the arithmetic; lane 0 of a ninth warp issues every TMA transfer and MMA
template <int D> struct Lay {
  static constexpr int kTile = TJ * D * 2;        // operand tile [128 clusters][D] bf16
  static constexpr int kRows = NR * D * 2;        // tile of 64 query rows
  static constexpr int oHi = 0, oLo = oHi + kTile, oNu = oLo + kTile;
  static constexpr int oQ = oNu + kTile, oDO = oQ + NP * kRows;
  static constexpr int oPt = oDO + NP * kRows, oGt = oPt + TJ * NR * 2;
  // gradient rows on their way out: dkappa is staged in the (consumed) P / G tiles, dnu in a tile of its own,
  // so that the three operand tiles are free for the next cluster tile as soon as the MMAs have finished
  static constexpr int oStK = oPt, oStN = oGt + TJ * NR * 2;
  static constexpr int oMask = oStN + kTile;      // [NP*NR rows][Ck/32] words follow
};
constexpr uint32_t cS = 0, cDP = 64, cDNU = 128, cDKA = 256, cDQ = 384;   // TMEM columns
constexpr float kLog2e = 1.4426950408889634f;
}  // namespace fb

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int D>
__global__ void __launch_bounds__(fb::THREADS, 1)
k_far_bwd_tc(Dims dm, const __grid_constant__ CUtensorMap tm_khi, const __grid_constant__ CUtensorMap tm_klo,
             const __grid_constant__ CUtensorMap tm_nu, const __grid_constant__ CUtensorMap tm_gka,
             const __grid_constant__ CUtensorMap tm_gnu, const bf16* __restrict__ Q, const bf16* __restrict__ dO,
             const float* __restrict__ qbar, const float* __restrict__ LSE, const float* __restrict__ delta,
             const int32_t* __restrict__ off_q, const int32_t* __restrict__ perm_q, const int32_t* __restrict__ sel,
             const float* __restrict__ beta, const float* __restrict__ mu, float* __restrict__ dQacc, bf16* __restrict__ dkappa,
             bf16* __restrict__ dnu, float* __restrict__ dS, int grad_by_key_cluster, int* __restrict__ status) {
  using namespace fb;
  typedef Lay<D> LY;
  constexpr int kTile = LY::kTile, kRows = LY::kRows, oHi = LY::oHi, oLo = LY::oLo, oNu = LY::oNu, oQ = LY::oQ, oDO = LY::oDO,
                oPt = LY::oPt, oGt = LY::oGt, oStK = LY::oStK, oStN = LY::oStN, oMask = LY::oMask, G = D / 64, CPR = D / 8;
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  // bar_full: kappa tiles landed; bar_nu: nu tile landed; bar1: S / dPnu products done; bar2: dnu / dkappa
  // products done; bar3: dq products done as well; bar_st: the previous tile's stores have read their staging
  __shared__ uint64_t bar_full, bar_nu, bar1, bar2, bar3, bar_st;
  __shared__ uint32_t tbase_s;
  __shared__ int32_t rows[NP * NR];
  __shared__ __align__(16) float Ls[NP * NR], ds[NP * NR], qb[D], part[2][TJ], dsid[2][TJ];
  const int i = blockIdx.x, pl = blockIdx.y, pq = blockIdx.z;
  const int blk = dm.causal ? pl + 1 : 0, Ck = dm.Ck, NJ = Ck / TJ, MW = Ck >> 5, m = dm.m;
  const int tid = threadIdx.x, warp = tid >> 5, wg = tid >> 7, L = tid & 127;
#ifdef MUSE_PHASE_CLOCKS
  const long long t_in_ = clock64();
  long long t_loop_ = 0, t_end_ = 0;
#endif
  const int32_t* oq = off_q + (size_t)pq * (dm.S * dm.Cq + 1) + (size_t)blk * dm.Cq + i;
  const int p0 = oq[0], p1 = oq[1];
  if (p0 >= p1) {
    // An empty segment: its gradient rows are zeros.  The key-side tensor-core pass (the reader of the
    // [plane][j][i] layout) takes whole tiles of rows without looking at which segments exist.
    if (grad_by_key_cluster) {
      const size_t row0 = ((size_t)pq * dm.SB + pl) * Ck;
      for (int e = tid; e < Ck * CPR; e += blockDim.x) {
        const size_t at = ((row0 + (e / CPR)) * dm.Cq + i) * D + (e % CPR) * 8;
        *reinterpret_cast<uint4*>(dkappa + at) = make_uint4(0u, 0u, 0u, 0u);
        *reinterpret_cast<uint4*>(dnu + at) = make_uint4(0u, 0u, 0u, 0u);
      }
      for (int j = tid; j < Ck; j += blockDim.x) dS[(row0 + j) * dm.Cq + i] = 0.f;
    }
    return;
  }
  unsigned char* sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);
  uint32_t* smask = reinterpret_cast<uint32_t*>(sm + oMask);
  const size_t ent0 = (((size_t)pq * dm.SB + pl) * dm.Cq + i) * Ck;
  const bf16* Qp = Q + (size_t)pq * dm.N * D;
  const bf16* dOp = dO + (size_t)pq * dm.N * D;
  const int32_t* pm = perm_q + (size_t)pq * dm.N;

  if (warp == 0) tc::tmem_alloc(&tbase_s, 512);
  if (tid == 0) { tc::mbar_init(&bar_full, 1); tc::mbar_init(&bar1, 1); tc::mbar_init(&bar2, 1); tc::mbar_init(&bar3, 1);
                  tc::mbar_init(&bar_nu, 1); tc::mbar_init(&bar_st, 1); tc::mbar_init_fence(); }
  if (tid < D) qb[tid] = qbar[((size_t)pq * dm.Cq + i) * D + tid];
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tbase = tbase_s, tlane = tbase + ((uint32_t)((warp & 3) * 32) << 16);
  uint32_t ph_full = 0, ph1 = 0, ph2 = 0, ph3 = 0, ph_st = 0;
  const bool cw = warp < 8;                               // compute warp
  bool ok = true;
  const uint32_t aHi = tc::smem_u32(sm + oHi), aLo = tc::smem_u32(sm + oLo), aNu = tc::smem_u32(sm + oNu),
                 aPt = tc::smem_u32(sm + oPt), aGt = tc::smem_u32(sm + oGt);

  auto issue_kappa = [&](int jt_) {                       // issuer: the two kappa tiles of cluster tile jt_
    tc::mbar_expect_tx(&bar_full, 2 * kTile);
    const int row = (int)(ent0 + (size_t)jt_ * TJ);
    for (int g = 0; g < G; ++g) {
      tc::tma_load_2d(sm + oHi + g * TJ * 128, &tm_khi, 64 * g, row, &bar_full);
      tc::tma_load_2d(sm + oLo + g * TJ * 128, &tm_klo, 64 * g, row, &bar_full);
    }
  };
  auto issue_nu = [&](int jt_) {                          // issuer: its nu tile
    tc::mbar_expect_tx(&bar_nu, kTile);
    const int row = (int)(ent0 + (size_t)jt_ * TJ);
    for (int g = 0; g < G; ++g) tc::tma_load_2d(sm + oNu + g * TJ * 128, &tm_nu, 64 * g, row, &bar_nu);
  };
  for (int s0 = p0; s0 < p1 && ok; s0 += NP * NR) {        // sweep: up to 64 rows
    const int ns = min(NP * NR, p1 - s0), np = (ns + NR - 1) / NR;
    __syncthreads();
    // the operand tiles are free (every product of the previous sweep has completed): the first cluster
    // tile travels while the rows are gathered
    if (tid == ISSUER) { issue_kappa(0); issue_nu(0); }
    if (tid < NP * NR) {
      int t = tid < ns && MUSE_IN_RANGE(s0 + tid, dm.N) ? pm[s0 + tid] : -1;
      if (t >= 0 && !MUSE_IN_RANGE(t, dm.N)) t = -1;
      rows[tid] = t;
      Ls[tid] = t >= 0 ? LSE[(size_t)pq * dm.N + t] * kLog2e : 0.f;
      ds[tid] = t >= 0 ? delta[(size_t)pq * dm.N + t] : 0.f;
    }
    for (int e = tid; e < 2 * Ck; e += THREADS) smask[e] = 0u;
    __syncthreads();
    for (int e = tid; e < NP * NR * CPR; e += THREADS) {
      const int r = e / CPR, ck = e % CPR, kb = ck >> 3, c = ck & 7, p = r / NR, rr = r % NR;
      uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;
      if (r < ns && rows[r] >= 0) {
        a = reinterpret_cast<const uint4*>(Qp + (size_t)rows[r] * D)[ck];
        b = reinterpret_cast<const uint4*>(dOp + (size_t)rows[r] * D)[ck];
      }
      *reinterpret_cast<uint4*>(sm + oQ + p * kRows + kb * NR * 128 + tc::sw128_off(rr, c)) = a;
      *reinterpret_cast<uint4*>(sm + oDO + p * kRows + kb * NR * 128 + tc::sw128_off(rr, c)) = b;
    }
    for (int e = tid; e < ns * m; e += THREADS) {
      const int r = e / m, k = e % m;
      const int c = rows[r] >= 0 ? sel[((size_t)pq * dm.N + rows[r]) * m + k] : -1;
      if (c >= 0 && c < Ck) atomicOr(&smask[2 * c + (r >> 5)], 1u << (r & 31));     // [cluster][row bits]
    }
    tc::fence_async_smem();
    __syncthreads();

#ifdef MUSE_PHASE_CLOCKS
    long long pc[6] = {0, 0, 0, 0, 0, 0};
#endif
    // L and delta of this warpgroup's 32 rows stay in registers for the whole sweep
    static_assert(NP == 1, "one pass per sweep");
    float Lc[32], dc[32];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float4 a = *reinterpret_cast<const float4*>(Ls + 32 * (wg & 1) + 4 * k), b = *reinterpret_cast<const float4*>(ds + 32 * (wg & 1) + 4 * k);
      Lc[4 * k] = a.x; Lc[4 * k + 1] = a.y; Lc[4 * k + 2] = a.z; Lc[4 * k + 3] = a.w;
      dc[4 * k] = b.x; dc[4 * k + 1] = b.y; dc[4 * k + 2] = b.z; dc[4 * k + 3] = b.w;
    }
    float bnext = beta[ent0 + L];
    const bool later_sweep = s0 > p0;                       // gradients of earlier sweeps are already stored: add to them
    if (later_sweep) {
      if (tid == ISSUER) tc::tma_store_wait_all();
      __syncthreads();
    }
#ifdef MUSE_PHASE_CLOCKS
    t_loop_ = clock64();
#endif
    for (int jt = 0; jt < NJ && ok; ++jt) {
      const int j = jt * TJ + L;
#ifdef MUSE_PHASE_CLOCKS
      long long k0_ = clock64(), k1_ = 0, k2_ = 0, k3_ = 0, k4_ = 0;
#endif
      const float bj = bnext;                               // loaded one tile ahead
      const bool alive = bj != -INFINITY;                   // an empty cluster has beta = mu = -inf
      const float sig2 = dm.sigma * kLog2e, bj2 = alive ? bj * kLog2e : 0.f;
      if (jt + 1 < NJ) bnext = beta[ent0 + j + TJ];
      float gsum = 0.f, gt2 = 0.f, pdp = 0.f;
      const float mu1 = 1.f + mu[ent0 + j];                               // 1 + accumulated log-mass of cluster j
      for (int p = 0; p < np && ok; ++p) {
        const uint32_t aQ = tc::smem_u32(sm + oQ + p * kRows), aDO = tc::smem_u32(sm + oDO + p * kRows);
        if (tid == ISSUER) {
          if (p == 0) {
            if (!tc::mbar_wait(&bar_full, ph_full)) ok = false;
            if (!tc::mbar_wait(&bar_nu, ph_full)) ok = false;
          }
          tc::fence_after_sync();
          const uint32_t idesc = tc::idesc_bf16(TJ, NR, 0, 0);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            tc::mma_bf16_ss(tbase + cS, tc::smem_desc_sw128(aHi + (ks / 4) * TJ * 128 + (ks % 4) * 32, 16, 1024),
                            tc::smem_desc_sw128(aQ + (ks / 4) * NR * 128 + (ks % 4) * 32, 16, 1024), idesc, ks > 0);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            tc::mma_bf16_ss(tbase + cS, tc::smem_desc_sw128(aLo + (ks / 4) * TJ * 128 + (ks % 4) * 32, 16, 1024),
                            tc::smem_desc_sw128(aQ + (ks / 4) * NR * 128 + (ks % 4) * 32, 16, 1024), idesc, 1);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            tc::mma_bf16_ss(tbase + cDP, tc::smem_desc_sw128(aNu + (ks / 4) * TJ * 128 + (ks % 4) * 32, 16, 1024),
                            tc::smem_desc_sw128(aDO + (ks / 4) * NR * 128 + (ks % 4) * 32, 16, 1024), idesc, ks > 0);
          tc::mma_commit(&bar1);
          if (p == 0) {
            tc::tma_store_wait_read();        // the previous tile's stores have read the staging tiles, which the
            tc::mbar_arrive(&bar_st);         // compute warps write again (P / G tiles first)
          }
          if (!tc::mbar_wait(&bar1, ph1)) ok = false;
          if (p + 1 == np && jt + 1 < NJ && ok) issue_nu(jt + 1);     // the nu tile is only read by the products above
        }
        if (cw && !tc::mbar_wait(&bar1, ph1)) ok = false;
        ph1 ^= 1;
        tc::fence_after_sync();
#ifdef MUSE_PHASE_CLOCKS
        if (p == 0) k1_ = clock64();
#endif
        if (cw) {
          float s[32], dp[32];
          tc::tmem_ld32(tlane + cS + 32 * wg, s);
          tc::tmem_ld32(tlane + cDP + 32 * wg, dp);
#ifdef MUSE_PHASE_CLOCKS
          if (p == 0 && tid == 0 && blockIdx.x == 5 && blockIdx.y == 3 && blockIdx.z == 0 && jt == 3) status[32] = (int)(clock64() - k1_);
#endif
          uint32_t pw[16], gw[16];
          // bit r of `near`: row r of this warpgroup's 32 is not in the far set of cluster j (retrieved,
          // past the end of the segment, or the cluster is empty)
          const int nv = ns - (p * NR + 32 * wg);
          const uint32_t near = alive ? (smask[2 * j + wg] | (nv >= 32 ? 0u : nv <= 0 ? 0xffffffffu : 0xffffffffu << nv)) : 0xffffffffu;
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            float pv[2], gv[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const float t2 = fmaf(s[c + h], sig2, bj2);                 // Eq. 6 score in log2 units
              const float e = fast_exp2(t2 - Lc[c + h]);
              pv[h] = (near >> (c + h)) & 1u ? 0.f : e;
              gv[h] = pv[h] * (dp[c + h] - dc[c + h]);
              gsum += gv[h];
              gt2 = fmaf(gv[h], t2, gt2);
              pdp = fmaf(pv[h], dp[c + h], pdp);
            }
            __nv_bfloat162 a = __floats2bfloat162_rn(pv[0], pv[1]), b = __floats2bfloat162_rn(dm.sigma * gv[0], dm.sigma * gv[1]);
            pw[c >> 1] = *reinterpret_cast<uint32_t*>(&a);
            gw[c >> 1] = *reinterpret_cast<uint32_t*>(&b);
          }
#ifdef MUSE_PHASE_CLOCKS
          if (p == 0 && tid == 0 && blockIdx.x == 5 && blockIdx.y == 3 && blockIdx.z == 0 && jt == 3) status[33] = (int)(clock64() - k1_);
#endif
          if (p == 0) {
            if (!tc::mbar_wait(&bar_st, ph_st)) ok = false;
            ph_st ^= 1;
          }
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            *reinterpret_cast<uint4*>(sm + oPt + tc::sw128_off(L, 4 * wg + ch)) = make_uint4(pw[4 * ch], pw[4 * ch + 1], pw[4 * ch + 2], pw[4 * ch + 3]);
            *reinterpret_cast<uint4*>(sm + oGt + tc::sw128_off(L, 4 * wg + ch)) = make_uint4(gw[4 * ch], gw[4 * ch + 1], gw[4 * ch + 2], gw[4 * ch + 3]);
          }
        }
#ifdef MUSE_PHASE_CLOCKS
        if (p == 0) k2_ = clock64();
#endif
        tc::fence_async_smem();
        tc::fence_before_sync();
        __syncthreads();
        if (tid == ISSUER) {
          tc::fence_after_sync();
          const uint32_t id_row = tc::idesc_bf16(TJ, D, 0, 1);      // A K-major (P / G), B = query rows, MN-major
          // A = kappa tile MN-major, B = G MN-major.  M = 128 output dims even when D = 64: the second 64-dim group of the
          // operand is then the tile that follows in shared memory, and output lanes 64..127 hold numbers that nobody reads
          const uint32_t id_dq = tc::idesc_bf16(128, NR, 1, 1);
#pragma unroll
          for (int ks = 0; ks < NR / 16; ++ks)
            tc::mma_bf16_ss(tbase + cDNU, tc::smem_desc_sw128(aPt + ks * 32, 16, 1024),
                            tc::smem_desc_sw128(aDO + ks * 16 * 128, NR * 128, 1024), id_row, !(p == 0 && ks == 0));
#pragma unroll
          for (int ks = 0; ks < NR / 16; ++ks)
            tc::mma_bf16_ss(tbase + cDKA, tc::smem_desc_sw128(aGt + ks * 32, 16, 1024),
                            tc::smem_desc_sw128(aQ + ks * 16 * 128, NR * 128, 1024), id_row, !(p == 0 && ks == 0));
          tc::mma_commit(&bar2);              // the read-out of dnu / dkappa can start while the dq products still run
#pragma unroll
          for (int ks = 0; ks < TJ / 16; ++ks)
            tc::mma_bf16_ss(tbase + cDQ + p * NR, tc::smem_desc_sw128(aHi + ks * 16 * 128, TJ * 128, 1024),
                            tc::smem_desc_sw128(aGt + ks * 16 * 128, TJ * 128, 1024), id_dq, !(jt == 0 && ks == 0));
#pragma unroll
          for (int ks = 0; ks < TJ / 16; ++ks)
            tc::mma_bf16_ss(tbase + cDQ + p * NR, tc::smem_desc_sw128(aLo + ks * 16 * 128, TJ * 128, 1024),
                            tc::smem_desc_sw128(aGt + ks * 16 * 128, TJ * 128, 1024), id_dq, 1);
          tc::mma_commit(&bar3);
          // every MMA on the operand tiles has completed: the next cluster tile may overwrite them
          if (!tc::mbar_wait(&bar3, ph3)) ok = false;
          if (p + 1 == np && jt + 1 < NJ && ok) issue_kappa(jt + 1);
        }
        if (cw && !tc::mbar_wait(&bar2, ph2)) ok = false;
        // a further pass writes the P / G tiles again: the dq products must have read them
        if (cw && p + 1 < np && !tc::mbar_wait(&bar3, ph3)) ok = false;
        ph2 ^= 1;
        ph3 ^= 1;
        tc::fence_after_sync();
      }
      ph_full ^= 1;
#ifdef MUSE_PHASE_CLOCKS
      k3_ = clock64();
#endif
      // ---- tile read-out: warpgroup 0 -> dnu, warpgroup 1 -> dkappa; both need sum_r g
      float gtot = 0.f;
      if (cw) {
        // dS = sum_r g (1 + mu - score) - sum_r p (dO.nu): the same quantity as
        // sum_r g - dkappa.kappa - dnu.nu, without the two row dot products
        part[wg][L] = gsum; dsid[wg][L] = alive ? fmaf(mu1, gsum, fmaf(-0.6931471805599453f, gt2, -pdp)) : 0.f;
        tc::named_bar_sync(1, CW);                          // the issuer is still waiting for the dq products
        gtot = part[0][L] + part[1][L];
      }
#ifdef MUSE_PHASE_CLOCKS
      const bool rec_ = (tid == 0 || tid == 128) && blockIdx.x == 5 && blockIdx.y == 3 && blockIdx.z == 0 && jt == 3;
      if (rec_) status[34 + 3 * wg] = (int)(clock64() - k3_);
#endif
      // gradient entry: [plane][i][j] like the summaries, or [plane][j][i] so that the key-side
      // pass finds the 128 query clusters of one key cluster in one contiguous tile
      const size_t gent = grad_by_key_cluster ? (((size_t)pq * dm.SB + pl) * Ck + j) * dm.Cq + i : ent0 + j;
      // this thread's row, 32 dims per step, rounded into its own row of the staging tile (which then leaves
      // as one TMA box).  The G tile carried sigma, so dkappa = acc - (sigma sum_r g) qbar_i.  (Few instructions
      // per element matter more here than overlapping the TMEM loads: eight warps share the issue slots.)
      if (cw) {
        const uint32_t tsrc = tlane + (wg == 0 ? cDNU : cDKA);
        unsigned char* stg = sm + (wg == 0 ? oStN : oStK) + L * 128;
        const float gq = -dm.sigma * gtot;
#pragma unroll 1
        for (int u = 0; u < D / 32; ++u) {
          float x[32];
          tc::tmem_ld32(tsrc + 32 * u, x);
          // the second half of the dkappa staging is the G tile, which the dq products read
          if (u == 2 && wg == 1 && !tc::mbar_wait(&bar3, ph3 ^ 1)) ok = false;
          if (wg == 1) {
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {
              const float4 q = *reinterpret_cast<const float4*>(qb + 32 * u + 4 * ch);
              x[4 * ch] = fmaf(gq, q.x, x[4 * ch]); x[4 * ch + 1] = fmaf(gq, q.y, x[4 * ch + 1]);
              x[4 * ch + 2] = fmaf(gq, q.z, x[4 * ch + 2]); x[4 * ch + 3] = fmaf(gq, q.w, x[4 * ch + 3]);
            }
          }
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            const int d = 32 * u + 8 * ch;
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              __nv_bfloat162 b2 = __floats2bfloat162_rn(x[8 * ch + 2 * e], x[8 * ch + 2 * e + 1]);
              w[e] = *reinterpret_cast<uint32_t*>(&b2);
            }
            *reinterpret_cast<uint4*>(stg + (d >> 6) * (TJ * 128) + (((((d & 63) >> 3)) ^ (L & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
#ifdef MUSE_PHASE_CLOCKS
      if (rec_) status[35 + 3 * wg] = (int)(clock64() - k3_);
#endif
      // the two gradient tiles leave by TMA: 128 rows of 256 bytes each, Cq entries apart in the
      // [plane][j][i] layout (adjacent in the [plane][i][j] one)
      tc::fence_async_smem();
      __syncthreads();
#ifdef MUSE_PHASE_CLOCKS
      if (rec_) status[36 + 3 * wg] = (int)(clock64() - k3_);
#endif
      if (tid == ISSUER && ok) {
        const int c1 = grad_by_key_cluster ? i : 0;
        const int c2 = grad_by_key_cluster ? (pq * dm.SB + pl) * Ck + jt * TJ : (int)(ent0 + (size_t)jt * TJ);
        if (!later_sweep) {
          for (int g = 0; g < G; ++g) {
            tc::tma_store_3d(&tm_gnu, sm + oStN + g * TJ * 128, 64 * g, c1, c2);
            tc::tma_store_3d(&tm_gka, sm + oStK + g * TJ * 128, 64 * g, c1, c2);
          }
        } else {                              // a further sweep of a long segment adds to the stored rows
          for (int g = 0; g < G; ++g) {
            tc::tma_reduce_add_3d(&tm_gnu, sm + oStN + g * TJ * 128, 64 * g, c1, c2);
            tc::tma_reduce_add_3d(&tm_gka, sm + oStK + g * TJ * 128, 64 * g, c1, c2);
          }
        }
        tc::tma_store_commit();
      }
      tc::fence_before_sync();
      if (wg == 0 && ok) dS[gent] = (later_sweep ? dS[gent] : 0.f) + dsid[0][L] + dsid[1][L];
#ifdef MUSE_PHASE_CLOCKS
      k4_ = clock64();
      pc[0] += k1_ - k0_; pc[1] += k2_ - k1_; pc[2] += k3_ - k2_; pc[3] += k4_ - k3_; pc[4] += 1; pc[5] = np;
#endif
    }
#ifdef MUSE_PHASE_CLOCKS
    if (tid == 0 && blockIdx.x == 5 && blockIdx.y == 3 && blockIdx.z == 0 && s0 == p0)
      for (int k = 0; k < 6; ++k) status[24 + k] = (int)pc[k];
    t_end_ = clock64();
#endif
    // ---- dq: warpgroup p reads pass p (thread = output dim), adds into the fp32 accumulator
    if (cw && !tc::mbar_wait(&bar3, ph3 ^ 1)) ok = false;     // the last tile's dq products
    tc::fence_after_sync();
    for (int p = 0; cw && p < np; ++p) {
      for (int c0 = 32 * wg; c0 < NR; c0 += 64) {
        float v[32];
        tc::tmem_ld32(tlane + cDQ + p * NR + c0, v);
        if (ok && L < D) {
#pragma unroll
          for (int r = 0; r < 32; ++r) {
            const int rr = p * NR + c0 + r;
            if (rr < ns && rows[rr] >= 0) atomicAdd(dQacc + ((size_t)pq * dm.N + rows[rr]) * D + L, v[r]);   // (result unused: no round trip)
          }
        }
      }
    }
    tc::fence_before_sync();
  }
  tc::fence_before_sync();
  __syncthreads();
  if (tid == ISSUER) tc::tma_store_wait_read();             // the staging tiles must outlive the stores' reads only
  if (warp == 0) tc::tmem_dealloc(tbase, 512);
  if (!ok && tid == 0) report_status(status, 4);
#ifdef MUSE_PHASE_CLOCKS
  if (tid == 0 && blockIdx.x == 5 && blockIdx.y == 3 && blockIdx.z == 0) {
    status[56] = (int)(t_loop_ - t_in_); status[57] = (int)(t_end_ - t_loop_); status[58] = (int)(clock64() - t_end_);
  }
#endif
}

bool far_bwd_tc_supported(const Dims& d, int dtype) {
  // (the far-set mask, 8 bytes per key cluster, shares the CTA's shared memory with 200 KB of tiles)
  return dtype == MUSE_BF16 && (d.D == 64 || d.D == 128) && d.Ck % fb::TJ == 0 && d.Ck <= 2048;
}

int far_bwd_tc(const Dims& d, const SummPtrs& sp, const void* Q, const void* dO, const float* qbar, const float* LSE,
               const float* delta, const int32_t* off_q, const int32_t* perm_q, const int32_t* sel, float* dQacc,
               void* dkappa, void* dnu, float* dS, int grad_by_key_cluster, int* status, cudaStream_t st) {
  const uint64_t ent = (uint64_t)d.B * d.Hq * d.SB * d.Cq * d.Ck;
  CUtensorMap khi, klo, nu;
  const uint64_t Dd = (uint64_t)d.D;
  int rc = make_tmap_bf16_rows(&khi, sp.khi, ent, d.D, fb::TJ);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&klo, sp.klo, ent, d.D, fb::TJ);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&nu, sp.nu, ent, d.D, fb::TJ);
  // gradient tensors for the tiled stores: (d, i, plane * Ck + j) when grouped by key cluster, else (d, 1, entry)
  CUtensorMap gka, gnu;
  const uint64_t rows_j = (uint64_t)d.B * d.Hq * d.SB * d.Ck;
  const uint64_t dims_a[3] = {Dd, (uint64_t)d.Cq, rows_j}, str_a[2] = {Dd * 2, (uint64_t)d.Cq * Dd * 2};
  const uint64_t dims_b[3] = {Dd, 1, ent}, str_b[2] = {Dd * 2, Dd * 2};
  const uint32_t box[3] = {64, 1, (uint32_t)fb::TJ};
  if (rc == MUSE_OK) rc = make_tmap_bf16_nd(&gka, dkappa, 3, grad_by_key_cluster ? dims_a : dims_b, grad_by_key_cluster ? str_a : str_b, box);
  if (rc == MUSE_OK) rc = make_tmap_bf16_nd(&gnu, dnu, 3, grad_by_key_cluster ? dims_a : dims_b, grad_by_key_cluster ? str_a : str_b, box);
  if (rc != MUSE_OK) return rc;
  if (ent >= (1ull << 31)) return MUSE_ERR_UNSUPPORTED;      // 32-bit tile coordinates
  const size_t mask_bytes = (size_t)fb::NP * fb::NR * (d.Ck / 32) * 4;
  prof_mark("k_far_bwd_tc", st);
  if (d.D == 128) {
    const size_t smem = (size_t)fb::Lay<128>::oMask + mask_bytes + 1024;
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_far_bwd_tc<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_far_bwd_tc<128><<<dim3(d.Cq, d.SB, d.B * d.Hq), fb::THREADS, smem, st>>>(
        d, khi, klo, nu, gka, gnu, (const bf16*)Q, (const bf16*)dO, qbar, LSE, delta, off_q, perm_q, sel, sp.beta, sp.mu, dQacc, (bf16*)dkappa,
        (bf16*)dnu, dS, grad_by_key_cluster, status);
  } else {
    const size_t smem = (size_t)fb::Lay<64>::oMask + mask_bytes + 1024;
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_far_bwd_tc<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_far_bwd_tc<64><<<dim3(d.Cq, d.SB, d.B * d.Hq), fb::THREADS, smem, st>>>(
        d, khi, klo, nu, gka, gnu, (const bf16*)Q, (const bf16*)dO, qbar, LSE, delta, off_q, perm_q, sel, sp.beta, sp.mu, dQacc, (bf16*)dkappa,
        (bf16*)dnu, dS, grad_by_key_cluster, status);
  }
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

}  // namespace muse
