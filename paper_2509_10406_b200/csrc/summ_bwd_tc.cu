// Key-side pass of the backward through the accumulated summaries, on the tensor cores
// (bf16 mode, D = 64 or 128, Cq a multiple of 8).  One CTA per (key cluster j, head).  For every
// plane pl the summary (i, j, pl) was built from the keys u of cluster j in blocks <= pl, with
// weights w_iu = exp(sigma qbar_i.k_u - mu_ij(pl)) <= 1.  Given the far-field gradients
// (dkappa, dnu, dS) of that plane:
//   c_iu  = dS_i + dkappa_i.k_u + dnu_i.v_u
//   dK_u += sum_i w_iu dkappa_i + [agg_grad] sum_i (w_iu c_iu) (sigma qbar_i),   dV_u += sum_i w_iu dnu_i
// (the shared-memory qbar tiles already carry the factor sigma)
// Query clusters sit on the MMA M side for the three D-contractions (one thread per i computes
// w and w*c) and on the K side for the three i-contractions, whose outputs are transposed
// ([d][u]) so that the read-out is coalesced over d.  Planes are handled independently and
// accumulate, together with the query-cluster tiles, in tensor memory; the far-field backward
// stores its gradients [plane][j][i] so that each (plane, j, 128 i) tile is one contiguous TMA box.
#include <cuda.h>
#include "common.cuh"
#include "tc05.cuh"

namespace muse {

typedef __nv_bfloat16 bf16;

namespace sb {
constexpr int TI = 128, NU = 64;
constexpr int THREADS = 288, ISSUER = 256;     // warps 0-7 do the arithmetic; lane 0 of a ninth warp issues every TMA load and MMA
template <int D> struct Lay {
  static constexpr int kTile = TI * D * 2;     // [128 query clusters][D] bf16
  static constexpr int kKeys = NU * D * 2;     // [64 keys][D] bf16
  // The low half of the centroid tile is only needed for the tilt logits, which do not depend on
  // the plane: once they are in TMEM its space serves as the second dkappa buffer.
  static constexpr int oQhi = 0, oQlo = oQhi + kTile, oDka0 = oQlo + kTile, oDnu0 = oDka0 + kTile, oDnu1 = oDnu0 + kTile;
  static constexpr int oK = oDnu1 + kTile, oV = oK + kKeys, oW = oV + kKeys, oWc = oW + TI * NU * 2;
  static constexpr int total = oWc + TI * NU * 2 + 1024;
};
constexpr uint32_t cL = 0, cX1 = 64, cX2 = 128, cDK = 192, cDV = 256;
}  // namespace sb

// 2-D tensor map over a bf16 matrix with an arbitrary row pitch (bytes), 128B swizzle, box [box_rows][64]
int make_tmap_bf16_pitched(void* out_map, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch_bytes, uint32_t box_rows);

template <int D>
__global__ void __launch_bounds__(sb::THREADS, 1)
k_summ_bwd_tc(Dims dm, const __grid_constant__ CUtensorMap tm_dka, const __grid_constant__ CUtensorMap tm_dnu,
              const __grid_constant__ CUtensorMap tm_K, const __grid_constant__ CUtensorMap tm_V,
              const __grid_constant__ CUtensorMap tm_qhi, const __grid_constant__ CUtensorMap tm_qlo,
              const int32_t* __restrict__ off_k, const int32_t* __restrict__ off_q,
              const float* __restrict__ mu, const float* __restrict__ dS, float* __restrict__ dK_perm,
              float* __restrict__ dV_perm, int per_block, int* __restrict__ status) {
  // per_block = 1 (two-level retrieval): mu and the gradients belong to the PER-BLOCK summaries, plane pl holds the summary
  // of bucket pl alone; a key chunk then meets only the planes whose bucket it overlaps, and the weights of a plane are
  // masked to that bucket's keys.
  using namespace sb;
  typedef Lay<D> LY;
  constexpr int kTile = LY::kTile, kKeys = LY::kKeys, oQhi = LY::oQhi, oQlo = LY::oQlo, oDka0 = LY::oDka0, oDnu0 = LY::oDnu0,
                oDnu1 = LY::oDnu1, oK = LY::oK, oV = LY::oV, oW = LY::oW, oWc = LY::oWc, G = D / 64;
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ uint64_t bar_g[2], bar_kv, bar_q, bar_l, bar1, bar2;
  __shared__ uint32_t tbase_s;
  const int j = blockIdx.x, pq = blockIdx.y;
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int tid = threadIdx.x, warp = tid >> 5, wg = tid >> 7, L = tid & 127;
  const bool cw = warp < 8;                               // compute warp (the ninth warp only issues)
  const int32_t* ok_ = off_k + (size_t)pk * (dm.Ck * dm.S + 1) + (size_t)j * dm.S;
  const int32_t* oq = off_q + (size_t)pq * (dm.S * dm.Cq + 1);
  const int kbeg = ok_[0];
  (void)MUSE_IN_RANGE(ok_[dm.SB], dm.N + 1); (void)MUSE_IN_RANGE(kbeg, ok_[dm.SB] + 1);   // (the tiles come through tensor maps, which clip)
  if (kbeg >= ok_[dm.SB]) return;                       // no key of this cluster is ever summarised
  unsigned char* sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);
  if (warp == 0) tc::tmem_alloc(&tbase_s, 512);
  if (tid == 0) {
    tc::mbar_init(&bar_g[0], 1); tc::mbar_init(&bar_g[1], 1); tc::mbar_init(&bar_kv, 1); tc::mbar_init(&bar_q, 1); tc::mbar_init(&bar_l, 1);
    tc::mbar_init(&bar1, 1); tc::mbar_init(&bar2, 1); tc::mbar_init_fence();
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tbase = tbase_s, tlane = tbase + ((uint32_t)((warp & 3) * 32) << 16);
  uint32_t ph_g[2] = {0, 0}, ph_kv = 0, ph_q = 0, ph_l = 0, ph1 = 0, ph2 = 0;
  bool ok = true;
  const uint32_t aQhi = tc::smem_u32(sm + oQhi), aQlo = tc::smem_u32(sm + oQlo), aK = tc::smem_u32(sm + oK),
                 aV = tc::smem_u32(sm + oV), aW = tc::smem_u32(sm + oW), aWc = tc::smem_u32(sm + oWc);

  const int kvis = ok_[dm.SB];
#ifdef MUSE_PHASE_CLOCKS
  long long pc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  long long t_ = clock64();
#define PCLK(k) { long long n_ = clock64(); pc[k] += n_ - t_; t_ = n_; }
#else
#define PCLK(k)
#endif
  for (int c0 = kbeg; c0 < kvis && ok; c0 += NU) {        // 64 keys of the cluster at a time (usually one chunk)
    __syncthreads();
    if (tid == ISSUER) {
      tc::mbar_expect_tx(&bar_kv, 2 * kKeys);
      const int row = (int)((size_t)pk * dm.N + c0);
      for (int g = 0; g < G; ++g) {
        tc::tma_load_2d(sm + oK + g * NU * 128, &tm_K, 64 * g, row, &bar_kv);
        tc::tma_load_2d(sm + oV + g * NU * 128, &tm_V, 64 * g, row, &bar_kv);
      }
    }
    int pl0 = 0;                                          // planes [pl0, pl_end) see this chunk (bucket ends grow with the plane)
    while (pl0 < dm.SB && ok_[pl0 + 1] <= c0) ++pl0;
    int pl_end = dm.SB;
    if (per_block) { pl_end = pl0; while (pl_end < dm.SB && ok_[pl_end] < c0 + NU) ++pl_end; }
    if (!tc::mbar_wait(&bar_kv, ph_kv)) ok = false;
    ph_kv ^= 1;
    bool started = false;                                 // dK^T / dV^T accumulate in TMEM over all (i tile, plane)
    for (int i0 = 0; i0 < dm.Cq && ok; i0 += TI) {
      const int i = i0 + L;
      const bool in_range = cw && i < dm.Cq;
      const int ic = in_range ? i : 0;
      auto issue_grad = [&](int pl, int buf) {            // thread 0: both gradient tiles of (plane, j, i0..i0+127)
        tc::mbar_expect_tx(&bar_g[buf], 2 * kTile);
        const int row = (int)((((size_t)pq * dm.SB + pl) * dm.Ck + j) * dm.Cq + i0);
        unsigned char* dka = sm + (buf ? oQlo : oDka0);
        unsigned char* dnu = sm + (buf ? oDnu1 : oDnu0);
        for (int g = 0; g < G; ++g) {
          tc::tma_load_2d(dka + g * TI * 128, &tm_dka, 64 * g, row, &bar_g[buf]);
          tc::tma_load_2d(dnu + g * TI * 128, &tm_dnu, 64 * g, row, &bar_g[buf]);
        }
      };
      PCLK(7)
      __syncthreads();                                    // every MMA that read the centroid tiles has completed (bar2 waited)
      if (tid == ISSUER) {
        // sigma * qbar tile as bf16 hi + lo operands (split once per layer), and the first gradient tiles
        tc::mbar_expect_tx(&bar_q, 2 * kTile);
        const int r = pq * dm.Cq + i0;
        for (int g = 0; g < G; ++g) {
          tc::tma_load_2d(sm + oQhi + g * TI * 128, &tm_qhi, 64 * g, r, &bar_q);
          tc::tma_load_2d(sm + oQlo + g * TI * 128, &tm_qlo, 64 * g, r, &bar_q);
        }
        if (pl0 < pl_end) issue_grad(pl0, 0);
      }
      // which planes hold a non-empty segment of query cluster i (others were never written by the far-field pass)
      uint32_t livemask = 0u;
      for (int pl = pl0; pl < pl_end; ++pl) {
        const int blk = dm.causal ? pl + 1 : 0;
        // (per-block gradients are zero-filled before they are accumulated: every plane's rows are valid)
        if (in_range && (per_block || oq[(size_t)blk * dm.Cq + i + 1] > oq[(size_t)blk * dm.Cq + i])) livemask |= 1u << pl;
      }
      // tilt logits l_iu = sigma qbar_i . k_u, the same for every plane: once per centroid tile
      if (tid == ISSUER) {
        if (!tc::mbar_wait(&bar_q, ph_q)) ok = false;
        tc::fence_after_sync();
        const uint32_t idesc = tc::idesc_bf16(TI, NU, 0, 0);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc::mma_bf16_ss(tbase + cL, tc::smem_desc_sw128(aQhi + (ks / 4) * TI * 128 + (ks % 4) * 32, 16, 1024),
                          tc::smem_desc_sw128(aK + (ks / 4) * NU * 128 + (ks % 4) * 32, 16, 1024), idesc, ks > 0);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc::mma_bf16_ss(tbase + cL, tc::smem_desc_sw128(aQlo + (ks / 4) * TI * 128 + (ks % 4) * 32, 16, 1024),
                          tc::smem_desc_sw128(aK + (ks / 4) * NU * 128 + (ks % 4) * 32, 16, 1024), idesc, 1);
        tc::mma_commit(&bar_l);
      }
      ph_q ^= 1;
      __syncwarp();
      if (!tc::mbar_wait(&bar_l, ph_l)) ok = false;       // from here on the low tile's space is free
      ph_l ^= 1;
      tc::fence_after_sync();
      PCLK(0)
      float lg[32];
      if (cw) {                                                   // this thread's logits: row i, keys 32 wg .. 32 wg + 31 (log2 units)
        tc::tmem_ld32(tlane + cL + 32 * wg, lg);
#pragma unroll
        for (int c = 0; c < 32; ++c) lg[c] *= 1.4426950408889634f;
      }
      // per-plane scalars, loaded one plane ahead
      auto ent_of = [&](int pl) { return (((size_t)pq * dm.SB + pl) * dm.Cq + ic) * dm.Ck + j; };        // summaries: [plane][i][j]
      auto gent_of = [&](int pl) { return (((size_t)pq * dm.SB + pl) * dm.Ck + j) * dm.Cq + ic; };      // gradients: [plane][j][i]
      float mu_n = 0.f, dS_n = 0.f;
      if (pl0 < pl_end && ((livemask >> pl0) & 1u)) { mu_n = mu[ent_of(pl0)]; dS_n = dS[gent_of(pl0)]; }
      for (int pl = pl0, k = 0; pl < pl_end && ok; ++pl, ++k) {
        const int buf = k & 1;
        const int nk = min(NU, ok_[pl + 1] - c0);
        const int klo = per_block ? max(0, ok_[pl] - c0) : 0;      // first key of the chunk that this plane weighs
        const bool live = (livemask >> pl) & 1u;
        const float mu_i = mu_n * 1.4426950408889634f, dS_i = dS_n;
        const int oDka = buf ? oQlo : oDka0, oDnu = buf ? oDnu1 : oDnu0;
        const uint32_t aDka = tc::smem_u32(sm + oDka), aDnu = tc::smem_u32(sm + oDnu);
        if (pl + 1 < pl_end && ((livemask >> (pl + 1)) & 1u)) { mu_n = mu[ent_of(pl + 1)]; dS_n = dS[gent_of(pl + 1)]; }
        // The far-field pass wrote every row of the gradient tensors (zeros for an empty segment), so the
        // tiles go to the tensor cores as they land.  The D-contractions of this plane do not depend on the
        // previous plane's i-contractions: they are issued first, and only the W / Wc tiles and the other
        // gradient buffer wait for those.
        if (tid == ISSUER) {
          if (!tc::mbar_wait(&bar_g[buf], ph_g[buf])) ok = false;
          tc::fence_after_sync();
          const uint32_t idesc = tc::idesc_bf16(TI, NU, 0, 0);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            tc::mma_bf16_ss(tbase + cX1, tc::smem_desc_sw128(aDka + (ks / 4) * TI * 128 + (ks % 4) * 32, 16, 1024),
                            tc::smem_desc_sw128(aK + (ks / 4) * NU * 128 + (ks % 4) * 32, 16, 1024), idesc, ks > 0);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            tc::mma_bf16_ss(tbase + cX2, tc::smem_desc_sw128(aDnu + (ks / 4) * TI * 128 + (ks % 4) * 32, 16, 1024),
                            tc::smem_desc_sw128(aV + (ks / 4) * NU * 128 + (ks % 4) * 32, 16, 1024), idesc, ks > 0);
          tc::mma_commit(&bar1);
          if (k > 0 && !tc::mbar_wait(&bar2, ph2)) ok = false;      // the previous plane's MMAs are done with the other buffer
          if (pl + 1 < pl_end && ok) issue_grad(pl + 1, buf ^ 1);
        }
        ph_g[buf] ^= 1;
        PCLK(1)
        if (cw && !tc::mbar_wait(&bar1, ph1)) ok = false;
        ph1 ^= 1;
        tc::fence_after_sync();
        PCLK(3)
        if (cw) {
          float x1[32], x2[32];
          tc::tmem_ld32(tlane + cX1 + 32 * wg, x1);
          tc::tmem_ld32(tlane + cX2 + 32 * wg, x2);
          uint32_t ww[16], wc[16];
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            float w0 = 0.f, w1 = 0.f, c0_ = 0.f, c1_ = 0.f;
            if (live && 32 * wg + c < nk && 32 * wg + c >= klo) { w0 = tc::fast_exp2(lg[c] - mu_i); c0_ = w0 * (dS_i + x1[c] + x2[c]); }
            if (live && 32 * wg + c + 1 < nk && 32 * wg + c + 1 >= klo) { w1 = tc::fast_exp2(lg[c + 1] - mu_i); c1_ = w1 * (dS_i + x1[c + 1] + x2[c + 1]); }
            __nv_bfloat162 a = __floats2bfloat162_rn(w0, w1), b = __floats2bfloat162_rn(c0_, c1_);
            ww[c >> 1] = *reinterpret_cast<uint32_t*>(&a); wc[c >> 1] = *reinterpret_cast<uint32_t*>(&b);
          }
          if (k > 0 && !tc::mbar_wait(&bar2, ph2)) ok = false;      // the previous plane's MMAs have read W / Wc
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            *reinterpret_cast<uint4*>(sm + oW + tc::sw128_off(L, 4 * wg + ch)) = make_uint4(ww[4 * ch], ww[4 * ch + 1], ww[4 * ch + 2], ww[4 * ch + 3]);
            *reinterpret_cast<uint4*>(sm + oWc + tc::sw128_off(L, 4 * wg + ch)) = make_uint4(wc[4 * ch], wc[4 * ch + 1], wc[4 * ch + 2], wc[4 * ch + 3]);
          }
        }
        if (k > 0) ph2 ^= 1;
        tc::fence_async_smem();
        tc::fence_before_sync();
        __syncthreads();
        if (tid == ISSUER) {
          tc::fence_after_sync();
          // A [i][d] and B [i][u]: both contract over rows.  M = 128 output dims even when D = 64: the second 64-dim group
          // of the A operand is then the tile that follows in shared memory, and output lanes 64..127 hold numbers that nobody reads
          const uint32_t idesc = tc::idesc_bf16(128, NU, 1, 1);
#pragma unroll
          for (int ks = 0; ks < TI / 16; ++ks)
            tc::mma_bf16_ss(tbase + cDK, tc::smem_desc_sw128(aDka + ks * 16 * 128, TI * 128, 1024),
                            tc::smem_desc_sw128(aW + ks * 16 * 128, TI * 128, 1024), idesc, started || ks > 0);
          if (dm.agg_grad) {
#pragma unroll
            for (int ks = 0; ks < TI / 16; ++ks)
              tc::mma_bf16_ss(tbase + cDK, tc::smem_desc_sw128(aQhi + ks * 16 * 128, TI * 128, 1024),
                              tc::smem_desc_sw128(aWc + ks * 16 * 128, TI * 128, 1024), idesc, 1);
          }
#pragma unroll
          for (int ks = 0; ks < TI / 16; ++ks)
            tc::mma_bf16_ss(tbase + cDV, tc::smem_desc_sw128(aDnu + ks * 16 * 128, TI * 128, 1024),
                            tc::smem_desc_sw128(aW + ks * 16 * 128, TI * 128, 1024), idesc, started || ks > 0);
          tc::mma_commit(&bar2);
        }
        started = true;
        __syncwarp();
        PCLK(4)
#ifdef MUSE_PHASE_CLOCKS
        pc[6] += 1;
#endif
      }
      if (pl0 < pl_end) {                                 // last plane's MMAs
        if (!tc::mbar_wait(&bar2, ph2)) ok = false;
        ph2 ^= 1;
        tc::fence_after_sync();
      }
    }
    PCLK(5)
    // read-out once per key chunk: thread = d, warpgroup = half of the keys; add into the fp32 accumulators
    const int nkc = min(NU, kvis - c0);
    if (cw) {
      float a[32], b[32];
      tc::tmem_ld32(tlane + cDK + 32 * wg, a);
      tc::tmem_ld32(tlane + cDV + 32 * wg, b);
      if (ok && started && L < D) {
#pragma unroll
        for (int u = 0; u < 32; ++u) {
          if (32 * wg + u < nkc) {
            const size_t at = ((size_t)pq * dm.N + c0 + 32 * wg + u) * D + L;
            atomicAdd(dK_perm + at, a[u]);                 // (result unused: no round trip; one CTA owns the element)
            atomicAdd(dV_perm + at, b[u]);
          }
        }
      }
    }
    tc::fence_before_sync();
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tbase, 512);
#ifdef MUSE_PHASE_CLOCKS
  if (tid == 0 && blockIdx.x == 5 && blockIdx.y == 0) for (int k = 0; k < 8; ++k) status[56 + k] = (int)pc[k];
#endif
  if (!ok && tid == 0) report_status(status, 5);
}

bool summ_bwd_tc_supported(const Dims& d, int dtype) {
  return dtype == MUSE_BF16 && (d.D == 64 || d.D == 128) && d.Cq % 8 == 0;
}

int make_tmap_bf16_rows(void* out_map, const void* base, uint64_t rows, uint32_t cols, uint32_t box_rows);

int summ_bwd_tc(const Dims& d, const void* Kp, const void* Vp, const int32_t* off_k, const int32_t* off_q, const float* qbar,
                const float* mu, const void* dkappa, const void* dnu, const float* dS, float* dK_perm, float* dV_perm,
                void* qsplit, int per_block, int* status, cudaStream_t st) {
  // qsplit: 2 * B*Hq*Cq*D bf16 of scratch for the split centroids
  bf16* qhi = (bf16*)qsplit;
  bf16* qlo = qhi + (size_t)d.B * d.Hq * d.Cq * d.D;
  int rcq = split_qbar(d, qbar, qhi, qlo, st);
  if (rcq != MUSE_OK) return rcq;
  CUtensorMap tqh, tql;
  rcq = make_tmap_bf16_rows(&tqh, qhi, (uint64_t)d.B * d.Hq * d.Cq, d.D, sb::TI);
  if (rcq == MUSE_OK) rcq = make_tmap_bf16_rows(&tql, qlo, (uint64_t)d.B * d.Hq * d.Cq, d.D, sb::TI);
  if (rcq != MUSE_OK) return rcq;
  CUtensorMap tdka, tdnu, tK, tV;
  const uint64_t grows = (uint64_t)d.B * d.Hq * d.SB * d.Ck * d.Cq;       // gradient entries, [plane][j][i]
  int rc = make_tmap_bf16_rows(&tdka, dkappa, grows, d.D, sb::TI);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&tdnu, dnu, grows, d.D, sb::TI);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&tK, Kp, (uint64_t)d.B * d.Hkv * d.N, d.D, sb::NU);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&tV, Vp, (uint64_t)d.B * d.Hkv * d.N, d.D, sb::NU);
  if (rc != MUSE_OK) return rc;
  prof_mark("k_summ_bwd_tc", st);
  if (d.D == 128) {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_summ_bwd_tc<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, sb::Lay<128>::total));
    k_summ_bwd_tc<128><<<dim3(d.Ck, d.B * d.Hq), sb::THREADS, sb::Lay<128>::total, st>>>(d, tdka, tdnu, tK, tV, tqh, tql, off_k, off_q, mu, dS,
                                                                                    dK_perm, dV_perm, per_block, status);
  } else {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_summ_bwd_tc<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, sb::Lay<64>::total));
    k_summ_bwd_tc<64><<<dim3(d.Ck, d.B * d.Hq), sb::THREADS, sb::Lay<64>::total, st>>>(d, tdka, tdnu, tK, tV, tqh, tql, off_k, off_q, mu, dS,
                                                                                  dK_perm, dV_perm, per_block, status);
  }
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

}  // namespace muse
