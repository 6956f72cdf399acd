// Accumulated tilted summaries on the tensor cores (bf16 mode, D = 128): Eq. 3-5 and the
// exclusive causal accumulation of Algorithm 1 in one online-softmax walk over the buckets of a
// key cluster.  One CTA = (key cluster j, 128 query clusters, head), 256 threads: thread
// (row i, warpgroup w) keeps the running max / mass of centroid i and 128 fp32 accumulators:
// dims [64 w, 64 w + 64) of kappa and of nu.
//   L   = sigma qbar K^T        tcgen05, qbar as bf16 hi + lo, keys TMA-loaded 64 at a time
//   w_u = exp(l_u - running max)  per thread, written as a bf16 hi + lo operand pair
//   U   = W [K | V]             tcgen05 (keys contracted), folded into the accumulators with the
//                               online-softmax rescale
// After each bucket the normalised snapshot (mu, beta, kappa hi/lo, nu) of plane = bucket index
// is staged in shared memory as three swizzled tiles that leave by TMA stores while the next
// plane is being computed.
#include <cuda.h>
#include "common.cuh"
#include "tc05.cuh"

namespace muse {

typedef __nv_bfloat16 bf16;
int make_tmap_bf16_rows(void* out_map, const void* base, uint64_t rows, uint32_t cols, uint32_t box_rows);
int make_tmap_bf16_nd(void* out_map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                      const uint32_t* box);

namespace st {
constexpr int TI = 128, NU = 64, THREADS = 256;
template <int D> struct Lay {                     // shared-memory offsets and TMEM columns for head dimension D (64 or 128)
  static constexpr int G = D / 64;                // 64-element (128-byte) column groups of a row
  static constexpr int kTile = TI * D * 2, kKeys = NU * D * 2, kW = TI * NU * 2;
  static constexpr int oQhi = 0, oQlo = oQhi + kTile, oK = oQlo + kTile, oV = oK + kKeys, oWhi = oV + kKeys, oWlo = oWhi + kW;
  static constexpr int oStage = oWlo + kW;        // three snapshot tiles (kappa hi, kappa lo, nu) leaving by TMA
  static constexpr int total = oStage + 3 * kTile + 1024;
  static constexpr uint32_t cL = 0, cUk = 64, cUv = 64 + D;
};
}  // namespace st

__global__ void k_split_qbar(const float* __restrict__ qbar, long long n, float sigma, bf16* __restrict__ hi, bf16* __restrict__ lo) {
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= n) return;
  const float x = qbar[e] * sigma;
  const bf16 h = __float2bfloat16_rn(x);
  hi[e] = h;
  lo[e] = __float2bfloat16_rn(x - __bfloat162float(h));
}

int split_qbar(const Dims& d, const float* qbar, void* qhi, void* qlo, cudaStream_t st) {
  const long long n = (long long)d.B * d.Hq * d.Cq * d.D;
  prof_mark("k_split_qbar", st);
  k_split_qbar<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(qbar, n, d.sigma, (bf16*)qhi, (bf16*)qlo);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

template <int D>
__global__ void __launch_bounds__(st::THREADS, 1)
k_summarize_tc(Dims dm, const __grid_constant__ CUtensorMap tm_K, const __grid_constant__ CUtensorMap tm_V,
               const __grid_constant__ CUtensorMap tm_okhi, const __grid_constant__ CUtensorMap tm_oklo,
               const __grid_constant__ CUtensorMap tm_onu, const __grid_constant__ CUtensorMap tm_qhi,
               const __grid_constant__ CUtensorMap tm_qlo, const int32_t* __restrict__ off_k, SummPtrs sp, int per_block,
               int* __restrict__ status) {
  using namespace st;
  typedef Lay<D> LY;
  constexpr int G = LY::G, HD = D / 2, kTile = LY::kTile;
  constexpr int oQhi = LY::oQhi, oQlo = LY::oQlo, oK = LY::oK, oV = LY::oV, oWhi = LY::oWhi, oWlo = LY::oWlo, oStage = LY::oStage;
  constexpr uint32_t cL = LY::cL, cUk = LY::cUk, cUv = LY::cUv;
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ uint64_t bar_kv, bar_q, bar1, bar2;
  __shared__ uint32_t tbase_s;
  const int j = blockIdx.x, i0 = blockIdx.y * TI, pq = blockIdx.z;
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int tid = threadIdx.x, warp = tid >> 5, wg = tid >> 7, row = tid & 127, i = i0 + row;
  unsigned char* sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);
  const int32_t* off = off_k + (size_t)pk * (dm.Ck * dm.S + 1) + (size_t)j * dm.S;
  if (warp == 0) tc::tmem_alloc(&tbase_s, 512);
  if (tid == 0) { tc::mbar_init(&bar_kv, 1); tc::mbar_init(&bar_q, 1); tc::mbar_init(&bar1, 1); tc::mbar_init(&bar2, 1); tc::mbar_init_fence(); }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  // sigma * qbar tile as bf16 hi and lo operands, split once per layer and loaded here by TMA
  if (tid == 0) {
    tc::mbar_expect_tx(&bar_q, 2 * kTile);
    const int r = pq * dm.Cq + i0;
    for (int g = 0; g < G; ++g) {
      tc::tma_load_2d(sm + oQhi + g * TI * 128, &tm_qhi, 64 * g, r, &bar_q);
      tc::tma_load_2d(sm + oQlo + g * TI * 128, &tm_qlo, 64 * g, r, &bar_q);
    }
  }
  const uint32_t tbase = tbase_s, tlane = tbase + ((uint32_t)((warp & 3) * 32) << 16);
  const uint32_t aQhi = tc::smem_u32(sm + oQhi), aQlo = tc::smem_u32(sm + oQlo), aK = tc::smem_u32(sm + oK),
                 aV = tc::smem_u32(sm + oV), aWhi = tc::smem_u32(sm + oWhi), aWlo = tc::smem_u32(sm + oWlo);
  uint32_t ph_kv = 0, ph1 = 0, ph2 = 0;
  bool ok = true, q_ready = false;
  float acc[D];
#pragma unroll
  for (int d = 0; d < D; ++d) acc[d] = 0.f;
  float M = -INFINITY, s = 0.f, T = 0.f;           // running max, mass and sum of w * logit (all relative to M)
#ifdef MUSE_PHASE_CLOCKS
  long long pc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  long long t_ = clock64();
#define PCLK(k) { long long n_ = clock64(); pc[k] += n_ - t_; t_ = n_; }
#else
#define PCLK(k)
#endif

  // The cluster's keys are contiguous in bucket order, so its chunks (at most 64 keys, never across a
  // bucket boundary) form one sequence; thread 32 starts the load of chunk n + 1 as soon as the MMAs of
  // chunk n have released the key / value tiles, so that it lands while the snapshot is written.
  // A bucket usually holds far fewer than 64 keys: only the 16-key groups in use are loaded and contracted.
  auto issue_kv = [&](int c0, int nk) {
    const int ng_ = (nk + 15) >> 4;
    tc::mbar_expect_tx(&bar_kv, ng_ * 2 * G * (16 * 128));
    const int r = (int)((size_t)pk * dm.N + c0);
    for (int g = 0; g < ng_; ++g)
      for (int cg = 0; cg < G; ++cg) {
        tc::tma_load_2d(sm + oK + cg * NU * 128 + g * 16 * 128, &tm_K, 64 * cg, r + 16 * g, &bar_kv);
        tc::tma_load_2d(sm + oV + cg * NU * 128 + g * 16 * 128, &tm_V, 64 * cg, r + 16 * g, &bar_kv);
      }
  };
  auto issue_after = [&](int c_end) {                  // the chunk that starts at key c_end, if any
    int npl = 0;
    while (npl < dm.SB && off[npl + 1] <= c_end) ++npl;
    if (npl < dm.SB) issue_kv(c_end, min(NU, off[npl + 1] - c_end));
  };
  if (tid == 32) issue_after(off[0]);
  for (int pl = 0; pl < dm.SB && ok; ++pl) {
    const int p0 = off[pl], p1 = off[pl + 1];
    (void)MUSE_IN_RANGE(p1, dm.N + 1); (void)MUSE_IN_RANGE(p0, p1 + 1);     // (the tiles come through tensor maps, which clip)
    if (per_block) {                                     // the summary of block pl alone: the running state starts afresh
      M = -INFINITY; s = 0.f; T = 0.f;
#pragma unroll
      for (int d = 0; d < D; ++d) acc[d] = 0.f;
    }
    for (int c0 = p0; c0 < p1 && ok; c0 += NU) {
      const int nk = min(NU, p1 - c0);
      PCLK(0)
      __syncthreads();
      const int ng = (nk + 15) >> 4;
      if (tid == 0) {
        if (!q_ready) { if (!tc::mbar_wait(&bar_q, 0)) ok = false; q_ready = true; }
        if (!tc::mbar_wait(&bar_kv, ph_kv)) ok = false;
        tc::fence_after_sync();
        const uint32_t idesc = tc::idesc_bf16(TI, 16 * ng, 0, 0);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc::mma_bf16_ss(tbase + cL, tc::smem_desc_sw128(aQhi + (ks / 4) * TI * 128 + (ks % 4) * 32, 16, 1024),
                          tc::smem_desc_sw128(aK + (ks / 4) * NU * 128 + (ks % 4) * 32, 16, 1024), idesc, ks > 0);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc::mma_bf16_ss(tbase + cL, tc::smem_desc_sw128(aQlo + (ks / 4) * TI * 128 + (ks % 4) * 32, 16, 1024),
                          tc::smem_desc_sw128(aK + (ks / 4) * NU * 128 + (ks % 4) * 32, 16, 1024), idesc, 1);
        tc::mma_commit(&bar1);
      }
      ph_kv ^= 1;
      __syncwarp();
      if (!tc::mbar_wait(&bar1, ph1)) ok = false;
      ph1 ^= 1;
      tc::fence_after_sync();
      PCLK(1)
      // two sweeps over the logits in TMEM (max, then weights) keep the register footprint small
      float cm = -INFINITY;
      for (int g = 0; g < ng; ++g) {
        float v[16];
        tc::tmem_ld16(tlane + cL + 16 * g, v);
#pragma unroll
        for (int u = 0; u < 16; ++u) if (16 * g + u < nk) cm = fmaxf(cm, v[u]);
      }
      const float Mn = fmaxf(M, cm);
      const float sc = __expf(M - Mn);                 // 0 on the first keys (M = -inf)
      float ws = 0.f, wl = 0.f;
      for (int g = 0; g < ng; ++g) {
        float v[16];
        tc::tmem_ld16(tlane + cL + 16 * g, v);
        uint32_t pk_[8];
#pragma unroll
        for (int u = 0; u < 16; u += 2) {
          const bool in0 = 16 * g + u < nk, in1 = 16 * g + u + 1 < nk;
          const float w0 = in0 ? __expf(v[u] - Mn) : 0.f, w1 = in1 ? __expf(v[u + 1] - Mn) : 0.f;
          ws += w0 + w1;
          wl += (in0 ? w0 * v[u] : 0.f) + (in1 ? w1 * v[u + 1] : 0.f);
          __nv_bfloat162 hb = __floats2bfloat162_rn(w0, w1);
          __nv_bfloat162 lb = __floats2bfloat162_rn(w0 - __low2float(hb), w1 - __high2float(hb));
          pk_[u >> 1] = wg == 0 ? *reinterpret_cast<uint32_t*>(&hb) : *reinterpret_cast<uint32_t*>(&lb);
        }
#pragma unroll
        for (int ch = 0; ch < 2; ++ch)
          *reinterpret_cast<uint4*>(sm + (wg == 0 ? oWhi : oWlo) + tc::sw128_off(row, 2 * g + ch)) = make_uint4(pk_[4 * ch], pk_[4 * ch + 1], pk_[4 * ch + 2], pk_[4 * ch + 3]);
      }
      s = s * sc + ws; T = T * sc + wl; M = Mn;
      tc::fence_async_smem();
      tc::fence_before_sync();
      __syncthreads();
      PCLK(2)
      if (tid == 0) {
        tc::fence_after_sync();
        const uint32_t idesc = tc::idesc_bf16(TI, D, 0, 1);          // A = W (K-major over keys), B = key rows (MN-major)
        for (int ks = 0; ks < ng; ++ks) {
          tc::mma_bf16_ss(tbase + cUk, tc::smem_desc_sw128(aWhi + ks * 32, 16, 1024), tc::smem_desc_sw128(aK + ks * 16 * 128, NU * 128, 1024), idesc, ks > 0);
          tc::mma_bf16_ss(tbase + cUv, tc::smem_desc_sw128(aWhi + ks * 32, 16, 1024), tc::smem_desc_sw128(aV + ks * 16 * 128, NU * 128, 1024), idesc, ks > 0);
        }
        for (int ks = 0; ks < ng; ++ks) {
          tc::mma_bf16_ss(tbase + cUk, tc::smem_desc_sw128(aWlo + ks * 32, 16, 1024), tc::smem_desc_sw128(aK + ks * 16 * 128, NU * 128, 1024), idesc, 1);
          tc::mma_bf16_ss(tbase + cUv, tc::smem_desc_sw128(aWlo + ks * 32, 16, 1024), tc::smem_desc_sw128(aV + ks * 16 * 128, NU * 128, 1024), idesc, 1);
        }
        tc::mma_commit(&bar2);
      }
      __syncwarp();
      if (!tc::mbar_wait(&bar2, ph2)) ok = false;
      ph2 ^= 1;
      tc::fence_after_sync();
      if (tid == 32 && ok) issue_after(c0 + nk);         // key / value tiles are free again (not thread 0: it issues the MMAs)
      PCLK(3)
#pragma unroll
      for (int d0 = 0; d0 < D; d0 += 32) {              // acc[0..D/2): kappa dims (D/2) wg.., acc[D/2..D): nu dims (D/2) wg..
        float v[32];
        tc::tmem_ld32(tlane + (d0 < D / 2 ? cUk : cUv) + (D / 2) * wg + (d0 & (D / 2 - 1)), v);
#pragma unroll
        for (int e = 0; e < 32; ++e) acc[d0 + e] = fmaf(acc[d0 + e], sc, v[e]);
      }
      tc::fence_before_sync();
      PCLK(4)
#ifdef MUSE_PHASE_CLOCKS
      pc[7] += 1;
#endif
    }
    // ---- snapshot of plane pl: three 128 x 256-byte row tiles (kappa hi, kappa lo, nu) staged in the W region
    const bool some = s > 0.f;
    const float inv = some ? 1.f / s : 0.f;
    const size_t ent_row0 = ((size_t)pq * dm.SB + pl) * dm.Cq;       // entry = (ent_row0 + i) * Ck + j
    if (wg == 0 && i < dm.Cq) {
      const float m_ = some ? M + __logf(s) : -INFINITY;
      const size_t ent = (ent_row0 + i) * dm.Ck + j;
      sp.mu[ent] = m_;
      sp.beta[ent] = some ? m_ - T * inv : -INFINITY;
    }
    // kappa hi / lo (warpgroup 0) and nu (warpgroup 1) as swizzled [128 rows][2 x 128 B] tiles; they leave
    // by TMA (rows of consecutive query clusters are Ck entries apart in memory) while the next plane is computed
    if (tid == 0) tc::tma_store_wait_read();                           // the previous plane's stores have read the tiles
    __syncthreads();
    // this warpgroup's half of the row (dims [HD wg, HD wg + HD)) in 16-byte chunks of 8 dims: chunk c of column group gq
#pragma unroll
    for (int ck = 0; ck < HD / 8; ++ck) {
      uint32_t w[4], wl_[4], wn[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float x0 = acc[ck * 8 + 2 * e] * inv, x1 = acc[ck * 8 + 2 * e + 1] * inv;
        __nv_bfloat162 hh = __floats2bfloat162_rn(x0, x1);
        __nv_bfloat162 ll = __floats2bfloat162_rn(x0 - __low2float(hh), x1 - __high2float(hh));
        __nv_bfloat162 nn = __floats2bfloat162_rn(acc[HD + ck * 8 + 2 * e] * inv, acc[HD + ck * 8 + 2 * e + 1] * inv);
        w[e] = *reinterpret_cast<uint32_t*>(&hh); wl_[e] = *reinterpret_cast<uint32_t*>(&ll); wn[e] = *reinterpret_cast<uint32_t*>(&nn);
      }
      const int dch = wg * (HD / 8) + ck;                                  // 16-byte chunk of the whole row
      const uint32_t off = (dch >> 3) * TI * 128 + tc::sw128_off(row, dch & 7);
      *reinterpret_cast<uint4*>(sm + oStage + off) = make_uint4(w[0], w[1], w[2], w[3]);
      *reinterpret_cast<uint4*>(sm + oStage + kTile + off) = make_uint4(wl_[0], wl_[1], wl_[2], wl_[3]);
      *reinterpret_cast<uint4*>(sm + oStage + 2 * kTile + off) = make_uint4(wn[0], wn[1], wn[2], wn[3]);
    }
    tc::fence_async_smem();
    __syncthreads();
    if (tid == 0 && ok) {
      const int P = pq * dm.SB + pl;
      for (int g = 0; g < G; ++g) {
        tc::tma_store_4d(&tm_okhi, sm + oStage + g * TI * 128, 64 * g, j, i0, P);
        tc::tma_store_4d(&tm_oklo, sm + oStage + kTile + g * TI * 128, 64 * g, j, i0, P);
        tc::tma_store_4d(&tm_onu, sm + oStage + 2 * kTile + g * TI * 128, 64 * g, j, i0, P);
      }
      tc::tma_store_commit();
    }
    PCLK(5)
  }
#ifdef MUSE_PHASE_CLOCKS
  if (tid == 0 && blockIdx.x == 5 && blockIdx.y == 0 && blockIdx.z == 0) for (int k = 0; k < 8; ++k) status[56 + k] = (int)pc[k];
#endif
  if (tid == 0) tc::tma_store_wait_all();
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tbase, 512);
  if (!ok && tid == 0) report_status(status, 7);
}

bool summarize_tc_supported(const Dims& d, int dtype) { return dtype == MUSE_BF16 && (d.D == 64 || d.D == 128); }

int summarize_tc(const Dims& d, const void* Kp, const void* Vp, const int32_t* off_k, const float* qbar, const SummPtrs& sp,
                 int per_block, void* qsplit, int* status, cudaStream_t stream) {
  // qsplit: 2 * B*Hq*Cq*D bf16 of scratch for the split centroids
  bf16* qhi = (bf16*)qsplit;
  bf16* qlo = qhi + (size_t)d.B * d.Hq * d.Cq * d.D;
  int rcq = split_qbar(d, qbar, qhi, qlo, stream);
  if (rcq != MUSE_OK) return rcq;
  CUtensorMap tqh, tql;
  rcq = make_tmap_bf16_rows(&tqh, qhi, (uint64_t)d.B * d.Hq * d.Cq, d.D, st::TI);
  if (rcq == MUSE_OK) rcq = make_tmap_bf16_rows(&tql, qlo, (uint64_t)d.B * d.Hq * d.Cq, d.D, st::TI);
  if (rcq != MUSE_OK) return rcq;
  CUtensorMap tK, tV;
  int rc = make_tmap_bf16_rows(&tK, Kp, (uint64_t)d.B * d.Hkv * d.N, d.D, 16);       // boxes of 16 keys
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&tV, Vp, (uint64_t)d.B * d.Hkv * d.N, d.D, 16);
  // outputs as 4-D tensors (d, j, i, head * planes + plane); a box is 128 query clusters of one key cluster
  CUtensorMap okhi, oklo, onu;
  const uint64_t dims[4] = {(uint64_t)d.D, (uint64_t)d.Ck, (uint64_t)d.Cq, (uint64_t)d.B * d.Hq * d.SB};
  const uint64_t strides[3] = {(uint64_t)d.D * 2, (uint64_t)d.Ck * d.D * 2, (uint64_t)d.Cq * d.Ck * d.D * 2};
  const uint32_t box[4] = {64, 1, (uint32_t)st::TI, 1};
  if (rc == MUSE_OK) rc = make_tmap_bf16_nd(&okhi, sp.khi, 4, dims, strides, box);
  if (rc == MUSE_OK) rc = make_tmap_bf16_nd(&oklo, sp.klo, 4, dims, strides, box);
  if (rc == MUSE_OK) rc = make_tmap_bf16_nd(&onu, sp.nu, 4, dims, strides, box);
  if (rc != MUSE_OK) return rc;
  prof_mark("k_summarize_tc", stream);
  const dim3 grid(d.Ck, cdiv(d.Cq, st::TI), d.B * d.Hq);
  if (d.D == 128) {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_summarize_tc<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, st::Lay<128>::total));
    k_summarize_tc<128><<<grid, st::THREADS, st::Lay<128>::total, stream>>>(d, tK, tV, okhi, oklo, onu, tqh, tql, off_k, sp, per_block, status);
  } else {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_summarize_tc<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, st::Lay<64>::total));
    k_summarize_tc<64><<<grid, st::THREADS, st::Lay<64>::total, stream>>>(d, tK, tV, okhi, oklo, onu, tqh, tql, off_k, sp, per_block, status);
  }
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

}  // namespace muse
