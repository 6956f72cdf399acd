// Far-field forward on the tensor cores (bf16 mode, D = 128, Ck a multiple of 128, Ck <= 2048).
// One CTA per (query cluster i, plane, head) segment; its queries (32 on average at the headline
// sizes, up to 64 per pass) share the Ck accumulated summaries of (i, plane).  The summaries sit
// on the MMA M side (128 clusters per tile, one TMEM lane each) and the queries on the N side
// (64 columns), so the segment streams its summaries once:
//   A  scores^T[j][r] = (kappa_hi[j] + kappa_lo[j]) . q[r]   two accumulating MMAs per tile,
//      kappa tiles streamed by TMA through a ring that spans the whole operand area;
//      score = sigma * that + beta[j] (Eq. 6).  All 64 x Ck scores stay in TMEM (512 columns).
//   B  16 queries at a time: TMEM -> shared memory transposed to [r][j] fp32
//   C  per query (one warp each): top-m selection, far-set softmax, P written as a bf16 operand
//   D  out^T[d][r] = sum_j nu[j][d] P[r][j]      nu tiles (MN-major A operand) streamed by TMA,
//      brought into L2 ahead of time while phase C runs
//   E  TMEM -> o_far (thread = d, coalesced over d for each query)
#include <cuda.h>
#include "common.cuh"
#include "tc05.cuh"

namespace muse {

typedef __nv_bfloat16 bf16;
int make_tmap_bf16_rows(void* out_map, const void* base, uint64_t rows, uint32_t cols, uint32_t box_rows);

constexpr int kFD = 128, kFJ = 128;                 // head dim, clusters per tile
// Queries per pass FR and per selection step FQ (one warp each) are template parameters: 64 / 16 up to 1024
// key clusters, 32 / 8 up to 2048 (all FR x Ck scores of a pass live in the 512 TMEM columns, P and the score
// rows of a step in shared memory).
constexpr int kTileBytes = kFJ * kFD * 2;           // 32 KB: one [128][128] bf16 operand tile
constexpr int kFarTcCols = 512;
constexpr int kMaxStA = 6, kMaxStD = 4;
constexpr int kCandMax = 128;                       // candidates kept by the compacting selection (4 per lane)

struct FarBars { uint64_t fullA[kMaxStA], emptyA[kMaxStA], fullD[kMaxStD], emptyD[kMaxStD], done; };


// Top-m of one query's scores s[0..Ck) (one warp; Ck <= 32 NKMAX).  Writes the chosen clusters to
// so[0..m) (-1 padded), and removes them from the far set by setting their score to -inf.
// Order-preserving integer keys; the key T of the m-th largest is found by bisection with warp
// reductions, everything above T is taken and, among ties at T, the lowest cluster indices.
// When few scores can reach the top m (bounded below by the m-th largest lane maximum), they are
// first compacted into `cand` (kCandMax keys then kCandMax indices, 128-byte segments `seg`
// bytes apart) so that every bisection round touches 4 keys per lane instead of Ck / 32.
template <int NKMAX>
__device__ __forceinline__ void select_top_m(float* s, int Ck, int m, int32_t* so, int lane, unsigned char* cand, int seg,
                                             bool may_compact) {
  const int NK = Ck >> 5;                       // scores per lane (<= NKMAX)
  uint32_t key[NKMAX];
#pragma unroll
  for (int k = 0; k < NKMAX; ++k) {
    const uint32_t b = __float_as_uint(k < NK ? s[lane + 32 * k] : -INFINITY);
    key[k] = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
  }
  const uint32_t kFinite = 0x00800000u;         // smallest key above key(-inf) = 0x007fffff
  const uint32_t lt = (1u << lane) - 1u;
  auto count_ge = [&](uint32_t thr) {           // lane-local count, then one warp reduction
    int c = 0;
#pragma unroll
    for (int k = 0; k < NKMAX; ++k) c += key[k] >= thr ? 1 : 0;
    return (int)__reduce_add_sync(0xffffffffu, (unsigned)c);
  };
  // lane-local statistics in one sweep: finite count, largest and second largest key, smallest finite key
  uint32_t m1 = 0u, m2 = 0u, kmn = 0xffffffffu;
  int nfin = 0;
#pragma unroll
  for (int k = 0; k < NKMAX; ++k) {
    m2 = max(m2, min(m1, key[k]));
    m1 = max(m1, key[k]);
    const bool fin = key[k] >= kFinite;
    nfin += fin ? 1 : 0;
    kmn = min(kmn, fin ? key[k] : 0xffffffffu);
  }
  const bool take_all = (int)__reduce_add_sync(0xffffffffu, (unsigned)nfin) <= m;
  uint32_t T = kFinite;
  bool compacted = false;
  int ncand = 0;
  uint32_t ck[4] = {0u, 0u, 0u, 0u};
  if (!take_all) {
    const uint32_t kmx = __reduce_max_sync(0xffffffffu, m1);
    kmn = __reduce_min_sync(0xffffffffu, kmn);
    if (m <= 64) {
      // the m-th largest of the 64 per-lane top-two keys bounds the m-th largest score from below
      // (tightly: about m + 4 scores reach it on random data), by bisection over the bits below
      // the prefix shared by the largest and the smallest finite key
      const int sh0 = __clz((int)(kmx ^ kmn));
      uint32_t lb = sh0 >= 32 ? kmx : (kmx & ~(0xffffffffu >> sh0));
      for (int bit = 31 - sh0; bit >= 0; --bit) {
        const uint32_t c2 = lb | (1u << bit);
        if ((int)__reduce_add_sync(0xffffffffu, (unsigned)((m1 >= c2) + (m2 >= c2))) >= m) lb = c2;
      }
      kmn = max(kmn, lb);
      if (may_compact) {
        ncand = count_ge(kmn);
        compacted = ncand <= kCandMax;
      }
    }
    const int shared = __clz((int)(kmx ^ kmn));            // 32 if the interval is a single key
    T = shared >= 32 ? kmx : (kmx & ~(0xffffffffu >> shared));
    if (compacted) {
      int base = 0;
#pragma unroll
      for (int k = 0; k < NKMAX; ++k) {
        if (k < NK) {
          const bool in = key[k] >= kmn;
          const uint32_t mb = __ballot_sync(0xffffffffu, in);
          if (in) {
            const int pos = base + __popc(mb & lt);
            *reinterpret_cast<uint32_t*>(cand + (pos >> 5) * seg + (pos & 31) * 4) = key[k];
            *reinterpret_cast<int32_t*>(cand + (4 + (pos >> 5)) * seg + (pos & 31) * 4) = lane + 32 * k;
          }
          base += __popc(mb);
        }
      }
      __syncwarp();
#pragma unroll
      for (int q = 0; q < 4; ++q)
        ck[q] = lane + 32 * q < ncand ? *reinterpret_cast<const uint32_t*>(cand + q * seg + lane * 4) : 0u;
      for (int bit = 31 - shared; bit >= 0; --bit) {
        const uint32_t c2 = T | (1u << bit);
        const int c = (int)__reduce_add_sync(0xffffffffu, (unsigned)((ck[0] >= c2) + (ck[1] >= c2) + (ck[2] >= c2) + (ck[3] >= c2)));
        if (c >= m) { T = c2; if (c == m) break; }
      }
    } else {
      for (int bit = 31 - shared; bit >= 0; --bit) {
        const uint32_t c2 = T | (1u << bit);
        const int c = count_ge(c2);
        if (c >= m) { T = c2; if (c == m) break; }
      }
    }
  }
  int base = 0, ties_seen = 0;
  if (compacted) {
    const uint32_t T1 = T + 1u;
    const int need = m - (int)__reduce_add_sync(0xffffffffu, (unsigned)((ck[0] >= T1) + (ck[1] >= T1) + (ck[2] >= T1) + (ck[3] >= T1)));
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const bool tie = ck[q] == T, gt = ck[q] > T;
      const uint32_t mt = __ballot_sync(0xffffffffu, tie);
      const bool take = gt || (tie && ties_seen + __popc(mt & lt) < need);
      ties_seen += __popc(mt);
      const uint32_t ms = __ballot_sync(0xffffffffu, take);
      if (take) {
        const int j = *reinterpret_cast<const int32_t*>(cand + (4 + q) * seg + lane * 4);
        so[base + __popc(ms & lt)] = j;
        s[j] = -INFINITY;
      }
      base += __popc(ms);
    }
  } else {
    const int need = take_all ? 0 : m - count_ge(T + 1u);
#pragma unroll
    for (int k = 0; k < NKMAX; ++k) {
      if (k < NK) {
        const bool tie = !take_all && key[k] == T;
        const bool gt = take_all ? key[k] >= kFinite : key[k] > T;
        const uint32_t mt = __ballot_sync(0xffffffffu, tie);
        const bool take = gt || (tie && ties_seen + __popc(mt & lt) < need);
        ties_seen += __popc(mt);
        const uint32_t ms = __ballot_sync(0xffffffffu, take);
        if (take) { so[base + __popc(ms & lt)] = lane + 32 * k; s[lane + 32 * k] = -INFINITY; }
        base += __popc(ms);
      }
    }
  }
  for (int k = base + lane; k < m; k += 32) so[k] = -1;
}

template <int FR, int FQ>
__global__ void __launch_bounds__(FQ * 32, 1)
k_far_fwd_tc(Dims dm, const __grid_constant__ CUtensorMap tm_khi, const __grid_constant__ CUtensorMap tm_klo,
             const __grid_constant__ CUtensorMap tm_nu, const bf16* __restrict__ Q, const int32_t* __restrict__ off_q,
             const int32_t* __restrict__ perm_q, const float* __restrict__ mu, const float* __restrict__ beta,
             const int32_t* __restrict__ sel_in, int32_t* __restrict__ sel_out, float* __restrict__ o_far,
             float* __restrict__ lse_far, int p_bytes, int sc_bytes, int nsA, int nsD, int* __restrict__ status) {
  constexpr int NT = FQ * 32, NTG = FQ / 4, KT = 16 / NTG;   // threads; tile groups in the TMEM read-out; cluster tiles per group
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ FarBars bars;
  __shared__ uint32_t tbase_s;
  __shared__ int32_t rows[FR];
  __shared__ float rinv[FR];
  __shared__ int32_t selq[kMaxM];
  const int i = blockIdx.x, pl = blockIdx.y, pq = blockIdx.z;
  const int blk = dm.causal ? pl + 1 : 0, Ck = dm.Ck, NJ = Ck / kFJ, m = dm.m;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int32_t* oq = off_q + (size_t)pq * (dm.S * dm.Cq + 1) + (size_t)blk * dm.Cq + i;
  const int p0 = oq[0], p1 = oq[1];
  if (p0 >= p1) return;
  // operand area: phase A uses all of it as the kappa ring; afterwards P (bf16 [64][Ck]) sits at
  // its start and the score rows of the current 16 queries, later the nu ring, behind it
  unsigned char* sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);
  unsigned char* Pm = sm;
  float* sc = reinterpret_cast<float*>(sm + p_bytes);
  unsigned char* Qs = sm + p_bytes + sc_bytes;
  const size_t ent0 = (((size_t)pq * dm.SB + pl) * dm.Cq + i) * Ck;
  const float* mup = mu + ent0;
  const float* bep = beta + ent0;
  const bf16* Qp = Q + (size_t)pq * dm.N * kFD;
  const int32_t* pm = perm_q + (size_t)pq * dm.N;

  if (warp == 0) tc::tmem_alloc(&tbase_s, kFarTcCols);
  if (tid == 0) {
    for (int s = 0; s < kMaxStA; ++s) { tc::mbar_init(&bars.fullA[s], 1); tc::mbar_init(&bars.emptyA[s], 1); }
    for (int s = 0; s < kMaxStD; ++s) { tc::mbar_init(&bars.fullD[s], 1); tc::mbar_init(&bars.emptyD[s], 1); }
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
  uint32_t cntA = 0, cntD = 0, done_ph = 0;   // tiles produced (thread 0) / consumed (thread 32) so far; phase of `done`
  bool ok = true;
  const int lq = warp & 3, tg = warp >> 2;            // TMEM lane quarter of this warp, tile group

  for (int r0 = p0; r0 < p1 && ok; r0 += FR) {
    const int n = min(FR, p1 - r0);
#ifdef MUSE_PHASE_CLOCKS
    long long ck0 = clock64(), ck1 = 0, ck3 = 0, ck4 = 0;
#endif
    if (tid < FR) rows[tid] = tid < n ? pm[r0 + tid] : -1;
    // query rows -> K-major swizzled tile [64][128] bf16 (2 blocks of [64][128 B])
    for (int e = tid; e < FR * (kFD / 8); e += NT) {
      const int r = e >> 4, ck = e & 15, kb = ck >> 3, c = ck & 7;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (r < n) v = reinterpret_cast<const uint4*>(Qp + (size_t)pm[r0 + r] * kFD)[ck];
      *reinterpret_cast<uint4*>(Qs + kb * FR * 128 + tc::sw128_off(r, c)) = v;
    }
    tc::fence_async_smem();
    tc::fence_before_sync();
    __syncthreads();
    // ---- A: scores^T for all clusters, kappa_hi / kappa_lo tiles through an nsA-stage TMA ring;
    //         thread 0 produces (TMA), thread 32 consumes (MMA), so neither waits for the other's latency
    if (tid == 0) {
      const int T = 2 * NJ;
      for (int t = 0; t < T; ++t, ++cntA) {
        const int s = cntA % nsA;
        if (!tc::mbar_wait(&bars.emptyA[s], ((cntA / nsA) & 1) ^ 1)) { ok = false; break; }
        tc::mbar_expect_tx(&bars.fullA[s], kTileBytes);
        const void* map = (t & 1) ? (const void*)&tm_klo : (const void*)&tm_khi;
        const int row = (int)(ent0 + (size_t)(t >> 1) * kFJ);
        tc::tma_load_2d(sm + s * kTileBytes, map, 0, row, &bars.fullA[s]);
        tc::tma_load_2d(sm + s * kTileBytes + kFJ * 128, map, 64, row, &bars.fullA[s]);
      }
      // bring the nu tiles of this segment into L2 while the selection runs
      for (int t = 0; t < NJ; ++t) {
        tc::tma_prefetch_2d(&tm_nu, 0, (int)(ent0 + (size_t)t * kFJ));
        tc::tma_prefetch_2d(&tm_nu, 64, (int)(ent0 + (size_t)t * kFJ));
      }
    } else if (tid == 32) {
      tc::fence_after_sync();
      const uint32_t idesc = tc::idesc_bf16(kFJ, FR, 0, 0);
      const uint32_t qa = tc::smem_u32(Qs);
      const int T = 2 * NJ;
      for (int u = 0; u < T; ++u, ++cntA) {
        const int s = cntA % nsA;
        if (!tc::mbar_wait(&bars.fullA[s], (cntA / nsA) & 1)) { ok = false; break; }
        tc::fence_after_sync();
        const uint32_t a0 = tc::smem_u32(sm + s * kTileBytes);
#pragma unroll
        for (int ks = 0; ks < kFD / 16; ++ks)
          tc::mma_bf16_ss(tbase + (u >> 1) * FR, tc::smem_desc_sw128(a0 + (ks / 4) * kFJ * 128 + (ks % 4) * 32, 16, 1024),
                          tc::smem_desc_sw128(qa + (ks / 4) * FR * 128 + (ks % 4) * 32, 16, 1024), idesc, (u & 1) || ks > 0);
        tc::mma_commit(&bars.emptyA[s]);
      }
      if (ok) tc::mma_commit(&bars.done);
    }
    float bq[KT];                                       // beta of this thread's clusters, loaded ahead of the TMEM reads
#pragma unroll
    for (int k = 0; k < KT; ++k) { const int jt = tg + NTG * k; bq[k] = jt < NJ ? bep[jt * kFJ + (tid & 127)] : 0.f; }
    __syncwarp();     // lanes 1..31 of warp 0 park here instead of spinning beside the issuing lane
    if (!tc::mbar_wait(&bars.done, done_ph)) ok = false;
    done_ph ^= 1;
    tc::fence_after_sync();
#ifdef MUSE_PHASE_CLOCKS
    ck1 = clock64();
#endif
    for (int qs = 0; qs * FQ < n; ++qs) {
      // ---- B: TMEM -> sc[r][j] for the 16 queries of this step
#ifdef MUSE_PHASE_CLOCKS
      long long cb0 = clock64(), cb1 = 0, cb2 = 0, cb3 = 0;
#endif
#pragma unroll
      for (int k = 0; k < KT; ++k) {
        const int jt = tg + NTG * k;
        if (jt >= NJ) break;
        float v[FQ];
        if constexpr (FQ == 16) tc::tmem_ld16(tbase + ((uint32_t)(lq * 32) << 16) + jt * FR + qs * FQ, v);
        else tc::tmem_ld8(tbase + ((uint32_t)(lq * 32) << 16) + jt * FR + qs * FQ, v);
        const int j = jt * kFJ + (tid & 127);
        const float b = bq[k];
#pragma unroll
        for (int r = 0; r < FQ; ++r) sc[r * Ck + j] = b == -INFINITY ? -INFINITY : fmaf(v[r], dm.sigma, b);
      }
      __syncthreads();
#ifdef MUSE_PHASE_CLOCKS
      cb1 = clock64();
#endif
      // ---- C: selection + softmax of the far set; P (bf16) as a K-major operand [64][Ck]
      const int r = qs * FQ + warp;                    // one query per warp
      float* s = sc + warp * Ck;
      float sum = 0.f, mx = -INFINITY;
      if (r < n) {
        const int t = rows[r];
        int32_t* so = sel_out + ((size_t)pq * dm.N + t) * m;
        if (sel_in != nullptr) {
          const int32_t* si = sel_in + ((size_t)pq * dm.N + t) * m;
          for (int k = lane; k < m; k += 32) { int c = si[k]; so[k] = c; if (c >= 0 && c < Ck) s[c] = -INFINITY; }
        } else if (dm.sel_mode == MUSE_SEL_PER_QCLUSTER) {
          for (int k = lane; k < m; k += 32) { int c = selq[k]; so[k] = c; if (c >= 0) s[c] = -INFINITY; }
        } else if (m > 0) {
          // this query's own (not yet written) P row doubles as the candidate scratch
          select_top_m<(FR == 64 ? 32 : 64)>(s, Ck, m, so, lane, Pm + r * 128, FR * 128, Ck >= 512);
        }
        __syncwarp();
#ifdef MUSE_PHASE_CLOCKS
        cb2 = clock64();
#endif
        for (int j = lane; j < Ck; j += 32) mx = fmaxf(mx, s[j]);
        mx = warp_max(mx);
      }
      // probabilities, 8 consecutive clusters (one 16-byte chunk) per lane and step
      for (int q = lane; q < Ck / 8; q += 32) {
        const float4 s0 = *reinterpret_cast<const float4*>(s + q * 8), s1 = *reinterpret_cast<const float4*>(s + q * 8 + 4);
        const float sv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          float p0_ = 0.f, p1_ = 0.f;
          if (mx != -INFINITY) { p0_ = __expf(sv[2 * k] - mx); p1_ = __expf(sv[2 * k + 1] - mx); }
          __nv_bfloat162 b = __floats2bfloat162_rn(p0_, p1_);
          sum += __low2float(b) + __high2float(b);
          w[k] = *reinterpret_cast<uint32_t*>(&b);
        }
        *reinterpret_cast<uint4*>(Pm + (q >> 3) * (FR * 128) + tc::sw128_off(r, q & 7)) = make_uint4(w[0], w[1], w[2], w[3]);
      }
      sum = warp_sum(sum);
      if (lane == 0) {
        rinv[r] = sum > 0.f ? 1.f / sum : 0.f;
        if (r < n) lse_far[(size_t)pq * dm.N + rows[r]] = sum > 0.f ? mx + logf(sum) : -INFINITY;
      }
#ifdef MUSE_PHASE_CLOCKS
      cb3 = clock64();
      if (tid == 0 && blockIdx.x == 5 && blockIdx.y == 3 && blockIdx.z == 0 && r0 == p0 && qs == 0) {
        status[9] = (int)(cb1 - cb0); status[13] = (int)(cb2 - cb1); status[14] = (int)(cb3 - cb2);
      }
#endif
      __syncthreads();
    }
    tc::fence_async_smem();
    tc::fence_before_sync();
    __syncthreads();
#ifdef MUSE_PHASE_CLOCKS
    ck3 = clock64();
#endif
    // ---- D: out^T = nu^T P^T, nu tiles through an nsD-stage TMA ring in the score region
    if (tid == 0 && ok) {
      unsigned char* ring = sm + p_bytes;
      for (int t = 0; t < NJ; ++t, ++cntD) {
        const int s = cntD % nsD;
        if (!tc::mbar_wait(&bars.emptyD[s], ((cntD / nsD) & 1) ^ 1)) { ok = false; break; }
        tc::mbar_expect_tx(&bars.fullD[s], kTileBytes);
        const int row = (int)(ent0 + (size_t)t * kFJ);
        tc::tma_load_2d(ring + s * kTileBytes, &tm_nu, 0, row, &bars.fullD[s]);
        tc::tma_load_2d(ring + s * kTileBytes + kFJ * 128, &tm_nu, 64, row, &bars.fullD[s]);
      }
    } else if (tid == 32 && ok) {
      tc::fence_after_sync();
      const uint32_t idesc = tc::idesc_bf16(kFD, FR, 1, 0);
      const uint32_t pa = tc::smem_u32(Pm);
      unsigned char* ring = sm + p_bytes;
      for (int u = 0; u < NJ; ++u, ++cntD) {
        const int s = cntD % nsD;
        if (!tc::mbar_wait(&bars.fullD[s], (cntD / nsD) & 1)) { ok = false; break; }
        tc::fence_after_sync();
        const uint32_t a0 = tc::smem_u32(ring + s * kTileBytes);
#pragma unroll
        for (int ks = 0; ks < kFJ / 16; ++ks)
          tc::mma_bf16_ss(tbase, tc::smem_desc_sw128(a0 + ks * 16 * 128, kFJ * 128, 1024),
                          tc::smem_desc_sw128(pa + (2 * u + ks / 4) * (FR * 128) + (ks % 4) * 32, 16, 1024), idesc,
                          u > 0 || ks > 0);
        tc::mma_commit(&bars.emptyD[s]);
      }
      if (ok) tc::mma_commit(&bars.done);
    }
    __syncwarp();
    if (!tc::mbar_wait(&bars.done, done_ph)) ok = false;
    done_ph ^= 1;
    tc::fence_after_sync();
#ifdef MUSE_PHASE_CLOCKS
    ck4 = clock64();
    if (tid == 0 && blockIdx.x == 5 && blockIdx.y == 3 && blockIdx.z == 0 && r0 == p0) {
      status[8] = (int)(ck1 - ck0); status[9] = 0; status[10] = (int)(ck3 - ck1); status[11] = (int)(ck4 - ck3);
      status[12] = n;
    }
#endif
    // ---- E: thread = output dim d; warps 0-3 read queries 0..31, warps 4-7 queries 32..63
    if (warp < FR / 8) {
      const int half = warp >> 2;
      float v[32];
      tc::tmem_ld32(tbase + ((uint32_t)(lq * 32) << 16) + 32 * half, v);
      if (ok) {
#pragma unroll
        for (int r = 0; r < 32; ++r)
          if (32 * half + r < n) o_far[((size_t)pq * dm.N + rows[32 * half + r]) * kFD + (tid & 127)] = v[r] * rinv[32 * half + r];
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
  return dtype == MUSE_BF16 && d.D == kFD && d.Ck % kFJ == 0 && d.Ck <= 2048 && d.Ck >= kFJ;
}

int far_fwd_tc(const Dims& d, const SummPtrs& sp, const void* Q, const int32_t* off_q, const int32_t* perm_q,
               const int32_t* sel_in, int32_t* sel_out, float* o_far, float* lse_far, int* status, cudaStream_t st) {
  const uint64_t ent = (uint64_t)d.B * d.Hq * d.SB * d.Cq * d.Ck;
  CUtensorMap khi, klo, nu;
  int rc = make_tmap_bf16_rows(&khi, sp.khi, ent, kFD, kFJ);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&klo, sp.klo, ent, kFD, kFJ);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&nu, sp.nu, ent, kFD, kFJ);
  if (rc != MUSE_OK) return rc;
  const bool wide = d.Ck > 1024;                                         // 32 queries per pass, 8 per selection step
  const int FR = wide ? 32 : 64, FQ = wide ? 8 : 16;
  const int p_bytes = FR * d.Ck * 2;                                     // P: bf16 [FR][Ck]
  int sc_bytes = FQ * d.Ck * 4;                                          // FQ score rows, later the nu ring
  if (sc_bytes < 2 * kTileBytes) sc_bytes = 2 * kTileBytes;
  int nsA = (p_bytes + sc_bytes) / kTileBytes, nsD = sc_bytes / kTileBytes;
  nsA = nsA > kMaxStA ? kMaxStA : nsA;
  nsD = nsD > kMaxStD ? kMaxStD : nsD;
  const size_t smem = (size_t)p_bytes + sc_bytes + FR * kFD * 2 + 1024;
  prof_mark("k_far_fwd_tc", st);
  if (wide) {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_far_fwd_tc<32, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_far_fwd_tc<32, 8><<<dim3(d.Cq, d.SB, d.B * d.Hq), 256, smem, st>>>(d, khi, klo, nu, (const bf16*)Q, off_q, perm_q, sp.mu, sp.beta,
                                                                 sel_in, sel_out, o_far, lse_far, p_bytes, sc_bytes, nsA, nsD, status);
  } else {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_far_fwd_tc<64, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_far_fwd_tc<64, 16><<<dim3(d.Cq, d.SB, d.B * d.Hq), 512, smem, st>>>(d, khi, klo, nu, (const bf16*)Q, off_q, perm_q, sp.mu, sp.beta,
                                                                   sel_in, sel_out, o_far, lse_far, p_bytes, sc_bytes, nsA, nsD, status);
  }
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

}  // namespace muse
