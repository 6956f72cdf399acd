// Far-field forward on the tensor cores (bf16 mode, D = 64 or 128, Ck a multiple of 128, Ck <= 2048).
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

constexpr int kFJ = 128;                            // clusters per tile
// Queries per pass FR and per selection step FQ (one warp each) are template parameters: 64 / 16 up to 1024
// key clusters, 32 / 8 up to 2048 (all FR x Ck scores of a pass live in the 512 TMEM columns, P and the score
// rows of a step in shared memory).
constexpr int kMaxStA = 6, kMaxStD = 4;
constexpr int kCandMax = 128;                       // candidates kept by the compacting selection (4 per lane)

struct FarBars { uint64_t fullA[kMaxStA], emptyA[kMaxStA], fullD[kMaxStD], emptyD[kMaxStD], done; };


// Top-m of one query's scores s[0..Ck) (one warp; Ck <= 32 NKMAX).  Writes the chosen clusters to
// so[0..m) (-1 padded, in no particular order), and removes them from the far set by setting
// their score to -inf.  Scores become order-preserving integer keys; everything above the key T
// of the m-th largest is taken and, among ties at T, the lowest cluster indices.
//
// Fast path (m <= 64, `may_compact`): the m-th largest of the 64 per-lane top-two keys, found by a
// bitonic sort across the warp (two keys per lane, shuffles only), bounds the m-th largest score
// from below, and on random data only about m + 4 scores reach it.  Those candidates are
// compacted into `cand` (kCandMax keys then kCandMax indices, 128-byte segments `seg` bytes apart;
// a lane-prefix sum gives every lane its slots, so the scatter needs no votes) and T is found by
// bisection over 4 keys per lane.  The code is laid out for instruction-level parallelism: a
// warp's chain of dependent votes and reductions, not the issue rate, bounds the selection.
// General path (any m, many equal scores, fewer than m finite scores): bisection over all keys.
template <int NKMAX>
__device__ __forceinline__ void select_top_m(float* s, int Ck, int m, int32_t* so, int lane, unsigned char* cand, int seg,
                                             bool may_compact, int* dbg = nullptr) {
#ifdef MUSE_PHASE_CLOCKS
  long long c0_ = clock64(), c1_ = 0, c2_ = 0, c3_ = 0, c4_ = 0;
#define MUSE_SEL_CLOCK(x) x = clock64()
#else
#define MUSE_SEL_CLOCK(x)
#endif
  const int NK = Ck >> 5;                       // scores per lane (<= NKMAX)
  auto to_key = [](float x) {
    const uint32_t b = __float_as_uint(x);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
  };
  float v[NKMAX];
#pragma unroll
  for (int k = 0; k < NKMAX; ++k) v[k] = k < NK ? s[lane + 32 * k] : -INFINITY;
  const uint32_t kFinite = 0x00800000u;         // smallest key above key(-inf) = 0x007fffff
  const uint32_t lt = (1u << lane) - 1u;
  float f1 = -INFINITY, f2 = -INFINITY;         // the lane's largest and second largest score
#pragma unroll
  for (int k = 0; k < NKMAX; ++k) {
    f2 = fmaxf(f2, fminf(f1, v[k]));
    f1 = fmaxf(f1, v[k]);
  }
  const uint32_t m1 = to_key(f1), m2 = to_key(f2);
  MUSE_SEL_CLOCK(c1_);
  if (may_compact && m >= 1 && m <= 64) {
    // bitonic sort, descending, of the 64 keys e = 2 lane + r held as (v0, v1)
    uint32_t v0 = m1, v1 = m2;
    const int e2 = lane << 1;
#pragma unroll
    for (int k = 2; k <= 64; k <<= 1) {
      const bool desc = (e2 & k) == 0;
#pragma unroll
      for (int j = k >> 1; j >= 2; j >>= 1) {
        const uint32_t p0 = __shfl_xor_sync(0xffffffffu, v0, j >> 1), p1 = __shfl_xor_sync(0xffffffffu, v1, j >> 1);
        const bool keep_max = ((e2 & j) == 0) == desc;
        v0 = keep_max ? max(v0, p0) : min(v0, p0);
        v1 = keep_max ? max(v1, p1) : min(v1, p1);
      }
      const uint32_t hi = max(v0, v1), lo = min(v0, v1);
      v0 = desc ? hi : lo;
      v1 = desc ? lo : hi;
    }
    const uint32_t lb = __shfl_sync(0xffffffffu, ((m - 1) & 1) ? v1 : v0, (m - 1) >> 1);
    const uint32_t kmx = __shfl_sync(0xffffffffu, v0, 0);
    MUSE_SEL_CLOCK(c2_);
    uint32_t msk[(NKMAX + 31) / 32] = {};                     // this lane's candidates, one bit per score
    // (float comparison: the same set as by key, plus -0 beside +0, which does no harm)
    const uint32_t lbb = (lb & 0x80000000u) ? (lb & 0x7fffffffu) : ~lb;
    const float lbf = __uint_as_float(lbb);
#pragma unroll
    for (int k = 0; k < NKMAX; ++k) msk[k >> 5] |= v[k] >= lbf ? 1u << (k & 31) : 0u;
    int cl = 0;
#pragma unroll
    for (int w = 0; w < (NKMAX + 31) / 32; ++w) cl += __popc(msk[w]);
    int incl = cl;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += t;
    }
    const int ncand = __shfl_sync(0xffffffffu, incl, 31);
    if (lb >= kFinite && ncand <= kCandMax) {
      // a lane holds one or two candidates as a rule: walk its mask and fetch the scores again
      int pos = incl - cl;
#pragma unroll
      for (int w = 0; w < (NKMAX + 31) / 32; ++w) {
        for (uint32_t mm = msk[w]; mm != 0u; mm &= mm - 1u, ++pos) {
          const int j = lane + 32 * (32 * w + __ffs((int)mm) - 1);
          *reinterpret_cast<uint32_t*>(cand + (pos >> 5) * seg + (pos & 31) * 4) = to_key(s[j]);
          *reinterpret_cast<int32_t*>(cand + (4 + (pos >> 5)) * seg + (pos & 31) * 4) = j;
        }
      }
      __syncwarp();
      MUSE_SEL_CLOCK(c3_);
      uint32_t ck[4];
      int32_t ci[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const bool in = lane + 32 * q < ncand;
        ck[q] = in ? *reinterpret_cast<const uint32_t*>(cand + q * seg + lane * 4) : 0u;
        ci[q] = in ? *reinterpret_cast<const int32_t*>(cand + (4 + q) * seg + lane * 4) : 0x7fffffff;
      }
      auto count4 = [&](uint32_t thr) {
        return (int)__reduce_add_sync(0xffffffffu, (unsigned)((ck[0] >= thr) + (ck[1] >= thr) + (ck[2] >= thr) + (ck[3] >= thr)));
      };
      const int shared = __clz((int)(kmx ^ lb));              // 32 if the interval is a single key
      uint32_t T = shared >= 32 ? kmx : (kmx & ~(0xffffffffu >> shared));
      for (int bit = 31 - shared; bit >= 0; --bit) {
        const uint32_t c2 = T | (1u << bit);
        const int c = count4(c2);
        if (c >= m) { T = c2; if (c == m) break; }
      }
      MUSE_SEL_CLOCK(c4_);
#ifdef MUSE_PHASE_CLOCKS
      if (dbg && lane == 0) { dbg[0] = (int)(c1_ - c0_); dbg[1] = (int)(c2_ - c1_); dbg[2] = (int)(c3_ - c2_); dbg[3] = (int)(c4_ - c3_); dbg[4] = ncand; dbg[5] = 1; }
#endif
      int need = m - count4(T + 1u);                            // ties at T still to take (>= 0)
      const int ntie = (int)__reduce_add_sync(0xffffffffu, (unsigned)((ck[0] == T) + (ck[1] == T) + (ck[2] == T) + (ck[3] == T)));
      bool take[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) take[q] = ck[q] > T || (ntie <= need && ck[q] == T);
      if (ntie > need) {
        // more ties than places: lowest cluster indices first
        for (; need > 0; --need) {
          int jm = 0x7fffffff;
#pragma unroll
          for (int q = 0; q < 4; ++q) jm = min(jm, (ck[q] == T && !take[q]) ? ci[q] : 0x7fffffff);
          jm = __reduce_min_sync(0xffffffffu, jm);
#pragma unroll
          for (int q = 0; q < 4; ++q) take[q] = take[q] || (ck[q] == T && ci[q] == jm);
        }
      }
      int base = 0;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (32 * q < ncand) {
          const uint32_t ms = __ballot_sync(0xffffffffu, take[q]);
          if (take[q]) { so[base + __popc(ms & lt)] = ci[q]; s[ci[q]] = -INFINITY; }
          base += __popc(ms);
        }
      }
      for (int k = base + lane; k < m; k += 32) so[k] = -1;
      return;
    }
  }

  uint32_t key[NKMAX];
#pragma unroll
  for (int k = 0; k < NKMAX; ++k) key[k] = to_key(v[k]);
  auto count_ge = [&](uint32_t thr) {           // lane-local count, then one warp reduction
    int c = 0;
#pragma unroll
    for (int k = 0; k < NKMAX; ++k) c += key[k] >= thr ? 1 : 0;
    return (int)__reduce_add_sync(0xffffffffu, (unsigned)c);
  };
  uint32_t kmn = 0xffffffffu;                   // smallest finite key
  int nfin = 0;
#pragma unroll
  for (int k = 0; k < NKMAX; ++k) {
    const bool fin = key[k] >= kFinite;
    nfin += fin ? 1 : 0;
    kmn = min(kmn, fin ? key[k] : 0xffffffffu);
  }
  const bool take_all = (int)__reduce_add_sync(0xffffffffu, (unsigned)nfin) <= m;
  uint32_t T = kFinite;
  if (!take_all) {
    const uint32_t kmx = __reduce_max_sync(0xffffffffu, m1);
    kmn = __reduce_min_sync(0xffffffffu, kmn);
    const int shared = __clz((int)(kmx ^ kmn));            // 32 if the interval is a single key
    T = shared >= 32 ? kmx : (kmx & ~(0xffffffffu >> shared));
    for (int bit = 31 - shared; bit >= 0; --bit) {
      const uint32_t c2 = T | (1u << bit);
      const int c = count_ge(c2);
      if (c >= m) { T = c2; if (c == m) break; }
    }
  }
  int base = 0, ties_seen = 0;
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
  for (int k = base + lane; k < m; k += 32) so[k] = -1;
}

// NKMAX: scores per lane that the selection keeps in registers (Ck <= 32 NKMAX); MINB: CTAs per SM the register
// budget is set for.  With few key clusters the per-query selection, a chain of dependent warp operations, is what
// takes the time: small instances (few registers, few TMEM columns) put several CTAs on an SM.
template <int FR, int FQ, int D, int NKMAX, int MINB>
__global__ void __launch_bounds__(FQ * 32, MINB)
k_far_fwd_tc(Dims dm, const __grid_constant__ CUtensorMap tm_khi, const __grid_constant__ CUtensorMap tm_klo,
             const __grid_constant__ CUtensorMap tm_nu, const bf16* __restrict__ Q, const int32_t* __restrict__ off_q,
             const int32_t* __restrict__ perm_q, const float* __restrict__ mu, const float* __restrict__ beta,
             const int32_t* __restrict__ sel_in, int32_t* __restrict__ sel_out, float* __restrict__ o_far,
             float* __restrict__ lse_far, int p_bytes, int sc_bytes, int nsA, int nsD, int tcols, int* __restrict__ status) {
  constexpr int NT = FQ * 32, NTG = FQ / 4, KT = 16 / NTG;   // threads; tile groups in the TMEM read-out; cluster tiles per group
  constexpr int kTileBytes = kFJ * D * 2, G = D / 64;        // one [128 clusters][D] bf16 operand tile; 128-byte column groups of a row
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
  const bf16* Qp = Q + (size_t)pq * dm.N * D;
  const int32_t* pm = perm_q + (size_t)pq * dm.N;

  if (warp == 0) tc::tmem_alloc(&tbase_s, tcols);
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
  uint32_t cntA = 0, cntD = 0, done_ph = 0;   // tiles of the earlier passes (same in every thread); phase of `done`
  bool ok = true;
  // TMA producers: lane 0 of warps 0, 2, 3, 4.  One thread sustains only about 30 bytes per clock
  // (every bulk-tensor instruction holds it for some 270 clocks per 16 KB box, every wait after one
  // for some 500), several threads add up.  Producer p serves the tiles whose running index is
  // p modulo the producer count, and that count divides the ring depth, so a ring stage always
  // belongs to one producer and its waits on the stage's barrier never fall a phase behind.
  const int prod = lane != 0 ? -1 : warp == 0 ? 0 : (warp >= 2 && warp <= 4) ? warp - 1 : -1;
  const int WA = nsA % 4 == 0 ? 4 : nsA % 3 == 0 ? 3 : nsA % 2 == 0 ? 2 : 1;
  const int WD = nsD % 4 == 0 ? 4 : nsD % 2 == 0 ? 2 : 1;
  const int lq = warp & 3, tg = warp >> 2;            // TMEM lane quarter of this warp, tile group

  for (int r0 = p0; r0 < p1 && ok; r0 += FR) {
    const int n = min(FR, p1 - r0);
#ifdef MUSE_PHASE_CLOCKS
    long long ck0 = clock64(), ck1 = 0, ck3 = 0, ck4 = 0;
#endif
    // ---- A: scores^T for all clusters, kappa_hi / kappa_lo tiles through an nsA-stage TMA ring;
    //         the producers load (TMA), thread 32 consumes (MMA), so neither waits for the other's latency.
    //         The first ring-full of tiles is requested before the query rows are gathered.
    // (ring stage, phase and owning producer of a tile advance by increments: no division per tile)
    const int sA0 = cntA % nsA, phA0 = (cntA / nsA) & 1, sD0 = cntD % nsD, phD0 = (cntD / nsD) & 1;
    int sa = sA0, pha = phA0, wa = sA0 % WA;             // of the next tile this producer looks at
    auto next_a = [&]() {
      if (++sa == nsA) { sa = 0; pha ^= 1; }
      if (++wa == WA) wa = 0;
    };
    auto produce_a = [&](int t) {
      const int s = sa;
      if (!tc::mbar_wait(&bars.emptyA[s], pha ^ 1)) { ok = false; return; }
      tc::mbar_expect_tx(&bars.fullA[s], kTileBytes);
      const void* map = (t & 1) ? (const void*)&tm_klo : (const void*)&tm_khi;
      const int row = (int)(ent0 + (size_t)(t >> 1) * kFJ);
      for (int g = 0; g < G; ++g) tc::tma_load_2d(sm + s * kTileBytes + g * kFJ * 128, map, 64 * g, row, &bars.fullA[s]);
    };
    const int TA = 2 * NJ, TA0 = min(nsA, TA);
    if (prod >= 0 && prod < WA)
      for (int t = 0; t < TA0 && ok; ++t, next_a())
        if (wa == prod) produce_a(t);
    if (tid < FR) rows[tid] = tid < n ? pm[r0 + tid] : -1;
    // query rows -> K-major swizzled tile [FR][D] bf16 (G blocks of [FR][128 B])
    for (int e = tid; e < FR * (D / 8); e += NT) {
      const int r = e / (D / 8), ck = e % (D / 8), kb = ck >> 3, c = ck & 7;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (r < n && MUSE_IN_RANGE(r0 + r, dm.N) && MUSE_IN_RANGE(pm[r0 + r], dm.N)) v = reinterpret_cast<const uint4*>(Qp + (size_t)pm[r0 + r] * D)[ck];
      *reinterpret_cast<uint4*>(Qs + kb * FR * 128 + tc::sw128_off(r, c)) = v;
    }
    tc::fence_async_smem();
    tc::fence_before_sync();
    __syncthreads();
    if (prod >= 0) {
      if (prod < WA)
        for (int t = TA0; t < TA && ok; ++t, next_a())
          if (wa == prod) produce_a(t);
      // bring the nu tiles of this segment into L2 while the selection runs
      for (int t = prod; t < NJ; t += 4) {
        for (int g = 0; g < G; ++g) tc::tma_prefetch_2d(&tm_nu, 64 * g, (int)(ent0 + (size_t)t * kFJ));
      }
    } else if (tid == 32) {
      tc::fence_after_sync();
      const uint32_t idesc = tc::idesc_bf16(kFJ, FR, 0, 0);
      const uint64_t dq0 = tc::smem_desc_sw128(tc::smem_u32(Qs), 16, 1024), da0 = tc::smem_desc_sw128(tc::smem_u32(sm), 16, 1024);
      const int T = 2 * NJ;
#ifdef MUSE_PHASE_CLOCKS
      long long ta0_ = clock64();
#endif
      for (int u = 0, s = sA0, ph = phA0; u < T; ++u) {
        if (!tc::mbar_wait(&bars.fullA[s], ph)) { ok = false; break; }
#ifdef MUSE_PHASE_CLOCKS
        if (blockIdx.x == 200 && blockIdx.y == 5 && blockIdx.z == 1 && r0 == p0) {
          if (u == 0) status[62] = (int)(clock64() - ta0_);
          if (u == T - 1) status[63] = (int)(clock64() - ta0_);
        }
#endif
        const uint64_t da = tc::desc_step(da0, (uint32_t)s * kTileBytes);
        const uint32_t dcol = tbase + (u >> 1) * FR;

#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc::mma_bf16_ss(dcol, tc::desc_step(da, (ks / 4) * kFJ * 128 + (ks % 4) * 32),
                          tc::desc_step(dq0, (ks / 4) * FR * 128 + (ks % 4) * 32), idesc, (u & 1) || ks > 0);
        tc::mma_commit(&bars.emptyA[s]);
        if (++s == nsA) { s = 0; ph ^= 1; }
      }
      if (ok) tc::mma_commit(&bars.done);
    }
    float bq[KT];                                       // beta of this thread's clusters, loaded ahead of the TMEM reads
#pragma unroll
    for (int k = 0; k < KT; ++k) { const int jt = tg + NTG * k; bq[k] = jt < NJ ? bep[jt * kFJ + (tid & 127)] : 0.f; }
    // only the consumer polls the mbarrier; everyone else sleeps at the hardware barrier
    if (tid == 32) {
      if (!tc::mbar_wait(&bars.done, done_ph)) ok = false;
      tc::fence_before_sync();
    }
    ok = __syncthreads_and(ok);
    done_ph ^= 1;
    cntA += TA;
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
          for (int k = lane; k < m; k += 32) { int c = si[k]; c = (c >= 0 && c < Ck) ? c : -1; so[k] = c; if (c >= 0) s[c] = -INFINITY; }
        } else if (dm.sel_mode == MUSE_SEL_PER_QCLUSTER) {
          for (int k = lane; k < m; k += 32) { int c = selq[k]; so[k] = c; if (c >= 0) s[c] = -INFINITY; }
        } else if (m > 0) {
          // this query's own (not yet written) P row doubles as the candidate scratch
          int* dbg = nullptr;
#ifdef MUSE_PHASE_CLOCKS
          if (warp == 0 && blockIdx.x == 200 && blockIdx.y == 5 && blockIdx.z == 1 && r0 == p0 && qs == 0) dbg = status + 56;
#endif
          select_top_m<NKMAX>(s, Ck, m, so, lane, Pm + r * 128, FR * 128, Ck >= 512, dbg);
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
      if (tid == 0 && blockIdx.x == 200 && blockIdx.y == 5 && blockIdx.z == 1 && r0 == p0 && qs == 0) {
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
    if (prod >= 0 && prod < WD && ok) {
      unsigned char* ring = sm + p_bytes;
      for (int t = 0, s = sD0, ph = phD0, w = sD0 % WD; t < NJ; ++t) {
        const int s_ = s, ph_ = ph, w_ = w;
        if (++s == nsD) { s = 0; ph ^= 1; }
        if (++w == WD) w = 0;
        if (w_ != prod) continue;
        if (!tc::mbar_wait(&bars.emptyD[s_], ph_ ^ 1)) { ok = false; break; }
        tc::mbar_expect_tx(&bars.fullD[s_], kTileBytes);
        const int row = (int)(ent0 + (size_t)t * kFJ);
        for (int g = 0; g < G; ++g) tc::tma_load_2d(ring + s_ * kTileBytes + g * kFJ * 128, &tm_nu, 64 * g, row, &bars.fullD[s_]);
      }
    } else if (tid == 32 && ok) {
      tc::fence_after_sync();
      // M = 128 output dims even when D = 64: the second 64-dim group of the MN-major operand then reads whatever
      // follows the tile in shared memory, and output lanes 64..127 hold numbers that nobody reads
      const uint32_t idesc = tc::idesc_bf16(128, FR, 1, 0);
      const uint64_t dp0 = tc::smem_desc_sw128(tc::smem_u32(Pm), 16, 1024);
      const uint64_t dn0 = tc::smem_desc_sw128(tc::smem_u32(sm + p_bytes), kFJ * 128, 1024);
#ifdef MUSE_PHASE_CLOCKS
      long long td0_ = clock64();
#endif
      for (int u = 0, s = sD0, ph = phD0; u < NJ; ++u) {
        if (!tc::mbar_wait(&bars.fullD[s], ph)) { ok = false; break; }
#ifdef MUSE_PHASE_CLOCKS
        if (blockIdx.x == 200 && blockIdx.y == 5 && blockIdx.z == 1 && r0 == p0) {
          if (u == 0) status[15] = (int)(clock64() - td0_);
          if (u == NJ - 1) status[16] = (int)(clock64() - td0_);
        }
#endif
        const uint64_t da = tc::desc_step(dn0, (uint32_t)s * kTileBytes), dp = tc::desc_step(dp0, (uint32_t)(2 * u) * (FR * 128));
#pragma unroll
        for (int ks = 0; ks < kFJ / 16; ++ks)
          tc::mma_bf16_ss(tbase, tc::desc_step(da, ks * 16 * 128), tc::desc_step(dp, (ks / 4) * (FR * 128) + (ks % 4) * 32), idesc,
                          u > 0 || ks > 0);
        tc::mma_commit(&bars.emptyD[s]);
        if (++s == nsD) { s = 0; ph ^= 1; }
      }
      if (ok) tc::mma_commit(&bars.done);
    }
    if (tid == 32) {
      if (!tc::mbar_wait(&bars.done, done_ph)) ok = false;
      tc::fence_before_sync();
    }
    ok = __syncthreads_and(ok);
    done_ph ^= 1;
    cntD += NJ;
    tc::fence_after_sync();
#ifdef MUSE_PHASE_CLOCKS
    ck4 = clock64();
    if (tid == 0 && blockIdx.x == 200 && blockIdx.y == 5 && blockIdx.z == 1 && r0 == p0) {
      status[8] = (int)(ck1 - ck0); status[9] = 0; status[10] = (int)(ck3 - ck1); status[11] = (int)(ck4 - ck3);
      status[12] = n;
    }
#endif
    // ---- E: thread = output dim d; warps 0-3 read queries 0..31, warps 4-7 queries 32..63
    if (warp < FR / 8) {
      const int half = warp >> 2;
      float v[32];
      tc::tmem_ld32(tbase + ((uint32_t)(lq * 32) << 16) + 32 * half, v);
      if (ok && (tid & 127) < D) {
#pragma unroll
        for (int r = 0; r < 32; ++r)
          if (32 * half + r < n) o_far[((size_t)pq * dm.N + rows[32 * half + r]) * D + (tid & 127)] = v[r] * rinv[32 * half + r];
      }
    }
    tc::fence_before_sync();
    __syncthreads();
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tbase, tcols);
  if (!ok && tid == 0) report_status(status, 3);
}

bool far_fwd_tc_supported(const Dims& d, int dtype) {
  return dtype == MUSE_BF16 && (d.D == 64 || d.D == 128) && d.Ck % kFJ == 0 && d.Ck <= 2048 && d.Ck >= kFJ;
}

int far_fwd_tc(const Dims& d, const SummPtrs& sp, const void* Q, const int32_t* off_q, const int32_t* perm_q,
               const int32_t* sel_in, int32_t* sel_out, float* o_far, float* lse_far, int* status, cudaStream_t st) {
  const uint64_t ent = (uint64_t)d.B * d.Hq * d.SB * d.Cq * d.Ck;
  CUtensorMap khi, klo, nu;
  int rc = make_tmap_bf16_rows(&khi, sp.khi, ent, d.D, kFJ);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&klo, sp.klo, ent, d.D, kFJ);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&nu, sp.nu, ent, d.D, kFJ);
  if (rc != MUSE_OK) return rc;
  const bool wide = d.Ck > 1024;                                         // 32 queries per pass, 8 per selection step
  const int FR = wide ? 32 : 64, FQ = wide ? 8 : 16;
  const int tile_bytes = kFJ * d.D * 2;
  const int p_bytes = FR * d.Ck * 2;                                     // P: bf16 [FR][Ck]
  int sc_bytes = FQ * d.Ck * 4;                                          // FQ score rows, later the nu ring
  if (sc_bytes < 2 * tile_bytes) sc_bytes = 2 * tile_bytes;
  int nsA = (p_bytes + sc_bytes) / tile_bytes, nsD = sc_bytes / tile_bytes;
  nsA = nsA > kMaxStA ? kMaxStA : nsA;
  nsD = nsD > kMaxStD ? kMaxStD : nsD;
  // (D = 64: one more tile of room behind the ring, which the padded 128-row products of phase D read past)
  const size_t smem = (size_t)p_bytes + sc_bytes + FR * d.D * 2 + 1024 + (d.D == 64 ? tile_bytes : 0);
  prof_mark("k_far_fwd_tc", st);
  // TMEM columns: all FR x Ck scores of a pass (the output of phase D reuses them), a power of two >= 32
  int tcols = 32;
  while (tcols < FR * (d.Ck / kFJ)) tcols *= 2;
#define MUSE_FAR_FWD_LAUNCH(FR_, FQ_, D_, NK_, MB_)                                                                              \
  do {                                                                                                                         \
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_far_fwd_tc<FR_, FQ_, D_, NK_, MB_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
    k_far_fwd_tc<FR_, FQ_, D_, NK_, MB_><<<dim3(d.Cq, d.SB, d.B * d.Hq), FQ_ * 32, smem, st>>>(                                   \
        d, khi, klo, nu, (const bf16*)Q, off_q, perm_q, sp.mu, sp.beta, sel_in, sel_out, o_far, lse_far, p_bytes, sc_bytes, nsA, nsD, tcols, status); \
  } while (0)
  if (wide) { if (d.D == 128) MUSE_FAR_FWD_LAUNCH(32, 8, 128, 64, 1); else MUSE_FAR_FWD_LAUNCH(32, 8, 64, 64, 1); }
  else if (d.Ck <= 256) { if (d.D == 128) MUSE_FAR_FWD_LAUNCH(64, 16, 128, 8, 2); else MUSE_FAR_FWD_LAUNCH(64, 16, 64, 8, 2); }
  else { if (d.D == 128) MUSE_FAR_FWD_LAUNCH(64, 16, 128, 32, 1); else MUSE_FAR_FWD_LAUNCH(64, 16, 64, 32, 1); }
#undef MUSE_FAR_FWD_LAUNCH
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

}  // namespace muse
