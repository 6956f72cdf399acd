// Seeded k-means++ start points on the GPU (an alternative to the strided start of Appendix "Centroid Computation",
// step 1; the paper does not use it).  The first start point is position 0 of the seeded shuffle; draw c = 1 .. C - 1
// picks one vector with probability proportional to d2 = its squared distance to the nearest start point so far.
// The draw is an exponential race: vector t gets u_t in (0, 1) from an integer hash of (seed, stream, c, t),
// e_t = -log(u_t), and the largest d2_t / e_t wins (lowest index on ties) -- the same law as sampling the
// cumulative sum of d2, but a maximum instead of a prefix sum, so every draw is one pass over the vectors.
//
// One problem (head, side) = one thread-block cluster of up to 8 CTAs, each owning a contiguous slice of the vectors;
// the C - 1 draws are sequential, each ends with one candidate per CTA written into every CTA's shared memory and a
// hardware cluster barrier.  A draw reads every vector once (distance to the newest start point only; the running
// minima stay in shared memory when the slice fits, else in scratch), so the stage moves (C - 1) N D e bytes per
// problem.  At the headline size its instructions per vector take about as long as the HBM read: the
// kernel sits between the issue limit and the bandwidth limit.
#include <cooperative_groups.h>
#include <type_traits>

#include "common.cuh"
#include "feistel.cuh"
#include "tc05.cuh"

namespace cg = cooperative_groups;

namespace muse {

constexpr int kPpThreads = 256, kPpCluster = 8, kPpWarps = kPpThreads / 32;

__device__ __forceinline__ bool pp_better(float k, int i, float bk, int bi) { return k > bk || (k == bk && i < bi); }

// contiguous global -> shared bulk copy (16-byte aligned, size a multiple of 16), completion counted on an mbarrier
__device__ __forceinline__ void pp_bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(tc::smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(tc::smem_u32(bar)) : "memory");
}

// Every warp streams its own groups of GR consecutive vectors through a private ring of kPpStages shared-memory
// stages filled by bulk copies (plain loads top out near 25 bytes per clock per SM here, bulk copies do not); the ring
// keeps running across draws, since every draw reads the same slice in the same order.
template <class T, int D, int kPpStages, int kPpGroupBytes>
__global__ void __launch_bounds__(kPpThreads)
k_kmeanspp(const T* __restrict__ X, int N, int C, uint64_t seed, int kind, float* __restrict__ mind2,
           int32_t* __restrict__ idx_out, int md_shared, int* __restrict__ status) {
  cg::cluster_group cluster = cg::this_cluster();
  const int CS = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  const int prob = blockIdx.x / CS, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int EPL = 16 / (int)sizeof(T);      // elements per 16-byte load
  constexpr int LPR = D / EPL, RPW = 32 / LPR;  // lanes per vector, vectors per warp and load
  constexpr int GR = (kPpGroupBytes / (D * (int)sizeof(T))) < 32 ? (kPpGroupBytes / (D * (int)sizeof(T))) : 32;   // vectors per group
  constexpr int GB = GR * D * (int)sizeof(T);   // bytes per stage (<= 8 KB)
  constexpr int NL = GR / RPW;                  // loads per lane and group
  extern __shared__ __align__(128) unsigned char pp_smem[];
  __shared__ float cs[D];
  __shared__ float exk[2][kPpCluster], wk[kPpWarps], dpark[kPpWarps][32];
  __shared__ int exi[2][kPpCluster], wi[kPpWarps];
  __shared__ uint64_t full[kPpWarps][kPpStages];
  unsigned char* ring = pp_smem + (size_t)warp * kPpStages * GB;
  float* mds = reinterpret_cast<float*>(pp_smem + (size_t)kPpWarps * kPpStages * GB);   // the slice's running minima, when they fit
  const T* Xp = X + (size_t)prob * N * D;
  float* md = mind2 + (size_t)prob * N;
  const uint64_t stream = (uint64_t)prob * 2 + (uint64_t)kind;
  const int per = (N + CS - 1) / CS, lo = rank * per, hi = min(N, lo + per);
  const int sub = lane % LPR, grp = lane / LPR;
  // this warp's groups of one draw: group k covers vectors [lo + (k * kPpWarps + warp) * GR, ... + GR)
  const int ngroups = hi > lo ? (hi - lo + GR - 1) / GR : 0;
  const int mine = ngroups > warp ? (ngroups - warp + kPpWarps - 1) / kPpWarps : 0;
  const bool norms = md_shared != 0 && C > 1;   // squared norms kept beside the minima: the cheaper distance form
  const int total = mine * (C - 1 + (norms ? 1 : 0));      // at most (N / 256) * (kMaxC + 1): fits
  // Every CTA walks its slice from a different starting group (the order inside a draw does not matter: the draw is
  // a maximum with an explicit tie rule).  Without it all CTAs read the same offset of their 2^k-spaced slices at the
  // same moment, and the copies crowd onto a few memory channels.
  const int shift = mine > 0 ? (int)((blockIdx.x * 37u + 11u) % (unsigned)mine) : 0;
  // running positions instead of divisions: kc / sc = group and stage consumed next, ki / si = group and stage filled next
  int kc = shift, sc = 0, ki = shift, si = 0, issued = 0;
  uint32_t phase = 0;                           // bit s = parity of stage s's next completion
  auto issue = [&]() {                          // lane 0: start the copy of the warp's next group
    const int k = ki, s = si;
    ki = ki + 1 == mine ? 0 : ki + 1; si = si + 1 == kPpStages ? 0 : si + 1; ++issued;
    const int t0 = lo + (k * kPpWarps + warp) * GR;
    const uint32_t bytes = (uint32_t)min(GR, hi - t0) * (uint32_t)(D * sizeof(T));
    tc::mbar_expect_tx(&full[warp][s], bytes);
    pp_bulk_load(ring + s * GB, Xp + (size_t)t0 * D, bytes, &full[warp][s]);
  };
  if (lane == 0) {
    for (int s = 0; s < kPpStages; ++s) tc::mbar_init(&full[warp][s], 1);
    tc::mbar_init_fence();
  }
  __syncwarp();
  if (lane == 0)
    while (issued < kPpStages - 1 && issued < total) issue();
  bool ok = true;
  // Running minima d2 (and, with them, the squared norms): in shared memory when the slice fits beside the ring
  // (md_shared); otherwise the minima live in global scratch and are loaded one group ahead.
  float* xns = mds + per;                       // squared norms of the slice's vectors (md_shared only)
  float mcur = INFINITY;
  float cen[EPL];
  float cn = 0.f;                               // squared norm of the newest start point
  uint64_t key_c = 0;
  float bk = -1.f; int bi = 0x7fffffff;
  int last = feistel_permute(0, N, seed, stream);
  // One group of the warp: refill the ring, wait for the group's bytes, reduce every vector against `cen`, finish one
  // vector per lane.  MODE 0: squared norms (once, before the first draw); MODE 1: draw with d2 = sum (x - c)^2;
  // MODE 2: draw with d2 = |x|^2 + |c|^2 - 2 x.c from the stored norms (a third fewer instructions per element; the
  // cancellation error, about 1e-7 of |x|^2 + |c|^2, is far below what separates the race's leaders).
  auto consume = [&](auto mode_tag, int c, bool more_in_pass) -> bool {
    constexpr int MODE = decltype(mode_tag)::value;
    const int s = sc, k = kc;
    // (the stage read in the previous iteration is free: its loads delivered their values before that iteration's
    // closing __syncwarp)
    if (lane == 0 && issued < total) issue();
    // the outcome of the bounded wait is made the same for the whole warp before anyone acts on it
    if (!__all_sync(0xffffffffu, tc::mbar_wait(&full[warp][s], (phase >> s) & 1u) ? 1 : 0)) return false;
    phase ^= 1u << s;
    kc = kc + 1 == mine ? 0 : kc + 1; sc = sc + 1 == kPpStages ? 0 : sc + 1;
    float mnext = INFINITY;
    if (MODE != 0 && !md_shared && more_in_pass && c > 1) {
      const int tn = lo + (kc * kPpWarps + warp) * GR + lane;
      if (lane < GR && tn < hi) mnext = md[tn];
    }
    const unsigned char* st = ring + s * GB;
    const int w0 = lo + (k * kPpWarps + warp) * GR;
#pragma unroll
    for (int h = 0; h < NL; h += 8) {
      uint4 raw[8];
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (h + u < NL) raw[u] = *reinterpret_cast<const uint4*>(st + ((size_t)((h + u) * RPW + grp) * D + sub * EPL) * sizeof(T));
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        if (h + u >= NL) continue;
        float x[EPL];
        if (sizeof(T) == 2) {
          const uint32_t wv[4] = {raw[u].x, raw[u].y, raw[u].z, raw[u].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) { x[2 * e] = __uint_as_float(wv[e] << 16); x[2 * e + 1] = __uint_as_float(wv[e] & 0xffff0000u); }
        } else {
          x[0] = __uint_as_float(raw[u].x); x[1] = __uint_as_float(raw[u].y);
          x[EPL - 2] = __uint_as_float(raw[u].z); x[EPL - 1] = __uint_as_float(raw[u].w);
        }
        float d = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
          if (MODE == 0) d = fmaf(x[e], x[e], d);
          else if (MODE == 1) { const float a = x[e] - cen[e]; d = fmaf(a, a, d); }
          else d = fmaf(x[e], cen[e], d);
        }
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
        if (sub == 0) dpark[warp][(h + u) * RPW + grp] = d;
      }
    }
    __syncwarp();
    const int t = w0 + lane;
    if (lane < GR && t < hi) {                  // rows past the slice's end hold stale bytes: never looked at
      float d = dpark[warp][lane];
      if (MODE == 0) xns[t - lo] = d;
      else {
        if (MODE == 2) d = t == last ? 0.f : fmaxf(xns[t - lo] + cn - 2.f * d, 0.f);
        if (md_shared) { if (c > 1) d = fminf(d, mds[t - lo]); mds[t - lo] = d; }
        else { d = fminf(d, mcur); md[t] = d; }
        const uint64_t h = splitmix64(key_c ^ (uint64_t)t);
        const float u = ((float)(uint32_t)(h >> 41) + 0.5f) * (1.f / 8388608.f);
        const float key = d / -logf(u);
        if (pp_better(key, t, bk, bi)) { bk = key; bi = t; }
      }
    }
    __syncwarp();
    mcur = mnext;
    return true;
  };
  if (rank == 0 && tid == 0) idx_out[(size_t)prob * C] = last;
  cluster.sync();                               // every CTA of the problem is running before any of them writes into another's shared memory
  if (norms)
    for (int kk = 0; kk < mine && ok; ++kk) ok = consume(std::integral_constant<int, 0>(), 0, kk + 1 < mine);
  for (int c = 1; c < C; ++c) {
    if (tid < D) cs[tid] = MUSE_IN_RANGE(last, N) ? to_f(Xp[(size_t)last * D + tid]) : 0.f;
    __syncthreads();
    cn = 0.f;
#pragma unroll
    for (int k = 0; k < EPL; ++k) { cen[k] = cs[sub * EPL + k]; cn = fmaf(cen[k], cen[k], cn); }
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) cn += __shfl_xor_sync(0xffffffffu, cn, o);
    key_c = splitmix64(seed ^ (stream << 32) ^ (0xA5ull << 56) ^ (uint64_t)c);
    bk = -1.f; bi = 0x7fffffff;
    for (int kk = 0; kk < mine && ok; ++kk)
      ok = norms ? consume(std::integral_constant<int, 2>(), c, kk + 1 < mine) : consume(std::integral_constant<int, 1>(), c, kk + 1 < mine);
    if (!md_shared && mine > 0 && ok) {         // first group of the next draw (this lane wrote its value during this draw)
      const int tn = lo + (kc * kPpWarps + warp) * GR + lane;
      mcur = lane < GR && tn < hi ? md[tn] : INFINITY;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ok_ = __shfl_xor_sync(0xffffffffu, bk, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (pp_better(ok_, oi, bk, bi)) { bk = ok_; bi = oi; }
    }
    if (lane == 0) { wk[warp] = bk; wi[warp] = bi; }
    __syncthreads();
    const int par = c & 1;
    if (warp == 0) {
      bk = lane < kPpWarps ? wk[lane] : -1.f; bi = lane < kPpWarps ? wi[lane] : 0x7fffffff;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ok_ = __shfl_xor_sync(0xffffffffu, bk, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (pp_better(ok_, oi, bk, bi)) { bk = ok_; bi = oi; }
      }
      if (lane < CS) {                          // lane r delivers this CTA's candidate to CTA r
        *cluster.map_shared_rank(&exk[par][rank], lane) = bk;
        *cluster.map_shared_rank(&exi[par][rank], lane) = bi;
      }
    }
    cluster.sync();                             // every CTA's candidate has arrived (and the previous draw's have been read)
    bk = -1.f; bi = 0x7fffffff;
    for (int r = 0; r < CS; ++r)
      if (pp_better(exk[par][r], exi[par][r], bk, bi)) { bk = exk[par][r]; bi = exi[par][r]; }
    last = min(max(bi, 0), N - 1);
    if (rank == 0 && tid == 0) idx_out[(size_t)prob * C + c] = last;
  }
  if (!ok) {
    // a wait gave up: say so, and let the (at most kPpStages - 1) copies still in flight land before the CTA's
    // shared memory is released
    if (lane == 0) report_status(status, MUSE_STATUS_ASSIGN_TIMEOUT);
    const long long t0 = clock64();
    while (clock64() - t0 < (1ll << 24)) { }
  }
  cluster.sync();                               // no CTA leaves while another may still write into its shared memory
}

size_t kmeanspp_ws_floats(int problems, int N) { return (size_t)problems * N; }

template <class T, int D>
struct PpPlan { int stages; int md_shared; size_t smem; };

// Ring depth and where the running minima live for a slice of `per` vectors: three stages when the minima then still
// fit in shared memory (or do not fit either way), two stages when that is what makes them fit.
template <class T, int D>
static PpPlan<T, D> pp_plan(int per) {
  constexpr int GR = (8192 / (D * (int)sizeof(T))) < 32 ? (8192 / (D * (int)sizeof(T))) : 32;
  const size_t stage = (size_t)kPpWarps * GR * D * sizeof(T), md_bytes = 2 * (size_t)per * sizeof(float), budget = 224 * 1024;   // minima + norms
  if (3 * stage + md_bytes <= budget) return {3, 1, 3 * stage + md_bytes};
  if (2 * stage + md_bytes <= budget) return {2, 1, 2 * stage + md_bytes};
  return {3, 0, 3 * stage};
}

template <class T, int D, int ST>
static int kmeanspp_v(const T* X, int problems, int N, int C, int kind, uint64_t seed, float* mind2, int32_t* idx_out,
                      int cs, int md_shared, size_t smem, bool query_only, int* max_clusters, int* status, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cfg.stream = st;
  cfg.gridDim = dim3(problems * cs);
  cfg.blockDim = dim3(kPpThreads);
  cfg.dynamicSmemBytes = smem;
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_kmeanspp<T, D, ST, 8192>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  if (query_only) {
    MUSE_CUDA_OK(cudaOccupancyMaxActiveClusters(max_clusters, k_kmeanspp<T, D, ST, 8192>, &cfg));
    return MUSE_OK;
  }
  prof_mark("k_kmeanspp", st);
  MUSE_CUDA_OK(cudaLaunchKernelEx(&cfg, k_kmeanspp<T, D, ST, 8192>, X, N, C, seed, kind, mind2, idx_out, md_shared, status));
  return MUSE_OK;
}

template <class T, int D>
static int kmeanspp_t(const T* X, int problems, int N, int C, int kind, uint64_t seed, float* mind2, int32_t* idx_out,
                      int* status, cudaStream_t st) {
  // CTAs per problem: the most (up to 8, slices of at least 1024 vectors) for which all problems' clusters can be resident
  // at once.  The draws are sequential, so a cluster that has to wait for a free slot doubles the stage's time; a GPU
  // whose processor groups leave no room for every cluster of 8 does better with clusters of 7 or 6.
  int cs_max = 1;
  while (cs_max < kPpCluster && N >= 1024 * (cs_max + 1)) ++cs_max;
  int cs = cs_max;
  for (int c = cs_max; c >= 1; --c) {
    const PpPlan<T, D> pl = pp_plan<T, D>((N + c - 1) / c);
    int active = 0;
    int rc = pl.stages == 3 ? kmeanspp_v<T, D, 3>(X, problems, N, C, kind, seed, mind2, idx_out, c, pl.md_shared, pl.smem, true, &active, status, st)
                            : kmeanspp_v<T, D, 2>(X, problems, N, C, kind, seed, mind2, idx_out, c, pl.md_shared, pl.smem, true, &active, status, st);
    if (rc != MUSE_OK) return rc;
    if (active >= problems) { cs = c; break; }
    if (c == 1 || active * c < 64) { cs = cs_max; break; }       // more problems than the GPU holds: several rounds either way
  }
  const PpPlan<T, D> pl = pp_plan<T, D>((N + cs - 1) / cs);
  if (pl.stages == 3) return kmeanspp_v<T, D, 3>(X, problems, N, C, kind, seed, mind2, idx_out, cs, pl.md_shared, pl.smem, false, nullptr, status, st);
  return kmeanspp_v<T, D, 2>(X, problems, N, C, kind, seed, mind2, idx_out, cs, pl.md_shared, pl.smem, false, nullptr, status, st);
}

// Start indices [problems, C] of every problem; mind2 is scratch of kmeanspp_ws_floats(problems, N) floats.
int kmeanspp(int dtype, const void* X, int problems, int N, int D, int C, int kind, uint64_t seed, float* mind2,
             int32_t* idx_out, int* status, cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  if (dtype == MUSE_F32) {
    if (D == 64) return kmeanspp_t<float, 64>((const float*)X, problems, N, C, kind, seed, mind2, idx_out, status, st);
    return kmeanspp_t<float, 128>((const float*)X, problems, N, C, kind, seed, mind2, idx_out, status, st);
  }
  if (D == 64) return kmeanspp_t<bf, 64>((const bf*)X, problems, N, C, kind, seed, mind2, idx_out, status, st);
  return kmeanspp_t<bf, 128>((const bf*)X, problems, N, C, kind, seed, mind2, idx_out, status, st);
}

}  // namespace muse
