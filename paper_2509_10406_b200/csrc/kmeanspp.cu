// Seeded k-means++ start points on the GPU (an alternative to the strided start of Appendix "Centroid Computation",
// step 1; the paper does not use it).  The first start point is position 0 of the seeded shuffle; draw c = 1 .. C - 1
// picks one vector with probability proportional to d2 = its squared distance to the nearest start point so far.
// The draw is an exponential race: vector t gets u_t in (0, 1) from an integer hash of (seed, stream, c, t),
// e_t = -log(u_t), and the largest d2_t / e_t wins (lowest index on ties) -- the same law as sampling the
// cumulative sum of d2, but a maximum instead of a prefix sum, so every draw is one pass over the vectors.
//
// One problem (head, side) = one thread-block cluster of up to 8 CTAs, each owning a contiguous slice of the vectors;
// the C - 1 draws are sequential, each ends with one candidate per CTA written into every CTA's shared memory and a
// hardware cluster barrier.  A draw reads every vector once (distance to the newest start point only, the running
// minimum lives in scratch), so the stage moves (C - 1) N D e bytes per problem and is bound by L2 / HBM bandwidth.
#include <cooperative_groups.h>

#include "common.cuh"
#include "feistel.cuh"

namespace cg = cooperative_groups;

namespace muse {

constexpr int kPpThreads = 512, kPpCluster = 8, kPpWarps = kPpThreads / 32;

__device__ __forceinline__ bool pp_better(float k, int i, float bk, int bi) { return k > bk || (k == bk && i < bi); }

template <class T, int D>
__global__ void __launch_bounds__(kPpThreads)
k_kmeanspp(const T* __restrict__ X, int N, int C, uint64_t seed, int kind, float* __restrict__ mind2,
           int32_t* __restrict__ idx_out) {
  cg::cluster_group cluster = cg::this_cluster();
  const int CS = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  const int prob = blockIdx.x / CS, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  __shared__ float cs[D];
  __shared__ float exk[2][kPpCluster], wk[kPpWarps];
  __shared__ int exi[2][kPpCluster], wi[kPpWarps];
  const T* Xp = X + (size_t)prob * N * D;
  float* md = mind2 + (size_t)prob * N;
  const uint64_t stream = (uint64_t)prob * 2 + (uint64_t)kind;
  const int per = (N + CS - 1) / CS, lo = rank * per, hi = min(N, lo + per);
  constexpr int EPL = D / 8;                    // elements per lane: 8 lanes share one vector
  const int sub = lane & 7, grp = lane >> 3;
  int last = feistel_permute(0, N, seed, stream);
  if (rank == 0 && tid == 0) idx_out[(size_t)prob * C] = last;
  cluster.sync();                               // every CTA of the problem is running before any of them writes into another's shared memory
  for (int c = 1; c < C; ++c) {
    if (tid < D) cs[tid] = MUSE_IN_RANGE(last, N) ? to_f(Xp[(size_t)last * D + tid]) : 0.f;
    __syncthreads();
    float cen[EPL];
#pragma unroll
    for (int k = 0; k < EPL / 4; ++k) {
      const float4 v = *reinterpret_cast<const float4*>(&cs[k * 32 + sub * 4]);
      cen[k * 4] = v.x; cen[k * 4 + 1] = v.y; cen[k * 4 + 2] = v.z; cen[k * 4 + 3] = v.w;
    }
    const uint64_t key_c = splitmix64(seed ^ (stream << 32) ^ (0xA5ull << 56) ^ (uint64_t)c);
    float bk = -1.f; int bi = 0x7fffffff;
#pragma unroll 2
    for (int t0 = lo + warp * 4; t0 < hi; t0 += kPpWarps * 4) {
      const int t = t0 + grp;
      float d = 0.f;
      if (t < hi) {
#pragma unroll
        for (int k = 0; k < EPL / 4; ++k) {
          const float4 v = ld4(Xp + (size_t)t * D + k * 32 + sub * 4);
          const float a = v.x - cen[k * 4], b = v.y - cen[k * 4 + 1], e = v.z - cen[k * 4 + 2], f = v.w - cen[k * 4 + 3];
          d = fmaf(a, a, d); d = fmaf(b, b, d); d = fmaf(e, e, d); d = fmaf(f, f, d);
        }
      }
      d += __shfl_xor_sync(0xffffffffu, d, 1);
      d += __shfl_xor_sync(0xffffffffu, d, 2);
      d += __shfl_xor_sync(0xffffffffu, d, 4);
      if (sub == 0 && t < hi) {
        if (c > 1) d = fminf(d, md[t]);
        md[t] = d;
        const uint64_t h = splitmix64(key_c ^ (uint64_t)t);
        const float u = ((float)(uint32_t)(h >> 41) + 0.5f) * (1.f / 8388608.f);
        const float key = d / -logf(u);
        if (pp_better(key, t, bk, bi)) { bk = key; bi = t; }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ok = __shfl_xor_sync(0xffffffffu, bk, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (pp_better(ok, oi, bk, bi)) { bk = ok; bi = oi; }
    }
    if (lane == 0) { wk[warp] = bk; wi[warp] = bi; }
    __syncthreads();
    const int par = c & 1;
    if (warp == 0) {
      bk = lane < kPpWarps ? wk[lane] : -1.f; bi = lane < kPpWarps ? wi[lane] : 0x7fffffff;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ok = __shfl_xor_sync(0xffffffffu, bk, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (pp_better(ok, oi, bk, bi)) { bk = ok; bi = oi; }
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
    last = bi;
    if (rank == 0 && tid == 0) idx_out[(size_t)prob * C + c] = last;
  }
  cluster.sync();                               // no CTA leaves while another may still write into its shared memory
}

size_t kmeanspp_ws_floats(int problems, int N) { return (size_t)problems * N; }

template <class T, int D>
static int kmeanspp_t(const T* X, int problems, int N, int C, int kind, uint64_t seed, float* mind2, int32_t* idx_out,
                      cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cfg.stream = st;
  // CTAs per problem: as many as keep a slice of at least 1024 vectors, up to 8
  int cs = 1;
  while (cs < kPpCluster && N >= 2048 * cs) cs *= 2;
  cfg.gridDim = dim3(problems * cs);
  cfg.blockDim = dim3(kPpThreads);
  cfg.dynamicSmemBytes = 0;
  attr[0].val.clusterDim.x = cs;
  prof_mark("k_kmeanspp", st);
  MUSE_CUDA_OK(cudaLaunchKernelEx(&cfg, k_kmeanspp<T, D>, X, N, C, seed, kind, mind2, idx_out));
  return MUSE_OK;
}

// Start indices [problems, C] of every problem; mind2 is scratch of kmeanspp_ws_floats(problems, N) floats.
int kmeanspp(int dtype, const void* X, int problems, int N, int D, int C, int kind, uint64_t seed, float* mind2,
             int32_t* idx_out, cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  if (dtype == MUSE_F32) {
    if (D == 64) return kmeanspp_t<float, 64>((const float*)X, problems, N, C, kind, seed, mind2, idx_out, st);
    return kmeanspp_t<float, 128>((const float*)X, problems, N, C, kind, seed, mind2, idx_out, st);
  }
  if (D == 64) return kmeanspp_t<bf, 64>((const bf*)X, problems, N, C, kind, seed, mind2, idx_out, st);
  return kmeanspp_t<bf, 128>((const bf*)X, problems, N, C, kind, seed, mind2, idx_out, st);
}

}  // namespace muse
