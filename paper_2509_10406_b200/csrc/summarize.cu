// Summaries stage: bucket keys by (cluster, block), then build the exclusive causal
// accumulation of the exponentially tilted per-block summaries (Section "Summary Computation
// and Causal Accumulation", Eq. 3-5; Algorithm 1 "Causal accumulation along spatial axis").
#include "common.cuh"


namespace muse {

bool summarize_tc_supported(const Dims& d, int dtype);
int summarize_tc(const Dims& d, const void* Kp, const void* Vp, const int32_t* off_k, const float* qbar, const SummPtrs& sp,
                 int per_block, void* qsplit, int* status, cudaStream_t stream);

SummLayout summ_layout(const Dims& d, int dtype) {
  const size_t es = dtype == MUSE_F32 ? 4 : 2;
  const size_t ent = (size_t)d.B * d.Hq * d.SB * d.Cq * d.Ck;
  auto up = [](size_t x) { return (x + 255) & ~size_t(255); };
  SummLayout L;
  L.mu = 0;
  L.beta = up(L.mu + ent * sizeof(float));
  L.khi = up(L.beta + ent * sizeof(float));
  L.klo = up(L.khi + ent * d.D * es);
  L.nu = dtype == MUSE_F32 ? L.klo : up(L.klo + ent * d.D * es);
  L.Kp = up(L.nu + ent * d.D * es);
  L.Vp = up(L.Kp + (size_t)d.B * d.Hkv * d.N * d.D * es);
  L.cbar = up(L.Vp + (size_t)d.B * d.Hkv * d.N * d.D * es);
  // dipole: merged matrices (fp32 next to retrieval, where retrieved clusters are subtracted from them), then the
  // shared covariances (per kv head; per query head when tilted), the centroid weights and the sums of the weights
  const size_t ecb = d.m > 0 ? 4 : es, covh = d.dipole == 2 ? d.Hq : d.Hkv;
  L.cov = up(L.cbar + (d.dipole ? (size_t)d.B * d.Hq * d.SB * d.Cq * d.D * d.D * ecb : 0));
  L.pw = up(L.cov + (d.dipole ? (size_t)d.B * covh * d.SB * d.Ck * d.D * d.D * es : 0));
  L.zall = up(L.pw + (d.dipole ? ent * es : 0));
  L.qstar = up(L.zall + (d.dipole ? (size_t)d.B * d.Hq * d.SB * d.Cq * sizeof(float) : 0));
  L.blk = up(L.qstar + (d.dipole == 2 ? (size_t)d.B * d.Hq * d.D * sizeof(float) : 0));
  L.blk_beta = L.blk_khi = L.blk_klo = L.blk_nu = L.blk;
  L.total = L.blk;
  if (d.k2 > 0) {                                       // per-block summaries beside the accumulated ones
    L.blk_beta = up(L.blk + ent * sizeof(float));
    L.blk_khi = up(L.blk_beta + ent * sizeof(float));
    L.blk_klo = up(L.blk_khi + ent * d.D * es);
    L.blk_nu = dtype == MUSE_F32 ? L.blk_klo : up(L.blk_klo + ent * d.D * es);
    L.total = up(L.blk_nu + ent * d.D * es);
  }
  return L;
}

// out[p] = in[perm[p]] for whole rows of D elements (16 bytes per thread).
template <class T>
__global__ void k_gather_rows(const T* __restrict__ in, const int32_t* __restrict__ perm, int N, int D,
                              T* __restrict__ out) {
  const int vpr = D * (int)sizeof(T) / 16;           // 16-byte vectors per row
  const int prob = blockIdx.y;
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= (long long)N * vpr) return;
  const int p = (int)(e / vpr), v = (int)(e % vpr);
  const int t = perm[(size_t)prob * N + p];
  if (!MUSE_IN_RANGE(t, N)) return;
  const uint4* src = reinterpret_cast<const uint4*>(in + ((size_t)prob * N + t) * D);
  uint4* dst = reinterpret_cast<uint4*>(out + ((size_t)prob * N + p) * D);
  dst[v] = src[v];
}

// Untilted per-bucket statistics (Section "Summary Computation": the zero-tilt case of Eq. 3-5):
// counts n_jb and the plain sums of the keys and of the values of bucket (j, b).  One warp per
// bucket walks its rows of the bucketed copies in order (fixed summation order).
template <class T, int D>
__global__ void k_bucket_sums(const T* __restrict__ Kp, const T* __restrict__ Vp, const int32_t* __restrict__ off_k, int N,
                              int nbuckets, int32_t* __restrict__ counts, float* __restrict__ ksum, float* __restrict__ vsum) {
  const int prob = blockIdx.y, lane = threadIdx.x & 31;
  const int bk = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (bk >= nbuckets) return;
  const int32_t* o = off_k + (size_t)prob * (nbuckets + 1) + bk;
  const int p0 = o[0], p1 = MUSE_IN_RANGE(o[1], N + 1) && MUSE_IN_RANGE(o[0], o[1] + 1) ? o[1] : o[0];
  constexpr int EPL = D / 32;
  float ak[EPL], av[EPL];
#pragma unroll
  for (int k = 0; k < EPL; ++k) ak[k] = av[k] = 0.f;
  for (int p = p0; p < p1; ++p) {
    float x[EPL], y[EPL];
    ldv<EPL>(Kp + ((size_t)prob * N + p) * D + lane * EPL, x);
    ldv<EPL>(Vp + ((size_t)prob * N + p) * D + lane * EPL, y);
#pragma unroll
    for (int k = 0; k < EPL; ++k) { ak[k] += x[k]; av[k] += y[k]; }
  }
  const size_t e = (size_t)prob * nbuckets + bk;
  stv<EPL>(ksum + e * D + lane * EPL, ak);
  stv<EPL>(vsum + e * D + lane * EPL, av);
  if (lane == 0) counts[e] = p1 - p0;
}

// One CTA = (key cluster j, tile of 64 query clusters, query head).  It walks the cluster's
// buckets in block order, keeping for each query centroid i a running (max, mass, weighted
// sums of [k|v]) exactly like an online softmax, and emits a normalised snapshot after each
// bucket: the snapshot after bucket b is the accumulated summary seen by queries of block b+1.
constexpr int kSumI = 64, kSumKC = 16, kSumThreads = 256;

template <class T, int D>
__global__ void __launch_bounds__(kSumThreads)
k_summarize(Dims dm, const T* __restrict__ Kp, const T* __restrict__ Vp, const int32_t* __restrict__ off_k,
            const float* __restrict__ qbar, SummPtrs sp, int per_block) {
  constexpr int LDQ = D + 4, LDKV = 2 * D + 4, LDL = kSumKC + 1, NV = 2 * D / 32;
  extern __shared__ float smf[];
  float* qb = smf;                         // [64][LDQ]  sigma * qbar tile
  float* kv = qb + kSumI * LDQ;            // [KC][LDKV] rows [k | v]
  float* Ls = kv + kSumKC * LDKV;          // [64][LDL]  tilt logits
  const int j = blockIdx.x, i0 = blockIdx.y * kSumI, pq = blockIdx.z;
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int tid = threadIdx.x;
  const float* qsrc = qbar + (size_t)pq * dm.Cq * D;
  for (int e = tid; e < kSumI * (D / 4); e += kSumThreads) {
    int r = e / (D / 4), q = e % (D / 4);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i0 + r < dm.Cq) v = ld4(qsrc + (size_t)(i0 + r) * D + q * 4);
    v.x *= dm.sigma; v.y *= dm.sigma; v.z *= dm.sigma; v.w *= dm.sigma;
    st4(qb + r * LDQ + q * 4, v);
  }
  const int32_t* off = off_k + (size_t)pk * (dm.Ck * dm.S + 1) + (size_t)j * dm.S;
  const T* Kb = Kp + (size_t)pk * dm.N * D;
  const T* Vb = Vp + (size_t)pk * dm.N * D;
  const int ip = tid >> 3, sl = tid & 7;           // phase 2: i pair, dim slice
  const int li = tid >> 2, ug = tid & 3;           // phase 1: i, group of 4 keys
  float acc[2][NV][4];
  float M[2] = {-INFINITY, -INFINITY}, s[2] = {0.f, 0.f};
#pragma unroll
  for (int a = 0; a < 2; ++a)
#pragma unroll
    for (int k = 0; k < NV; ++k)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[a][k][c] = 0.f;

  for (int b = 0; b < dm.SB; ++b) {
    const int p0 = off[b], p1 = off[b + 1];
    if (per_block) {                                    // the summary of block b alone: the running state starts afresh
#pragma unroll
      for (int a = 0; a < 2; ++a) {
        M[a] = -INFINITY; s[a] = 0.f;
#pragma unroll
        for (int k = 0; k < NV; ++k)
#pragma unroll
          for (int c = 0; c < 4; ++c) acc[a][k][c] = 0.f;
      }
    }
    for (int c0 = p0; c0 < p1; c0 += kSumKC) {
      const int n = min(kSumKC, p1 - c0);
      __syncthreads();
      for (int e = tid; e < n * (2 * D / 4); e += kSumThreads) {
        int r = e / (2 * D / 4), q = e % (2 * D / 4);
        float4 v = q < D / 4 ? ld4(Kb + (size_t)(c0 + r) * D + q * 4)
                             : ld4(Vb + (size_t)(c0 + r) * D + (q - D / 4) * 4);
        st4(kv + r * LDKV + q * 4, v);
      }
      __syncthreads();
      {
        float dot[4] = {0.f, 0.f, 0.f, 0.f};
        if (ug * 4 < n) {
#pragma unroll 4
          for (int dd = 0; dd < D; dd += 4) {
            float4 qv = ld4(qb + li * LDQ + dd);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              float4 kk = ld4(kv + (ug * 4 + u) * LDKV + dd);   // rows >= n hold stale finite data; unused
              dot[u] = fmaf(qv.x, kk.x, dot[u]); dot[u] = fmaf(qv.y, kk.y, dot[u]);
              dot[u] = fmaf(qv.z, kk.z, dot[u]); dot[u] = fmaf(qv.w, kk.w, dot[u]);
            }
          }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) Ls[li * LDL + ug * 4 + u] = dot[u];
      }
      __syncthreads();
#pragma unroll
      for (int a = 0; a < 2; ++a) {
        const float* Lr = Ls + (ip * 2 + a) * LDL;
        float cm = -INFINITY;
        for (int u = 0; u < n; ++u) cm = fmaxf(cm, Lr[u]);
        const float Mn = fmaxf(M[a], cm);
        const float sc = expf(M[a] - Mn);            // exp(-inf) = 0 on the first keys
        M[a] = Mn; s[a] *= sc;
#pragma unroll
        for (int k = 0; k < NV; ++k)
#pragma unroll
          for (int c = 0; c < 4; ++c) acc[a][k][c] *= sc;
        for (int u = 0; u < n; ++u) {
          const float w = expf(Lr[u] - Mn);
          s[a] += w;
#pragma unroll
          for (int k = 0; k < NV; ++k) {
            float4 x = ld4(kv + u * LDKV + sl * 4 + 32 * k);
            acc[a][k][0] = fmaf(w, x.x, acc[a][k][0]); acc[a][k][1] = fmaf(w, x.y, acc[a][k][1]);
            acc[a][k][2] = fmaf(w, x.z, acc[a][k][2]); acc[a][k][3] = fmaf(w, x.w, acc[a][k][3]);
          }
        }
      }
    }
    // snapshot -> plane b
#pragma unroll
    for (int a = 0; a < 2; ++a) {
      const int i = i0 + ip * 2 + a;
      const bool live = i < dm.Cq;          // no early exit: the shuffles below need the whole warp
      const size_t ent = (((size_t)pq * dm.SB + b) * dm.Cq + i) * dm.Ck + j;
      const bool some = s[a] > 0.f;
      const float inv = some ? 1.f / s[a] : 0.f;
      // beta = mu - sigma qbar_i . kappa: partial dot over this thread's kappa dims, summed over the 8 slices
      float qk = 0.f;
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        const int c4 = sl * 4 + 32 * k;
        float4 v = make_float4(acc[a][k][0] * inv, acc[a][k][1] * inv, acc[a][k][2] * inv, acc[a][k][3] * inv);
        if (c4 < D) {
          if (live) st_kappa4<T>(sp, ent * D + c4, v);
          float4 q = ld4(qb + (ip * 2 + a) * LDQ + c4);
          qk += q.x * kappa_repr<T>(v.x) + q.y * kappa_repr<T>(v.y) + q.z * kappa_repr<T>(v.z) + q.w * kappa_repr<T>(v.w);
        } else if (live) {
          st_nu4<T>(sp, ent * D + (c4 - D), v);
        }
      }
      qk += __shfl_xor_sync(0xffffffffu, qk, 1); qk += __shfl_xor_sync(0xffffffffu, qk, 2); qk += __shfl_xor_sync(0xffffffffu, qk, 4);
      if (sl == 0 && live) {
        const float m_ = some ? M[a] + logf(s[a]) : -INFINITY;
        sp.mu[ent] = m_;
        sp.beta[ent] = some ? m_ - qk : -INFINITY;
      }
    }
  }
}

template <class T, int D>
static int summarize_planes(const Dims& d, int dtype, const T* Kp, const T* Vp, const int32_t* off_k, const float* qbar,
                            const SummPtrs& sp, int per_block, void* qsplit, int32_t* status, cudaStream_t st);

// assign_k == nullptr: off_k and perm_k are inputs (the keys are already bucketed: the backward pass
// rebuilding the summaries it was not given); `status` then points at the caller's status words.
template <class T, int D>
static int summarize_t(const Dims& d, int dtype, const T* K, const T* V, const int32_t* assign_k,
                       const float* qbar, int32_t* off_k, int32_t* perm_k, int32_t* counts, float* ksum, float* vsum,
                       void* summaries, void* ws, int32_t* status_in, cudaStream_t st) {
  const int pk = d.B * d.Hkv;
  Arena ar(ws);
  int32_t* status = ar.take<int32_t>(kStatusWords);      // cleared by the entry point
  if (status_in != nullptr) status = status_in;
  int32_t* sort_scratch = ar.take<int32_t>(sort_ws_elems(d.N, d.Ck * d.S) * (size_t)pk);
  int rc = MUSE_OK;
  if (assign_k != nullptr) rc = bucket_sort(0, assign_k, pk, d.N, d.Ck, d.S, d.Bs, 1, off_k, perm_k, sort_scratch, st);
  if (rc != MUSE_OK) return rc;
  SummLayout L = summ_layout(d, dtype);
  char* base = (char*)summaries;
  T* Kp = (T*)(base + L.Kp); T* Vp = (T*)(base + L.Vp);
  const int vpr = D * (int)sizeof(T) / 16;
  dim3 gg(cdiv(d.N * vpr, 256), pk);
  prof_mark("k_gather_rows", st);
  k_gather_rows<T><<<gg, 256, 0, st>>>(K, perm_k, d.N, D, Kp);
  MUSE_LAUNCH_OK();
  prof_mark("k_gather_rows", st);
  k_gather_rows<T><<<gg, 256, 0, st>>>(V, perm_k, d.N, D, Vp);
  MUSE_LAUNCH_OK();
  if (counts != nullptr) {
    prof_mark("k_bucket_sums", st);
    k_bucket_sums<T, D><<<dim3(cdiv(d.Ck * d.S, 8), pk), 256, 0, st>>>(Kp, Vp, off_k, d.N, d.Ck * d.S, counts, ksum, vsum);
    MUSE_LAUNCH_OK();
  }
  if (d.SB == 0) return MUSE_OK;
  void* qsplit = ar.take<__nv_bfloat16>(2 * (size_t)d.B * d.Hq * d.Cq * d.D);   // split centroids for the tensor kernel
  rc = summarize_planes<T, D>(d, dtype, Kp, Vp, off_k, qbar, summ_ptrs(L, base), 0, qsplit, status, st);
  if (rc == MUSE_OK && d.k2 > 0) rc = summarize_planes<T, D>(d, dtype, Kp, Vp, off_k, qbar, summ_ptrs_blk(L, base), 1, qsplit, status, st);
  if (rc != MUSE_OK || !d.dipole || d.SB == 0) return rc;     // one causal block: no far field, nothing to correct
  return dipole_build(d, dtype, Kp, Vp, off_k, summ_ptrs(L, base).mu, dipole_ptrs(L, base), status, st);
}

template <class T, int D>
static int summarize_planes(const Dims& d, int dtype, const T* Kp, const T* Vp, const int32_t* off_k, const float* qbar,
                            const SummPtrs& sp, int per_block, void* qsplit, int32_t* status, cudaStream_t st) {
  if (summarize_tc_supported(d, dtype) && !path_forced(kForceSummFwdSimt))
    return summarize_tc(d, Kp, Vp, off_k, qbar, sp, per_block, qsplit, status, st);
  const size_t smem = (size_t)(kSumI * (D + 4) + kSumKC * (2 * D + 4) + kSumI * (kSumKC + 1)) * sizeof(float);
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_summarize<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  dim3 grid(d.Ck, cdiv(d.Cq, kSumI), d.B * d.Hq);
  prof_mark("k_summarize", st);
  k_summarize<T, D><<<grid, kSumThreads, smem, st>>>(d, Kp, Vp, off_k, qbar, sp, per_block);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

size_t summarize_ws_bytes(const Dims& d, int dtype) {
  Arena ar(nullptr);
  ar.take<int32_t>(kStatusWords);
  ar.take<int32_t>((size_t)d.B * d.Hkv * sort_ws_elems(d.N, d.Ck * d.S));
  ar.take<__nv_bfloat16>(2 * (size_t)d.B * d.Hq * d.Cq * d.D);
  return ar.used;
}

int summarize(const Dims& d, int dtype, const void* K, const void* V, const int32_t* assign_k,
              const float* qbar, int32_t* off_k, int32_t* perm_k, int32_t* counts, float* ksum, float* vsum,
              void* summaries, void* ws, int32_t* status, cudaStream_t st) {
  if (dtype == MUSE_F32) {
    if (d.D == 64) return summarize_t<float, 64>(d, dtype, (const float*)K, (const float*)V, assign_k, qbar, off_k, perm_k, counts, ksum, vsum, summaries, ws, status, st);
    return summarize_t<float, 128>(d, dtype, (const float*)K, (const float*)V, assign_k, qbar, off_k, perm_k, counts, ksum, vsum, summaries, ws, status, st);
  }
  typedef __nv_bfloat16 bf;
  if (d.D == 64) return summarize_t<bf, 64>(d, dtype, (const bf*)K, (const bf*)V, assign_k, qbar, off_k, perm_k, counts, ksum, vsum, summaries, ws, status, st);
  return summarize_t<bf, 128>(d, dtype, (const bf*)K, (const bf*)V, assign_k, qbar, off_k, perm_k, counts, ksum, vsum, summaries, ws, status, st);
}

}  // namespace muse
