// Dipole correction of the far field (Appendix "Error Analysis": "Dipole Correction" and
// "Untilted (Partially Specialized) Covariances").  Three steps at summary time and one per query:
//   1. Cov_0jb(v,k): shared, untilted cross-covariance of values and keys over the keys of
//      cluster j in blocks before b (one D x D matrix per key cluster and plane)
//   2. p_ib(j) = softmax_j of the accumulated log-masses (the monopole's own centroid weights)
//   3. Cbar_ib = sum_j p_ib(j) Cov_0jb   -- one GEMM [Cq x Ck] x [Ck x D^2] per (head, plane);
//      tcgen05 kernel in dipole_tc.cu, plain kernel here for fp32 mode and odd shapes
//   4. o_far_t += Cbar_ib * sigma (q_t - qbar_i)   (value shift only; the mass is unchanged)
#include "common.cuh"


namespace muse {

bool dipole_merge_tc_supported(const Dims& d, int dtype);
int dipole_merge_tc(const Dims& d, const void* P, const void* cov, void* cbar, int* status, cudaStream_t st);

// ---- 1. untilted accumulated covariance ------------------------------------------------------
// One CTA per (key cluster j, kv head): walks the cluster's buckets in block order with running
// raw moments (sum v k'^T, sum v, sum k', n) and writes the centred covariance after each bucket;
// k' = k - (first key of the cluster), which leaves the covariance unchanged and keeps the raw
// moments small.  Thread (ty, tx) owns a TV x TV sub-block: value dims ty*TV.., key dims tx*TV...
constexpr int kCovKeys = 8;

template <class T, class ST, int D>
__global__ void __launch_bounds__(256)
k_dipole_cov(Dims dm, const T* __restrict__ Kp, const T* __restrict__ Vp, const int32_t* __restrict__ off_k,
             ST* __restrict__ cov) {
  constexpr int TV = D / 16;
  __shared__ float ks[kCovKeys][D], vs[kCovKeys][D], k0[D];
  const int j = blockIdx.x, pk = blockIdx.y, tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int32_t* off = off_k + (size_t)pk * (dm.Ck * dm.S + 1) + (size_t)j * dm.S;
  const T* Kb = Kp + (size_t)pk * dm.N * D;
  const T* Vb = Vp + (size_t)pk * dm.N * D;
  const int first = off[0];
  if (tid < D) k0[tid] = first < off[dm.S] ? to_f(Kb[(size_t)first * D + tid]) : 0.f;
  float A[TV][TV], sv[TV], sk[TV];
#pragma unroll
  for (int a = 0; a < TV; ++a) {
    sv[a] = 0.f; sk[a] = 0.f;
#pragma unroll
    for (int c = 0; c < TV; ++c) A[a][c] = 0.f;
  }
  int n = 0;
  __syncthreads();
  for (int pl = 0; pl < dm.SB; ++pl) {
    const int u0 = off[pl], u1 = off[pl + 1];
    for (int c0 = u0; c0 < u1; c0 += kCovKeys) {
      const int nk = min(kCovKeys, u1 - c0);
      __syncthreads();
      for (int e = tid; e < kCovKeys * (D / 4); e += 256) {
        const int r = e / (D / 4), q = e % (D / 4);
        if (r < nk) {
          float4 kk = ld4(Kb + (size_t)(c0 + r) * D + q * 4), vv = ld4(Vb + (size_t)(c0 + r) * D + q * 4);
          kk.x -= k0[q * 4]; kk.y -= k0[q * 4 + 1]; kk.z -= k0[q * 4 + 2]; kk.w -= k0[q * 4 + 3];
          st4(&ks[r][q * 4], kk); st4(&vs[r][q * 4], vv);
        }
      }
      __syncthreads();
      for (int r = 0; r < nk; ++r) {
        float kv_[TV], vv_[TV];
#pragma unroll
        for (int a = 0; a < TV; ++a) { kv_[a] = ks[r][tx * TV + a]; vv_[a] = vs[r][ty * TV + a]; }
#pragma unroll
        for (int a = 0; a < TV; ++a) {
          sv[a] += vv_[a]; sk[a] += kv_[a];
#pragma unroll
          for (int c = 0; c < TV; ++c) A[a][c] = fmaf(vv_[a], kv_[c], A[a][c]);
        }
      }
      n += nk;
    }
    // centred covariance of everything seen so far = what queries of block pl + 1 see
    const float inv = n > 0 ? 1.f / (float)n : 0.f;
    ST* out = cov + (((size_t)pk * dm.SB + pl) * dm.Ck + j) * D * D;
#pragma unroll
    for (int a = 0; a < TV; ++a) {
      const float vm = sv[a] * inv;
#pragma unroll
      for (int c = 0; c < TV; c += 4) {
        float4 o = make_float4(A[a][c] * inv - vm * sk[c] * inv, A[a][c + 1] * inv - vm * sk[c + 1] * inv,
                               A[a][c + 2] * inv - vm * sk[c + 2] * inv, A[a][c + 3] * inv - vm * sk[c + 3] * inv);
        st4(out + (size_t)(ty * TV + a) * D + tx * TV + c, o);
      }
    }
  }
}

// ---- 2. merge weights: one warp per (head, plane, query cluster) row of log-masses ---------------
template <class ST>
__global__ void k_dipole_weights(const float* __restrict__ mu, long long rows, int Ck, ST* __restrict__ P) {
  const long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const float* mr = mu + row * Ck;
  float mx = -INFINITY;
  for (int j = lane; j < Ck; j += 32) mx = fmaxf(mx, mr[j]);
  mx = warp_max(mx);
  float s = 0.f;
  if (mx != -INFINITY)
    for (int j = lane; j < Ck; j += 32) s += expf(mr[j] - mx);
  s = warp_sum(s);
  const float inv = s > 0.f ? 1.f / s : 0.f;
  for (int j = lane; j < Ck; j += 32) P[row * Ck + j] = from_f<ST>(mx == -INFINITY ? 0.f : expf(mr[j] - mx) * inv);
}

// ---- 3. merge, plain version: thread = one of 256 columns of the D*D axis, 16 query clusters ------
constexpr int kMrgI = 16, kMrgJ = 64;

template <class ST>
__global__ void __launch_bounds__(256)
k_dipole_merge(Dims dm, const ST* __restrict__ P, const ST* __restrict__ cov, ST* __restrict__ cbar) {
  __shared__ float ps[kMrgI][kMrgJ];
  const int DD = dm.D * dm.D;
  const int x = blockIdx.x * 256 + threadIdx.x, i0 = blockIdx.y * kMrgI;
  const int pp = blockIdx.z, pq = pp / dm.SB, pl = pp % dm.SB;
  const int pk = (pq / dm.Hq) * dm.Hkv + dm.hm.g[pq % dm.Hq];
  const ST* Pb = P + ((size_t)pp * dm.Cq) * dm.Ck;
  const ST* cb = cov + (((size_t)pk * dm.SB + pl) * dm.Ck) * DD;
  float acc[kMrgI];
#pragma unroll
  for (int a = 0; a < kMrgI; ++a) acc[a] = 0.f;
  for (int j0 = 0; j0 < dm.Ck; j0 += kMrgJ) {
    __syncthreads();
    for (int e = threadIdx.x; e < kMrgI * kMrgJ; e += 256) {
      const int a = e / kMrgJ, jj = e % kMrgJ;
      ps[a][jj] = (i0 + a < dm.Cq && j0 + jj < dm.Ck) ? to_f(Pb[(size_t)(i0 + a) * dm.Ck + j0 + jj]) : 0.f;
    }
    __syncthreads();
    const int nj = min(kMrgJ, dm.Ck - j0);
    for (int jj = 0; jj < nj; ++jj) {
      const float c = to_f(cb[(size_t)(j0 + jj) * DD + x]);
#pragma unroll
      for (int a = 0; a < kMrgI; ++a) acc[a] = fmaf(ps[a][jj], c, acc[a]);
    }
  }
#pragma unroll
  for (int a = 0; a < kMrgI; ++a)
    if (i0 + a < dm.Cq) cbar[((size_t)pp * dm.Cq + i0 + a) * DD + x] = from_f<ST>(acc[a]);
}

// ---- 4. consumption: one CTA per (query cluster, plane, head) segment ------------------------------
constexpr int kApplyQ = 8;

template <class T, class ST, int D>
__global__ void __launch_bounds__(256)
k_dipole_apply(Dims dm, const T* __restrict__ Q, const float* __restrict__ qbar, const int32_t* __restrict__ off_q,
               const int32_t* __restrict__ perm_q, const ST* __restrict__ cbar, const float* __restrict__ lse_far,
               float* __restrict__ o_far) {
  extern __shared__ float smd[];
  float* Ct = smd;                              // [D key dims][D + 1]: transposed matrix, value dim fastest
  float* qs = Ct + D * (D + 1);                 // [2 * kApplyQ][D] residuals
  const int i = blockIdx.x, pl = blockIdx.y, pq = blockIdx.z, tid = threadIdx.x;
  const int blk = dm.causal ? pl + 1 : 0;
  const int32_t* oq = off_q + (size_t)pq * (dm.S * dm.Cq + 1) + (size_t)blk * dm.Cq + i;
  const int p0 = oq[0], p1 = oq[1];
  if (p0 >= p1) return;
  const ST* cb = cbar + (((size_t)pq * dm.SB + pl) * dm.Cq + i) * D * D;
  for (int e = tid; e < D * D / 4; e += 256) {
    const int dv = e / (D / 4), c4 = (e % (D / 4)) * 4;
    const float4 v = ld4(cb + (size_t)dv * D + c4);
    Ct[(c4 + 0) * (D + 1) + dv] = v.x; Ct[(c4 + 1) * (D + 1) + dv] = v.y;
    Ct[(c4 + 2) * (D + 1) + dv] = v.z; Ct[(c4 + 3) * (D + 1) + dv] = v.w;
  }
  const float* qb = qbar + ((size_t)pq * dm.Cq + i) * D;
  const T* Qp = Q + (size_t)pq * dm.N * D;
  const int32_t* pm = perm_q + (size_t)pq * dm.N;
  constexpr int G = 256 / D;                    // query groups working side by side (2 or 4)
  const int grp = tid / D, dv = tid % D;
  for (int r0 = p0; r0 < p1; r0 += G * kApplyQ) {
    __syncthreads();
    for (int e = tid; e < G * kApplyQ * D; e += 256) {
      const int r = e / D, dk = e % D;
      qs[e] = r0 + r < p1 ? dm.sigma * (to_f(Qp[(size_t)pm[r0 + r] * D + dk]) - qb[dk]) : 0.f;
    }
    __syncthreads();
    float acc[kApplyQ];
#pragma unroll
    for (int a = 0; a < kApplyQ; ++a) acc[a] = 0.f;
    const float* qg = qs + grp * kApplyQ * D;
    for (int dk = 0; dk < D; ++dk) {
      const float c = Ct[dk * (D + 1) + dv];
#pragma unroll
      for (int a = 0; a < kApplyQ; ++a) acc[a] = fmaf(c, qg[a * D + dk], acc[a]);
    }
#pragma unroll
    for (int a = 0; a < kApplyQ; ++a) {
      const int r = r0 + grp * kApplyQ + a;
      if (r < p1) {
        const size_t t = (size_t)pq * dm.N + pm[r];
        if (lse_far[t] != -INFINITY) o_far[t * D + dv] += acc[a];
      }
    }
  }
}

// ---- host side ------------------------------------------------------------------------------------
size_t dipole_ws_bytes(const Dims& d, int dtype) {
  if (!d.dipole || d.SB == 0) return 0;
  const size_t es = dtype == MUSE_F32 ? 4 : 2;
  Arena ar(nullptr);
  ar.take<char>((size_t)d.B * d.Hkv * d.SB * d.Ck * d.D * d.D * es);
  ar.take<char>((size_t)d.B * d.Hq * d.SB * d.Cq * d.Ck * es);
  return ar.used;
}

template <class T, class ST, int D>
static int dipole_build_t(const Dims& d, int dtype, const T* Kp, const T* Vp, const int32_t* off_k, const float* mu,
                          ST* cbar, void* ws, int* status, cudaStream_t st) {
  Arena ar(ws);
  ST* cov = ar.take<ST>((size_t)d.B * d.Hkv * d.SB * d.Ck * D * D);
  ST* P = ar.take<ST>((size_t)d.B * d.Hq * d.SB * d.Cq * d.Ck);
  prof_mark("k_dipole_cov", st);
  k_dipole_cov<T, ST, D><<<dim3(d.Ck, d.B * d.Hkv), 256, 0, st>>>(d, Kp, Vp, off_k, cov);
  MUSE_LAUNCH_OK();
  const long long rows = (long long)d.B * d.Hq * d.SB * d.Cq;
  prof_mark("k_dipole_weights", st);
  k_dipole_weights<ST><<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(mu, rows, d.Ck, P);
  MUSE_LAUNCH_OK();
  if (dipole_merge_tc_supported(d, dtype) && !path_forced(kForceDipoleSimt))
    return dipole_merge_tc(d, P, cov, cbar, status, st);
  prof_mark("k_dipole_merge", st);
  k_dipole_merge<ST><<<dim3(D * D / 256, cdiv(d.Cq, kMrgI), d.B * d.Hq * d.SB), 256, 0, st>>>(d, P, cov, cbar);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

int dipole_build(const Dims& d, int dtype, const void* Kp, const void* Vp, const int32_t* off_k, const float* mu,
                 void* cbar, void* ws, int* status, cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  if (dtype == MUSE_F32) {
    if (d.D == 64) return dipole_build_t<float, float, 64>(d, dtype, (const float*)Kp, (const float*)Vp, off_k, mu, (float*)cbar, ws, status, st);
    return dipole_build_t<float, float, 128>(d, dtype, (const float*)Kp, (const float*)Vp, off_k, mu, (float*)cbar, ws, status, st);
  }
  if (d.D == 64) return dipole_build_t<bf, bf, 64>(d, dtype, (const bf*)Kp, (const bf*)Vp, off_k, mu, (bf*)cbar, ws, status, st);
  return dipole_build_t<bf, bf, 128>(d, dtype, (const bf*)Kp, (const bf*)Vp, off_k, mu, (bf*)cbar, ws, status, st);
}

template <class T, class ST, int D>
static int dipole_apply_t(const Dims& d, const T* Q, const float* qbar, const int32_t* off_q, const int32_t* perm_q,
                          const ST* cbar, const float* lse_far, float* o_far, cudaStream_t st) {
  const size_t smem = (size_t)(D * (D + 1) + (256 / D) * kApplyQ * D) * sizeof(float);
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_dipole_apply<T, ST, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  prof_mark("k_dipole_apply", st);
  k_dipole_apply<T, ST, D><<<dim3(d.Cq, d.SB, d.B * d.Hq), 256, smem, st>>>(d, Q, qbar, off_q, perm_q, cbar, lse_far, o_far);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

int dipole_apply(const Dims& d, int dtype, const void* Q, const float* qbar, const int32_t* off_q, const int32_t* perm_q,
                 const void* cbar, const float* lse_far, float* o_far, cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  if (dtype == MUSE_F32) {
    if (d.D == 64) return dipole_apply_t<float, float, 64>(d, (const float*)Q, qbar, off_q, perm_q, (const float*)cbar, lse_far, o_far, st);
    return dipole_apply_t<float, float, 128>(d, (const float*)Q, qbar, off_q, perm_q, (const float*)cbar, lse_far, o_far, st);
  }
  if (d.D == 64) return dipole_apply_t<bf, bf, 64>(d, (const bf*)Q, qbar, off_q, perm_q, (const bf*)cbar, lse_far, o_far, st);
  return dipole_apply_t<bf, bf, 128>(d, (const bf*)Q, qbar, off_q, perm_q, (const bf*)cbar, lse_far, o_far, st);
}

}  // namespace muse
