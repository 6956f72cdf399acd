// Dipole correction of the far field (Appendix "Error Analysis": "Dipole Correction" and
// "Untilted (Partially Specialized) Covariances").  Three steps at summary time and one per query:
//   1. Cov_0jb(v,k): shared, untilted cross-covariance of values and keys over the keys of
//      cluster j in blocks before b (one D x D matrix per key cluster and plane)
//   2. p_ib(j) = softmax_j of the accumulated log-masses (the monopole's own centroid weights)
//   3. Cbar_ib = sum_j p_ib(j) Cov_0jb   -- one GEMM [Cq x Ck] x [Ck x D^2] per (head, plane);
//      tcgen05 kernel in dipole_tc.cu, plain kernel here for fp32 mode and odd shapes
//   4. o_far_t += Cbar_ib * sigma (q_t - qbar_i)   (value shift only; the mass is unchanged)
// Next to retrieval (m > 0; Appendix "Compatibility with Retrieval") the clusters a query retrieved are attended
// exactly, so their share leaves the merged matrix and the centroid weights are renormalised over the rest:
//   c_t = (Cbar_ib qres_t - sum_{j in sel_t} p_ib(j) Cov_0jb qres_t) / (sum_j p_ib(j) - sum_{j in sel_t} p_ib(j)).
// The subtraction only cancels cleanly if both sides hold the same numbers, so in this mode Cbar is kept in fp32
// (the fp32 accumulation of exactly the stored, rounded weights and covariances) and the weight sums are taken
// over the stored weights.  The retrieved clusters' terms are computed per (cluster, plane) group of the
// retrieval's inverse index (one covariance in shared memory, its (query, slot) pairs streamed) and added
// into a per-query row with floating-point atomics.
#include "common.cuh"


namespace muse {

bool dipole_merge_tc_supported(const Dims& d, int dtype);
int dipole_merge_tc(const Dims& d, const void* P, const void* cov, void* cbar, int out_f32, int* status, cudaStream_t st);
bool dipole_sub_tc_supported(const Dims& d, int dtype);
int dipole_sub_tc(const Dims& d, const void* Q, const float* qbar, const int32_t* assign_q, const int32_t* goff, const int32_t* pairs,
                  const void* cov, const void* pw, float* csub, int* status, cudaStream_t st);

// ---- 1. untilted accumulated covariance ------------------------------------------------------
// One CTA per (key cluster j, kv head): walks the cluster's buckets in block order with running
// raw moments (sum v k'^T, sum v, sum k', n) and writes the centred covariance after each bucket;
// k' = k - (first key of the cluster), which leaves the covariance unchanged and keeps the raw
// moments small.  Thread (ty, tx) owns a TV x TV sub-block: value dims ty*TV.., key dims tx*TV...
constexpr int kCovKeys = 8;

// TILT (dipole == 2): one covariance set per QUERY head, its members weighted by w_u ~ exp(sigma qstar . k_u) with
// qstar the head's shared tilt point; the weights are carried relative to a running maximum of the logits and all
// running moments are rescaled when it grows.
template <class T, class ST, int D, bool TILT>
__global__ void __launch_bounds__(256)
k_dipole_cov(Dims dm, const T* __restrict__ Kp, const T* __restrict__ Vp, const int32_t* __restrict__ off_k,
             const float* __restrict__ qstar, ST* __restrict__ cov) {
  constexpr int TV = D / 16;
  __shared__ float ks[kCovKeys][D], vs[kCovKeys][D], k0[D], qs_[D], wl[kCovKeys];
  const int j = blockIdx.x, pc = blockIdx.y, tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int pk = TILT ? (pc / dm.Hq) * dm.Hkv + dm.hm.g[pc % dm.Hq] : pc;
  const int32_t* off = off_k + (size_t)pk * (dm.Ck * dm.S + 1) + (size_t)j * dm.S;
  const T* Kb = Kp + (size_t)pk * dm.N * D;
  const T* Vb = Vp + (size_t)pk * dm.N * D;
  const int first = off[0];
  if (tid < D) {
    k0[tid] = first < off[dm.S] ? to_f(Kb[(size_t)first * D + tid]) : 0.f;
    qs_[tid] = TILT ? dm.sigma * qstar[(size_t)pc * D + tid] : 0.f;
  }
  float A[TV][TV], sv[TV], sk[TV];
  float wsum = 0.f, wmax = -INFINITY;             // TILT: sum of the weights, and the logit they are relative to
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
      if (TILT) {
        // logits of the chunk's keys (shifted keys: a constant per cluster, which cancels in the normalised weights)
        const int wq = tid >> 5, ln = tid & 31;
        float l = 0.f;
        if (wq < nk)
          for (int c = ln; c < D; c += 32) l = fmaf(qs_[c], ks[wq][c], l);
        l = warp_sum(l);
        if (ln == 0) wl[wq] = wq < nk ? l : -INFINITY;
        __syncthreads();
        float mx = wmax;
        for (int r = 0; r < nk; ++r) mx = fmaxf(mx, wl[r]);
        if (mx > wmax) {
          const float f = wmax == -INFINITY ? 0.f : expf(wmax - mx);
          wsum *= f;
#pragma unroll
          for (int a = 0; a < TV; ++a) {
            sv[a] *= f; sk[a] *= f;
#pragma unroll
            for (int c = 0; c < TV; ++c) A[a][c] *= f;
          }
          wmax = mx;
        }
      }
      for (int r = 0; r < nk; ++r) {
        const float wr = TILT ? expf(wl[r] - wmax) : 1.f;
        float kv_[TV], vv_[TV];
#pragma unroll
        for (int a = 0; a < TV; ++a) { kv_[a] = ks[r][tx * TV + a]; vv_[a] = wr * vs[r][ty * TV + a]; }
#pragma unroll
        for (int a = 0; a < TV; ++a) {
          sv[a] += vv_[a]; sk[a] = fmaf(wr, kv_[a], sk[a]);
#pragma unroll
          for (int c = 0; c < TV; ++c) A[a][c] = fmaf(vv_[a], kv_[c], A[a][c]);
        }
        wsum += wr;
      }
      n += nk;
    }
    // centred covariance of everything seen so far = what queries of block pl + 1 see
    const float inv = n > 0 ? 1.f / (TILT ? wsum : (float)n) : 0.f;
    ST* out = cov + (((size_t)pc * dm.SB + pl) * dm.Ck + j) * D * D;
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
__global__ void k_dipole_weights(const float* __restrict__ mu, long long rows, int Ck, ST* __restrict__ P, float* __restrict__ zall) {
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
  float z = 0.f;
  for (int j = lane; j < Ck; j += 32) {
    const ST v = from_f<ST>(mx == -INFINITY ? 0.f : expf(mr[j] - mx) * inv);
    P[row * Ck + j] = v;
    z += to_f(v);
  }
  z = warp_sum(z);
  if (lane == 0) zall[row] = z;                  // sum of the weights as stored (1 up to their rounding)
}

// ---- 3. merge, plain version: thread = one of 256 columns of the D*D axis, 16 query clusters ------
constexpr int kMrgI = 16, kMrgJ = 64;

template <class ST, class OT>
__global__ void __launch_bounds__(256)
k_dipole_merge(Dims dm, const ST* __restrict__ P, const ST* __restrict__ cov, OT* __restrict__ cbar) {
  __shared__ float ps[kMrgI][kMrgJ];
  const int DD = dm.D * dm.D;
  const int x = blockIdx.x * 256 + threadIdx.x, i0 = blockIdx.y * kMrgI;
  const int pp = blockIdx.z, pq = pp / dm.SB, pl = pp % dm.SB;
  const int pk = dm.dipole == 2 ? pq : (pq / dm.Hq) * dm.Hkv + dm.hm.g[pq % dm.Hq];     // head that owns the covariances
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
    if (i0 + a < dm.Cq) cbar[((size_t)pp * dm.Cq + i0 + a) * DD + x] = from_f<OT>(acc[a]);
}

// ---- 4a. the retrieved clusters' share (m > 0): one CTA per (key cluster j, plane, head) group of the inverse index ----
// Register tile: a thread owns 4 consecutive value dims of kSubQ pairs; the covariance sits transposed in shared memory
// in its storage type (Ct[key dim][value dim], rows 16-byte aligned), so that per 4 key dims a thread reads 4 vectors of
// the matrix and kSubQ broadcast vectors of residuals for 16 * kSubQ multiply-adds -- with one value dim per thread the
// kernel was bound by shared-memory reads at a fifth of the FMA rate.
constexpr int kSubQ = 8;

template <class T, class ST, int D>
__global__ void __launch_bounds__(256)
k_dipole_sub(Dims dm, const T* __restrict__ Q, const float* __restrict__ qbar, const int32_t* __restrict__ assign_q,
             const int32_t* __restrict__ goff, const int32_t* __restrict__ pairs, const ST* __restrict__ cov,
             const ST* __restrict__ pw, float* __restrict__ csub) {
  constexpr int TG = D / 4, G = 256 / TG, R = G * kSubQ;      // threads per pair group, groups, pairs per pass
  constexpr int P = D + 16 / (int)sizeof(ST);                 // pitch of a Ct row (elements)
  extern __shared__ __align__(16) unsigned char smd_raw[];
  float* qs = reinterpret_cast<float*>(smd_raw);              // [R][D] residuals
  ST* Ct = reinterpret_cast<ST*>(qs + R * D);                 // [D key dims][P]
  __shared__ int t_s[R], i_s[R];
  __shared__ float p_s[R];
  const int j = blockIdx.x, pl = blockIdx.y, pq = blockIdx.z, tid = threadIdx.x;
  const int32_t* go = goff + (size_t)pq * (dm.SB * dm.Ck + 1) + (size_t)j * dm.SB + pl;
  const int g0 = go[0], g1 = go[1];
  if (g0 >= g1) return;
  const int pk = (pq / dm.Hq) * dm.Hkv + dm.hm.g[pq % dm.Hq];
  const int pc = dm.dipole == 2 ? pq : pk;      // the tilted covariance belongs to a query head
  const ST* cb = cov + (((size_t)pc * dm.SB + pl) * dm.Ck + j) * D * D;
  for (int e = tid; e < D * D; e += 256) Ct[(e % D) * P + e / D] = cb[e];          // cov[dv][dk] -> Ct[dk][dv]
  const T* Qp = Q + (size_t)pq * dm.N * D;
  const int32_t* aq = assign_q + (size_t)pq * dm.N;
  const int32_t* pr = pairs + (size_t)pq * dm.N * dm.m;
  const ST* pwb = pw + ((size_t)pq * dm.SB + pl) * dm.Cq * dm.Ck;
  const int grp = tid / TG, d4 = (tid % TG) * 4;
  for (int r0 = g0; r0 < g1; r0 += R) {
    __syncthreads();
    if (tid < R) {
      int t = -1, i = 0;
      if (r0 + tid < g1) {
        t = pr[r0 + tid] / dm.m;
        if (!MUSE_IN_RANGE(t, dm.N)) t = -1;
      }
      if (t >= 0) { i = aq[t]; if (!MUSE_IN_RANGE(i, dm.Cq)) { t = -1; i = 0; } }
      t_s[tid] = t; i_s[tid] = i;
      p_s[tid] = t >= 0 ? to_f(pwb[(size_t)i * dm.Ck + j]) : 0.f;
    }
    __syncthreads();
    for (int e = tid; e < R * (D / 4); e += 256) {
      const int r = e / (D / 4), c4 = (e % (D / 4)) * 4, t = t_s[r];
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (t >= 0) {
        const float4 q = ld4(Qp + (size_t)t * D + c4), b = ld4(qbar + ((size_t)pq * dm.Cq + i_s[r]) * D + c4);
        v = make_float4(dm.sigma * (q.x - b.x), dm.sigma * (q.y - b.y), dm.sigma * (q.z - b.z), dm.sigma * (q.w - b.w));
      }
      st4(qs + r * D + c4, v);
    }
    __syncthreads();
    float acc[kSubQ][4];
#pragma unroll
    for (int a = 0; a < kSubQ; ++a) { acc[a][0] = 0.f; acc[a][1] = 0.f; acc[a][2] = 0.f; acc[a][3] = 0.f; }
    const float* qg = qs + grp * kSubQ * D;
#pragma unroll 2
    for (int dk = 0; dk < D; dk += 4) {
      const float4 c0 = ld4(Ct + (dk + 0) * P + d4), c1 = ld4(Ct + (dk + 1) * P + d4);
      const float4 c2 = ld4(Ct + (dk + 2) * P + d4), c3 = ld4(Ct + (dk + 3) * P + d4);
#pragma unroll
      for (int a = 0; a < kSubQ; ++a) {
        const float4 q = *reinterpret_cast<const float4*>(qg + a * D + dk);
        acc[a][0] = fmaf(c0.x, q.x, fmaf(c1.x, q.y, fmaf(c2.x, q.z, fmaf(c3.x, q.w, acc[a][0]))));
        acc[a][1] = fmaf(c0.y, q.x, fmaf(c1.y, q.y, fmaf(c2.y, q.z, fmaf(c3.y, q.w, acc[a][1]))));
        acc[a][2] = fmaf(c0.z, q.x, fmaf(c1.z, q.y, fmaf(c2.z, q.z, fmaf(c3.z, q.w, acc[a][2]))));
        acc[a][3] = fmaf(c0.w, q.x, fmaf(c1.w, q.y, fmaf(c2.w, q.z, fmaf(c3.w, q.w, acc[a][3]))));
      }
    }
#pragma unroll
    for (int a = 0; a < kSubQ; ++a) {
      const int r = grp * kSubQ + a, t = t_s[r];
      const float p = p_s[r];
      if (t >= 0)
        atomicAdd(reinterpret_cast<float4*>(&csub[((size_t)pq * dm.N + t) * D + d4]),
                  make_float4(p * acc[a][0], p * acc[a][1], p * acc[a][2], p * acc[a][3]));
    }
  }
}

// ---- 4b. consumption: one CTA per (query cluster, plane, head) segment --------------------------------
// m == 0: o_far += Cbar qres.  m > 0: o_far += (Cbar qres - csub) / Z with Z = the stored weights' sum minus the
// retrieved clusters' weights; corr / zq (optional) receive the correction and Z for the backward pass.
template <class T, class ST, class CT, int D>
__global__ void __launch_bounds__(256)
k_dipole_apply(Dims dm, const T* __restrict__ Q, const float* __restrict__ qbar, const int32_t* __restrict__ off_q,
               const int32_t* __restrict__ perm_q, const CT* __restrict__ cbar, const float* __restrict__ lse_far,
               const int32_t* __restrict__ sel, const ST* __restrict__ pw, const float* __restrict__ zall,
               const float* __restrict__ csub, int round_q, float* __restrict__ o_far, float* __restrict__ corr, float* __restrict__ zq) {
  // same register tile as k_dipole_sub: a thread owns 4 consecutive value dims of kSubQ queries
  constexpr int TG = D / 4, G = 256 / TG, R = G * kSubQ;
  constexpr int P = D + 16 / (int)sizeof(CT);
  extern __shared__ __align__(16) unsigned char smd_raw[];
  float* qs = reinterpret_cast<float*>(smd_raw);              // [R][D] residuals
  CT* Ct = reinterpret_cast<CT*>(qs + R * D);                 // [D key dims][P]: transposed matrix
  __shared__ float z_s[R];
  __shared__ int t_s[R];
  const int i = blockIdx.x, pl = blockIdx.y, pq = blockIdx.z, tid = threadIdx.x;
  const int blk = dm.causal ? pl + 1 : 0;
  const int32_t* oq = off_q + (size_t)pq * (dm.S * dm.Cq + 1) + (size_t)blk * dm.Cq + i;
  const int p0 = oq[0], p1 = oq[1];
  if (p0 >= p1) return;
  const size_t row = ((size_t)pq * dm.SB + pl) * dm.Cq + i;
  const CT* cb = cbar + row * D * D;
  for (int e = tid; e < D * D; e += 256) Ct[(e % D) * P + e / D] = cb[e];          // Cbar[dv][dk] -> Ct[dk][dv]
  const float* qb = qbar + ((size_t)pq * dm.Cq + i) * D;
  const T* Qp = Q + (size_t)pq * dm.N * D;
  const int32_t* pm = perm_q + (size_t)pq * dm.N;
  const int grp = tid / TG, d4 = (tid % TG) * 4;
  for (int r0 = p0; r0 < p1; r0 += R) {
    __syncthreads();
    if (tid < R) {
      float z = 1.f;
      int t = -1;
      if (r0 + tid < p1) {
        t = pm[r0 + tid];
        if (!MUSE_IN_RANGE(t, dm.N)) t = -1;
      }
      if (dm.m > 0 && t >= 0) {
        z = zall[row];
        for (int s = 0; s < dm.m; ++s) {
          const int jj = sel[((size_t)pq * dm.N + t) * dm.m + s];
          if (jj >= 0 && MUSE_IN_RANGE(jj, dm.Ck)) z -= to_f(pw[row * dm.Ck + jj]);
        }
      }
      z_s[tid] = z; t_s[tid] = t;
    }
    __syncthreads();
    for (int e = tid; e < R * (D / 4); e += 256) {
      const int r = e / (D / 4), c4 = (e % (D / 4)) * 4, t = t_s[r];
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (t >= 0) {
        const float4 q = ld4(Qp + (size_t)t * D + c4), b = ld4(qb + c4);
        v = make_float4(dm.sigma * (q.x - b.x), dm.sigma * (q.y - b.y), dm.sigma * (q.z - b.z), dm.sigma * (q.w - b.w));
        if (round_q) {                          // the same residuals as the tensor-core kernel that made csub
          v.x = __bfloat162float(__float2bfloat16_rn(v.x)); v.y = __bfloat162float(__float2bfloat16_rn(v.y));
          v.z = __bfloat162float(__float2bfloat16_rn(v.z)); v.w = __bfloat162float(__float2bfloat16_rn(v.w));
        }
      }
      st4(qs + r * D + c4, v);
    }
    __syncthreads();
    float acc[kSubQ][4];
#pragma unroll
    for (int a = 0; a < kSubQ; ++a) { acc[a][0] = 0.f; acc[a][1] = 0.f; acc[a][2] = 0.f; acc[a][3] = 0.f; }
    const float* qg = qs + grp * kSubQ * D;
#pragma unroll 2
    for (int dk = 0; dk < D; dk += 4) {
      const float4 c0 = ld4(Ct + (dk + 0) * P + d4), c1 = ld4(Ct + (dk + 1) * P + d4);
      const float4 c2 = ld4(Ct + (dk + 2) * P + d4), c3 = ld4(Ct + (dk + 3) * P + d4);
#pragma unroll
      for (int a = 0; a < kSubQ; ++a) {
        const float4 q = *reinterpret_cast<const float4*>(qg + a * D + dk);
        acc[a][0] = fmaf(c0.x, q.x, fmaf(c1.x, q.y, fmaf(c2.x, q.z, fmaf(c3.x, q.w, acc[a][0]))));
        acc[a][1] = fmaf(c0.y, q.x, fmaf(c1.y, q.y, fmaf(c2.y, q.z, fmaf(c3.y, q.w, acc[a][1]))));
        acc[a][2] = fmaf(c0.z, q.x, fmaf(c1.z, q.y, fmaf(c2.z, q.z, fmaf(c3.z, q.w, acc[a][2]))));
        acc[a][3] = fmaf(c0.w, q.x, fmaf(c1.w, q.y, fmaf(c2.w, q.z, fmaf(c3.w, q.w, acc[a][3]))));
      }
    }
#pragma unroll
    for (int a = 0; a < kSubQ; ++a) {
      const int r = grp * kSubQ + a, tl = t_s[r];
      if (tl < 0) continue;
      const size_t t = (size_t)pq * dm.N + tl;
      const float z = z_s[r];
      float4 c = make_float4(0.f, 0.f, 0.f, 0.f);
      if (lse_far[t] != -INFINITY && z > 1e-30f) {
        c = make_float4(acc[a][0], acc[a][1], acc[a][2], acc[a][3]);
        if (dm.m > 0) {
          const float4 sb = ld4(csub + t * D + d4);
          const float iz = 1.f / z;
          c = make_float4((c.x - sb.x) * iz, (c.y - sb.y) * iz, (c.z - sb.z) * iz, (c.w - sb.w) * iz);
        }
      }
      if (o_far) {
        float4 o = ld4(o_far + t * D + d4);
        o.x += c.x; o.y += c.y; o.z += c.z; o.w += c.w;
        st4(o_far + t * D + d4, o);
      }
      if (corr) { st4(corr + t * D + d4, c); if (d4 == 0) zq[t] = z; }
    }
  }
}

// ---- the shared tilt point of dipole == 2: the mean of a head's query centroids weighted by their member counts ----
// ("Untilted (Partially Specialized) Covariances": centring the shared tilt at the mass-weighted mean query centroid.)
// One CTA per query head: integer histogram of the assignments, then a fixed-order weighted sum.
__global__ void __launch_bounds__(256)
k_dipole_qstar(Dims dm, const int32_t* __restrict__ assign_q, const float* __restrict__ qbar, float* __restrict__ qstar) {
  __shared__ int cnt[kMaxC];
  const int pq = blockIdx.x, tid = threadIdx.x;
  for (int i = tid; i < dm.Cq; i += 256) cnt[i] = 0;
  __syncthreads();
  const int32_t* aq = assign_q + (size_t)pq * dm.N;
  for (int t = tid; t < dm.N; t += 256) {
    const int i = aq[t];
    if (MUSE_IN_RANGE(i, dm.Cq)) atomicAdd(&cnt[i], 1);
  }
  __syncthreads();
  for (int c = tid; c < dm.D; c += 256) {
    float s = 0.f;
    for (int i = 0; i < dm.Cq; ++i) s = fmaf((float)cnt[i], qbar[((size_t)pq * dm.Cq + i) * dm.D + c], s);
    qstar[(size_t)pq * dm.D + c] = s / (float)dm.N;
  }
}

int dipole_tilt_point(const Dims& d, const int32_t* assign_q, const float* qbar, float* qstar, cudaStream_t st) {
  prof_mark("k_dipole_qstar", st);
  k_dipole_qstar<<<d.B * d.Hq, 256, 0, st>>>(d, assign_q, qbar, qstar);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

// ---- host side ------------------------------------------------------------------------------------
// Scratch of the forward pass (and of the backward's recomputation): the retrieved clusters' rows.
size_t dipole_fwd_ws_bytes(const Dims& d) {
  if (!d.dipole || d.m == 0 || d.SB == 0) return 0;
  Arena ar(nullptr);
  ar.take<float>((size_t)d.B * d.Hq * d.N * d.D);
  return ar.used;
}

template <class T, class ST, int D>
static int dipole_build_t(const Dims& d, int dtype, const T* Kp, const T* Vp, const int32_t* off_k, const float* mu,
                          const DipolePtrs& dp, int* status, cudaStream_t st) {
  ST* cov = (ST*)dp.cov; ST* P = (ST*)dp.pw;
  prof_mark("k_dipole_cov", st);
  if (d.dipole == 2) k_dipole_cov<T, ST, D, true><<<dim3(d.Ck, d.B * d.Hq), 256, 0, st>>>(d, Kp, Vp, off_k, dp.qstar, cov);
  else k_dipole_cov<T, ST, D, false><<<dim3(d.Ck, d.B * d.Hkv), 256, 0, st>>>(d, Kp, Vp, off_k, nullptr, cov);
  MUSE_LAUNCH_OK();
  const long long rows = (long long)d.B * d.Hq * d.SB * d.Cq;
  prof_mark("k_dipole_weights", st);
  k_dipole_weights<ST><<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(mu, rows, d.Ck, P, dp.zall);
  MUSE_LAUNCH_OK();
  const bool f32out = d.m > 0 && sizeof(ST) == 2;        // next to retrieval the merged matrices stay in fp32
  if (dipole_merge_tc_supported(d, dtype) && !path_forced(kForceDipoleSimt))
    return dipole_merge_tc(d, P, cov, dp.cbar, f32out ? 1 : 0, status, st);
  prof_mark("k_dipole_merge", st);
  const dim3 grid(D * D / 256, cdiv(d.Cq, kMrgI), d.B * d.Hq * d.SB);
  if (f32out) k_dipole_merge<ST, float><<<grid, 256, 0, st>>>(d, P, cov, (float*)dp.cbar);
  else k_dipole_merge<ST, ST><<<grid, 256, 0, st>>>(d, P, cov, (ST*)dp.cbar);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

int dipole_build(const Dims& d, int dtype, const void* Kp, const void* Vp, const int32_t* off_k, const float* mu,
                 const DipolePtrs& dp, int* status, cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  if (dtype == MUSE_F32) {
    if (d.D == 64) return dipole_build_t<float, float, 64>(d, dtype, (const float*)Kp, (const float*)Vp, off_k, mu, dp, status, st);
    return dipole_build_t<float, float, 128>(d, dtype, (const float*)Kp, (const float*)Vp, off_k, mu, dp, status, st);
  }
  if (d.D == 64) return dipole_build_t<bf, bf, 64>(d, dtype, (const bf*)Kp, (const bf*)Vp, off_k, mu, dp, status, st);
  return dipole_build_t<bf, bf, 128>(d, dtype, (const bf*)Kp, (const bf*)Vp, off_k, mu, dp, status, st);
}

template <class T, class ST, int D>
static int dipole_apply_t(const Dims& d, const T* Q, const float* qbar, const int32_t* assign_q, const int32_t* off_q,
                          const int32_t* perm_q, const DipolePtrs& dp, const float* lse_far, const int32_t* sel,
                          const int32_t* goff, const int32_t* pairs, float* csub, float* o_far, float* corr, float* zq,
                          int* status, cudaStream_t st) {
  const size_t rows_b = (size_t)(256 / (D / 4)) * kSubQ * D * sizeof(float);      // the residual rows of one pass
  const dim3 grid(d.Cq, d.SB, d.B * d.Hq);
  int round_q = 0;
  if (d.m > 0) {
    const size_t ssub = (size_t)(256 / (D / 4)) * kSubQ * D * sizeof(float) + (size_t)D * (D + 16 / sizeof(ST)) * sizeof(ST);
    MUSE_CUDA_OK(cudaMemsetAsync(csub, 0, (size_t)d.B * d.Hq * d.N * D * sizeof(float), st));
    const bool tensor = sizeof(ST) == 2 && dipole_sub_tc_supported(d, MUSE_BF16) && !path_forced(kForceDipoleSimt);
    if (tensor) {
      int rc = dipole_sub_tc(d, Q, qbar, assign_q, goff, pairs, dp.cov, dp.pw, csub, status, st);
      if (rc != MUSE_OK) return rc;
    } else {
      MUSE_CUDA_OK(cudaFuncSetAttribute(k_dipole_sub<T, ST, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ssub));
      prof_mark("k_dipole_sub", st);
      k_dipole_sub<T, ST, D><<<dim3(d.Ck, d.SB, d.B * d.Hq), 256, ssub, st>>>(d, Q, qbar, assign_q, goff, pairs, (const ST*)dp.cov,
                                                                              (const ST*)dp.pw, csub);
      MUSE_LAUNCH_OK();
    }
    round_q = tensor ? 1 : 0;
    if (sizeof(ST) == 2) {
      const size_t smem = rows_b + (size_t)D * (D + 4) * sizeof(float);
      MUSE_CUDA_OK(cudaFuncSetAttribute(k_dipole_apply<T, ST, float, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      prof_mark("k_dipole_apply", st);
      k_dipole_apply<T, ST, float, D><<<grid, 256, smem, st>>>(d, Q, qbar, off_q, perm_q, (const float*)dp.cbar, lse_far, sel,
                                                               (const ST*)dp.pw, dp.zall, csub, round_q, o_far, corr, zq);
      MUSE_LAUNCH_OK();
      return MUSE_OK;
    }
  }
  const size_t smem = rows_b + (size_t)D * (D + 16 / sizeof(ST)) * sizeof(ST);
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_dipole_apply<T, ST, ST, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  prof_mark("k_dipole_apply", st);
  k_dipole_apply<T, ST, ST, D><<<grid, 256, smem, st>>>(d, Q, qbar, off_q, perm_q, (const ST*)dp.cbar, lse_far, sel, (const ST*)dp.pw,
                                                        dp.zall, csub, round_q, o_far, corr, zq);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

// o_far += correction (forward); corr / zq non-null: the correction and its weight sum are written out instead
// (o_far may then be NULL).  sel, goff, pairs, csub are used with m > 0 only.
int dipole_apply(const Dims& d, int dtype, const void* Q, const float* qbar, const int32_t* assign_q, const int32_t* off_q,
                 const int32_t* perm_q, const DipolePtrs& dp, const float* lse_far, const int32_t* sel, const int32_t* goff,
                 const int32_t* pairs, float* csub, float* o_far, float* corr, float* zq, int* status, cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  if (dtype == MUSE_F32) {
    if (d.D == 64) return dipole_apply_t<float, float, 64>(d, (const float*)Q, qbar, assign_q, off_q, perm_q, dp, lse_far, sel, goff, pairs, csub, o_far, corr, zq, status, st);
    return dipole_apply_t<float, float, 128>(d, (const float*)Q, qbar, assign_q, off_q, perm_q, dp, lse_far, sel, goff, pairs, csub, o_far, corr, zq, status, st);
  }
  if (d.D == 64) return dipole_apply_t<bf, bf, 64>(d, (const bf*)Q, qbar, assign_q, off_q, perm_q, dp, lse_far, sel, goff, pairs, csub, o_far, corr, zq, status, st);
  return dipole_apply_t<bf, bf, 128>(d, (const bf*)Q, qbar, assign_q, off_q, perm_q, dp, lse_far, sel, goff, pairs, csub, o_far, corr, zq, status, st);
}

}  // namespace muse
