// Backward through the dipole correction of the far field (Appendix "Error Analysis": "Dipole Correction",
// "Untilted (Partially Specialized) Covariances", "Compatibility with Retrieval"; the paper states the forward only,
// the gradient rules follow the ones it gives for the monopole: assignments, selections and query centroids are
// constants, the aggregation weights are differentiated unless agg_grad = 0).
//
// Forward, per query t of segment (query cluster i, plane b):  every far cluster's value is nu_j + c_t with
//   c_t = M_t qres_t / Z_t,   M_t = Cbar_ib - sum_{j in sel_t} p_ib(j) Cov_jb,   Z_t = sum_j p_ib(j) - sum_{j in sel_t} p_ib(j).
// With w_far = exp(lse_far - L), dc = w_far dO and x_t = dc / Z_t:
//   far logits     g_tj = p_tj (dO.nu_j + dO.c_t - delta_t)            -> the far-field backward runs with delta - dO.c
//   residual       dqres_t  = M_t^T x_t                                -> dQ (times sigma)
//   merged matrix  dCbar_ib = sum_t x_t qres_t^T,   dZ_t = -(x_t . c_t)
//   covariances    dCov_jb  = sum_i p_ib(j) dCbar_ib  -  sum_{t: j in sel_t} p_ib(j) x_t qres_t^T
//   weights        dp_ib(j) = <Cov_jb, dCbar_ib> + sum_t dZ_t  -  sum_{t: j in sel_t} (x_t^T Cov_jb qres_t + dZ_t)
//   log-masses     dmu_ijb  = p (dp - sum_k p_k dp_k)                  -> added to the summary gradient of the monopole
//   keys, values   Cov_jb = mean((v - vm)(k - km)^T) over blocks <= b of cluster j:
//                  dV_u = sum_{b >= block(u)} dCov_jb (k_u - km_b) / n_b,  dK_u = sum_b dCov_jb^T (v_u - vm_b) / n_b.
//                  dipole == 2 (weights w_ub = exp(l_u - lse_b), l_u = sigma qstar.k_u, in place of 1 / n_b): the same
//                  with w_ub, plus, unless agg_grad = 0, dl_u = sum_b w_ub [(v_u - vm_b)^T dCov_jb (k_u - km_b)
//                  - <dCov_jb, Cov_jb>] and dK_u += sigma qstar dl_u.
// Kernels: k_dipole_bwd_prep (per query), k_dipole_bwd_seg (per query segment), k_dipole_bwd_pairs (per group of the
// retrieval's inverse index, m > 0), k_dipole_dcov / k_dipole_dpw (the two dense contractions over the query and key
// clusters), k_dipole_dmu (softmax backward), k_dipole_cov_bwd (per key cluster: suffix sums over planes, then one
// matrix-vector product per key).  All FFMA.
#include "common.cuh"

namespace muse {

constexpr int kDbQ = 8;                         // queries (or keys) per thread group and pass

// ---- per query: x_t = w_far dO / Z, delta for the far field, dZ_t -------------------------------------------------
template <class T, int D>
__global__ void k_dipole_bwd_prep(const T* __restrict__ dO, const float* __restrict__ LSE, const float* __restrict__ lse_far,
                                  const float* __restrict__ delta, const float* __restrict__ corr, const float* __restrict__ zq,
                                  long long rows, float* __restrict__ xq, float* __restrict__ delta_far, float* __restrict__ dz) {
  const long long r = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= rows) return;
  const float lf = lse_far[r];
  const float z = lf != -INFINITY ? zq[r] : 0.f;
  const bool valid = lf != -INFINITY && z > 1e-30f;
  const float wf = valid ? expf(lf - LSE[r]) : 0.f;
  float g[D / 32], dot = 0.f;
#pragma unroll
  for (int k = 0; k < D / 32; ++k) {
    g[k] = to_f(dO[r * D + lane + 32 * k]);
    if (valid) dot = fmaf(g[k], corr[r * D + lane + 32 * k], dot);
  }
  dot = warp_sum(dot);
  const float s = valid ? wf / z : 0.f;
#pragma unroll
  for (int k = 0; k < D / 32; ++k) xq[r * D + lane + 32 * k] = s * g[k];
  if (lane == 0) { delta_far[r] = delta[r] - dot; dz[r] = -s * dot; }
}

// ---- per query segment (i, plane, head): dQ += sigma Cbar^T x,  dCbar = sum x qres^T,  sum of dZ -------------------
// The merged matrix sits in shared memory as stored ([value dim][key dim], rows 16-byte aligned); a thread owns 4
// consecutive key dims of kSegQ queries for Cbar^T x, and a TV x TV block of the segment's outer-product sum.
constexpr int kSegQ = 8;

template <class T, class CT, int D>
__global__ void __launch_bounds__(256)
k_dipole_bwd_seg(Dims dm, const T* __restrict__ Q, const float* __restrict__ qbar, const int32_t* __restrict__ off_q,
                 const int32_t* __restrict__ perm_q, const CT* __restrict__ cbar, const float* __restrict__ xq,
                 const float* __restrict__ dz, float* __restrict__ dQacc, float* __restrict__ dcbar, float* __restrict__ dzs) {
  constexpr int TG = D / 4, G = 256 / TG, R = G * kSegQ, TV = D / 16;
  constexpr int P = D + 16 / (int)sizeof(CT);
  extern __shared__ __align__(16) unsigned char smd_raw[];
  float* qs = reinterpret_cast<float*>(smd_raw);              // [R][D] residuals
  float* xs = qs + R * D;                                     // [R][D] x rows
  CT* Cs = reinterpret_cast<CT*>(xs + R * D);                 // [D value dims][P]
  __shared__ float zsum_s[R];
  __shared__ int t_s[R];
  const int i = blockIdx.x, pl = blockIdx.y, pq = blockIdx.z, tid = threadIdx.x;
  const int blk = dm.causal ? pl + 1 : 0;
  const int32_t* oq = off_q + (size_t)pq * (dm.S * dm.Cq + 1) + (size_t)blk * dm.Cq + i;
  const int p0 = oq[0], p1 = oq[1];
  if (p0 >= p1) return;                         // dCbar and the dZ sum of an empty segment stay at their cleared zero
  const size_t row = ((size_t)pq * dm.SB + pl) * dm.Cq + i;
  {
    const CT* cb = cbar + row * D * D;
    constexpr int V = 16 / (int)sizeof(CT);
    for (int e = tid; e < D * D / V; e += 256) {
      const int dv = e / (D / V), c = (e % (D / V)) * V;
      *reinterpret_cast<uint4*>(Cs + dv * P + c) = *reinterpret_cast<const uint4*>(cb + (size_t)dv * D + c);
    }
  }
  const float* qb = qbar + ((size_t)pq * dm.Cq + i) * D;
  const T* Qp = Q + (size_t)pq * dm.N * D;
  const int32_t* pm = perm_q + (size_t)pq * dm.N;
  const int grp = tid / TG, d4 = (tid % TG) * 4, ty = tid >> 4, tx = tid & 15;
  float A[TV][TV];
#pragma unroll
  for (int a = 0; a < TV; ++a)
#pragma unroll
    for (int c = 0; c < TV; ++c) A[a][c] = 0.f;
  float zacc = 0.f;
  for (int r0 = p0; r0 < p1; r0 += R) {
    __syncthreads();
    if (tid < R) {
      int t = -1;
      if (r0 + tid < p1) {
        t = pm[r0 + tid];
        if (!MUSE_IN_RANGE(t, dm.N)) t = -1;
      }
      t_s[tid] = t;
      if (t >= 0) zacc += dz[(size_t)pq * dm.N + t];
    }
    __syncthreads();
    for (int e = tid; e < R * (D / 4); e += 256) {
      const int r = e / (D / 4), c4 = (e % (D / 4)) * 4, t = t_s[r];
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f), x = v;
      if (t >= 0) {
        const float4 q = ld4(Qp + (size_t)t * D + c4), b = ld4(qb + c4);
        v = make_float4(dm.sigma * (q.x - b.x), dm.sigma * (q.y - b.y), dm.sigma * (q.z - b.z), dm.sigma * (q.w - b.w));
        x = ld4(xq + ((size_t)pq * dm.N + t) * D + c4);
      }
      st4(qs + r * D + c4, v); st4(xs + r * D + c4, x);
    }
    __syncthreads();
    // dqres[dk] = sum_dv Cbar[dv][dk] x[dv]
    float acc[kSegQ][4];
#pragma unroll
    for (int a = 0; a < kSegQ; ++a) { acc[a][0] = 0.f; acc[a][1] = 0.f; acc[a][2] = 0.f; acc[a][3] = 0.f; }
    const float* xg = xs + grp * kSegQ * D;
#pragma unroll 2
    for (int dv = 0; dv < D; dv += 4) {
      const float4 c0 = ld4(Cs + (dv + 0) * P + d4), c1 = ld4(Cs + (dv + 1) * P + d4);
      const float4 c2 = ld4(Cs + (dv + 2) * P + d4), c3 = ld4(Cs + (dv + 3) * P + d4);
#pragma unroll
      for (int a = 0; a < kSegQ; ++a) {
        const float4 x = *reinterpret_cast<const float4*>(xg + a * D + dv);
        acc[a][0] = fmaf(c0.x, x.x, fmaf(c1.x, x.y, fmaf(c2.x, x.z, fmaf(c3.x, x.w, acc[a][0]))));
        acc[a][1] = fmaf(c0.y, x.x, fmaf(c1.y, x.y, fmaf(c2.y, x.z, fmaf(c3.y, x.w, acc[a][1]))));
        acc[a][2] = fmaf(c0.z, x.x, fmaf(c1.z, x.y, fmaf(c2.z, x.z, fmaf(c3.z, x.w, acc[a][2]))));
        acc[a][3] = fmaf(c0.w, x.x, fmaf(c1.w, x.y, fmaf(c2.w, x.z, fmaf(c3.w, x.w, acc[a][3]))));
      }
    }
#pragma unroll
    for (int a = 0; a < kSegQ; ++a) {
      const int t = t_s[grp * kSegQ + a];
      if (t < 0) continue;
      float* dst = dQacc + ((size_t)pq * dm.N + t) * D + d4;      // this segment owns the query: plain read-modify-write
      float4 o = ld4(dst);
      o.x += dm.sigma * acc[a][0]; o.y += dm.sigma * acc[a][1]; o.z += dm.sigma * acc[a][2]; o.w += dm.sigma * acc[a][3];
      st4(dst, o);
    }
    // dCbar[dv][dk] += x[dv] qres[dk]; thread (ty, tx) owns value dims ty*TV.., key dims tx*TV..
    for (int r = 0; r < R; ++r) {
      float xv[TV], qv[TV];
#pragma unroll
      for (int a = 0; a < TV; ++a) { xv[a] = xs[r * D + ty * TV + a]; qv[a] = qs[r * D + tx * TV + a]; }
#pragma unroll
      for (int a = 0; a < TV; ++a)
#pragma unroll
        for (int c = 0; c < TV; ++c) A[a][c] = fmaf(xv[a], qv[c], A[a][c]);
    }
  }
  float* out = dcbar + row * D * D;
#pragma unroll
  for (int a = 0; a < TV; ++a)
#pragma unroll
    for (int c = 0; c < TV; c += 4)
      st4(out + (size_t)(ty * TV + a) * D + tx * TV + c, make_float4(A[a][c], A[a][c + 1], A[a][c + 2], A[a][c + 3]));
  if (tid < R) zsum_s[tid] = zacc;
  __syncthreads();
  if (tid == 0) {
    float s = 0.f;
    for (int r = 0; r < R; ++r) s += zsum_s[r];
    dzs[row] = s;
  }
}

// ---- per (key cluster j, plane, head) group of the inverse index: what the retrieved clusters take back -----------
// The covariance sits in shared memory as stored ([value dim][key dim], rows 16-byte aligned); a thread owns 4 consecutive
// key dims of kPairQ pairs for v = Cov^T x (4 matrix vectors + kPairQ broadcast vectors per 16 * kPairQ multiply-adds),
// and a TV x TV block of the group's outer-product sum.
constexpr int kPairQ = 8;

template <class T, class ST, int D>
__global__ void __launch_bounds__(256)
k_dipole_bwd_pairs(Dims dm, const T* __restrict__ Q, const float* __restrict__ qbar, const int32_t* __restrict__ assign_q,
                   const int32_t* __restrict__ goff, const int32_t* __restrict__ pairs, const ST* __restrict__ cov,
                   const ST* __restrict__ pw, const float* __restrict__ xq, const float* __restrict__ dz,
                   float* __restrict__ dQacc, float* __restrict__ dcov, float* __restrict__ dpw) {
  constexpr int TG = D / 4, G = 256 / TG, R = G * kPairQ, TV = D / 16;
  constexpr int P = D + 16 / (int)sizeof(ST);
  extern __shared__ __align__(16) unsigned char smd_raw[];
  float* qs = reinterpret_cast<float*>(smd_raw);              // [R][D] residuals
  float* xs = qs + R * D;                                     // [R][D] x rows
  ST* Cs = reinterpret_cast<ST*>(xs + R * D);                 // [D value dims][P]
  __shared__ int t_s[R], i_s[R];
  __shared__ float p_s[R], s_s[R];
  const int j = blockIdx.x, pl = blockIdx.y, pq = blockIdx.z, tid = threadIdx.x;
  const int32_t* go = goff + (size_t)pq * (dm.SB * dm.Ck + 1) + (size_t)j * dm.SB + pl;
  const int g0 = go[0], g1 = go[1];
  const int pk = (pq / dm.Hq) * dm.Hkv + dm.hm.g[pq % dm.Hq];
  const int pc = dm.dipole == 2 ? pq : pk;
  const int grp = tid / TG, d4 = (tid % TG) * 4, ty = tid >> 4, tx = tid & 15;
  float A[TV][TV];
#pragma unroll
  for (int a = 0; a < TV; ++a)
#pragma unroll
    for (int c = 0; c < TV; ++c) A[a][c] = 0.f;
  if (g0 < g1) {
    const ST* cb = cov + (((size_t)pc * dm.SB + pl) * dm.Ck + j) * D * D;
    constexpr int V = 16 / (int)sizeof(ST);                   // elements per 16-byte copy
    for (int e = tid; e < D * D / V; e += 256) {
      const int dv = e / (D / V), c = (e % (D / V)) * V;
      *reinterpret_cast<uint4*>(Cs + dv * P + c) = *reinterpret_cast<const uint4*>(cb + (size_t)dv * D + c);
    }
  }
  const T* Qp = Q + (size_t)pq * dm.N * D;
  const int32_t* aq = assign_q + (size_t)pq * dm.N;
  const int32_t* pr = pairs + (size_t)pq * dm.N * dm.m;
  const size_t prow = ((size_t)pq * dm.SB + pl) * dm.Cq;
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
      p_s[tid] = t >= 0 ? to_f(pw[(prow + i) * dm.Ck + j]) : 0.f;
    }
    __syncthreads();
    for (int e = tid; e < R * (D / 4); e += 256) {
      const int r = e / (D / 4), c4 = (e % (D / 4)) * 4, t = t_s[r];
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f), x = v;
      if (t >= 0) {
        const float4 q = ld4(Qp + (size_t)t * D + c4), b = ld4(qbar + ((size_t)pq * dm.Cq + i_s[r]) * D + c4);
        v = make_float4(dm.sigma * (q.x - b.x), dm.sigma * (q.y - b.y), dm.sigma * (q.z - b.z), dm.sigma * (q.w - b.w));
        x = ld4(xq + ((size_t)pq * dm.N + t) * D + c4);
      }
      st4(qs + r * D + c4, v); st4(xs + r * D + c4, x);
    }
    __syncthreads();
    // v[dk] = sum_dv Cov[dv][dk] x[dv]:  dqres -= p v,  x^T Cov qres = v . qres
    float acc[kPairQ][4];
#pragma unroll
    for (int a = 0; a < kPairQ; ++a) { acc[a][0] = 0.f; acc[a][1] = 0.f; acc[a][2] = 0.f; acc[a][3] = 0.f; }
    const float* xg = xs + grp * kPairQ * D;
#pragma unroll 2
    for (int dv = 0; dv < D; dv += 4) {
      const float4 c0 = ld4(Cs + (dv + 0) * P + d4), c1 = ld4(Cs + (dv + 1) * P + d4);
      const float4 c2 = ld4(Cs + (dv + 2) * P + d4), c3 = ld4(Cs + (dv + 3) * P + d4);
#pragma unroll
      for (int a = 0; a < kPairQ; ++a) {
        const float4 x = *reinterpret_cast<const float4*>(xg + a * D + dv);
        acc[a][0] = fmaf(c0.x, x.x, fmaf(c1.x, x.y, fmaf(c2.x, x.z, fmaf(c3.x, x.w, acc[a][0]))));
        acc[a][1] = fmaf(c0.y, x.x, fmaf(c1.y, x.y, fmaf(c2.y, x.z, fmaf(c3.y, x.w, acc[a][1]))));
        acc[a][2] = fmaf(c0.z, x.x, fmaf(c1.z, x.y, fmaf(c2.z, x.z, fmaf(c3.z, x.w, acc[a][2]))));
        acc[a][3] = fmaf(c0.w, x.x, fmaf(c1.w, x.y, fmaf(c2.w, x.z, fmaf(c3.w, x.w, acc[a][3]))));
      }
    }
#pragma unroll
    for (int a = 0; a < kPairQ; ++a) {
      const int r = grp * kPairQ + a, t = t_s[r];
      const float4 q = *reinterpret_cast<const float4*>(qs + r * D + d4);
      float part = acc[a][0] * q.x + acc[a][1] * q.y + acc[a][2] * q.z + acc[a][3] * q.w;
#pragma unroll
      for (int o = TG / 2; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
      if (tid % TG == 0) s_s[r] = part;
      const float f = -dm.sigma * p_s[r];
      if (t >= 0)
        atomicAdd(reinterpret_cast<float4*>(&dQacc[((size_t)pq * dm.N + t) * D + d4]),
                  make_float4(f * acc[a][0], f * acc[a][1], f * acc[a][2], f * acc[a][3]));
    }
    for (int r = 0; r < R; ++r) {
      const float p = p_s[r];
      float xv[TV], qv[TV];
#pragma unroll
      for (int a = 0; a < TV; ++a) { xv[a] = p * xs[r * D + ty * TV + a]; qv[a] = qs[r * D + tx * TV + a]; }
#pragma unroll
      for (int a = 0; a < TV; ++a)
#pragma unroll
        for (int c = 0; c < TV; ++c) A[a][c] = fmaf(xv[a], qv[c], A[a][c]);
    }
    __syncthreads();
    if (tid < R && t_s[tid] >= 0)
      atomicAdd(&dpw[(prow + i_s[tid]) * dm.Ck + j], -(s_s[tid] + dz[(size_t)pq * dm.N + t_s[tid]]));
  }
  // the group's share, negated; the dense part (k_dipole_dcov) is added on top of it afterwards
  float* out = dcov + (((size_t)pq * dm.SB + pl) * dm.Ck + j) * D * D;
#pragma unroll
  for (int a = 0; a < TV; ++a)
#pragma unroll
    for (int c = 0; c < TV; c += 4)
      st4(out + (size_t)(ty * TV + a) * D + tx * TV + c, make_float4(-A[a][c], -A[a][c + 1], -A[a][c + 2], -A[a][c + 3]));
}

// ---- dCov[j][x] += sum_i P[i][j] dCbar[i][x]   (x over D*D; thread = one x, 16 key clusters per CTA) ---------------
constexpr int kDcJ = 16, kDcI = 64;

template <class ST>
__global__ void __launch_bounds__(256)
k_dipole_dcov(Dims dm, const ST* __restrict__ P, const float* __restrict__ dcbar, float* __restrict__ dcov) {
  __shared__ __align__(16) float ps[kDcI][kDcJ];
  const int DD = dm.D * dm.D;
  const int x = blockIdx.x * 256 + threadIdx.x, j0 = blockIdx.y * kDcJ;
  const size_t pp = blockIdx.z;
  float acc[kDcJ];
#pragma unroll
  for (int a = 0; a < kDcJ; ++a) acc[a] = 0.f;
  for (int i0 = 0; i0 < dm.Cq; i0 += kDcI) {
    __syncthreads();
    for (int e = threadIdx.x; e < kDcI * kDcJ; e += 256) {
      const int ii = e / kDcJ, jj = e % kDcJ;
      ps[ii][jj] = (i0 + ii < dm.Cq && j0 + jj < dm.Ck) ? to_f(P[(pp * dm.Cq + i0 + ii) * dm.Ck + j0 + jj]) : 0.f;
    }
    __syncthreads();
    const int ni = min(kDcI, dm.Cq - i0);
    for (int ii = 0; ii < ni; ++ii) {
      const float c = dcbar[(pp * dm.Cq + i0 + ii) * DD + x];
#pragma unroll
      for (int a = 0; a < kDcJ; a += 4) {
        const float4 p4 = *reinterpret_cast<const float4*>(&ps[ii][a]);
        acc[a] = fmaf(p4.x, c, acc[a]); acc[a + 1] = fmaf(p4.y, c, acc[a + 1]);
        acc[a + 2] = fmaf(p4.z, c, acc[a + 2]); acc[a + 3] = fmaf(p4.w, c, acc[a + 3]);
      }
    }
  }
#pragma unroll
  for (int a = 0; a < kDcJ; ++a)
    if (j0 + a < dm.Ck) dcov[(pp * dm.Ck + j0 + a) * DD + x] += acc[a];
}

// ---- dP[i][j] += <dCbar_i, Cov_j> + sum of dZ over the segment   (64 x 64 tile per CTA, 4 x 4 per thread) -----------
template <class ST>
__global__ void __launch_bounds__(256)
k_dipole_dpw(Dims dm, const float* __restrict__ dcbar, const ST* __restrict__ cov, const float* __restrict__ dzs,
             float* __restrict__ dpw) {
  __shared__ float as[64][33], bs[64][33];
  const int DD = dm.D * dm.D;
  const int j0 = blockIdx.x * 64, i0 = blockIdx.y * 64, tid = threadIdx.x;
  const int pp = blockIdx.z, pq = pp / dm.SB, pl = pp % dm.SB;
  const int pk = (pq / dm.Hq) * dm.Hkv + dm.hm.g[pq % dm.Hq];
  const int pc = dm.dipole == 2 ? pq : pk;
  const float* ab = dcbar + ((size_t)pp * dm.Cq) * DD;
  const ST* bb = cov + (((size_t)pc * dm.SB + pl) * dm.Ck) * DD;
  const int ty = tid >> 4, tx = tid & 15;
  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
  for (int x0 = 0; x0 < DD; x0 += 32) {
    __syncthreads();
    for (int e = tid; e < 64 * 8; e += 256) {
      const int r = e / 8, c4 = (e % 8) * 4;
      float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
      if (i0 + r < dm.Cq) a = ld4(ab + (size_t)(i0 + r) * DD + x0 + c4);
      if (j0 + r < dm.Ck) b = ld4(bb + (size_t)(j0 + r) * DD + x0 + c4);
      as[r][c4] = a.x; as[r][c4 + 1] = a.y; as[r][c4 + 2] = a.z; as[r][c4 + 3] = a.w;
      bs[r][c4] = b.x; bs[r][c4 + 1] = b.y; bs[r][c4 + 2] = b.z; bs[r][c4 + 3] = b.w;
    }
    __syncthreads();
#pragma unroll 8
    for (int x = 0; x < 32; ++x) {
      float av_[4], bv_[4];
#pragma unroll
      for (int a = 0; a < 4; ++a) { av_[a] = as[ty + 16 * a][x]; bv_[a] = bs[tx + 16 * a][x]; }
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(av_[a], bv_[b], acc[a][b]);
    }
  }
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int i = i0 + ty + 16 * a, j = j0 + tx + 16 * b;
      if (i < dm.Cq && j < dm.Ck) dpw[((size_t)pp * dm.Cq + i) * dm.Ck + j] += acc[a][b] + dzs[(size_t)pp * dm.Cq + i];
    }
}

// ---- softmax backward of the centroid weights into the summary gradient (one warp per (head, plane, i)) -----------
template <class ST>
__global__ void k_dipole_dmu(Dims dm, const ST* __restrict__ P, const float* __restrict__ dpw, long long rows,
                             float* __restrict__ dS, int grad_by_key_cluster) {
  const long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const ST* pr = P + row * dm.Ck;
  const float* dr = dpw + row * dm.Ck;
  float dot = 0.f;
  for (int j = lane; j < dm.Ck; j += 32) dot = fmaf(to_f(pr[j]), dr[j], dot);
  dot = warp_sum(dot);
  const long long pp = row / dm.Cq;
  const int i = (int)(row % dm.Cq);
  for (int j = lane; j < dm.Ck; j += 32) {
    const float p = to_f(pr[j]);
    if (p == 0.f) continue;                     // empty cluster: no entry
    const size_t at = grad_by_key_cluster ? ((size_t)pp * dm.Ck + j) * dm.Cq + i : (size_t)row * dm.Ck + j;
    dS[at] += p * (dr[j] - dot);
  }
}

// ---- through the covariances to keys and values: one CTA per (key cluster, query head) ----------------------------
// With w_ub = f_u / W_b (f_u = exp(l_u - max logit of the cluster), W_b = sum of f over the plane's members):
//   dV_u = f_u (A k_u - a_k),  dK_u = f_u (A^T v_u - a_v),  A = sum_{b >= block(u)} dCov_b / W_b,
//   a_k = sum_b dCov_b km_b / W_b,  a_v = sum_b dCov_b^T vm_b / W_b,
//   dl_u = f_u (v_u.(A k_u - a_k) - a_v.k_u + s),  s = sum_b (vm_b^T dCov_b km_b - <dCov_b, Cov_b>) / W_b
// (untilted: f = 1, W_b = n_b, no dl).  Keys enter shifted by the cluster's first key, which changes none of these.
template <class T, class ST, int D, bool TILT>
__global__ void __launch_bounds__(256)
k_dipole_cov_bwd(Dims dm, const T* __restrict__ Kp, const T* __restrict__ Vp, const int32_t* __restrict__ off_k,
                 const float* __restrict__ dcov, const float* __restrict__ qstar, const ST* __restrict__ cov,
                 float* __restrict__ dK_perm, float* __restrict__ dV_perm) {
  extern __shared__ float smd[];
  float* As = smd;                              // As[dv][dk], pitch D + 1: sum over later planes of dCov / n
  float* avp = As + D * (D + 1);                // [8 warps][D] partial column sums of a plane
  float* kb = avp + 8 * D;                      // [SB][D] prefix means of k - k0
  float* vb = kb + dm.SB * D;                   // [SB][D] prefix means of v
  float* ks = vb + dm.SB * D;                   // [kDbQ][D]
  float* vs = ks + kDbQ * D;
  float* ak = vs + kDbQ * D;                    // [D] sum of dCov km / n
  float* av = ak + D;                           // [D] sum of dCov^T vm / n
  float* k0 = av + D;
  float* qs_ = k0 + D;                          // [D] sigma * tilt point
  float* wb = qs_ + D;                          // [SB] W_b
  __shared__ float red[8], fk[kDbQ], dl_s[kDbQ], s_suf, lmax_s;
  const int j = blockIdx.x, pq = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int pk = (pq / dm.Hq) * dm.Hkv + dm.hm.g[pq % dm.Hq];
  const int32_t* off = off_k + (size_t)pk * (dm.Ck * dm.S + 1) + (size_t)j * dm.S;
  const T* Kb = Kp + (size_t)pk * dm.N * D;
  const T* Vb = Vp + (size_t)pk * dm.N * D;
  const int first = off[0];
  if (first >= off[dm.SB]) return;              // no key of this cluster is visible to anyone
  if (tid < D) {
    k0[tid] = to_f(Kb[(size_t)first * D + tid]); ak[tid] = 0.f; av[tid] = 0.f;
    qs_[tid] = TILT ? dm.sigma * qstar[(size_t)pq * D + tid] : 0.f;
  }
  for (int e = tid; e < D * (D + 1); e += 256) As[e] = 0.f;
  if (tid == 0) { s_suf = 0.f; lmax_s = 0.f; }
  __syncthreads();
  // logit of a key relative to the cluster's first key: one warp, all lanes return it
  auto logit = [&](int u) {
    float l = 0.f;
    for (int c = lane; c < D; c += 32) l = fmaf(qs_[c], to_f(Kb[(size_t)u * D + c]) - k0[c], l);
    return warp_sum(l);
  };
  if (TILT) {                                   // largest logit over the visible members
    float mx = -INFINITY;
    for (int u = first + warp; u < off[dm.SB]; u += 8) mx = fmaxf(mx, logit(u));
    if (lane == 0) red[warp] = mx;
    __syncthreads();
    if (tid == 0) { float m = red[0]; for (int w = 1; w < 8; ++w) m = fmaxf(m, red[w]); lmax_s = m; }
    __syncthreads();
  }
  const float lmax = lmax_s;
  // prefix means per plane (plane pl = blocks 0..pl), weighted by f_u; with the tilt the weights of eight keys at a
  // time are computed by the eight warps (one dot product each) and shared
  {
    const bool isv = tid >= D;
    const int c = tid % D;
    float s = 0.f, wsum = 0.f;
    for (int pl = 0; pl < dm.SB; ++pl) {
      if (TILT) {
        for (int u0 = off[pl]; u0 < off[pl + 1]; u0 += 8) {
          const int nk = min(8, off[pl + 1] - u0);
          const float l = warp < nk ? logit(u0 + warp) : 0.f;
          if (lane == 0) fk[warp] = warp < nk ? expf(l - lmax) : 0.f;
          __syncthreads();
          if (tid < 2 * D)
            for (int r = 0; r < nk; ++r) {
              s = fmaf(fk[r], isv ? to_f(Vb[(size_t)(u0 + r) * D + c]) : to_f(Kb[(size_t)(u0 + r) * D + c]) - k0[c], s);
              wsum += fk[r];
            }
          __syncthreads();
        }
      } else if (tid < 2 * D) {
        for (int u = off[pl]; u < off[pl + 1]; ++u) s += isv ? to_f(Vb[(size_t)u * D + c]) : to_f(Kb[(size_t)u * D + c]) - k0[c];
        wsum = (float)(off[pl + 1] - first);
      }
      if (tid < 2 * D) (isv ? vb : kb)[pl * D + c] = wsum > 0.f ? s / wsum : 0.f;
      if (tid == 0) wb[pl] = wsum;
    }
  }
  __syncthreads();
  // a plane's dCov is fetched into registers one plane ahead, so that its latency runs under the previous plane's work
  constexpr int NG = D * D / 4 / 256;           // float4 per thread and plane
  float4 greg[NG];
  auto fetch = [&](int pl) {
    const float* g = dcov + (((size_t)pq * dm.SB + pl) * dm.Ck + j) * D * D;
#pragma unroll
    for (int k = 0; k < NG; ++k) {
      const int e = tid + 256 * k;
      greg[k] = ld4(g + (size_t)(e / (D / 4)) * D + (e % (D / 4)) * 4);
    }
  };
  fetch(dm.SB - 1);
  for (int pl = dm.SB - 1; pl >= 0; --pl) {
    const float n = wb[pl];
    if (n > 0.f) {
      // straight from the registers: A += G / n (every thread its own elements); row sums against km (the D / 4 lanes
      // that share a row reduce by shuffles) and column sums against vm (per-warp partials, then one pass over the warps)
      const float inv = 1.f / n;
      const ST* cv = cov + (((size_t)pq * dm.SB + pl) * dm.Ck + j) * D * D;
      float av4[4] = {0.f, 0.f, 0.f, 0.f}, cc = 0.f;
#pragma unroll
      for (int k = 0; k < NG; ++k) {
        const int e = tid + 256 * k, dv = e / (D / 4), c4 = (e % (D / 4)) * 4;
        const float4 g = make_float4(greg[k].x * inv, greg[k].y * inv, greg[k].z * inv, greg[k].w * inv);
        float* o = As + dv * (D + 1) + c4;
        o[0] += g.x; o[1] += g.y; o[2] += g.z; o[3] += g.w;
        const float* kp = kb + pl * D + c4;
        float part = g.x * kp[0] + g.y * kp[1] + g.z * kp[2] + g.w * kp[3];
#pragma unroll
        for (int o2 = D / 8; o2 > 0; o2 >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o2);
        const float vm = vb[pl * D + dv];
        if (lane % (D / 4) == 0) {
          ak[dv] += part;
          if (TILT && dm.agg_grad) cc = fmaf(part, vm, cc);          // vm^T (dCov / W) km
        }
        av4[0] = fmaf(g.x, vm, av4[0]); av4[1] = fmaf(g.y, vm, av4[1]); av4[2] = fmaf(g.z, vm, av4[2]); av4[3] = fmaf(g.w, vm, av4[3]);
        if (TILT && dm.agg_grad) {              // - <dCov / W, Cov> with the stored covariance
          const float4 c = ld4(cv + (size_t)dv * D + c4);
          cc -= g.x * c.x + g.y * c.y + g.z * c.z + g.w * c.w;
        }
      }
      if (D == 64) {                            // two rows per warp pass: the half-warps hold the same columns
#pragma unroll
        for (int i = 0; i < 4; ++i) av4[i] += __shfl_xor_sync(0xffffffffu, av4[i], 16);
      }
      if (lane < D / 4) { float* o = avp + warp * D + lane * 4; o[0] = av4[0]; o[1] = av4[1]; o[2] = av4[2]; o[3] = av4[3]; }
      if (TILT && dm.agg_grad) {
        cc = warp_sum(cc);
        if (lane == 0) atomicAdd(&s_suf, cc);
      }
    }
    if (pl > 0) fetch(pl - 1);
    __syncthreads();
    if (n > 0.f && tid < D) {
      float s = 0.f;
#pragma unroll
      for (int w2 = 0; w2 < 8; ++w2) s += avp[w2 * D + tid];
      av[tid] += s;
    }
    __syncthreads();
    // keys of bucket (j, block pl): every plane >= pl holds them
    for (int u0 = off[pl]; u0 < off[pl + 1]; u0 += kDbQ) {
      const int nk = min(kDbQ, off[pl + 1] - u0);
      for (int e = tid; e < kDbQ * D; e += 256) {
        const int r = e / D, c = e % D;
        ks[e] = r < nk ? to_f(Kb[(size_t)(u0 + r) * D + c]) - k0[c] : 0.f;
        vs[e] = r < nk ? to_f(Vb[(size_t)(u0 + r) * D + c]) : 0.f;
      }
      if (warp < kDbQ) {
        const float l = TILT && warp < nk ? logit(u0 + warp) : 0.f;
        if (lane == 0) { fk[warp] = TILT ? (warp < nk ? expf(l - lmax) : 0.f) : 1.f; dl_s[warp] = 0.f; }
      }
      __syncthreads();
      if (tid < D) {                            // dV_u[dv] = f_u (sum_dk As[dv][dk] k_u[dk] - ak[dv])
        float acc[kDbQ];
#pragma unroll
        for (int a = 0; a < kDbQ; ++a) acc[a] = -ak[tid];
        for (int dk = 0; dk < D; ++dk) {
          const float c = As[tid * (D + 1) + dk];
#pragma unroll
          for (int a = 0; a < kDbQ; ++a) acc[a] = fmaf(c, ks[a * D + dk], acc[a]);
        }
        for (int a = 0; a < nk; ++a) dV_perm[((size_t)pq * dm.N + u0 + a) * D + tid] += fk[a] * acc[a];
        if (TILT && dm.agg_grad) {
#pragma unroll
          for (int a = 0; a < kDbQ; ++a) {      // v_u.(A k_u - a_k) - a_v.k_u  (D == value dims == key dims)
            const float part = warp_sum(vs[a * D + tid] * acc[a] - av[tid] * ks[a * D + tid]);
            if (lane == 0) atomicAdd(&dl_s[a], part);
          }
        }
      } else if (tid < 2 * D) {                 // dK_u[dk] = f_u (sum_dv As[dv][dk] v_u[dv] - av[dk])
        const int dk = tid - D;
        float acc[kDbQ];
#pragma unroll
        for (int a = 0; a < kDbQ; ++a) acc[a] = -av[dk];
        for (int dv = 0; dv < D; ++dv) {
          const float c = As[dv * (D + 1) + dk];
#pragma unroll
          for (int a = 0; a < kDbQ; ++a) acc[a] = fmaf(c, vs[a * D + dv], acc[a]);
        }
        for (int a = 0; a < nk; ++a) dK_perm[((size_t)pq * dm.N + u0 + a) * D + dk] += fk[a] * acc[a];
      }
      __syncthreads();
      if (TILT && dm.agg_grad && tid < D) {     // dK_u += sigma qstar dl_u
        const float s = s_suf;
        for (int a = 0; a < nk; ++a) dK_perm[((size_t)pq * dm.N + u0 + a) * D + tid] += qs_[tid] * fk[a] * (dl_s[a] + s);
      }
      __syncthreads();
    }
  }
}

// ---- host side ------------------------------------------------------------------------------------------------------
DipoleBwdWs dipole_bwd_ws(const Dims& d, Arena& ar) {
  DipoleBwdWs w = {};
  if (!d.dipole || d.SB == 0) return w;
  const size_t pq = (size_t)d.B * d.Hq, rows = pq * d.N, segs = pq * d.SB * d.Cq;
  w.sel_tmp = ar.take<int32_t>(rows * (d.m > 0 ? d.m : 1));
  w.lse_far = ar.take<float>(rows);
  w.zq = ar.take<float>(rows);
  w.dz = ar.take<float>(rows);
  w.delta_far = ar.take<float>(rows);
  w.xq = ar.take<float>(rows * d.D);            // first the recomputed far output, then x_t
  w.corr = ar.take<float>(rows * d.D);
  w.csub = ar.take<float>(d.m > 0 ? rows * d.D : 0);
  w.dcbar = ar.take<float>(segs * d.D * d.D);
  w.dcov = ar.take<float>(pq * d.SB * d.Ck * d.D * d.D);
  w.dpw = ar.take<float>(segs * d.Ck);
  w.dzs = ar.take<float>(segs);
  w.dcbar_bf = ar.take<__nv_bfloat16>(segs * d.D * d.D);      // bf16 copy of dCbar for the tensor-core contractions
  return w;
}

bool dipole_bwd_supported(const Dims& d) {
  const size_t smem = (size_t)(d.D * (d.D + 1) + 8 * d.D + 2 * d.SB * d.D + 2 * kDbQ * d.D + 4 * d.D + d.SB) * sizeof(float);
  return smem <= 200 * 1024;
}

// Before the far-field backward: corr, zq, lse_far are the forward's correction, weight sum and far log-sum-exp.
// Leaves delta_far for the far-field backward, adds the residual path to dQacc and fills dcov and dpw.
template <class T, class ST, int D>
static int dipole_bwd_pre_t(const Dims& d, const T* Q, const T* dO, const float* qbar, const float* LSE, const float* delta,
                            const int32_t* assign_q, const int32_t* off_q, const int32_t* perm_q, const DipolePtrs& dp,
                            const int32_t* goff, const int32_t* pairs, const DipoleBwdWs& w, float* dQacc, int* status,
                            cudaStream_t st) {
  const size_t pq = (size_t)d.B * d.Hq, segs = pq * d.SB * d.Cq;
  const long long rows = (long long)pq * d.N;
  prof_mark("k_dipole_bwd_prep", st);
  k_dipole_bwd_prep<T, D><<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(dO, LSE, w.lse_far, delta, w.corr, w.zq, rows, w.xq, w.delta_far, w.dz);
  MUSE_LAUNCH_OK();
  prof_mark("memset", st);
  MUSE_CUDA_OK(cudaMemsetAsync(w.dcbar, 0, segs * D * D * sizeof(float), st));
  MUSE_CUDA_OK(cudaMemsetAsync(w.dzs, 0, segs * sizeof(float), st));
  MUSE_CUDA_OK(cudaMemsetAsync(w.dpw, 0, segs * d.Ck * sizeof(float), st));
  const size_t rows_b = (size_t)2 * (256 / (D / 4)) * kSegQ * D * sizeof(float);
  const bool f32bar = d.m > 0 || sizeof(ST) == 4;
  const size_t smem = rows_b + (f32bar ? (size_t)D * (D + 4) * sizeof(float) : (size_t)D * (D + 16 / sizeof(ST)) * sizeof(ST));
  prof_mark("k_dipole_bwd_seg", st);
  if (f32bar) {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_dipole_bwd_seg<T, float, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_dipole_bwd_seg<T, float, D><<<dim3(d.Cq, d.SB, (unsigned)pq), 256, smem, st>>>(d, Q, qbar, off_q, perm_q, (const float*)dp.cbar, w.xq,
                                                                                    w.dz, dQacc, w.dcbar, w.dzs);
  } else {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_dipole_bwd_seg<T, ST, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_dipole_bwd_seg<T, ST, D><<<dim3(d.Cq, d.SB, (unsigned)pq), 256, smem, st>>>(d, Q, qbar, off_q, perm_q, (const ST*)dp.cbar, w.xq, w.dz,
                                                                                 dQacc, w.dcbar, w.dzs);
  }
  MUSE_LAUNCH_OK();
  const bool tensor = dipole_bwd_tc_supported(d, sizeof(ST) == 2 ? MUSE_BF16 : MUSE_F32) && !path_forced(kForceDipoleSimt);
  if (d.m > 0 && sizeof(ST) == 2 && dipole_bwd_pairs_tc_supported(d, MUSE_BF16) && !path_forced(kForceDipoleSimt)) {
    int rc = dipole_bwd_pairs_tc(d, Q, qbar, assign_q, goff, pairs, dp.cov, dp.pw, w.xq, w.dz, dQacc, w.dcov, w.dpw, tensor ? 0 : 1,
                                 status, st);
    if (rc != MUSE_OK) return rc;
  } else if (d.m > 0) {
    const size_t spair = (size_t)2 * (256 / (D / 4)) * kPairQ * D * sizeof(float) + (size_t)D * (D + 16 / sizeof(ST)) * sizeof(ST);
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_dipole_bwd_pairs<T, ST, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)spair));
    prof_mark("k_dipole_bwd_pairs", st);
    k_dipole_bwd_pairs<T, ST, D><<<dim3(d.Ck, d.SB, (unsigned)pq), 256, spair, st>>>(d, Q, qbar, assign_q, goff, pairs, (const ST*)dp.cov,
                                                                                   (const ST*)dp.pw, w.xq, w.dz, dQacc, w.dcov, w.dpw);
    MUSE_LAUNCH_OK();
  }
  if (d.m == 0 && !tensor) {                              // the plain kernel adds to dCov; the tensor kernel can overwrite it
    prof_mark("memset", st);
    MUSE_CUDA_OK(cudaMemsetAsync(w.dcov, 0, pq * d.SB * d.Ck * D * D * sizeof(float), st));
  }
  if (tensor) return dipole_bwd_tc(d, dp.pw, dp.cov, w.dcbar, w.dcbar_bf, w.dzs, w.dcov, w.dpw, d.agg_grad, d.m > 0 ? goff : nullptr, status, st);
  prof_mark("k_dipole_dcov", st);
  k_dipole_dcov<ST><<<dim3(D * D / 256, cdiv(d.Ck, kDcJ), (unsigned)(pq * d.SB)), 256, 0, st>>>(d, (const ST*)dp.pw, w.dcbar, w.dcov);
  MUSE_LAUNCH_OK();
  if (d.agg_grad) {
    prof_mark("k_dipole_dpw", st);
    k_dipole_dpw<ST><<<dim3(cdiv(d.Ck, 64), cdiv(d.Cq, 64), (unsigned)(pq * d.SB)), 256, 0, st>>>(d, w.dcbar, (const ST*)dp.cov, w.dzs, w.dpw);
    MUSE_LAUNCH_OK();
  }
  return MUSE_OK;
}

int dipole_bwd_pre(const Dims& d, int dtype, const void* Q, const void* dO, const float* qbar, const float* LSE, const float* delta,
                   const int32_t* assign_q, const int32_t* off_q, const int32_t* perm_q, const DipolePtrs& dp, const int32_t* goff,
                   const int32_t* pairs, const DipoleBwdWs& w, float* dQacc, int* status, cudaStream_t st) {
  typedef __nv_bfloat16 bf;
#define MUSE_DB(TT, SS, DD) dipole_bwd_pre_t<TT, SS, DD>(d, (const TT*)Q, (const TT*)dO, qbar, LSE, delta, assign_q, off_q, perm_q, dp, goff, pairs, w, dQacc, status, st)
  if (dtype == MUSE_F32) return d.D == 64 ? MUSE_DB(float, float, 64) : MUSE_DB(float, float, 128);
  return d.D == 64 ? MUSE_DB(bf, bf, 64) : MUSE_DB(bf, bf, 128);
#undef MUSE_DB
}

// After the far-field backward (which wrote the summary gradient dS): the weights' gradient joins it.
int dipole_bwd_dmu(const Dims& d, int dtype, const DipolePtrs& dp, const DipoleBwdWs& w, float* dS, int grad_by_key_cluster,
                   cudaStream_t st) {
  if (!d.agg_grad) return MUSE_OK;
  const long long rows = (long long)d.B * d.Hq * d.SB * d.Cq;
  prof_mark("k_dipole_dmu", st);
  if (dtype == MUSE_F32) k_dipole_dmu<float><<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(d, (const float*)dp.pw, w.dpw, rows, dS, grad_by_key_cluster);
  else k_dipole_dmu<__nv_bfloat16><<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(d, (const __nv_bfloat16*)dp.pw, w.dpw, rows, dS, grad_by_key_cluster);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

template <class T, class ST, int D>
static int dipole_bwd_keys_t(const Dims& d, const T* Kp, const T* Vp, const int32_t* off_k, const DipolePtrs& dp, const DipoleBwdWs& w,
                             float* dK_perm, float* dV_perm, cudaStream_t st) {
  const size_t smem = (size_t)(D * (D + 1) + 8 * D + 2 * d.SB * D + 2 * kDbQ * D + 4 * D + d.SB) * sizeof(float);
  const dim3 grid(d.Ck, d.B * d.Hq);
  prof_mark("k_dipole_cov_bwd", st);
  if (d.dipole == 2) {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_dipole_cov_bwd<T, ST, D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_dipole_cov_bwd<T, ST, D, true><<<grid, 256, smem, st>>>(d, Kp, Vp, off_k, w.dcov, dp.qstar, (const ST*)dp.cov, dK_perm, dV_perm);
  } else {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_dipole_cov_bwd<T, ST, D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_dipole_cov_bwd<T, ST, D, false><<<grid, 256, smem, st>>>(d, Kp, Vp, off_k, w.dcov, nullptr, (const ST*)dp.cov, dK_perm, dV_perm);
  }
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

// After the key-side pass of the monopole: the covariances' gradient reaches the bucketed keys and values.
int dipole_bwd_keys(const Dims& d, int dtype, const void* Kp, const void* Vp, const int32_t* off_k, const DipolePtrs& dp,
                    const DipoleBwdWs& w, float* dK_perm, float* dV_perm, cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  if (dtype == MUSE_F32) {
    if (d.D == 64) return dipole_bwd_keys_t<float, float, 64>(d, (const float*)Kp, (const float*)Vp, off_k, dp, w, dK_perm, dV_perm, st);
    return dipole_bwd_keys_t<float, float, 128>(d, (const float*)Kp, (const float*)Vp, off_k, dp, w, dK_perm, dV_perm, st);
  }
  if (d.D == 64) return dipole_bwd_keys_t<bf, bf, 64>(d, (const bf*)Kp, (const bf*)Vp, off_k, dp, w, dK_perm, dV_perm, st);
  return dipole_bwd_keys_t<bf, bf, 128>(d, (const bf*)Kp, (const bf*)Vp, off_k, dp, w, dK_perm, dV_perm, st);
}

}  // namespace muse
