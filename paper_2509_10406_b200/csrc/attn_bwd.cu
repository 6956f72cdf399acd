// Backward attention stage.  The merged output is one softmax over {exact keys} U {far
// clusters}, so every component's gradient uses the merged log-sum-exp L and
// delta = dO . O.  Assignments, selections and query centroids are constants (Appendix
// "Centroid Gradient Flow"); agg_grad = 0 also freezes the tilted aggregation weights
// (Appendix "Aggregation Weight Gradient Flow").
#include "common.cuh"
#include "flash_core.cuh"

namespace muse {

int near_bwd(const Dims& d, int dtype, const void* Q, const void* dO, const float* qbar, const float* LSE, const float* delta,
             const int32_t* off_q, const int32_t* perm_q, const int32_t* sel, const int32_t* bsel, const SummPtrs& sp, float* dQacc,
             float* dkappa_b, float* dnu_b, float* dS_b, int grad_ji, cudaStream_t st);
int grad_to_bf16(const float* in, size_t n, void* out, cudaStream_t st);

__device__ __forceinline__ int query_plane_b(const Dims& d, int t) { return d.causal ? t / d.Bs - 1 : 0; }

template <int D>
__device__ __forceinline__ void zero_acc(float a[4][D / 64][4]) {
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int k = 0; k < D / 64; ++k)
#pragma unroll
      for (int c = 0; c < 4; ++c) a[r][k][c] = 0.f;
}

// Like load_tile but converts to fp32 ([64][D+4] floats).
template <class T, int D, class RowFn>
__device__ __forceinline__ void load_tile_f32(float* __restrict__ dst, const T* __restrict__ src, int n, RowFn row_index, int tid) {
  constexpr int LD = D + 4;
  for (int e = tid; e < kTile * (D / 4); e += kFlashThreads) {
    int r = e / (D / 4), q = e % (D / 4);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (r < n) v = ld4(src + (size_t)row_index(r) * D + q * 4);
    st4(dst + r * LD + q * 4, v);
  }
}

// delta_t = sum_d dO[t][d] * O[t][d]; one warp per row.
template <class T, int D>
__global__ void k_delta(const T* __restrict__ O, const T* __restrict__ dO, long long rows, float* __restrict__ delta) {
  const long long r = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= rows) return;
  float s = 0.f;
#pragma unroll
  for (int k = 0; k < D / 32; ++k) s = fmaf(to_f(O[r * D + lane + 32 * k]), to_f(dO[r * D + lane + 32 * k]), s);
  s = warp_sum(s);
  if (lane == 0) delta[r] = s;
}

// ---------------------------------------------------------------------------------------------
// Local (block-diagonal) attention backward.
// ---------------------------------------------------------------------------------------------
template <class T, int D>
__global__ void __launch_bounds__(kFlashThreads)
k_local_bwd_dkdv(Dims dm, const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
                 const T* __restrict__ dO, const float* __restrict__ LSE, const float* __restrict__ delta,
                 float* __restrict__ dK_orig, float* __restrict__ dV_orig) {
  constexpr int LD = D + Pad<T>::v;
  extern __shared__ __align__(16) unsigned char smraw[];
  T* Ks = (T*)smraw; T* Vs = Ks + kTile * LD; T* Qs = Vs + kTile * LD; T* dOs = Qs + kTile * LD;
  float* Ps = (float*)(dOs + kTile * LD);
  __shared__ float Ls[kTile], ds[kTile];
  const int tpb = cdiv(dm.Bs, kTile);
  const int blk = blockIdx.x / tpb, kt = blockIdx.x % tpb, pq = blockIdx.y;
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int bstart = blk * dm.Bs, bend = bstart + dm.Bs;
  const int k0 = bstart + kt * kTile, nk = min(kTile, bend - k0);
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const T* Qb = Q + (size_t)pq * dm.N * D; const T* dOb = dO + (size_t)pq * dm.N * D;
  const T* Kb = K + (size_t)pk * dm.N * D; const T* Vb = V + (size_t)pk * dm.N * D;
  load_tile<T, D>(Ks, Kb, nk, [&](int r) { return k0 + r; }, tid);
  load_tile<T, D>(Vs, Vb, nk, [&](int r) { return k0 + r; }, tid);
  float dk[4][D / 64][4], dv[4][D / 64][4];
  zero_acc<D>(dk); zero_acc<D>(dv);
  for (int q0 = k0; q0 < bend; q0 += kTile) {         // query tiles at or after the key tile
    const int nq = min(kTile, bend - q0);
    __syncthreads();
    load_tile<T, D>(Qs, Qb, nq, [&](int r) { return q0 + r; }, tid);
    load_tile<T, D>(dOs, dOb, nq, [&](int r) { return q0 + r; }, tid);
    if (tid < kTile) {
      Ls[tid] = tid < nq ? LSE[(size_t)pq * dm.N + q0 + tid] : 0.f;
      ds[tid] = tid < nq ? delta[(size_t)pq * dm.N + q0 + tid] : 0.f;
    }
    __syncthreads();
    float s[4][4], dp[4][4];
    mm_nt<T, D>(Qs, Ks, s, ty, tx);
    mm_nt<T, D>(dOs, Vs, dp, ty, tx);
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int row = ty * 4 + r, t = q0 + row;
      float p[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int u = k0 + tx * 4 + c;
        p[c] = (row < nq && tx * 4 + c < nk && u <= t) ? expf(s[r][c] * dm.sigma - Ls[row]) : 0.f;
        dp[r][c] = p[c] * (dp[r][c] - ds[row]);
      }
      st4(Ps + row * kLDP + tx * 4, make_float4(p[0], p[1], p[2], p[3]));
    }
    __syncthreads();
    mm_tn<T, D>(Ps, dOs, dv, ty, tx);
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 4; ++r) st4(Ps + (ty * 4 + r) * kLDP + tx * 4, make_float4(dp[r][0], dp[r][1], dp[r][2], dp[r][3]));
    __syncthreads();
    mm_tn<T, D>(Ps, Qs, dk, ty, tx);
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int row = ty * 4 + r;
    if (row < nk) {
      const size_t u = (size_t)pq * dm.N + k0 + row;
#pragma unroll
      for (int k = 0; k < D / 64; ++k) {
        st4(dK_orig + u * D + tx * 4 + 64 * k, make_float4(dk[r][k][0] * dm.sigma, dk[r][k][1] * dm.sigma, dk[r][k][2] * dm.sigma, dk[r][k][3] * dm.sigma));
        st4(dV_orig + u * D + tx * 4 + 64 * k, make_float4(dv[r][k][0], dv[r][k][1], dv[r][k][2], dv[r][k][3]));
      }
    }
  }
}

template <class T, int D>
__global__ void __launch_bounds__(kFlashThreads)
k_local_bwd_dq(Dims dm, const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
               const T* __restrict__ dO, const float* __restrict__ LSE, const float* __restrict__ delta,
               float* __restrict__ dQacc) {
  constexpr int LD = D + Pad<T>::v;
  extern __shared__ __align__(16) unsigned char smraw[];
  T* Ks = (T*)smraw; T* Vs = Ks + kTile * LD; T* Qs = Vs + kTile * LD; T* dOs = Qs + kTile * LD;
  float* Ps = (float*)(dOs + kTile * LD);
  const int tpb = cdiv(dm.Bs, kTile);
  const int blk = blockIdx.x / tpb, qt = blockIdx.x % tpb, pq = blockIdx.y;
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int bstart = blk * dm.Bs, bend = bstart + dm.Bs;
  const int q0 = bstart + qt * kTile, nq = min(kTile, bend - q0);
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const T* Qb = Q + (size_t)pq * dm.N * D; const T* dOb = dO + (size_t)pq * dm.N * D;
  const T* Kb = K + (size_t)pk * dm.N * D; const T* Vb = V + (size_t)pk * dm.N * D;
  load_tile<T, D>(Qs, Qb, nq, [&](int r) { return q0 + r; }, tid);
  load_tile<T, D>(dOs, dOb, nq, [&](int r) { return q0 + r; }, tid);
  float Lr[4], dr[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int row = ty * 4 + r;
    Lr[r] = row < nq ? LSE[(size_t)pq * dm.N + q0 + row] : 0.f;
    dr[r] = row < nq ? delta[(size_t)pq * dm.N + q0 + row] : 0.f;
  }
  float dq[4][D / 64][4];
  zero_acc<D>(dq);
  const int kend = q0 + nq;
  for (int c0 = bstart; c0 < kend; c0 += kTile) {
    const int nk = min(kTile, kend - c0);
    __syncthreads();
    load_tile<T, D>(Ks, Kb, nk, [&](int r) { return c0 + r; }, tid);
    load_tile<T, D>(Vs, Vb, nk, [&](int r) { return c0 + r; }, tid);
    __syncthreads();
    float s[4][4], dp[4][4];
    mm_nt<T, D>(Qs, Ks, s, ty, tx);
    mm_nt<T, D>(dOs, Vs, dp, ty, tx);
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int row = ty * 4 + r, t = q0 + row;
      float g[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int u = c0 + tx * 4 + c;
        const float p = (row < nq && u <= t && u < kend) ? expf(s[r][c] * dm.sigma - Lr[r]) : 0.f;
        g[c] = p * (dp[r][c] - dr[r]);
      }
      st4(Ps + row * kLDP + tx * 4, make_float4(g[0], g[1], g[2], g[3]));
    }
    __syncthreads();
    mm_pn<T, D>(Ps, Ks, dq, ty, tx);
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int row = ty * 4 + r;
    if (row < nq) {
      const size_t t = (size_t)pq * dm.N + q0 + row;
#pragma unroll
      for (int k = 0; k < D / 64; ++k)
        st4(dQacc + t * D + tx * 4 + 64 * k, make_float4(dq[r][k][0] * dm.sigma, dq[r][k][1] * dm.sigma, dq[r][k][2] * dm.sigma, dq[r][k][3] * dm.sigma));
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Retrieval backward: one CTA per (key cluster j, head).  Key chunks are the outer loop so that
// dK, dV of a chunk accumulate in registers over every plane and query tile that sees it; the
// per-pair dq partials are owned by this CTA (a pair retrieves exactly one cluster).
// ---------------------------------------------------------------------------------------------
template <class T, int D>
__global__ void __launch_bounds__(kFlashThreads)
k_ret_bwd(Dims dm, const T* __restrict__ Q, const T* __restrict__ dO, const T* __restrict__ Kp,
          const T* __restrict__ Vp, const float* __restrict__ LSE, const float* __restrict__ delta,
          const int32_t* __restrict__ off_k, const int32_t* __restrict__ goff, const int32_t* __restrict__ pairs,
          float* __restrict__ dq_part, float* __restrict__ dK_perm, float* __restrict__ dV_perm) {
  constexpr int LD = D + Pad<T>::v;
  extern __shared__ __align__(16) unsigned char smraw[];
  T* Ks = (T*)smraw; T* Vs = Ks + kTile * LD; T* Qs = Vs + kTile * LD; T* dOs = Qs + kTile * LD;
  float* Ps = (float*)(dOs + kTile * LD);
  __shared__ float Ls[kTile], ds[kTile];
  __shared__ int32_t pid_s[kTile];
  const int j = blockIdx.x, pq = blockIdx.y;
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int nkeys = dm.SB * dm.Ck;
  const int32_t* go = goff + (size_t)pq * (nkeys + 1);
  const int32_t* ok = off_k + (size_t)pk * (dm.Ck * dm.S + 1) + (size_t)j * dm.S;
  const int kbeg = ok[0], kvis = ok[dm.SB];          // keys some plane can see
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const T* Qb = Q + (size_t)pq * dm.N * D; const T* dOb = dO + (size_t)pq * dm.N * D;
  const T* Kb = Kp + (size_t)pk * dm.N * D; const T* Vb = Vp + (size_t)pk * dm.N * D;
  const int32_t* pr = pairs + (size_t)pq * dm.N * dm.m;
  for (int c0 = kbeg; c0 < kvis; c0 += kTile) {
    __syncthreads();
    const int nkc = min(kTile, kvis - c0);
    load_tile<T, D>(Ks, Kb, nkc, [&](int r) { return c0 + r; }, tid);
    load_tile<T, D>(Vs, Vb, nkc, [&](int r) { return c0 + r; }, tid);
    float dk[4][D / 64][4], dv[4][D / 64][4];
    zero_acc<D>(dk); zero_acc<D>(dv);
    for (int pl = 0; pl < dm.SB; ++pl) {
      const int vis_end = ok[pl + 1];
      if (c0 >= vis_end) continue;
      const int nk = min(kTile, vis_end - c0);
      const int g0 = go[(size_t)j * dm.SB + pl], g1 = go[(size_t)j * dm.SB + pl + 1];
      for (int t0 = g0; t0 < g1; t0 += kTile) {
        const int nq = min(kTile, g1 - t0);
        __syncthreads();
        if (tid < kTile) {
          const int pid = tid < nq ? pr[t0 + tid] : 0;
          pid_s[tid] = pid;
          const size_t t = (size_t)pq * dm.N + pid / dm.m;
          Ls[tid] = tid < nq ? LSE[t] : 0.f;
          ds[tid] = tid < nq ? delta[t] : 0.f;
        }
        __syncthreads();
        load_tile<T, D>(Qs, Qb, nq, [&](int r) { return pid_s[r] / dm.m; }, tid);
        load_tile<T, D>(dOs, dOb, nq, [&](int r) { return pid_s[r] / dm.m; }, tid);
        __syncthreads();
        float s[4][4], dp[4][4];
        mm_nt<T, D>(Qs, Ks, s, ty, tx);
        mm_nt<T, D>(dOs, Vs, dp, ty, tx);
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int row = ty * 4 + r;
          float p[4];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            p[c] = (row < nq && tx * 4 + c < nk) ? expf(s[r][c] * dm.sigma - Ls[row]) : 0.f;
            dp[r][c] = p[c] * (dp[r][c] - ds[row]);
          }
          st4(Ps + row * kLDP + tx * 4, make_float4(p[0], p[1], p[2], p[3]));
        }
        __syncthreads();
        mm_tn<T, D>(Ps, dOs, dv, ty, tx);
        __syncthreads();
#pragma unroll
        for (int r = 0; r < 4; ++r) st4(Ps + (ty * 4 + r) * kLDP + tx * 4, make_float4(dp[r][0], dp[r][1], dp[r][2], dp[r][3]));
        __syncthreads();
        mm_tn<T, D>(Ps, Qs, dk, ty, tx);
        float dq[4][D / 64][4];
        zero_acc<D>(dq);
        mm_pn<T, D>(Ps, Ks, dq, ty, tx);
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int row = ty * 4 + r;
          if (row < nq) {
            float* dst = dq_part + ((size_t)pq * dm.N * dm.m + pid_s[row]) * D + tx * 4;
#pragma unroll
            for (int k = 0; k < D / 64; ++k) {
              float4 v = make_float4(dq[r][k][0] * dm.sigma, dq[r][k][1] * dm.sigma, dq[r][k][2] * dm.sigma, dq[r][k][3] * dm.sigma);
              if (c0 != kbeg) { float4 o = ld4(dst + 64 * k); v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w; }
              st4(dst + 64 * k, v);
            }
          }
        }
      }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int row = ty * 4 + r;
      if (row < nkc) {
        const size_t u = (size_t)pq * dm.N + c0 + row;
#pragma unroll
        for (int k = 0; k < D / 64; ++k) {
          st4(dK_perm + u * D + tx * 4 + 64 * k, make_float4(dk[r][k][0] * dm.sigma, dk[r][k][1] * dm.sigma, dk[r][k][2] * dm.sigma, dk[r][k][3] * dm.sigma));
          st4(dV_perm + u * D + tx * 4 + 64 * k, make_float4(dv[r][k][0], dv[r][k][1], dv[r][k][2], dv[r][k][3]));
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Far-field backward: one CTA per (query cluster i, plane, head) segment.
//   p_tj = exp(score_tj - L_t) over the far set;  dnu_j += p dO;  g = p (dO.nu_j - delta);
//   dq' += g kappa_j;  dkappa_j += g qres;  dmu_j += g.
// It stores dkappa, dnu and dS := dmu - dkappa.kappa - dnu.nu (the gradient w.r.t. the log of
// the un-normalised mass at fixed un-normalised sums), which is what the key-side pass needs.
// ---------------------------------------------------------------------------------------------
template <class T, int D>
__global__ void __launch_bounds__(kFlashThreads)
k_far_bwd(Dims dm, const T* __restrict__ Q, const T* __restrict__ dO, const float* __restrict__ qbar,
          const float* __restrict__ LSE, const float* __restrict__ delta, const int32_t* __restrict__ off_q,
          const int32_t* __restrict__ perm_q, const int32_t* __restrict__ sel, SummPtrs sp, float* __restrict__ dQacc,
          float* __restrict__ dkappa, float* __restrict__ dnu, float* __restrict__ dS) {
  constexpr int LD = D + 4;
  extern __shared__ __align__(16) unsigned char smraw[];
  float* kap = (float*)smraw; float* nus = kap + kTile * LD; float* qr = nus + kTile * LD; float* dOs = qr + kTile * LD;
  float* Ps = dOs + kTile * LD;
  uint32_t* smask = (uint32_t*)(Ps + kTile * kLDP);   // [64][Ck/32 rounded up]
  __shared__ float Ls[kTile], ds[kTile], mus[kTile], colsum[kTile];
  __shared__ int32_t rows[kTile];
  const int i = blockIdx.x, pl = blockIdx.y, pq = blockIdx.z;
  const int blk = dm.causal ? pl + 1 : 0, Ck = dm.Ck, MW = cdiv(Ck, 32);
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int32_t* oq = off_q + (size_t)pq * (dm.S * dm.Cq + 1) + (size_t)blk * dm.Cq + i;
  const int p0 = oq[0], p1 = oq[1];
  if (p0 >= p1) return;
  const bool single = p1 - p0 <= kTile;
  const size_t ent0 = (((size_t)pq * dm.SB + pl) * dm.Cq + i) * Ck;
  const T* Qb = Q + (size_t)pq * dm.N * D; const T* dOb = dO + (size_t)pq * dm.N * D;
  const float* qb = qbar + ((size_t)pq * dm.Cq + i) * D;
  const int32_t* pm = perm_q + (size_t)pq * dm.N;

  auto load_rows = [&](int r0, int n) {
    if (tid < kTile) {
      const int t = tid < n ? pm[r0 + tid] : -1;
      rows[tid] = t;
      Ls[tid] = t >= 0 ? LSE[(size_t)pq * dm.N + t] : 0.f;
      ds[tid] = t >= 0 ? delta[(size_t)pq * dm.N + t] : 0.f;
    }
    for (int e = tid; e < kTile * MW; e += kFlashThreads) smask[e] = 0u;
    __syncthreads();
    for (int e = tid; e < kTile * (D / 4); e += kFlashThreads) {
      const int r = e / (D / 4), q = e % (D / 4);
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f), g = v;
      if (r < n) {
        float4 x = ld4(Qb + (size_t)rows[r] * D + q * 4), c = ld4(qb + q * 4);
        v = make_float4(dm.sigma * (x.x - c.x), dm.sigma * (x.y - c.y), dm.sigma * (x.z - c.z), dm.sigma * (x.w - c.w));
        g = ld4(dOb + (size_t)rows[r] * D + q * 4);
      }
      st4(qr + r * LD + q * 4, v);
      st4(dOs + r * LD + q * 4, g);
    }
    for (int e = tid; e < n * dm.m; e += kFlashThreads) {
      const int r = e / dm.m, k = e % dm.m;
      const int c = sel[((size_t)pq * dm.N + rows[r]) * dm.m + k];
      if (c >= 0 && c < Ck) atomicOr(&smask[r * MW + (c >> 5)], 1u << (c & 31));
    }
    __syncthreads();
  };

  float dq[4][D / 64][4];
  zero_acc<D>(dq);
  if (single) load_rows(p0, p1 - p0);
  for (int j0 = 0; j0 < Ck; j0 += kTile) {
    __syncthreads();
    for (int e = tid; e < kTile * (D / 4); e += kFlashThreads) {
      const int r = e / (D / 4), q = e % (D / 4);
      float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
      if (j0 + r < Ck) { a = ld_kappa4<T>(sp, (ent0 + j0 + r) * D + q * 4); b = ld_nu4<T>(sp, (ent0 + j0 + r) * D + q * 4); }
      st4(kap + r * LD + q * 4, a);
      st4(nus + r * LD + q * 4, b);
    }
    if (tid < kTile) mus[tid] = j0 + tid < Ck ? sp.mu[ent0 + j0 + tid] : -INFINITY;
    float dka[4][D / 64][4], dnv[4][D / 64][4];
    float dmu_acc = 0.f;                               // threads 0..63: column tid
    zero_acc<D>(dka); zero_acc<D>(dnv);
    for (int r0 = p0; r0 < p1; r0 += kTile) {
      const int n = min(kTile, p1 - r0);
      __syncthreads();
      if (!single) { load_rows(r0, n); zero_acc<D>(dq); }
      float s[4][4], dp[4][4];
      mm_nt<float, D>(qr, kap, s, ty, tx);
      mm_nt<float, D>(dOs, nus, dp, ty, tx);
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int row = ty * 4 + r;
        float p[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int jl = tx * 4 + c, jg = j0 + jl;
          const float mj = mus[jl];
          const bool far = row < n && mj != -INFINITY && !((smask[row * MW + (jg >> 5)] >> (jg & 31)) & 1u);
          p[c] = far ? expf(s[r][c] + mj - Ls[row]) : 0.f;
          dp[r][c] = p[c] * (dp[r][c] - ds[row]);
        }
        st4(Ps + row * kLDP + tx * 4, make_float4(p[0], p[1], p[2], p[3]));
      }
      __syncthreads();
      mm_tn<float, D>(Ps, dOs, dnv, ty, tx);
      __syncthreads();
#pragma unroll
      for (int r = 0; r < 4; ++r) st4(Ps + (ty * 4 + r) * kLDP + tx * 4, make_float4(dp[r][0], dp[r][1], dp[r][2], dp[r][3]));
      __syncthreads();
      mm_tn<float, D>(Ps, qr, dka, ty, tx);
      mm_pn<float, D>(Ps, kap, dq, ty, tx);
      if (tid < kTile) { float cs = 0.f; for (int r = 0; r < kTile; ++r) cs += Ps[r * kLDP + tid]; dmu_acc += cs; }
      if (!single) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int row = ty * 4 + r;
          if (row < n) {
            float* dst = dQacc + ((size_t)pq * dm.N + rows[row]) * D + tx * 4;
#pragma unroll
            for (int k = 0; k < D / 64; ++k) {
              float4 o = ld4(dst + 64 * k);
              o.x += dq[r][k][0] * dm.sigma; o.y += dq[r][k][1] * dm.sigma; o.z += dq[r][k][2] * dm.sigma; o.w += dq[r][k][3] * dm.sigma;
              st4(dst + 64 * k, o);
            }
          }
        }
      }
    }
    // dS_j = dmu_j - dkappa_j . kappa_j - dnu_j . nu_j ; store the chunk's gradients
    if (tid < kTile) colsum[tid] = dmu_acc;
    __syncthreads();
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const int jl = ty * 4 + jj, jg = j0 + jl;
      float dot = 0.f;
#pragma unroll
      for (int k = 0; k < D / 64; ++k) {
        float4 a = ld4(kap + jl * LD + tx * 4 + 64 * k), b = ld4(nus + jl * LD + tx * 4 + 64 * k);
        dot += dka[jj][k][0] * a.x + dka[jj][k][1] * a.y + dka[jj][k][2] * a.z + dka[jj][k][3] * a.w;
        dot += dnv[jj][k][0] * b.x + dnv[jj][k][1] * b.y + dnv[jj][k][2] * b.z + dnv[jj][k][3] * b.w;
      }
      dot = row_sum16(dot);
      if (jg < Ck) {
#pragma unroll
        for (int k = 0; k < D / 64; ++k) {
          st4(dkappa + (ent0 + jg) * D + tx * 4 + 64 * k, make_float4(dka[jj][k][0], dka[jj][k][1], dka[jj][k][2], dka[jj][k][3]));
          st4(dnu + (ent0 + jg) * D + tx * 4 + 64 * k, make_float4(dnv[jj][k][0], dnv[jj][k][1], dnv[jj][k][2], dnv[jj][k][3]));
        }
        if (tx == 0) dS[ent0 + jg] = colsum[jl] - dot;
      }
    }
  }
  if (single) {
    const int n = p1 - p0;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int row = ty * 4 + r;
      if (row < n) {
        float* dst = dQacc + ((size_t)pq * dm.N + rows[row]) * D + tx * 4;
#pragma unroll
        for (int k = 0; k < D / 64; ++k) {
          float4 o = ld4(dst + 64 * k);
          o.x += dq[r][k][0] * dm.sigma; o.y += dq[r][k][1] * dm.sigma; o.z += dq[r][k][2] * dm.sigma; o.w += dq[r][k][3] * dm.sigma;
          st4(dst + 64 * k, o);
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Key-side pass through the accumulated summaries: one CTA per (key cluster j, head).
// For bucket b' (keys of block b') the planes pl >= b' contain it.  With the running suffix
//   GU(b') = sum_{pl >= b'} exp(mu(b') - mu(pl)) dkappa(pl)   (GW, GS likewise from dnu, dS)
// and w_iu = exp(sigma qbar_i . k_u - mu_ij(b')) <= 1:
//   dK_u += sum_i w_iu [ GU_i + agg (GS_i + GU_i . k_u + GW_i . v_u) sigma qbar_i ],  dV_u += sum_i w_iu GW_i.
// ---------------------------------------------------------------------------------------------
template <class T, int D, class GT>     // GT: storage type of the summary gradients (float or bf16)
__global__ void __launch_bounds__(kFlashThreads)
k_summ_bwd(Dims dm, const T* __restrict__ Kp, const T* __restrict__ Vp, const int32_t* __restrict__ off_k,
           const int32_t* __restrict__ off_q, const float* __restrict__ qbar, const float* __restrict__ mu,
           const GT* __restrict__ dkappa, const GT* __restrict__ dnu, const float* __restrict__ dS,
           float* __restrict__ dK_perm, float* __restrict__ dV_perm, int per_block) {
  // per_block = 1: mu and the gradients belong to the PER-BLOCK summaries (two-level retrieval): bucket b' feeds only
  // its own summary, so there is no suffix over the planes (the factor below is zero)
  constexpr int LD = D + 4;
  extern __shared__ __align__(16) unsigned char smraw[];
  float* qb = (float*)smraw; float* GU = qb + kTile * LD; float* GW = GU + kTile * LD;
  float* Ks = GW + kTile * LD; float* Vs = Ks + kTile * LD; float* Ps = Vs + kTile * LD;
  __shared__ float GS[kTile], muref[kTile], fac[kTile];
  __shared__ int live[kTile];
  const int j = blockIdx.x, pq = blockIdx.y;
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int32_t* ok = off_k + (size_t)pk * (dm.Ck * dm.S + 1) + (size_t)j * dm.S;
  const int32_t* oq = off_q + (size_t)pq * (dm.S * dm.Cq + 1);
  const T* Kb = Kp + (size_t)pk * dm.N * D; const T* Vb = Vp + (size_t)pk * dm.N * D;
  if (ok[0] >= ok[dm.SB]) return;                    // no key of this cluster is ever summarised
  for (int i0 = 0; i0 < dm.Cq; i0 += kTile) {
    __syncthreads();
    for (int e = tid; e < kTile * (D / 4); e += kFlashThreads) {
      const int r = e / (D / 4), q = e % (D / 4);
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (i0 + r < dm.Cq) v = ld4(qbar + ((size_t)pq * dm.Cq + i0 + r) * D + q * 4);
      v.x *= dm.sigma; v.y *= dm.sigma; v.z *= dm.sigma; v.w *= dm.sigma;
      st4(qb + r * LD + q * 4, v);
      st4(GU + r * LD + q * 4, make_float4(0.f, 0.f, 0.f, 0.f));
      st4(GW + r * LD + q * 4, make_float4(0.f, 0.f, 0.f, 0.f));
    }
    if (tid < kTile) { GS[tid] = 0.f; muref[tid] = INFINITY; }
    for (int pl = dm.SB - 1; pl >= 0; --pl) {
      __syncthreads();
      // suffix update: G(pl) = grad(pl) + exp(mu(pl) - mu(pl+1)) G(pl+1)
      if (tid < kTile) {
        const int i = i0 + tid;
        float f = 0.f; int lv = 0; float m_here = -INFINITY;
        if (i < dm.Cq) {
          m_here = mu[(((size_t)pq * dm.SB + pl) * dm.Cq + i) * dm.Ck + j];
          f = (per_block || m_here == -INFINITY || muref[tid] == INFINITY) ? 0.f : expf(m_here - muref[tid]);
          const int blk = dm.causal ? pl + 1 : 0;
          lv = (per_block || oq[(size_t)blk * dm.Cq + i + 1] > oq[(size_t)blk * dm.Cq + i]) && m_here != -INFINITY;
        }
        fac[tid] = f; live[tid] = lv;
        if (m_here != -INFINITY) muref[tid] = m_here;
        else if (per_block) muref[tid] = INFINITY;       // an empty bucket has no weights of its own
      }
      __syncthreads();
      for (int e = tid; e < kTile * (D / 4); e += kFlashThreads) {
        const int r = e / (D / 4), q = e % (D / 4);
        float4 u = ld4(GU + r * LD + q * 4), w = ld4(GW + r * LD + q * 4);
        const float f = fac[r];
        u.x *= f; u.y *= f; u.z *= f; u.w *= f; w.x *= f; w.y *= f; w.z *= f; w.w *= f;
        if (live[r]) {
          const size_t ent = (((size_t)pq * dm.SB + pl) * dm.Cq + i0 + r) * dm.Ck + j;
          float4 a = ld4(dkappa + ent * D + q * 4), b = ld4(dnu + ent * D + q * 4);
          u.x += a.x; u.y += a.y; u.z += a.z; u.w += a.w; w.x += b.x; w.y += b.y; w.z += b.z; w.w += b.w;
        }
        st4(GU + r * LD + q * 4, u); st4(GW + r * LD + q * 4, w);
      }
      if (tid < kTile) {
        float g = GS[tid] * fac[tid];
        if (live[tid]) g += dS[(((size_t)pq * dm.SB + pl) * dm.Cq + i0 + tid) * dm.Ck + j];
        GS[tid] = g;
      }
      // keys of bucket pl
      const int kb0 = ok[pl], kb1 = ok[pl + 1];
      for (int c0 = kb0; c0 < kb1; c0 += kTile) {
        const int nk = min(kTile, kb1 - c0);
        __syncthreads();
        load_tile_f32<T, D>(Ks, Kb, nk, [&](int r) { return c0 + r; }, tid);
        load_tile_f32<T, D>(Vs, Vb, nk, [&](int r) { return c0 + r; }, tid);
        __syncthreads();
        float l[4][4], x1[4][4], x2[4][4];
        mm_nt<float, D>(qb, Ks, l, ty, tx);
        mm_nt<float, D>(GU, Ks, x1, ty, tx);
        mm_nt<float, D>(GW, Vs, x2, ty, tx);
        float wc[4][4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int il = ty * 4 + r;
          const float mr = muref[il];
          float w[4];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const bool ok_ = i0 + il < dm.Cq && tx * 4 + c < nk && mr != INFINITY;
            w[c] = ok_ ? expf(l[r][c] - mr) : 0.f;
            wc[r][c] = w[c] * (GS[il] + x1[r][c] + x2[r][c]);
          }
          st4(Ps + il * kLDP + tx * 4, make_float4(w[0], w[1], w[2], w[3]));
        }
        __syncthreads();
        float dk[4][D / 64][4], dv[4][D / 64][4];
        zero_acc<D>(dk); zero_acc<D>(dv);
        mm_tn<float, D>(Ps, GU, dk, ty, tx);
        mm_tn<float, D>(Ps, GW, dv, ty, tx);
        if (dm.agg_grad) {
          __syncthreads();
#pragma unroll
          for (int r = 0; r < 4; ++r) st4(Ps + (ty * 4 + r) * kLDP + tx * 4, make_float4(wc[r][0], wc[r][1], wc[r][2], wc[r][3]));
          __syncthreads();
          mm_tn<float, D>(Ps, qb, dk, ty, tx);
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int row = ty * 4 + r;
          if (row < nk) {
            const size_t u = ((size_t)pq * dm.N + c0 + row) * D + tx * 4;
#pragma unroll
            for (int k = 0; k < D / 64; ++k) {
              float4 a = ld4(dK_perm + u + 64 * k), b = ld4(dV_perm + u + 64 * k);
              a.x += dk[r][k][0]; a.y += dk[r][k][1]; a.z += dk[r][k][2]; a.w += dk[r][k][3];
              b.x += dv[r][k][0]; b.y += dv[r][k][1]; b.z += dv[r][k][2]; b.w += dv[r][k][3];
              st4(dK_perm + u + 64 * k, a); st4(dV_perm + u + 64 * k, b);
            }
          }
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Final assembly
// ---------------------------------------------------------------------------------------------
template <class T, int D, class PT>      // PT: element type of the per-(query, slot) dq partials
__global__ void k_final_dq(Dims dm, const float* __restrict__ dQacc, const PT* __restrict__ dq_part,
                           const int32_t* __restrict__ sel, const int32_t* __restrict__ bsel, int use_ret, T* __restrict__ dQ) {
  const int pq = blockIdx.y;
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (t >= dm.N) return;
  const size_t row = (size_t)pq * dm.N + t;
  float acc[D / 32];
#pragma unroll
  for (int k = 0; k < D / 32; ++k) acc[k] = dQacc[row * D + lane + 32 * k];
  if (use_ret && query_plane_b(dm, t) >= 0) {
    if (bsel == nullptr) {                                 // one partial row per slot
      for (int s = 0; s < dm.m; ++s) {
        const int c = sel[row * dm.m + s];
        if (c < 0 || c >= dm.Ck) continue;                 // "none", or an entry outside [0, Ck), which counts as none
#pragma unroll
        for (int k = 0; k < D / 32; ++k) acc[k] += to_f(dq_part[(row * dm.m + s) * D + lane + 32 * k]);
      }
    } else {                                               // two-level retrieval: one per (slot, chosen block)
      const int kk = dm.k2, pl = query_plane_b(dm, t);
      for (int s = 0; s < dm.m; ++s) {
        const int c = sel[row * dm.m + s];
        if (c < 0 || c >= dm.Ck) continue;
        for (int e = 0; e < kk; ++e) {
          const int bb = bsel[(row * dm.m + s) * kk + e];
          if (bb < 0 || bb > pl) continue;
#pragma unroll
          for (int k = 0; k < D / 32; ++k) acc[k] += to_f(dq_part[((row * dm.m + s) * kk + e) * D + lane + 32 * k]);
        }
      }
    }
  }
#pragma unroll
  for (int k = 0; k < D / 32; ++k) dQ[row * D + lane + 32 * k] = from_f<T>(acc[k]);
}

// dK[u] = sum over the query heads of the group of (local part at u + bucketed part at p), u = perm_k[p].
template <class T, int D>
__global__ void k_final_dkv(Dims dm, const int32_t* __restrict__ perm_k, const float* __restrict__ dK_orig,
                            const float* __restrict__ dV_orig, const float* __restrict__ dK_perm,
                            const float* __restrict__ dV_perm, int use_orig, T* __restrict__ dK, T* __restrict__ dV) {
  const int pk = blockIdx.y, b_ = pk / dm.Hkv, g = pk % dm.Hkv;
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= (long long)dm.N * (D / 4)) return;
  const int p = (int)(e / (D / 4)), q = (int)(e % (D / 4));
  const int u = perm_k[(size_t)pk * dm.N + p];
  if (!MUSE_IN_RANGE(u, dm.N)) return;
  float4 ak = make_float4(0.f, 0.f, 0.f, 0.f), av = ak;
  for (int h = 0; h < dm.Hq; ++h) {
    if (dm.hm.g[h] != g) continue;
    const size_t pq = (size_t)b_ * dm.Hq + h;
    float4 x = ld4(dK_perm + (pq * dm.N + p) * D + q * 4), y = ld4(dV_perm + (pq * dm.N + p) * D + q * 4);
    ak.x += x.x; ak.y += x.y; ak.z += x.z; ak.w += x.w; av.x += y.x; av.y += y.y; av.z += y.z; av.w += y.w;
    if (use_orig) {
      x = ld4(dK_orig + (pq * dm.N + u) * D + q * 4); y = ld4(dV_orig + (pq * dm.N + u) * D + q * 4);
      ak.x += x.x; ak.y += x.y; ak.z += x.z; ak.w += x.w; av.x += y.x; av.y += y.y; av.z += y.z; av.w += y.w;
    }
  }
  st4(dK + ((size_t)pk * dm.N + u) * D + q * 4, ak);
  st4(dV + ((size_t)pk * dm.N + u) * D + q * 4, av);
}

// ---------------------------------------------------------------------------------------------
int local_bwd_tc(const Dims& d, const void* Q, const void* K, const void* V, const void* dO, const float* LSE,
                 const float* delta, float* dQacc, float* dK_orig, float* dV_orig, int* status, cudaStream_t st);
int ret_bwd_tc(const Dims& d, const void* Q, const void* dO, const void* Kp, const void* Vp, const float* LSE,
               const float* delta, const int32_t* off_k, const int32_t* goff, const int32_t* pairs, void* dq_part,
               float* dK_perm, float* dV_perm, int* status, cudaStream_t st);

bool far_bwd_tc_supported(const Dims& d, int dtype);
int far_bwd_tc(const Dims& d, const SummPtrs& sp, const void* Q, const void* dO, const float* qbar, const float* LSE,
               const float* delta, const int32_t* off_q, const int32_t* perm_q, const int32_t* sel, float* dQacc,
               void* dkappa, void* dnu, float* dS, int grad_by_key_cluster, int* status, cudaStream_t st);

bool summ_bwd_tc_supported(const Dims& d, int dtype);
int summ_bwd_tc(const Dims& d, const void* Kp, const void* Vp, const int32_t* off_k, const int32_t* off_q, const float* qbar,
                const float* mu, const void* dkappa, const void* dnu, const float* dS, float* dK_perm, float* dV_perm,
                void* qsplit, int per_block, int* status, cudaStream_t st);

struct BwdWs {
  int32_t *status, *off_q, *perm_q, *sort_scratch, *ret_scratch;
  __nv_bfloat16* qsplit;
  float *delta, *dQacc, *dq_part, *dK_orig, *dV_orig, *dK_perm, *dV_perm, *dkappa, *dnu, *dS;
  float *dkappa_b, *dnu_b, *dS_b;           // gradients of the per-block summaries (two-level retrieval), fp32
  DipoleBwdWs dip;                          // dipole correction
};

static BwdWs bwd_ws(const Dims& d, Arena& ar) {
  BwdWs w;
  const size_t pq = (size_t)d.B * d.Hq, ent = pq * d.SB * d.Cq * d.Ck;
  w.status = ar.take<int32_t>(64);          // ws[0]: non-zero if a bounded device-side wait gave up
  w.off_q = ar.take<int32_t>(pq * (d.S * d.Cq + 1));
  w.perm_q = ar.take<int32_t>(pq * d.N);
  w.sort_scratch = ar.take<int32_t>(pq * sort_ws_elems(d.N, d.Cq * d.S));
  w.ret_scratch = ar.take<int32_t>(pq * ret_index_elems(d));
  w.delta = ar.take<float>(pq * d.N);
  w.dQacc = ar.take<float>(pq * d.N * d.D);
  w.dq_part = ar.take<float>(pq * d.N * d.m * (d.k2 > 0 ? d.k2 : 1) * d.D);
  w.dK_orig = ar.take<float>(pq * d.N * d.D);
  w.dV_orig = ar.take<float>(pq * d.N * d.D);
  w.dK_perm = ar.take<float>(pq * d.N * d.D);
  w.dV_perm = ar.take<float>(pq * d.N * d.D);
  w.dkappa = ar.take<float>(ent * d.D);
  w.dnu = ar.take<float>(ent * d.D);
  w.dS = ar.take<float>(ent);
  w.qsplit = ar.take<__nv_bfloat16>(2 * pq * d.Cq * d.D);
  w.dkappa_b = w.dnu_b = w.dS_b = nullptr;
  if (d.k2 > 0) {
    w.dkappa_b = ar.take<float>(ent * d.D);
    w.dnu_b = ar.take<float>(ent * d.D);
    w.dS_b = ar.take<float>(ent);
  }
  w.dip = dipole_bwd_ws(d, ar);
  return w;
}

size_t attn_bwd_ws_bytes(const Dims& d, int) { Arena ar(nullptr); bwd_ws(d, ar); return ar.used; }

template <class T, int D>
static int attn_bwd_t(const Dims& d, int dtype, const T* Q, const T* K, const T* V, const T* O, const float* LSE,
                      const T* dO, const int32_t* assign_q, const float* qbar, const int32_t* off_k,
                      const int32_t* perm_k, const void* summaries, const int32_t* sel, const int32_t* bsel, T* dQ, T* dK, T* dV,
                      void* ws, cudaStream_t st) {
  Arena ar(ws);
  BwdWs w = bwd_ws(d, ar);
  if (d.k2 == 0) bsel = nullptr;
  const int pq = d.B * d.Hq, pk = d.B * d.Hkv;
  SummLayout L = summ_layout(d, dtype);
  const char* base = (const char*)summaries;
  const T* Kp = (const T*)(base + L.Kp); const T* Vp = (const T*)(base + L.Vp);
  const SummPtrs sp = summ_ptrs(L, base);
  const float* mu = sp.mu;
  const size_t nd = (size_t)pq * d.N * d.D * sizeof(float);
  const long long rows = (long long)pq * d.N;
  prof_mark("k_delta", st);
  k_delta<T, D><<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(O, dO, rows, w.delta);
  MUSE_LAUNCH_OK();
  prof_mark("memset", st);
  MUSE_CUDA_OK(cudaMemsetAsync(w.dK_perm, 0, nd, st));
  MUSE_CUDA_OK(cudaMemsetAsync(w.dV_perm, 0, nd, st));
  const size_t sm4 = 4 * tile_bytes<T, D>() + ptile_bytes();
  constexpr bool kTensor = sizeof(T) == 2;      // bf16 mode runs the exact-attention parts on tcgen05
  if (d.causal && kTensor) {
    int rc = local_bwd_tc(d, Q, K, V, dO, LSE, w.delta, w.dQacc, w.dK_orig, w.dV_orig, w.status, st);
    if (rc != MUSE_OK) return rc;
  } else if (d.causal) {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_local_bwd_dkdv<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm4));
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_local_bwd_dq<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm4));
    dim3 grid(d.S * cdiv(d.Bs, kTile), pq);
    prof_mark("k_local_bwd_dkdv", st);
    k_local_bwd_dkdv<T, D><<<grid, kFlashThreads, sm4, st>>>(d, Q, K, V, dO, LSE, w.delta, w.dK_orig, w.dV_orig);
    MUSE_LAUNCH_OK();
    prof_mark("k_local_bwd_dq", st);
    k_local_bwd_dq<T, D><<<grid, kFlashThreads, sm4, st>>>(d, Q, K, V, dO, LSE, w.delta, w.dQacc);
    MUSE_LAUNCH_OK();
  } else {
    prof_mark("memset", st);
    MUSE_CUDA_OK(cudaMemsetAsync(w.dQacc, 0, nd, st));
  }
  int use_ret = 0;
  if (d.SB > 0) {
    int rc = bucket_sort(0, assign_q, pq, d.N, d.Cq, d.S, d.Bs, 0, w.off_q, w.perm_q, w.sort_scratch, st);
    if (rc != MUSE_OK) return rc;
    RetIndex ri = {};
    if (d.m > 0) {
      rc = build_ret_index(d, sel, bsel, w.ret_scratch, &ri, st);
      if (rc != MUSE_OK) return rc;
      if (kTensor) {
        rc = ret_bwd_tc(d, Q, dO, Kp, Vp, LSE, w.delta, off_k, ri.goff, ri.pairs, w.dq_part, w.dK_perm, w.dV_perm, w.status, st);
        if (rc != MUSE_OK) return rc;
      } else {
        MUSE_CUDA_OK(cudaFuncSetAttribute(k_ret_bwd<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm4));
        prof_mark("k_ret_bwd", st);
        k_ret_bwd<T, D><<<dim3(d.Ck, pq), kFlashThreads, sm4, st>>>(d, Q, dO, Kp, Vp, LSE, w.delta, off_k, ri.goff, ri.pairs,
                                                                  w.dq_part, w.dK_perm, w.dV_perm);
        MUSE_LAUNCH_OK();
      }
      use_ret = 1;
    }
    const float* delta_far = w.delta;
    if (d.dipole) {
      // the forward's far log-sum-exp, correction and weight sums again; then everything of the dipole's backward that
      // does not need the far-field backward's output
      const DipolePtrs dp = dipole_ptrs(L, base);
      rc = far_fwd_again(d, dtype, Q, qbar, w.off_q, w.perm_q, sp, sel, w.dip.sel_tmp, w.dip.xq, w.dip.lse_far, w.status, st);
      if (rc != MUSE_OK) return rc;
      rc = dipole_apply(d, dtype, Q, qbar, assign_q, w.off_q, w.perm_q, dp, w.dip.lse_far, sel, ri.goff, ri.pairs, w.dip.csub, nullptr,
                        w.dip.corr, w.dip.zq, w.status, st);
      if (rc != MUSE_OK) return rc;
      rc = dipole_bwd_pre(d, dtype, Q, dO, qbar, LSE, w.delta, assign_q, w.off_q, w.perm_q, dp, ri.goff, ri.pairs, w.dip, w.dQacc,
                          w.status, st);
      if (rc != MUSE_OK) return rc;
      delta_far = w.dip.delta_far;
    }
    const bool far_tc = far_bwd_tc_supported(d, dtype) && !path_forced(kForceFarSimt);
    const size_t fsm = (size_t)(4 * kTile * (D + 4) + kTile * kLDP) * sizeof(float) + (size_t)kTile * cdiv(d.Ck, 32) * sizeof(uint32_t);
    const bool summ_tc = far_tc && summ_bwd_tc_supported(d, dtype) && !path_forced(kForceSummBwdSimt);
    if (far_tc) {
      rc = far_bwd_tc(d, sp, Q, dO, qbar, LSE, delta_far, w.off_q, w.perm_q, sel, w.dQacc, w.dkappa, w.dnu, w.dS, summ_tc ? 1 : 0, w.status, st);
      if (rc != MUSE_OK) return rc;
    } else {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_far_bwd<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fsm));
    prof_mark("k_far_bwd", st);
    k_far_bwd<T, D><<<dim3(d.Cq, d.SB, pq), kFlashThreads, fsm, st>>>(d, Q, dO, qbar, LSE, delta_far, w.off_q, w.perm_q, sel, sp,
                                                                    w.dQacc, w.dkappa, w.dnu, w.dS);
    MUSE_LAUNCH_OK();
    }
    if (d.dipole) {
      rc = dipole_bwd_dmu(d, dtype, dipole_ptrs(L, base), w.dip, w.dS, summ_tc ? 1 : 0, st);
      if (rc != MUSE_OK) return rc;
    }
    const size_t ssm = (size_t)(5 * kTile * (D + 4) + kTile * kLDP) * sizeof(float);
    if (summ_tc) {
      rc = summ_bwd_tc(d, Kp, Vp, off_k, w.off_q, qbar, mu, w.dkappa, w.dnu, w.dS, w.dK_perm, w.dV_perm, w.qsplit, 0, w.status, st);
      if (rc != MUSE_OK) return rc;
    } else if (far_tc) {
      typedef __nv_bfloat16 GB;
      MUSE_CUDA_OK(cudaFuncSetAttribute(k_summ_bwd<T, D, GB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ssm));
      prof_mark("k_summ_bwd", st);
      k_summ_bwd<T, D, GB><<<dim3(d.Ck, pq), kFlashThreads, ssm, st>>>(d, Kp, Vp, off_k, w.off_q, qbar, mu, (const GB*)w.dkappa,
                                                                     (const GB*)w.dnu, w.dS, w.dK_perm, w.dV_perm, 0);
    } else {
      MUSE_CUDA_OK(cudaFuncSetAttribute(k_summ_bwd<T, D, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ssm));
      prof_mark("k_summ_bwd", st);
      k_summ_bwd<T, D, float><<<dim3(d.Ck, pq), kFlashThreads, ssm, st>>>(d, Kp, Vp, off_k, w.off_q, qbar, mu, w.dkappa, w.dnu, w.dS,
                                                                        w.dK_perm, w.dV_perm, 0);
    }
    MUSE_LAUNCH_OK();
    if (d.dipole) {
      rc = dipole_bwd_keys(d, dtype, Kp, Vp, off_k, dipole_ptrs(L, base), w.dip, w.dK_perm, w.dV_perm, st);
      if (rc != MUSE_OK) return rc;
    }
  }
  if (d.k2 > 0 && d.m > 0 && d.SB > 0) {
    // two-level retrieval: the stand-in keys of the non-retrieved blocks of the selected clusters.  Their gradient goes to dQ
    // directly and to the per-block summaries, from where the key-side pass (per-block mode) carries it to K and V.
    const size_t ent = (size_t)pq * d.SB * d.Cq * d.Ck;
    prof_mark("memset", st);
    MUSE_CUDA_OK(cudaMemsetAsync(w.dkappa_b, 0, ent * d.D * sizeof(float), st));
    MUSE_CUDA_OK(cudaMemsetAsync(w.dnu_b, 0, ent * d.D * sizeof(float), st));
    MUSE_CUDA_OK(cudaMemsetAsync(w.dS_b, 0, ent * sizeof(float), st));
    const SummPtrs spb = summ_ptrs_blk(L, base);
    const bool tcb = summ_bwd_tc_supported(d, dtype) && !path_forced(kForceSummBwdSimt);
    int rc = near_bwd(d, dtype, Q, dO, qbar, LSE, w.delta, w.off_q, w.perm_q, sel, bsel, spb, w.dQacc, w.dkappa_b, w.dnu_b, w.dS_b,
                      tcb ? 1 : 0, st);
    if (rc != MUSE_OK) return rc;
    if (tcb) {
      // tensor-core key-side kernel in per-block mode: its gradient tiles are bf16, laid out [plane][j][i]; the buffers of the
      // accumulated-summary gradients have been consumed by now and take the converted copies
      rc = grad_to_bf16(w.dkappa_b, ent * d.D, w.dkappa, st);
      if (rc == MUSE_OK) rc = grad_to_bf16(w.dnu_b, ent * d.D, w.dnu, st);
      if (rc == MUSE_OK)
        rc = summ_bwd_tc(d, Kp, Vp, off_k, w.off_q, qbar, spb.mu, w.dkappa, w.dnu, w.dS_b, w.dK_perm, w.dV_perm, w.qsplit, 1, w.status, st);
      if (rc != MUSE_OK) return rc;
    } else {
      const size_t ssm = (size_t)(5 * kTile * (D + 4) + kTile * kLDP) * sizeof(float);
      MUSE_CUDA_OK(cudaFuncSetAttribute(k_summ_bwd<T, D, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ssm));
      prof_mark("k_summ_bwd", st);
      k_summ_bwd<T, D, float><<<dim3(d.Ck, pq), kFlashThreads, ssm, st>>>(d, Kp, Vp, off_k, w.off_q, qbar, spb.mu, w.dkappa_b, w.dnu_b, w.dS_b,
                                                                        w.dK_perm, w.dV_perm, 1);
      MUSE_LAUNCH_OK();
    }
  }
  prof_mark("k_final_dq", st);
  if (kTensor)
    k_final_dq<T, D, __nv_bfloat16><<<dim3(cdiv(d.N, 8), pq), 256, 0, st>>>(d, w.dQacc, (const __nv_bfloat16*)w.dq_part, sel, bsel, use_ret, dQ);
  else
    k_final_dq<T, D, float><<<dim3(cdiv(d.N, 8), pq), 256, 0, st>>>(d, w.dQacc, w.dq_part, sel, bsel, use_ret, dQ);
  MUSE_LAUNCH_OK();
  prof_mark("k_final_dkv", st);
  k_final_dkv<T, D><<<dim3(cdiv(d.N * (D / 4), 256), pk), 256, 0, st>>>(d, perm_k, w.dK_orig, w.dV_orig, w.dK_perm, w.dV_perm,
                                                                       d.causal, dK, dV);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

int attn_bwd(const Dims& d, int dtype, const void* Q, const void* K, const void* V, const void* O, const float* LSE,
             const void* dO, const int32_t* assign_q, const float* qbar, const int32_t* off_k, const int32_t* perm_k,
             const void* summaries, const int32_t* sel, const int32_t* bsel, void* dQ, void* dK, void* dV, void* ws,
             cudaStream_t st) {
  typedef __nv_bfloat16 bf;
#define MUSE_BWD(TT, DD) attn_bwd_t<TT, DD>(d, dtype, (const TT*)Q, (const TT*)K, (const TT*)V, (const TT*)O, LSE, (const TT*)dO, \
                                            assign_q, qbar, off_k, perm_k, summaries, sel, bsel, (TT*)dQ, (TT*)dK, (TT*)dV, ws, st)
  if (dtype == MUSE_F32) return d.D == 64 ? MUSE_BWD(float, 64) : MUSE_BWD(float, 128);
  return d.D == 64 ? MUSE_BWD(bf, 64) : MUSE_BWD(bf, 128);
#undef MUSE_BWD
}

}  // namespace muse
