// The retrieved clusters' share of the dipole correction on the tensor cores (bf16 mode; Appendix "Error Analysis",
// "Compatibility with Retrieval"): per (key cluster j, plane, head) group of the retrieval's inverse index
//   out[pair][dv] = p_i(j) * sum_dk Cov_j[dv][dk] * qres[pair][dk]
// is one GEMM [pairs x D] x [D x D].  A CTA loads the group's covariance once by TMA (K-major B operand: rows = value
// dims), then walks the group's (query, slot) pairs in tiles of 128: the warps build the residual rows sigma (q - qbar_i)
// as bf16 in a 128-byte-swizzled shared-memory tile (A operand), one thread issues the D / 16 tcgen05 MMAs, and every
// thread reads its pair's row back from TMEM, scales it by the pair's centroid weight and adds it to the query's row
// with 16-byte vector reductions.  The residuals are rounded to bf16 here, so the kernel that forms
// (Cbar qres - this) / Z rounds them the same way (flag round_q of dipole_apply): the subtraction then still cancels
// exactly what it should.  Every wait is bounded.
#include <cuda.h>
#include "common.cuh"
#include "tc05.cuh"

namespace muse {

typedef __nv_bfloat16 bf16;
int make_tmap_bf16_rows(void* out_map, const void* base, uint64_t rows, uint32_t cols, uint32_t box_rows);

struct SubBars { uint64_t cov, mma; };

template <int D>
__global__ void __launch_bounds__(128)
k_dipole_sub_tc(Dims dm, const bf16* __restrict__ Q, const float* __restrict__ qbar, const int32_t* __restrict__ assign_q,
                const int32_t* __restrict__ goff, const int32_t* __restrict__ pairs, const __grid_constant__ CUtensorMap tm_cov,
                const bf16* __restrict__ pw, float* __restrict__ csub, int* __restrict__ status) {
  constexpr int KH = D / 64;                      // 64-column halves of the K dimension
  constexpr int TA = 128 * 128, TB = D * 128;     // bytes of one half of the A tile (128 pairs) / of the B tile (D value dims)
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ SubBars bars;
  __shared__ uint32_t tbase_s;
  __shared__ int t_s[128], i_s[128];
  __shared__ float p_s[128];
  unsigned char* sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);
  unsigned char* smA = sm;                        // [KH][128 pairs][128 B]
  unsigned char* smB = sm + KH * TA;              // [KH][D value dims][128 B]
  const int j = blockIdx.x, pl = blockIdx.y, pq = blockIdx.z, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int32_t* go = goff + (size_t)pq * (dm.SB * dm.Ck + 1) + (size_t)j * dm.SB + pl;
  const int g0 = go[0], g1 = go[1];
  if (g0 >= g1) return;
  const int pk = (pq / dm.Hq) * dm.Hkv + dm.hm.g[pq % dm.Hq];
  const int pc = dm.dipole == 2 ? pq : pk;
  if (warp == 0) tc::tmem_alloc(&tbase_s, D);
  if (tid == 0) {
    tc::mbar_init(&bars.cov, 1); tc::mbar_init(&bars.mma, 1);
    tc::mbar_init_fence();
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tbase = tbase_s;
  bool ok = true;
  if (tid == 0) {
    const int row = (((pc * dm.SB + pl) * dm.Ck) + j) * D;       // first row (value dim 0) of Cov_j
    tc::mbar_expect_tx(&bars.cov, KH * TB);
    for (int h = 0; h < KH; ++h) tc::tma_load_2d(smB + h * TB, &tm_cov, 64 * h, row, &bars.cov);
  }
  const bf16* Qp = Q + (size_t)pq * dm.N * D;
  const int32_t* aq = assign_q + (size_t)pq * dm.N;
  const int32_t* pr = pairs + (size_t)pq * dm.N * dm.m;
  const bf16* pwb = pw + ((size_t)pq * dm.SB + pl) * dm.Cq * dm.Ck;
  const uint32_t idesc = tc::idesc_bf16(128, D, 0, 0);
  uint32_t nmma = 0;
  for (int r0 = g0; r0 < g1; r0 += 128) {
    {                                             // the pairs of this tile: thread = pair
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
    // residual rows as bf16 into the swizzled A tile: D / 8 lanes per row, one 16-byte chunk each
    constexpr int LPRW = D / 8, RPI = 32 / LPRW;  // lanes per row, rows per warp iteration
    for (int rr = warp * 32; rr < warp * 32 + 32; rr += RPI) {
      const int r = rr + lane / LPRW, ch = lane % LPRW, t = t_s[r];
      uint4 o = make_uint4(0u, 0u, 0u, 0u);
      if (t >= 0) {
        const uint4 qv = *reinterpret_cast<const uint4*>(Qp + (size_t)t * D + ch * 8);
        const float* qb = qbar + ((size_t)pq * dm.Cq + i_s[r]) * D + ch * 8;
        const float4 b0 = ld4(qb), b1 = ld4(qb + 4);
        const uint32_t w[4] = {qv.x, qv.y, qv.z, qv.w};
        const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
        uint32_t ow[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float lo = dm.sigma * (__uint_as_float(w[e] << 16) - bb[2 * e]);
          const float hi = dm.sigma * (__uint_as_float(w[e] & 0xffff0000u) - bb[2 * e + 1]);
          __nv_bfloat162 pk2 = __floats2bfloat162_rn(lo, hi);
          ow[e] = *reinterpret_cast<uint32_t*>(&pk2);
        }
        o = make_uint4(ow[0], ow[1], ow[2], ow[3]);
      }
      *reinterpret_cast<uint4*>(smA + (ch >> 3) * TA + tc::sw128_off(r, ch & 7)) = o;
    }
    tc::fence_async_smem();                       // the tile was written by ordinary stores and is read by the tensor core
    __syncthreads();
    if (tid == 0) {
      if (nmma == 0 && !tc::mbar_wait(&bars.cov, 0)) ok = false;
      tc::fence_after_sync();
      if (ok) {
        const uint32_t a0 = tc::smem_u32(smA), b0 = tc::smem_u32(smB);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc::mma_bf16_ss(tbase, tc::smem_desc_sw128(a0 + (ks >> 2) * TA + (ks & 3) * 32, 16, 1024),
                          tc::smem_desc_sw128(b0 + (ks >> 2) * TB + (ks & 3) * 32, 16, 1024), idesc, ks > 0);
      }
      tc::mma_commit(&bars.mma);
    }
    __syncwarp();
    if (!__all_sync(0xffffffffu, tc::mbar_wait(&bars.mma, nmma & 1) ? 1 : 0)) ok = false;
    ++nmma;
    tc::fence_after_sync();
    const int t = t_s[tid];
    const float p = p_s[tid];
#pragma unroll
    for (int q = 0; q < D / 32; ++q) {
      float v[32];
      tc::tmem_ld32(tbase + ((uint32_t)(warp * 32) << 16) + 32 * q, v);
      if (ok && t >= 0) {
        float* dst = csub + ((size_t)pq * dm.N + t) * D + 32 * q;
#pragma unroll
        for (int c = 0; c < 32; c += 4)
          atomicAdd(reinterpret_cast<float4*>(dst + c), make_float4(p * v[c], p * v[c + 1], p * v[c + 2], p * v[c + 3]));
      }
    }
    tc::fence_before_sync();
    __syncthreads();                              // everyone has read the accumulator and the pair list before the next tile
    tc::fence_after_sync();
    if (!__syncthreads_and(ok ? 1 : 0)) { ok = false; break; }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tbase, D);
  if (!ok && tid == 0) report_status(status, MUSE_STATUS_FAR_FWD_TIMEOUT);
}

// ---- backward: what the retrieved clusters take back, per group of the inverse index (D = 128) -------------------
// Per tile of 128 pairs, with x = w_far dO / Z rows, qres rows and p = p_i(j):
//   v[pair][dk]  = sum_dv x[pair][dv] Cov[dv][dk]        (A = x tile K-major, B = the covariance tile read MN-major)
//   dCov[dv][dk] -= sum_pair p x[pair][dv] qres[pair][dk] (A = (p x) tile and B = qres tile, both read MN-major: K = pairs;
//                                                          accumulated in TMEM over all tiles of the group)
// and per pair dQ -= sigma p v (16-byte reductions), dp -= v . qres + dZ.  x, p x and qres enter as bf16.
struct PairBars { uint64_t cov, mma; };

__global__ void __launch_bounds__(128)
k_dipole_bwd_pairs_tc(Dims dm, const bf16* __restrict__ Q, const float* __restrict__ qbar, const int32_t* __restrict__ assign_q,
                      const int32_t* __restrict__ goff, const int32_t* __restrict__ pairs, const __grid_constant__ CUtensorMap tm_cov,
                      const bf16* __restrict__ pw, const float* __restrict__ xq, const float* __restrict__ dz,
                      float* __restrict__ dQacc, float* __restrict__ dcov, float* __restrict__ dpw, int fill_empty,
                      int* __restrict__ status) {
  constexpr int D = 128, TA = 128 * 128;          // one 64-column half of a [128 rows][D] bf16 tile
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ PairBars bars;
  __shared__ uint32_t tbase_s;
  __shared__ int t_s[128], i_s[128];
  __shared__ float p_s[128];
  unsigned char* sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);
  unsigned char* smX = sm;                        // x rows            [2][128 pairs][128 B]
  unsigned char* smP = sm + 2 * TA;               // p * x rows
  unsigned char* smQ = sm + 4 * TA;               // residual rows
  unsigned char* smB = sm + 6 * TA;               // covariance        [2][128 value dims][128 B]
  const int j = blockIdx.x, pl = blockIdx.y, pq = blockIdx.z, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int32_t* go = goff + (size_t)pq * (dm.SB * dm.Ck + 1) + (size_t)j * dm.SB + pl;
  const int g0 = go[0], g1 = go[1];
  float* out = dcov + (((size_t)pq * dm.SB + pl) * dm.Ck + j) * D * D;
  if (g0 >= g1) {                                 // no pair retrieved this cluster in this plane: its share is zero
    if (fill_empty)                               // (the tensor-core contraction that follows overwrites such rows itself)
      for (int e = tid; e < D * D / 4; e += 128) reinterpret_cast<float4*>(out)[e] = make_float4(0.f, 0.f, 0.f, 0.f);
    return;
  }
  const int pk = (pq / dm.Hq) * dm.Hkv + dm.hm.g[pq % dm.Hq];
  const int pc = dm.dipole == 2 ? pq : pk;
  if (warp == 0) tc::tmem_alloc(&tbase_s, 256);
  if (tid == 0) {
    tc::mbar_init(&bars.cov, 1); tc::mbar_init(&bars.mma, 1);
    tc::mbar_init_fence();
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tbase = tbase_s;
  bool ok = true;
  if (tid == 0) {
    const int row = (((pc * dm.SB + pl) * dm.Ck) + j) * D;
    tc::mbar_expect_tx(&bars.cov, 2 * TA);
    for (int h = 0; h < 2; ++h) tc::tma_load_2d(smB + h * TA, &tm_cov, 64 * h, row, &bars.cov);
  }
  const bf16* Qp = Q + (size_t)pq * dm.N * D;
  const int32_t* aq = assign_q + (size_t)pq * dm.N;
  const int32_t* pr = pairs + (size_t)pq * dm.N * dm.m;
  const size_t prow = ((size_t)pq * dm.SB + pl) * dm.Cq;
  const uint32_t idesc_a = tc::idesc_bf16(128, D, 0, 1), idesc_b = tc::idesc_bf16(128, D, 1, 1);
  uint32_t nmma = 0;
  for (int r0 = g0; r0 < g1; r0 += 128) {
    {
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
    // the three operand tiles, 16 lanes per pair row, one 16-byte chunk of 8 elements each
    for (int rr = warp * 32; rr < warp * 32 + 32; rr += 2) {
      const int r = rr + (lane >> 4), ch = lane & 15, t = t_s[r];
      uint4 ox = make_uint4(0u, 0u, 0u, 0u), op = ox, oq = ox;
      if (t >= 0) {
        const float p = p_s[r];
        const uint4 qv = *reinterpret_cast<const uint4*>(Qp + (size_t)t * D + ch * 8);
        const float* qb = qbar + ((size_t)pq * dm.Cq + i_s[r]) * D + ch * 8;
        const float* xr = xq + ((size_t)pq * dm.N + t) * D + ch * 8;
        const float4 b0 = ld4(qb), b1 = ld4(qb + 4), x0 = ld4(xr), x1 = ld4(xr + 4);
        const uint32_t w[4] = {qv.x, qv.y, qv.z, qv.w};
        const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
        const float xx[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
        uint32_t wq[4], wx[4], wp[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          __nv_bfloat162 a = __floats2bfloat162_rn(dm.sigma * (__uint_as_float(w[e] << 16) - bb[2 * e]),
                                                   dm.sigma * (__uint_as_float(w[e] & 0xffff0000u) - bb[2 * e + 1]));
          __nv_bfloat162 b = __floats2bfloat162_rn(xx[2 * e], xx[2 * e + 1]);
          __nv_bfloat162 c = __floats2bfloat162_rn(p * xx[2 * e], p * xx[2 * e + 1]);
          wq[e] = *reinterpret_cast<uint32_t*>(&a); wx[e] = *reinterpret_cast<uint32_t*>(&b); wp[e] = *reinterpret_cast<uint32_t*>(&c);
        }
        oq = make_uint4(wq[0], wq[1], wq[2], wq[3]); ox = make_uint4(wx[0], wx[1], wx[2], wx[3]); op = make_uint4(wp[0], wp[1], wp[2], wp[3]);
      }
      const uint32_t at = (ch >> 3) * TA + tc::sw128_off(r, ch & 7);
      *reinterpret_cast<uint4*>(smX + at) = ox;
      *reinterpret_cast<uint4*>(smP + at) = op;
      *reinterpret_cast<uint4*>(smQ + at) = oq;
    }
    tc::fence_async_smem();
    __syncthreads();
    if (tid == 0) {
      if (nmma == 0 && !tc::mbar_wait(&bars.cov, 0)) ok = false;
      tc::fence_after_sync();
      if (ok) {
        const uint32_t x0 = tc::smem_u32(smX), p0 = tc::smem_u32(smP), q0 = tc::smem_u32(smQ), b0 = tc::smem_u32(smB);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)            // v = x Cov: K = value dims
          tc::mma_bf16_ss(tbase, tc::smem_desc_sw128(x0 + (ks >> 2) * TA + (ks & 3) * 32, 16, 1024),
                          tc::smem_desc_sw128(b0 + ks * 16 * 128, TA, 1024), idesc_a, ks > 0);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)            // dCov += (p x)^T qres: K = pairs
          tc::mma_bf16_ss(tbase + 128, tc::smem_desc_sw128(p0 + ks * 16 * 128, TA, 1024),
                          tc::smem_desc_sw128(q0 + ks * 16 * 128, TA, 1024), idesc_b, nmma > 0 || ks > 0);
      }
      tc::mma_commit(&bars.mma);
    }
    __syncwarp();
    if (!__all_sync(0xffffffffu, tc::mbar_wait(&bars.mma, nmma & 1) ? 1 : 0)) ok = false;
    ++nmma;
    tc::fence_after_sync();
    const int t = t_s[tid];
    const float f = -dm.sigma * p_s[tid];
    float s = 0.f;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float v[32];
      tc::tmem_ld32(tbase + ((uint32_t)(warp * 32) << 16) + 32 * q, v);
      if (ok && t >= 0) {
        float* dst = dQacc + ((size_t)pq * dm.N + t) * D + 32 * q;
#pragma unroll
        for (int c = 0; c < 32; c += 8) {
          const int ch = (32 * q + c) >> 3;       // the pair's residuals back from its (swizzled) tile row
          const uint4 qq = *reinterpret_cast<const uint4*>(smQ + (ch >> 3) * TA + tc::sw128_off(tid, ch & 7));
          const uint32_t w[4] = {qq.x, qq.y, qq.z, qq.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            s = fmaf(v[c + 2 * e], __uint_as_float(w[e] << 16), s);
            s = fmaf(v[c + 2 * e + 1], __uint_as_float(w[e] & 0xffff0000u), s);
          }
          atomicAdd(reinterpret_cast<float4*>(dst + c), make_float4(f * v[c], f * v[c + 1], f * v[c + 2], f * v[c + 3]));
          atomicAdd(reinterpret_cast<float4*>(dst + c + 4), make_float4(f * v[c + 4], f * v[c + 5], f * v[c + 6], f * v[c + 7]));
        }
      }
    }
    if (ok && t >= 0) atomicAdd(&dpw[(prow + i_s[tid]) * dm.Ck + j], -(s + dz[(size_t)pq * dm.N + t]));
    tc::fence_before_sync();
    __syncthreads();                              // the tiles and the accumulator of v are free for the next tile
    tc::fence_after_sync();
    if (!__syncthreads_and(ok ? 1 : 0)) { ok = false; break; }
  }
  // the group's share, negated; the dense part is added on top of it afterwards.  thread = value dim
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    float v[32];
    tc::tmem_ld32(tbase + 128 + ((uint32_t)(warp * 32) << 16) + 32 * q, v);
#pragma unroll
    for (int c = 0; c < 32; c += 4)
      st4(out + (size_t)tid * D + 32 * q + c, ok ? make_float4(-v[c], -v[c + 1], -v[c + 2], -v[c + 3]) : make_float4(0.f, 0.f, 0.f, 0.f));
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tbase, 256);
  if (!ok && tid == 0) report_status(status, MUSE_STATUS_FAR_BWD_TIMEOUT);
}

bool dipole_bwd_pairs_tc_supported(const Dims& d, int dtype) {
  const long long rows = (long long)d.B * (d.dipole == 2 ? d.Hq : d.Hkv) * d.SB * d.Ck * d.D;
  return dtype == MUSE_BF16 && d.D == 128 && rows < (1ll << 31);
}

int dipole_bwd_pairs_tc(const Dims& d, const void* Q, const float* qbar, const int32_t* assign_q, const int32_t* goff,
                        const int32_t* pairs, const void* cov, const void* pw, const float* xq, const float* dz, float* dQacc,
                        float* dcov, float* dpw, int fill_empty, int* status, cudaStream_t st) {
  CUtensorMap tm;
  const uint64_t rows = (uint64_t)d.B * (d.dipole == 2 ? d.Hq : d.Hkv) * d.SB * d.Ck * d.D;
  int rc = make_tmap_bf16_rows(&tm, cov, rows, d.D, d.D);
  if (rc != MUSE_OK) return rc;
  const size_t smem = (size_t)8 * 128 * 128 + 1024;
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_dipole_bwd_pairs_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  prof_mark("k_dipole_bwd_pairs_tc", st);
  k_dipole_bwd_pairs_tc<<<dim3(d.Ck, d.SB, d.B * d.Hq), 128, smem, st>>>(d, (const bf16*)Q, qbar, assign_q, goff, pairs, tm, (const bf16*)pw,
                                                                        xq, dz, dQacc, dcov, dpw, fill_empty, status);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

bool dipole_sub_tc_supported(const Dims& d, int dtype) {
  const long long rows = (long long)d.B * (d.dipole == 2 ? d.Hq : d.Hkv) * d.SB * d.Ck * d.D;
  return dtype == MUSE_BF16 && rows < (1ll << 31);
}

template <int D>
static int dipole_sub_tc_t(const Dims& d, const void* Q, const float* qbar, const int32_t* assign_q, const int32_t* goff,
                           const int32_t* pairs, const void* cov, const void* pw, float* csub, int* status, cudaStream_t st) {
  CUtensorMap tm;
  const uint64_t rows = (uint64_t)d.B * (d.dipole == 2 ? d.Hq : d.Hkv) * d.SB * d.Ck * D;
  int rc = make_tmap_bf16_rows(&tm, cov, rows, D, D);
  if (rc != MUSE_OK) return rc;
  const size_t smem = (size_t)(D / 64) * (128 * 128 + D * 128) + 1024;
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_dipole_sub_tc<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  prof_mark("k_dipole_sub_tc", st);
  k_dipole_sub_tc<D><<<dim3(d.Ck, d.SB, d.B * d.Hq), 128, smem, st>>>(d, (const bf16*)Q, qbar, assign_q, goff, pairs, tm, (const bf16*)pw,
                                                                     csub, status);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

int dipole_sub_tc(const Dims& d, const void* Q, const float* qbar, const int32_t* assign_q, const int32_t* goff, const int32_t* pairs,
                  const void* cov, const void* pw, float* csub, int* status, cudaStream_t st) {
  if (d.D == 64) return dipole_sub_tc_t<64>(d, Q, qbar, assign_q, goff, pairs, cov, pw, csub, status, st);
  return dipole_sub_tc_t<128>(d, Q, qbar, assign_q, goff, pairs, cov, pw, csub, status, st);
}

}  // namespace muse
