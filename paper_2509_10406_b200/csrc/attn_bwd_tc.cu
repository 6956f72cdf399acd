// Exact-attention backward on the Blackwell tensor cores (bf16 inputs, fp32 accumulation in
// tensor memory), for the local block-diagonal component and the retrieved-cluster component.
// With L the merged log-sum-exp and delta = dO.O (Appendix "Centroid Gradient Flow" fixes what
// is constant):  P = exp(sigma q.k - L),  G = P (dO.v - delta),
//                dV = P^T dO,  dK = sigma G^T Q,  dQ = sigma G K.
// Two tile routines, one thread per accumulator row:
//   rows-on-M (dQ):      S = Q K^T, dP = dO V^T -> G (bf16, smem) -> dQ += G K      (TMEM)
//   keys-on-M (dK, dV):  S^T = K Q^T, dP^T = V dO^T -> P^T, G^T -> dV += P^T dO, dK += G^T Q
// Operand tiles are 128-byte-swizzled in shared memory; a [rows][D] tile serves both as a
// K-major operand (contraction over D) and as an MN-major operand (contraction over rows).
#include <cuda.h>
#include "common.cuh"
#include "tc05.cuh"


namespace muse {

typedef __nv_bfloat16 bf16;
int make_tmap_bf16_rows(void* out_map, const void* base, uint64_t rows, uint32_t cols, uint32_t box_rows);
constexpr int kBM = 128, kBN = 64;
constexpr float kLog2e = 1.4426950408889634f;

template <int D, int ROWS, int NT = 128, class RowPtr>
__device__ __forceinline__ void fill_tile(unsigned char* dst, int n, RowPtr row_ptr, int tid) {
  constexpr int CPR = D / 8;
  for (int e = tid; e < ROWS * CPR; e += NT) {
    const int r = e / CPR, ck = e % CPR, kb = ck >> 3, c = ck & 7;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (r < n) v = reinterpret_cast<const uint4*>(row_ptr(r))[ck];
    *reinterpret_cast<uint4*>(dst + kb * ROWS * 128 + tc::sw128_off(r, c)) = v;
  }
}

// A [ROWS][D] tile held in registers between its global loads and its shared-memory stores, so
// that the loads of the next tile are in flight while the tensor core works on the current one.
template <int D, int ROWS, int NT = 128> struct TileRegs { static constexpr int N = ROWS * (D / 8) / NT; uint4 v[N]; };
template <int D, int ROWS, int NT = 128, class RowPtr>
__device__ __forceinline__ void tile_ldg(TileRegs<D, ROWS, NT>& t, int n, RowPtr row_ptr, int tid) {
  constexpr int CPR = D / 8;
#pragma unroll
  for (int k = 0; k < TileRegs<D, ROWS, NT>::N; ++k) {
    const int e = tid + NT * k, r = e / CPR, ck = e % CPR;
    t.v[k] = r < n ? __ldg(reinterpret_cast<const uint4*>(row_ptr(r)) + ck) : make_uint4(0u, 0u, 0u, 0u);
  }
}
template <int D, int ROWS, int NT = 128>
__device__ __forceinline__ void tile_sts(const TileRegs<D, ROWS, NT>& t, unsigned char* dst, int tid) {
  constexpr int CPR = D / 8;
#pragma unroll
  for (int k = 0; k < TileRegs<D, ROWS, NT>::N; ++k) {
    const int e = tid + NT * k, r = e / CPR, ck = e % CPR;
    *reinterpret_cast<uint4*>(dst + (ck >> 3) * ROWS * 128 + tc::sw128_off(r, ck & 7)) = t.v[k];
  }
}

// K-major view of a [ROWS][D] tile at k-step ks (16 elements of D)
template <int ROWS> __device__ __forceinline__ uint64_t desc_k(uint32_t base, int ks) {
  return tc::smem_desc_sw128(base + (ks / 4) * ROWS * 128 + (ks % 4) * 32, 16, 1024);
}
// MN-major view of a [ROWS][D] tile at k-step ks (16 rows)
template <int ROWS> __device__ __forceinline__ uint64_t desc_mn(uint32_t base, int ks) {
  return tc::smem_desc_sw128(base + ks * 16 * 128, ROWS * 128, 1024);
}

struct BwdCtx {
#ifdef MUSE_PHASE_CLOCKS
  long long pc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#endif
  unsigned char* sm;
  uint64_t* bar;
  uint32_t tbase, ph0, ph1;
  bool ok;
};

__device__ __forceinline__ void bwd_setup(BwdCtx& c, unsigned char* sm_raw, uint64_t* bar, uint32_t* tbase_s, uint32_t cols, int tid) {
  c.sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);
  c.bar = bar; c.ph0 = c.ph1 = 0; c.ok = true;
  if ((tid >> 5) == 0) tc::tmem_alloc(tbase_s, cols);
  if (tid == 0) { tc::mbar_init(&bar[0], 1); tc::mbar_init(&bar[1], 1); tc::mbar_init_fence(); }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  c.tbase = *tbase_s;
}
__device__ __forceinline__ void bwd_teardown(BwdCtx& c, uint32_t cols, int tid, int* status) {
  tc::fence_before_sync();
  __syncthreads();
  if ((tid >> 5) == 0) tc::tmem_dealloc(c.tbase, cols);
  if (!c.ok && tid == 0) report_status(status, 2);
}

__device__ __forceinline__ void store_row64(unsigned char* tile, int row, const float (&x)[kBN]) {
#pragma unroll
  for (int ch = 0; ch < kBN / 8; ++ch) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      __nv_bfloat162 b = __floats2bfloat162_rn(x[ch * 8 + 2 * k], x[ch * 8 + 2 * k + 1]);
      w[k] = *reinterpret_cast<uint32_t*>(&b);
    }
    *reinterpret_cast<uint4*>(tile + tc::sw128_off(row, ch)) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// half a row (32 columns, chunks 4*half .. 4*half+3) of a [128][64] bf16 tile
__device__ __forceinline__ void store_row32(unsigned char* tile, int row, int half, const float (&x)[32]) {
#pragma unroll
  for (int ch = 0; ch < 4; ++ch) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      __nv_bfloat162 b = __floats2bfloat162_rn(x[ch * 8 + 2 * k], x[ch * 8 + 2 * k + 1]);
      w[k] = *reinterpret_cast<uint32_t*>(&b);
    }
    *reinterpret_cast<uint4*>(tile + tc::sw128_off(row, 4 * half + ch)) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// ================================================================================================
// rows-on-M: dQ of 128 rows (Q, dO tiles already in shared memory) against keys [k_lo, k_hi)
// ================================================================================================
constexpr int kRowsThreads = 256;       // rows-on-M kernels: two warpgroups share the 64 key columns

template <int D> struct RowsSmem {
  // the G tile reuses the V tile's bytes: V is dead once the S / dP products have completed
  static constexpr int q = 0, dO = q + kBM * D * 2, k = dO + kBM * D * 2, v = k + kBN * D * 2, g = v,
                       total = v + (kBN * D * 2 > kBM * kBN * 2 ? kBN * D * 2 : kBM * kBN * 2) + 1024;
  static constexpr uint32_t cols = 256;       // S 64 | dP 64 | dQ D
};

template <int D, class Limit>
__device__ __forceinline__ bool dq_rows_tc(BwdCtx& c, const bf16* __restrict__ Kb, const bf16* __restrict__ Vb, int k_lo,
                                           int k_hi, Limit limit, float scale2, float L2, float delta, int tid) {
  typedef RowsSmem<D> SM;
  const int warp = tid >> 5, wg = tid >> 7, row = tid & 127;       // 256 threads: warpgroup wg owns key columns [32 wg, +32)
  const uint32_t t_s = c.tbase + ((uint32_t)((warp & 3) * 32) << 16), t_dp = t_s + kBN;
  const uint32_t qa = tc::smem_u32(c.sm + SM::q), da = tc::smem_u32(c.sm + SM::dO), ka = tc::smem_u32(c.sm + SM::k),
                 va = tc::smem_u32(c.sm + SM::v), ga = tc::smem_u32(c.sm + SM::g);
  const int my_limit = limit(row);
  bool first = true;
  TileRegs<D, kBN, kRowsThreads> kreg, vreg;
  if (k_lo < k_hi) {
    tile_ldg<D, kBN, kRowsThreads>(kreg, min(kBN, k_hi - k_lo), [&](int r) { return Kb + (size_t)(k_lo + r) * D; }, tid);
    tile_ldg<D, kBN, kRowsThreads>(vreg, min(kBN, k_hi - k_lo), [&](int r) { return Vb + (size_t)(k_lo + r) * D; }, tid);
  }
  for (int c0 = k_lo; c0 < k_hi && c.ok; c0 += kBN) {
    const int nk = min(kBN, k_hi - c0);
    tile_sts<D, kBN, kRowsThreads>(kreg, c.sm + SM::k, tid);
    tile_sts<D, kBN, kRowsThreads>(vreg, c.sm + SM::v, tid);
    tc::fence_async_smem();
    tc::fence_before_sync();
    __syncthreads();
    if (tid == 0) {
      tc::fence_after_sync();
      const uint32_t idesc = tc::idesc_bf16(kBM, kBN, 0, 0);
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) tc::mma_bf16_ss(c.tbase, desc_k<kBM>(qa, ks), desc_k<kBN>(ka, ks), idesc, ks > 0);
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) tc::mma_bf16_ss(c.tbase + kBN, desc_k<kBM>(da, ks), desc_k<kBN>(va, ks), idesc, ks > 0);
      tc::mma_commit(&c.bar[0]);
    }
    if (c0 + kBN < k_hi) {                   // next key tile: loads fly while the MMAs and the softmax piece run
      const int cn = c0 + kBN, nn = min(kBN, k_hi - cn);
      tile_ldg<D, kBN, kRowsThreads>(kreg, nn, [&](int r) { return Kb + (size_t)(cn + r) * D; }, tid);
      tile_ldg<D, kBN, kRowsThreads>(vreg, nn, [&](int r) { return Vb + (size_t)(cn + r) * D; }, tid);
    }
    if (!tc::mbar_wait(&c.bar[0], c.ph0)) { c.ok = false; break; }
    c.ph0 ^= 1;
    tc::fence_after_sync();
    const int vis = min(nk, my_limit - c0 + 1);
    {
      float s[32], dp[32], g[32];
      tc::tmem_ld32(t_s + 32 * wg, s);
      tc::tmem_ld32(t_dp + 32 * wg, dp);
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const float e = tc::fast_exp2(s[i] * scale2 - L2);
        g[i] = ((32 * wg + i) < vis ? e : 0.f) * (dp[i] - delta);
      }
      store_row32(c.sm + SM::g, row, wg, g);
    }
    tc::fence_async_smem();
    tc::fence_before_sync();
    __syncthreads();
    if (tid == 0) {
      tc::fence_after_sync();
      const uint32_t idesc = tc::idesc_bf16(kBM, D, 0, 1);
#pragma unroll
      for (int ks = 0; ks < kBN / 16; ++ks)
        tc::mma_bf16_ss(c.tbase + 2 * kBN, tc::smem_desc_sw128(ga + ks * 32, 16, 1024), desc_mn<kBN>(ka, ks), idesc, !(first && ks == 0));
      tc::mma_commit(&c.bar[1]);
    }
    first = false;
    if (!tc::mbar_wait(&c.bar[1], c.ph1)) { c.ok = false; break; }
    c.ph1 ^= 1;
    tc::fence_after_sync();
  }
  return !first;          // false: no key tile was processed, the accumulator holds nothing
}

// Reads this thread's accumulator row (D columns starting at column `col`), scales it by `f`
// and, if `write`, stores it.  The TMEM load is warp-collective, so EVERY thread of the CTA
// must call this; only the global store is predicated.
template <int D>
__device__ __forceinline__ void read_acc_row(const BwdCtx& c, uint32_t col, float f, float* __restrict__ dst, bool write, int tid) {
  const uint32_t t = c.tbase + ((uint32_t)(((tid >> 5) & 3) * 32) << 16) + col;
#pragma unroll
  for (int d0 = 0; d0 < D; d0 += 32) {
    float v[32];
    tc::tmem_ld32(t + d0, v);
    if (write) {
#pragma unroll
      for (int i = 0; i < 32; i += 4)
        *reinterpret_cast<float4*>(dst + d0 + i) = make_float4(v[i] * f, v[i + 1] * f, v[i + 2] * f, v[i + 3] * f);
    }
  }
}

template <int D>
__global__ void __launch_bounds__(kRowsThreads)
k_local_bwd_dq_tc(Dims dm, const bf16* __restrict__ Q, const bf16* __restrict__ K, const bf16* __restrict__ V,
                  const bf16* __restrict__ dO, const float* __restrict__ LSE, const float* __restrict__ delta,
                  float* __restrict__ dQacc, int* __restrict__ status) {
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ uint64_t bar[2];
  __shared__ uint32_t tbase_s;
  const int tid = threadIdx.x, row = tid & 127, wg = tid >> 7;
  BwdCtx c;
  bwd_setup(c, sm_raw, bar, &tbase_s, RowsSmem<D>::cols, tid);
  const int tpb = cdiv(dm.Bs, kBM);
  const int lin = blockIdx.x, qt = tpb - 1 - lin / dm.S, blk = lin % dm.S, pq = blockIdx.y;
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int bstart = blk * dm.Bs, bend = bstart + dm.Bs;
  const int q0 = bstart + qt * kBM, nq = min(kBM, bend - q0);
  const bf16* Qb = Q + (size_t)pq * dm.N * D; const bf16* dOb = dO + (size_t)pq * dm.N * D;
  const bf16* Kb = K + (size_t)pk * dm.N * D; const bf16* Vb = V + (size_t)pk * dm.N * D;
  fill_tile<D, kBM, kRowsThreads>(c.sm + RowsSmem<D>::q, nq, [&](int r) { return Qb + (size_t)(q0 + r) * D; }, tid);
  fill_tile<D, kBM, kRowsThreads>(c.sm + RowsSmem<D>::dO, nq, [&](int r) { return dOb + (size_t)(q0 + r) * D; }, tid);
  const size_t t = (size_t)pq * dm.N + q0 + row;
  const float L2 = row < nq ? LSE[t] * kLog2e : 0.f, dl = row < nq ? delta[t] : 0.f;
  dq_rows_tc<D>(c, Kb, Vb, bstart, q0 + nq, [&](int r) { return q0 + r; }, dm.sigma * kLog2e, L2, dl, tid);
  if (c.ok) read_acc_row<D / 2>(c, 2 * kBN + wg * (D / 2), dm.sigma, dQacc + t * D + wg * (D / 2), row < nq, tid);   // each warpgroup half a row
  bwd_teardown(c, RowsSmem<D>::cols, tid, status);
}

constexpr int kRetSplitRows = 4;      // CTAs sharing the 128-pair tiles of one (cluster, plane) group

template <int D>
__global__ void __launch_bounds__(kRowsThreads)
k_ret_bwd_dq_tc(Dims dm, const bf16* __restrict__ Q, const bf16* __restrict__ dO, const bf16* __restrict__ Kp,
                const bf16* __restrict__ Vp, const float* __restrict__ LSE, const float* __restrict__ delta,
                const int32_t* __restrict__ off_k, const int32_t* __restrict__ goff, const int32_t* __restrict__ pairs,
                bf16* __restrict__ dq_part, int* __restrict__ status) {
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ uint64_t bar[2];
  __shared__ uint32_t tbase_s;
  __shared__ int32_t pid_s[2][kBM];
  const int tid = threadIdx.x, row = tid & 127, wg = tid >> 7;
  const int j = blockIdx.x, pl = blockIdx.y / kRetSplitRows, sub = blockIdx.y % kRetSplitRows, pq = blockIdx.z;
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int nkeys = dm.SB * dm.Ck;
  const int32_t* go = goff + (size_t)pq * (nkeys + 1) + (size_t)j * dm.SB + pl;
  const int g0 = go[0], g1 = go[1], ntiles = (g1 - g0 + kBM - 1) / kBM;
  if (sub >= ntiles) return;                          // this split has no pair tile
  const int32_t* ok = off_k + (size_t)pk * (dm.Ck * dm.S + 1) + (size_t)j * dm.S;
  const int k0 = ok[0], k1 = ok[pl + 1];
  BwdCtx c;
  bwd_setup(c, sm_raw, bar, &tbase_s, RowsSmem<D>::cols, tid);
  const bf16* Qb = Q + (size_t)pq * dm.N * D; const bf16* dOb = dO + (size_t)pq * dm.N * D;
  const bf16* Kb = Kp + (size_t)pk * dm.N * D; const bf16* Vb = Vp + (size_t)pk * dm.N * D;
  const int32_t* pr = pairs + (size_t)pq * dm.N * dm.m;
  // pair ids two tiles ahead (shared memory), the rows they point at one tile ahead (registers)
  TileRegs<D, kBM, kRowsThreads> qreg, oreg;
  float Lreg = 0.f, dreg = 0.f;
  int pidreg = 0;
  auto load_pids = [&](int t) {
    if (tid < kBM) { const int t0 = g0 + t * kBM; pidreg = (t < ntiles && t0 + tid < g1) ? __ldg(pr + t0 + tid) : 0; }
  };
  auto load_rows = [&](int t, const int32_t* pid) {
    const int t0 = g0 + t * kBM, nq = min(kBM, g1 - t0);
    tile_ldg<D, kBM, kRowsThreads>(qreg, nq, [&](int r) { return Qb + (size_t)(pid[r] / dm.m) * D; }, tid);
    tile_ldg<D, kBM, kRowsThreads>(oreg, nq, [&](int r) { return dOb + (size_t)(pid[r] / dm.m) * D; }, tid);
    const size_t tt = (size_t)pq * dm.N + pid[row] / dm.m;
    Lreg = row < nq ? LSE[tt] * kLog2e : 0.f;
    dreg = row < nq ? delta[tt] : 0.f;
  };
  load_pids(sub);
  if (tid < kBM) pid_s[0][tid] = pidreg;
  load_pids(sub + kRetSplitRows);
  __syncthreads();
  load_rows(sub, pid_s[0]);
  int buf = 0;
  for (int t = sub; t < ntiles && c.ok; t += kRetSplitRows, buf ^= 1) {
    const int t0 = g0 + t * kBM, nq = min(kBM, g1 - t0);
    tile_sts<D, kBM, kRowsThreads>(qreg, c.sm + RowsSmem<D>::q, tid);
    tile_sts<D, kBM, kRowsThreads>(oreg, c.sm + RowsSmem<D>::dO, tid);
    if (tid < kBM) pid_s[buf ^ 1][tid] = pidreg;                      // pair ids of the next tile
    const float L2 = Lreg, dl = dreg;
    const int my_pid = pid_s[buf][row];
    __syncthreads();                                                  // pid_s[buf ^ 1] visible before the prefetch below
    if (t + kRetSplitRows < ntiles) load_rows(t + kRetSplitRows, pid_s[buf ^ 1]);
    load_pids(t + 2 * kRetSplitRows);
    const bool any = dq_rows_tc<D>(c, Kb, Vb, k0, k1, [&](int) { return k1 - 1; }, dm.sigma * kLog2e, L2, dl, tid);
    if (c.ok) {
      // bf16 row per (query, slot); each warpgroup converts and stores half of it
      bf16* dst = dq_part + ((size_t)pq * dm.N * dm.m + my_pid) * D + wg * (D / 2);
      const uint32_t tq = c.tbase + ((uint32_t)(((tid >> 5) & 3) * 32) << 16) + 2 * kBN + wg * (D / 2);
#pragma unroll
      for (int d0 = 0; d0 < D / 2; d0 += 32) {
        float v[32];
        if (any) tc::tmem_ld32(tq + d0, v);
        if (row < nq) {
#pragma unroll
          for (int i = 0; i < 32; i += 8) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              __nv_bfloat162 b2 = any ? __floats2bfloat162_rn(v[i + 2 * e] * dm.sigma, v[i + 2 * e + 1] * dm.sigma) : __floats2bfloat162_rn(0.f, 0.f);
              w[e] = *reinterpret_cast<uint32_t*>(&b2);
            }
            *reinterpret_cast<uint4*>(dst + d0 + i) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
    tc::fence_before_sync();
  }
  bwd_teardown(c, RowsSmem<D>::cols, tid, status);
}

// ================================================================================================
// keys-on-M: dK, dV of 128 keys (K, V tiles already in shared memory), fed 64 query rows at a time
// ================================================================================================
template <int D> struct KeysSmem {
  static constexpr int k = 0, v = k + kBM * D * 2, q = v + kBM * D * 2, dO = q + kBN * D * 2, pt = dO + kBN * D * 2,
                       gt = pt + kBM * kBN * 2, total = gt + kBM * kBN * 2 + 1024;
  static constexpr uint32_t cols = D == 128 ? 512 : 256;   // S^T 64 | dP^T 64 | dV D | dK D
};

// One tile of 64 query rows (already in shared memory with their L2 / delta in Ls / ds).
// valid(u_row) = number of leading query columns ... see callers: mask(col) tells whether
// query column `col` sees this thread's key.
template <int D, class Mask, class Prefetch>
__device__ __forceinline__ void dkdv_step_tc(BwdCtx& c, const float* __restrict__ Ls, const float* __restrict__ ds,
                                             Mask mask, float scale2, bool& started, int tid, Prefetch prefetch) {
  typedef KeysSmem<D> SM;
  const int warp = tid >> 5, wg = tid >> 7, row = tid & 127;       // 256 threads: warpgroup wg owns columns [32 wg, 32 wg + 32)
  const uint32_t t_s = c.tbase + ((uint32_t)((warp & 3) * 32) << 16), t_dp = t_s + kBN;
  const uint32_t ka = tc::smem_u32(c.sm + SM::k), va = tc::smem_u32(c.sm + SM::v), qa = tc::smem_u32(c.sm + SM::q),
                 da = tc::smem_u32(c.sm + SM::dO), pa = tc::smem_u32(c.sm + SM::pt), ga = tc::smem_u32(c.sm + SM::gt);
#ifdef MUSE_PHASE_CLOCKS
  const long long z0 = clock64();
#endif
  tc::fence_async_smem();
  tc::fence_before_sync();
  __syncthreads();
#ifdef MUSE_PHASE_CLOCKS
  const long long z1 = clock64();
#endif
  if (tid == 0) {
    tc::fence_after_sync();
    const uint32_t idesc = tc::idesc_bf16(kBM, kBN, 0, 0);
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) tc::mma_bf16_ss(c.tbase, desc_k<kBM>(ka, ks), desc_k<kBN>(qa, ks), idesc, ks > 0);
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) tc::mma_bf16_ss(c.tbase + kBN, desc_k<kBM>(va, ks), desc_k<kBN>(da, ks), idesc, ks > 0);
    tc::mma_commit(&c.bar[0]);
  }
  prefetch();                                  // global loads of the next query tile, overlapped with the MMAs
#ifdef MUSE_PHASE_CLOCKS
  const long long z2 = clock64();
#endif
  if (!tc::mbar_wait(&c.bar[0], c.ph0)) { c.ok = false; return; }
  c.ph0 ^= 1;
  tc::fence_after_sync();
#ifdef MUSE_PHASE_CLOCKS
  const long long z3 = clock64();
#endif
  {
    const int h = wg;
    float s[32], dp[32], Lc[32], dc[32], p[32], g[32];
    tc::tmem_ld32(t_s + 32 * h, s);
    tc::tmem_ld32(t_dp + 32 * h, dp);
    // the per-column L and delta come out of shared memory in vector loads before the loop: with
    // one or two warps per scheduler a load inside each iteration would expose its latency every time
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float4 a = *reinterpret_cast<const float4*>(Ls + 32 * h + 4 * k), b = *reinterpret_cast<const float4*>(ds + 32 * h + 4 * k);
      Lc[4 * k] = a.x; Lc[4 * k + 1] = a.y; Lc[4 * k + 2] = a.z; Lc[4 * k + 3] = a.w;
      dc[4 * k] = b.x; dc[4 * k + 1] = b.y; dc[4 * k + 2] = b.z; dc[4 * k + 3] = b.w;
    }
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const float e = tc::fast_exp2(s[i] * scale2 - Lc[i]);
      const float pv = mask(32 * h + i) ? e : 0.f;
      p[i] = pv;
      g[i] = pv * (dp[i] - dc[i]);
    }
    store_row32(c.sm + SM::pt, row, h, p);
    store_row32(c.sm + SM::gt, row, h, g);
  }
#ifdef MUSE_PHASE_CLOCKS
  const long long z4 = clock64();
#endif
  tc::fence_async_smem();
  tc::fence_before_sync();
  __syncthreads();
  if (tid == 0) {
    tc::fence_after_sync();
    const uint32_t idesc = tc::idesc_bf16(kBM, D, 0, 1);
#pragma unroll
    for (int ks = 0; ks < kBN / 16; ++ks)
      tc::mma_bf16_ss(c.tbase + 2 * kBN, tc::smem_desc_sw128(pa + ks * 32, 16, 1024), desc_mn<kBN>(da, ks), idesc, !(!started && ks == 0));
#pragma unroll
    for (int ks = 0; ks < kBN / 16; ++ks)
      tc::mma_bf16_ss(c.tbase + 2 * kBN + D, tc::smem_desc_sw128(ga + ks * 32, 16, 1024), desc_mn<kBN>(qa, ks), idesc, !(!started && ks == 0));
    tc::mma_commit(&c.bar[1]);
  }
  started = true;
  if (!tc::mbar_wait(&c.bar[1], c.ph1)) { c.ok = false; return; }
  c.ph1 ^= 1;
  tc::fence_after_sync();
#ifdef MUSE_PHASE_CLOCKS
  const long long z5 = clock64();
  c.pc[0] += z1 - z0; c.pc[1] += z2 - z1; c.pc[2] += z3 - z2; c.pc[3] += z4 - z3; c.pc[4] += z5 - z4; c.pc[5] += 1;
#endif
}

constexpr int kKeysThreads = 256;       // keys-on-M kernels: two warpgroups share the 64 query columns

// Local (block-diagonal) dK, dV: one CTA = 128 keys of a block against the query tiles (64 rows) that see
// them.  Software pipeline over the query tiles t, all operand tiles by TMA:
//   MMA1(t+1) (S^T = K Q^T, dP^T = V dO^T into the second accumulator buffer) is issued as soon as
//   MMA1(t) has landed, so it runs while the threads turn S^T(t), dP^T(t) into P^T, G^T;
//   MMA2(t) (dV += P^T dO, dK += G^T Q) runs during the next iteration; Q / dO tiles sit in a ring of
//   three, refilled as soon as the MMAs that read a slot have completed.
template <int D> struct LdkSmem {
  static constexpr int k = 0, v = k + kBM * D * 2, qd = v + kBM * D * 2, tile = 2 * kBN * D * 2,       // ring slot = Q tile | dO tile
                       pt = qd + 3 * tile, gt = pt + kBM * kBN * 2, total = gt + kBM * kBN * 2 + 1024;
  static constexpr uint32_t cDV = 256, cDK = 256 + D, cols = 512;   // S^T / dP^T buffers at 0 / 64 and 128 / 192
};

// Warps 0-7 do the arithmetic; lane 0 of a ninth warp issues every TMA load and MMA, so that issuing never
// delays a warp that the others wait for at the barriers.
constexpr int kLdkThreads = kKeysThreads + 32, kLdkIssuer = kKeysThreads;

template <int D>
__global__ void __launch_bounds__(kLdkThreads, 1)
k_local_bwd_dkdv_tc(Dims dm, const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_do,
                    const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                    const float* __restrict__ LSE, const float* __restrict__ delta,
                    float* __restrict__ dK_orig, float* __restrict__ dV_orig, int* __restrict__ status) {
  typedef LdkSmem<D> SM;
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ uint64_t barKV, barQ[3], bar1[2], bar2;
  __shared__ uint32_t tbase_s;
  __shared__ __align__(16) float Ls[3][kBN], ds[3][kBN];
  const int tid = threadIdx.x, warp = tid >> 5, row = tid & 127, wg = tid >> 7;
  unsigned char* sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);
  if (warp == 0) tc::tmem_alloc(&tbase_s, SM::cols);
  if (tid == 0) {
    tc::mbar_init(&barKV, 1); tc::mbar_init(&bar2, 1);
    for (int k = 0; k < 3; ++k) tc::mbar_init(&barQ[k], 1);
    tc::mbar_init(&bar1[0], 1); tc::mbar_init(&bar1[1], 1);
    tc::mbar_init_fence();
  }
  const int lin = blockIdx.x, kt = lin / dm.S, blk = lin % dm.S, pq = blockIdx.y;   // early key tiles (most work) first
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int bstart = blk * dm.Bs, bend = bstart + dm.Bs;
  const int k0 = bstart + kt * kBM, nk = min(kBM, bend - k0);
  const int T = (bend - k0 + kBN - 1) / kBN;                // query tiles that see these keys
  const int u = k0 + row;
  // threads 0..63: L (log2 units) and delta of query tile t; loaded into registers one tile before they are
  // stored, so that no warp waits for global memory in front of a barrier
  // (nothing may depend on the loaded values before store_scalars: a dependent instruction placed earlier
  // would make these warps wait for global memory)
  float Lnext = 0.f, dnext = 0.f;
  auto fetch_scalars = [&](int t) {
    if (tid < kBN && t < T) {
      const int q = min(k0 + t * kBN + tid, bend - 1);
      Lnext = LSE[(size_t)pq * dm.N + q];
      dnext = delta[(size_t)pq * dm.N + q];
    }
  };
  auto store_scalars = [&](int t) {
    if (tid < kBN && t < T) {
      const bool in = k0 + t * kBN + tid < bend;
      Ls[t % 3][tid] = in ? Lnext * kLog2e : 0.f; ds[t % 3][tid] = in ? dnext : 0.f;
    }
  };
  fetch_scalars(0); store_scalars(0); fetch_scalars(1); store_scalars(1); fetch_scalars(2); store_scalars(2);
  fetch_scalars(3);
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tbase = tbase_s, tl = tbase + ((uint32_t)((warp & 3) * 32) << 16);
  const uint32_t ka = tc::smem_u32(sm + SM::k), va = tc::smem_u32(sm + SM::v), pa = tc::smem_u32(sm + SM::pt), ga = tc::smem_u32(sm + SM::gt);
  bool ok = true;
  // thread 0 only
  auto load_qd = [&](int t) {
    unsigned char* slot = sm + SM::qd + (t % 3) * SM::tile;
    tc::mbar_expect_tx(&barQ[t % 3], SM::tile);
    const int r = pq * dm.N + k0 + t * kBN;
    for (int g = 0; g < D / 64; ++g) {
      tc::tma_load_2d(slot + g * kBN * 128, &tm_q, 64 * g, r, &barQ[t % 3]);
      tc::tma_load_2d(slot + kBN * D * 2 + g * kBN * 128, &tm_do, 64 * g, r, &barQ[t % 3]);
    }
  };
  // one descriptor per operand buffer, stepped per MMA (K-major views; the MN-major views of the ring differ in lbo)
  const uint64_t dk0 = tc::smem_desc_sw128(ka, 16, 1024), dv0 = tc::smem_desc_sw128(va, 16, 1024),
                 dq0 = tc::smem_desc_sw128(tc::smem_u32(sm + SM::qd), 16, 1024),
                 dqm0 = tc::smem_desc_sw128(tc::smem_u32(sm + SM::qd), kBN * 128, 1024),
                 dp0 = tc::smem_desc_sw128(pa, 16, 1024), dg0 = tc::smem_desc_sw128(ga, 16, 1024);
  auto issue1 = [&](int t) {                                // S^T(t) = K Q_t^T, dP^T(t) = V dO_t^T into accumulator buffer t & 1
    if (!tc::mbar_wait(&barQ[t % 3], (t / 3) & 1)) ok = false;
    tc::fence_after_sync();
    const uint32_t slot = (uint32_t)(t % 3) * SM::tile;
    const uint32_t idesc = tc::idesc_bf16(kBM, kBN, 0, 0), cb = tbase + (t & 1) * 2 * kBN;
    const uint64_t qd = tc::desc_step(dq0, slot), dd = tc::desc_step(dq0, slot + kBN * D * 2);
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks)
      tc::mma_bf16_ss(cb, tc::desc_step(dk0, (ks / 4) * kBM * 128 + (ks % 4) * 32), tc::desc_step(qd, (ks / 4) * kBN * 128 + (ks % 4) * 32), idesc, ks > 0);
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks)
      tc::mma_bf16_ss(cb + kBN, tc::desc_step(dv0, (ks / 4) * kBM * 128 + (ks % 4) * 32), tc::desc_step(dd, (ks / 4) * kBN * 128 + (ks % 4) * 32), idesc, ks > 0);
    tc::mma_commit(&bar1[t & 1]);
  };
  if (tid == kLdkIssuer) {
    tc::mbar_expect_tx(&barKV, 2 * kBM * D * 2);
    for (int g = 0; g < D / 64; ++g) {
      tc::tma_load_2d(sm + SM::k + g * kBM * 128, &tm_k, 64 * g, pk * dm.N + k0, &barKV);
      tc::tma_load_2d(sm + SM::v + g * kBM * 128, &tm_v, 64 * g, pk * dm.N + k0, &barKV);
    }
    load_qd(0);
    if (T > 1) load_qd(1);
    if (T > 2) load_qd(2);
    if (!tc::mbar_wait(&barKV, 0)) ok = false;
    issue1(0);
  }
  const float scale2 = dm.sigma * kLog2e;
  // Two loops over the query tiles, one per role, that meet at one CTA-wide barrier per tile (P^T / G^T
  // written).  Each role's instructions are contiguous: no warp jumps over the other role's code.  Every warp
  // runs all T tiles whatever happens (after a wait ran out the remaining waits are skipped).
  if (warp == 8) {
    for (int t = 0; t < T; ++t) {
      if (tid == kLdkIssuer) {
        if (t + 1 < T) issue1(t + 1);                       // its accumulator buffer was read before the last barrier
        if (t > 0) {                                        // MMA2(t - 1) has completed: its ring slot is free
          if (ok && !tc::mbar_wait(&bar2, (t - 1) & 1)) ok = false;
          if (t + 2 < T) load_qd(t + 2);
        }
      }
      tc::fence_before_sync();
      __syncthreads();
      if (tid == kLdkIssuer) {
        tc::fence_after_sync();
        const uint32_t slot = (uint32_t)(t % 3) * SM::tile;
        const uint32_t idesc = tc::idesc_bf16(kBM, D, 0, 1);
        const uint64_t qm = tc::desc_step(dqm0, slot), dm_ = tc::desc_step(dqm0, slot + kBN * D * 2);
        const uint32_t acc = t > 0;
#pragma unroll
        for (int ks = 0; ks < kBN / 16; ++ks)
          tc::mma_bf16_ss(tbase + SM::cDV, tc::desc_step(dp0, ks * 32), tc::desc_step(dm_, ks * 16 * 128), idesc, ks > 0 ? 1u : acc);
#pragma unroll
        for (int ks = 0; ks < kBN / 16; ++ks)
          tc::mma_bf16_ss(tbase + SM::cDK, tc::desc_step(dg0, ks * 32), tc::desc_step(qm, ks * 16 * 128), idesc, ks > 0 ? 1u : acc);
        tc::mma_commit(&bar2);
      }
      __syncwarp();
    }
  } else {
    for (int t = 0; t < T; ++t) {
      const int q0 = k0 + t * kBN, nq = min(kBN, bend - q0);
      if (ok && !tc::mbar_wait(&bar1[t & 1], (t >> 1) & 1)) ok = false;
      tc::fence_after_sync();
      float p[32], g[32];
      {
        float s[32], dp[32];
        tc::tmem_ld32(tl + (t & 1) * 2 * kBN + 32 * wg, s);
        tc::tmem_ld32(tl + (t & 1) * 2 * kBN + kBN + 32 * wg, dp);
        const float* Lt = Ls[t % 3] + 32 * wg;
        const float* dt = ds[t % 3] + 32 * wg;
        // bit c of `vis`: query column 32 wg + c exists and sees this thread's key (causal, key inside the tile)
        const int lo = max(0, u - q0 - 32 * wg), hi = row < nk ? min(32, nq - 32 * wg) : 0;
        const uint32_t vis = hi > lo ? ((hi >= 32 ? 0xffffffffu : (1u << hi) - 1u) & (lo >= 32 ? 0u : 0xffffffffu << lo)) : 0u;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const float4 a = *reinterpret_cast<const float4*>(Lt + 4 * k), b = *reinterpret_cast<const float4*>(dt + 4 * k);
          const float Lc[4] = {a.x, a.y, a.z, a.w}, dc[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float ev = tc::fast_exp2(fmaf(s[4 * k + e], scale2, -Lc[e]));
            const float pv = (vis >> (4 * k + e)) & 1u ? ev : 0.f;
            p[4 * k + e] = pv;
            g[4 * k + e] = pv * (dp[4 * k + e] - dc[e]);
          }
        }
      }
      if (t > 0) {                                          // MMA2(t - 1) has completed: P^T / G^T are free
        if (ok && !tc::mbar_wait(&bar2, (t - 1) & 1)) ok = false;
        tc::fence_after_sync();
        store_scalars(t + 2);                               // fetched during the previous tile
        fetch_scalars(t + 3);
      }
      store_row32(sm + SM::pt, row, wg, p);
      store_row32(sm + SM::gt, row, wg, g);
      tc::fence_async_smem();
      tc::fence_before_sync();
      __syncthreads();
    }
  }
  ok = __syncthreads_and(ok);
  if (ok && T > 0) { if (!tc::mbar_wait(&bar2, (T - 1) & 1)) ok = false; }
  tc::fence_after_sync();
  if (warp < 8) {                                           // warpgroup 0 writes dV, warpgroup 1 writes dK (all their threads run the TMEM loads)
    const size_t at = ((size_t)pq * dm.N + k0 + row) * D;
    float* dst = (wg == 0 ? dV_orig : dK_orig) + at;
    const float f = wg == 0 ? 1.f : dm.sigma;
#pragma unroll
    for (int d0 = 0; d0 < D; d0 += 32) {
      float v[32];
      tc::tmem_ld32(tl + (wg == 0 ? SM::cDV : SM::cDK) + d0, v);
      if (ok && row < nk) {
#pragma unroll
        for (int i = 0; i < 32; i += 4)
          *reinterpret_cast<float4*>(dst + d0 + i) = make_float4(v[i] * f, v[i + 1] * f, v[i + 2] * f, v[i + 3] * f);
      }
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tbase, SM::cols);
  if (!ok && tid == 0) report_status(status, 2);
}

// One CTA per (key cluster j, plane, split, head): 128-key tiles of the run the plane sees, fed with
// every kRetSplit-th tile of 64 retrieving pairs.  Popular clusters are retrieved by thousands of
// queries, so the pair tiles are spread over kRetSplit CTAs and over the planes; each CTA adds
// its partial dK, dV with vector float atomics into the zero-initialised accumulators.
constexpr int kRetSplit = 8;

template <int D>
__device__ __forceinline__ void add_acc_row(const BwdCtx& c, uint32_t col, float f, float* __restrict__ dst, bool write, int tid) {
  const uint32_t t = c.tbase + ((uint32_t)(((tid >> 5) & 3) * 32) << 16) + col;
#pragma unroll
  for (int d0 = 0; d0 < D; d0 += 32) {
    float v[32];
    tc::tmem_ld32(t + d0, v);
    if (write) {
#pragma unroll
      for (int i = 0; i < 32; i += 4)
        atomicAdd(reinterpret_cast<float4*>(dst + d0 + i), make_float4(v[i] * f, v[i + 1] * f, v[i + 2] * f, v[i + 3] * f));
    }
  }
}

template <int D>
__global__ void __launch_bounds__(kKeysThreads)
k_ret_bwd_dkdv_tc(Dims dm, const bf16* __restrict__ Q, const bf16* __restrict__ dO, const bf16* __restrict__ Kp,
                  const bf16* __restrict__ Vp, const float* __restrict__ LSE, const float* __restrict__ delta,
                  const int32_t* __restrict__ off_k, const int32_t* __restrict__ goff, const int32_t* __restrict__ pairs,
                  float* __restrict__ dK_perm, float* __restrict__ dV_perm, int* __restrict__ status) {
  typedef KeysSmem<D> SM;
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ uint64_t bar[2];
  __shared__ uint32_t tbase_s;
  __shared__ __align__(16) float Ls[kBN], ds[kBN];
  __shared__ int32_t tok_s[2][kBN];
  const int tid = threadIdx.x, row = tid & 127, wg = tid >> 7;
  const int j = blockIdx.x, pl = blockIdx.y / kRetSplit, sub = blockIdx.y % kRetSplit, pq = blockIdx.z;
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int nkeys = dm.SB * dm.Ck;
  const int32_t* go = goff + (size_t)pq * (nkeys + 1) + (size_t)j * dm.SB + pl;
  const int32_t* ok = off_k + (size_t)pk * (dm.Ck * dm.S + 1) + (size_t)j * dm.S;
  const int kbeg = ok[0], kvis = ok[pl + 1];
  const int g0 = go[0], g1 = go[1], ntiles = (g1 - g0 + kBN - 1) / kBN;
  if (kbeg >= kvis || sub >= ntiles) return;          // nothing for this (plane, split): no TMEM taken
  BwdCtx c;
  bwd_setup(c, sm_raw, bar, &tbase_s, SM::cols, tid);
  const bf16* Qb = Q + (size_t)pq * dm.N * D; const bf16* dOb = dO + (size_t)pq * dm.N * D;
  const bf16* Kb = Kp + (size_t)pk * dm.N * D; const bf16* Vb = Vp + (size_t)pk * dm.N * D;
  const int32_t* pr = pairs + (size_t)pq * dm.N * dm.m;
  for (int c0 = kbeg; c0 < kvis && c.ok; c0 += kBM) {
    const int nkc = min(kBM, kvis - c0);
    __syncthreads();
    fill_tile<D, kBM, kKeysThreads>(c.sm + SM::k, nkc, [&](int r) { return Kb + (size_t)(c0 + r) * D; }, tid);
    fill_tile<D, kBM, kKeysThreads>(c.sm + SM::v, nkc, [&](int r) { return Vb + (size_t)(c0 + r) * D; }, tid);
    bool started = false;
    const bool mine = row < nkc;
    // Pair ids are fetched two tiles ahead (into tok_s), the rows they point at one tile ahead
    // (into registers), so neither dependent load sits on the critical path of a tile.
    TileRegs<D, kBN, kKeysThreads> qreg, oreg;
    float Lreg = 0.f, dreg = 0.f;
    int tokreg = 0;
    auto load_tokens = [&](int t) {            // thread < 64: token of pair (t, thread), 0 beyond the group
      if (tid < kBN) { const int t0 = g0 + t * kBN; tokreg = (t < ntiles && t0 + tid < g1) ? __ldg(pr + t0 + tid) / dm.m : 0; }
    };
    auto load_rows = [&](int t, const int32_t* tok) {       // tok: shared-memory tokens of tile t
      const int t0 = g0 + t * kBN, nq = min(kBN, g1 - t0);
      tile_ldg<D, kBN, kKeysThreads>(qreg, nq, [&](int r) { return Qb + (size_t)tok[r] * D; }, tid);
      tile_ldg<D, kBN, kKeysThreads>(oreg, nq, [&](int r) { return dOb + (size_t)tok[r] * D; }, tid);
      if (tid < kBN) {
        Lreg = tid < nq ? LSE[(size_t)pq * dm.N + tok[tid]] * kLog2e : 0.f;
        dreg = tid < nq ? delta[(size_t)pq * dm.N + tok[tid]] : 0.f;
      }
    };
    __syncthreads();
    load_tokens(sub);
    if (tid < kBN) tok_s[0][tid] = tokreg;
    load_tokens(sub + kRetSplit);
    __syncthreads();
    load_rows(sub, tok_s[0]);
    int buf = 0;
    for (int t = sub; t < ntiles && c.ok; t += kRetSplit, buf ^= 1) {
      const int t0 = g0 + t * kBN, nq = min(kBN, g1 - t0);
      tile_sts<D, kBN, kKeysThreads>(qreg, c.sm + SM::q, tid);
      tile_sts<D, kBN, kKeysThreads>(oreg, c.sm + SM::dO, tid);
      if (tid < kBN) { Ls[tid] = Lreg; ds[tid] = dreg; tok_s[buf ^ 1][tid] = tokreg; }     // tokens of the next tile
      dkdv_step_tc<D>(c, Ls, ds, [&](int col) { return col < nq && mine; }, dm.sigma * kLog2e, started, tid,
                      [&]() {                  // runs after the step's first barrier: tok_s[buf ^ 1] is visible
                        if (t + kRetSplit < ntiles) load_rows(t + kRetSplit, tok_s[buf ^ 1]);
                        load_tokens(t + 2 * kRetSplit);
                      });
    }
    if (c.ok && started) {                      // warpgroup 0 adds dV, warpgroup 1 adds dK
      const size_t at = ((size_t)pq * dm.N + c0 + row) * D;
      if (wg == 0) add_acc_row<D>(c, 2 * kBN, 1.f, dV_perm + at, row < nkc, tid);
      else add_acc_row<D>(c, 2 * kBN + D, dm.sigma, dK_perm + at, row < nkc, tid);
    }
    tc::fence_before_sync();
  }
#ifdef MUSE_PHASE_CLOCKS
  if (tid == 0 && c.pc[5] >= 8 && atomicCAS(status + 40, 0, 1) == 0)
    for (int k = 0; k < 7; ++k) status[41 + k] = (int)c.pc[k];
#endif
  bwd_teardown(c, SM::cols, tid, status);
}

// ---- launchers ------------------------------------------------------------------------------------
#define MUSE_TC_LAUNCH(KERNEL, SMEM, NT, GRID, ...)                                                                  \
  do {                                                                                                            \
    if (d.D == 128) {                                                                                             \
      MUSE_CUDA_OK(cudaFuncSetAttribute(KERNEL<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM<128>::total)); \
      KERNEL<128><<<GRID, NT, SMEM<128>::total, st>>>(__VA_ARGS__);                                              \
    } else {                                                                                                      \
      MUSE_CUDA_OK(cudaFuncSetAttribute(KERNEL<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM<64>::total));   \
      KERNEL<64><<<GRID, NT, SMEM<64>::total, st>>>(__VA_ARGS__);                                                 \
    }                                                                                                             \
    MUSE_LAUNCH_OK();                                                                                             \
  } while (0)

int local_bwd_tc(const Dims& d, const void* Q, const void* K, const void* V, const void* dO, const float* LSE,
                 const float* delta, float* dQacc, float* dK_orig, float* dV_orig, int* status, cudaStream_t st) {
  const int pq = d.B * d.Hq;
  dim3 grid(d.S * cdiv(d.Bs, kBM), pq);
  CUtensorMap tq, tdo, tk, tv;
  int rc = make_tmap_bf16_rows(&tq, Q, (uint64_t)pq * d.N, (uint32_t)d.D, kBN);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&tdo, dO, (uint64_t)pq * d.N, (uint32_t)d.D, kBN);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&tk, K, (uint64_t)d.B * d.Hkv * d.N, (uint32_t)d.D, kBM);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&tv, V, (uint64_t)d.B * d.Hkv * d.N, (uint32_t)d.D, kBM);
  if (rc != MUSE_OK) return rc;
  prof_mark("k_local_bwd_dkdv_tc", st);
  MUSE_TC_LAUNCH(k_local_bwd_dkdv_tc, LdkSmem, kLdkThreads, grid, d, tq, tdo, tk, tv, LSE, delta, dK_orig, dV_orig, status);
  prof_mark("k_local_bwd_dq_tc", st);
  MUSE_TC_LAUNCH(k_local_bwd_dq_tc, RowsSmem, kRowsThreads, grid, d, (const bf16*)Q, (const bf16*)K, (const bf16*)V, (const bf16*)dO, LSE,
                 delta, dQacc, status);
  return MUSE_OK;
}

int ret_bwd_pairs_tc(const Dims& d, const void* Q, const void* dO, const void* Kp, const void* Vp, const float* LSE,
                     const float* delta, const int32_t* off_k, const int32_t* goff, const int32_t* pairs, void* dq_part,
                     float* dK_perm, float* dV_perm, int* status, cudaStream_t st);

int ret_bwd_tc(const Dims& d, const void* Q, const void* dO, const void* Kp, const void* Vp, const float* LSE,
               const float* delta, const int32_t* off_k, const int32_t* goff, const int32_t* pairs, void* dq_part,
               float* dK_perm, float* dV_perm, int* status, cudaStream_t st) {
  const int pq = d.B * d.Hq;
  if (!path_forced(kForceRetBwdSplit) || d.k2 > 0)
    return ret_bwd_pairs_tc(d, Q, dO, Kp, Vp, LSE, delta, off_k, goff, pairs, dq_part, dK_perm, dV_perm, status, st);
  prof_mark("k_ret_bwd_dkdv_tc", st);
  MUSE_TC_LAUNCH(k_ret_bwd_dkdv_tc, KeysSmem, kKeysThreads, dim3(d.Ck, d.SB * kRetSplit, pq), d, (const bf16*)Q, (const bf16*)dO, (const bf16*)Kp,
                 (const bf16*)Vp, LSE, delta, off_k, goff, pairs, dK_perm, dV_perm, status);
  prof_mark("k_ret_bwd_dq_tc", st);
  MUSE_TC_LAUNCH(k_ret_bwd_dq_tc, RowsSmem, kRowsThreads, dim3(d.Ck, d.SB * kRetSplitRows, pq), d, (const bf16*)Q, (const bf16*)dO, (const bf16*)Kp,
                 (const bf16*)Vp, LSE, delta, off_k, goff, pairs, (bf16*)dq_part, status);
  return MUSE_OK;
}

}  // namespace muse
