// Exact-attention forward on the Blackwell tensor cores (bf16 inputs, fp32 accumulation in
// tensor memory): the local block-diagonal component and the retrieved-cluster component of
// Algorithm 1.  One CTA = 128 query rows (one thread per row); keys stream in tiles of 64.
//   S  = Q K^T      tcgen05.mma, A = Q tile, B = K tile, both K-major in 128B-swizzled smem
//   P  = softmax piece, one thread per row straight out of TMEM, written back as bf16 to smem
//   PV              tcgen05.mma, A = P tile (K-major), B = V tile (MN-major), read from TMEM
//                   and folded into the fp32 output registers with the online-softmax rescale.
#include <cuda.h>
#include "common.cuh"
#include "tc05.cuh"


namespace muse {

typedef __nv_bfloat16 bf16;
constexpr int kTcM = 128, kTcN = 64;

template <int D> struct FwdTcSmem {
  static constexpr int q_bytes = kTcM * D * 2, k_bytes = kTcN * D * 2, v_bytes = kTcN * D * 2, p_bytes = kTcM * kTcN * 2;
  static constexpr int total = q_bytes + k_bytes + v_bytes + p_bytes + 1024;
};

// rows of D bf16 -> K-major swizzled blocks: block kb (64 elements of K) is [nrows_tile][128 B]
template <int D, int ROWS, class RowPtr>
__device__ __forceinline__ void fill_kmajor(unsigned char* dst, int n, RowPtr row_ptr, int tid) {
  constexpr int CPR = D / 8;                       // 16-byte chunks per row
  for (int e = tid; e < ROWS * CPR; e += 128) {
    const int r = e / CPR, ck = e % CPR, kb = ck >> 3, c = ck & 7;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (r < n) v = reinterpret_cast<const uint4*>(row_ptr(r))[ck];
    *reinterpret_cast<uint4*>(dst + kb * ROWS * 128 + tc::sw128_off(r, c)) = v;
  }
}
// rows (k index) of D bf16 -> MN-major swizzled groups: group g (64 columns) is [ROWS][128 B]
template <int D, int ROWS, class RowPtr>
__device__ __forceinline__ void fill_mnmajor(unsigned char* dst, int n, RowPtr row_ptr, int tid) {
  constexpr int CPR = D / 8;
  for (int e = tid; e < ROWS * CPR; e += 128) {
    const int r = e / CPR, cn = e % CPR, g = cn >> 3, c = cn & 7;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (r < n) v = reinterpret_cast<const uint4*>(row_ptr(r))[cn];
    *reinterpret_cast<uint4*>(dst + g * ROWS * 128 + tc::sw128_off(r, c)) = v;
  }
}

struct TcCtx {
  unsigned char *Qs, *Ks, *Vs, *Ps;
  uint64_t* bar;          // [2]
  uint32_t tbase;
  uint32_t ph0, ph1;      // mbarrier phases
  bool ok;
};

// Attention of the 128 rows already in c.Qs over keys [k_lo, k_hi) of (Kb, Vb).  `limit(r)` is the
// last visible key index of row r (inclusive) for causal masking, or k_hi - 1.
// Results: o[D] un-normalised, m2 (running max, log2 units), l (running sum).
template <int D, class Limit>
__device__ __forceinline__ void attend_tc(TcCtx& c, const bf16* __restrict__ Kb, const bf16* __restrict__ Vb,
                                          int k_lo, int k_hi, Limit limit, float scale2, float (&o)[D], float& m2,
                                          float& l, int tid) {
  const int warp = tid >> 5;
  const uint32_t t_s = c.tbase + ((uint32_t)(warp * 32) << 16), t_o = t_s + kTcN;
  const int my_limit = limit(tid);
  for (int c0 = k_lo; c0 < k_hi && c.ok; c0 += kTcN) {
    const int nk = min(kTcN, k_hi - c0);
    fill_kmajor<D, kTcN>(c.Ks, nk, [&](int r) { return Kb + (size_t)(c0 + r) * D; }, tid);
    fill_mnmajor<D, kTcN>(c.Vs, nk, [&](int r) { return Vb + (size_t)(c0 + r) * D; }, tid);
    tc::fence_async_smem();
    tc::fence_before_sync();
    __syncthreads();
    if (tid == 0) {
      tc::fence_after_sync();
      const uint32_t idesc = tc::idesc_bf16(kTcM, kTcN, 0, 0);
      const uint32_t qa = tc::smem_u32(c.Qs), ka = tc::smem_u32(c.Ks);
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks)
        tc::mma_bf16_ss(c.tbase, tc::smem_desc_sw128(qa + (ks / 4) * kTcM * 128 + (ks % 4) * 32, 16, 1024),
                        tc::smem_desc_sw128(ka + (ks / 4) * kTcN * 128 + (ks % 4) * 32, 16, 1024), idesc, ks > 0);
      tc::mma_commit(&c.bar[0]);
    }
    if (!tc::mbar_wait(&c.bar[0], c.ph0)) { c.ok = false; break; }
    c.ph0 ^= 1;
    tc::fence_after_sync();
    float s[kTcN];
    {
      float v[32];
      tc::tmem_ld32(t_s, v);
#pragma unroll
      for (int i = 0; i < 32; ++i) s[i] = v[i];
      tc::tmem_ld32(t_s + 32, v);
#pragma unroll
      for (int i = 0; i < 32; ++i) s[32 + i] = v[i];
    }
    float mx = -INFINITY;
    const int vis = min(nk, my_limit - c0 + 1);            // visible columns of this tile for my row
#pragma unroll
    for (int i = 0; i < kTcN; ++i) { s[i] = i < vis ? s[i] * scale2 : -INFINITY; mx = fmaxf(mx, s[i]); }
    const float mn = fmaxf(m2, mx);
    const float base = mn == -INFINITY ? 0.f : mn;
    const float resc = exp2f(m2 - base);
    float rs = 0.f;
    uint32_t pk[kTcN / 2];
#pragma unroll
    for (int i = 0; i < kTcN; i += 2) {
      const float p0 = exp2f(s[i] - base), p1 = exp2f(s[i + 1] - base);
      __nv_bfloat162 b = __floats2bfloat162_rn(p0, p1);
      // accumulate the rounded values so that the normaliser matches what the PV product sees
      rs += __low2float(b) + __high2float(b);
      pk[i / 2] = *reinterpret_cast<uint32_t*>(&b);
    }
    l = l * resc + rs;
    m2 = mn;
    if (resc != 1.f) {
#pragma unroll
      for (int i = 0; i < D; ++i) o[i] *= resc;
    }
#pragma unroll
    for (int ch = 0; ch < kTcN / 8; ++ch)
      *reinterpret_cast<uint4*>(c.Ps + tc::sw128_off(tid, ch)) = make_uint4(pk[ch * 4], pk[ch * 4 + 1], pk[ch * 4 + 2], pk[ch * 4 + 3]);
    tc::fence_async_smem();
    tc::fence_before_sync();
    __syncthreads();
    if (tid == 0) {
      tc::fence_after_sync();
      const uint32_t idesc = tc::idesc_bf16(kTcM, D, 0, 1);
      const uint32_t pa = tc::smem_u32(c.Ps), va = tc::smem_u32(c.Vs);
#pragma unroll
      for (int ks = 0; ks < kTcN / 16; ++ks)
        tc::mma_bf16_ss(c.tbase + kTcN, tc::smem_desc_sw128(pa + ks * 32, 16, 1024),
                        tc::smem_desc_sw128(va + ks * 16 * 128, kTcN * 128, 1024), idesc, ks > 0);
      tc::mma_commit(&c.bar[1]);
    }
    if (!tc::mbar_wait(&c.bar[1], c.ph1)) { c.ok = false; break; }
    c.ph1 ^= 1;
    tc::fence_after_sync();
#pragma unroll
    for (int d0 = 0; d0 < D; d0 += 32) {
      float v[32];
      tc::tmem_ld32(t_o + d0, v);
#pragma unroll
      for (int i = 0; i < 32; ++i) o[d0 + i] += v[i];
    }
    tc::fence_before_sync();
  }
}

template <int D>
__device__ __forceinline__ void tc_setup(TcCtx& c, unsigned char* sm_raw, uint64_t* bar, uint32_t* tbase_s, int tid) {
  unsigned char* sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);
  c.Qs = sm; c.Ks = c.Qs + FwdTcSmem<D>::q_bytes; c.Vs = c.Ks + FwdTcSmem<D>::k_bytes; c.Ps = c.Vs + FwdTcSmem<D>::v_bytes;
  c.bar = bar; c.ph0 = c.ph1 = 0; c.ok = true;
  if ((tid >> 5) == 0) tc::tmem_alloc(tbase_s, D == 128 ? 256 : 128);
  if (tid == 0) { tc::mbar_init(&bar[0], 1); tc::mbar_init(&bar[1], 1); tc::mbar_init_fence(); }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  c.tbase = *tbase_s;
}

template <int D>
__device__ __forceinline__ void tc_teardown(TcCtx& c, int tid, int* status) {
  tc::fence_before_sync();
  __syncthreads();
  if ((tid >> 5) == 0) tc::tmem_dealloc(c.tbase, D == 128 ? 256 : 128);
  if (!c.ok && tid == 0) report_status(status, 1);
}

// ---- local (block-diagonal) attention ------------------------------------------------------------
// 256 threads: thread (row, warpgroup w) owns key columns [32 w, 32 w + 32) of every 64-key tile and
// output dims [D/2 w, D/2 w + D/2) of its row; the two halves of a row share the running maximum
// through shared memory.  Software pipeline over the key tiles t (K and V tiles arrive by TMA):
//   S(t+1) = Q K_{t+1}^T is issued as soon as S(t) has landed (two S buffers in TMEM, two K tiles in
//   shared memory), so it runs while the threads do the softmax of tile t; O(t) = P(t) V_t is
//   awaited at the start of iteration t + 1, which frees P and V for tile t + 1; O accumulates in TMEM.
constexpr int kLfThreads = 256;

template <int D> struct LfSmem {
  static constexpr int q = 0, k = q + kTcM * D * 2, v = k + 2 * kTcN * D * 2, p = v + kTcN * D * 2, total = p + kTcM * kTcN * 2 + 1024;
};

template <int D>
__global__ void __launch_bounds__(kLfThreads, 2)
k_local_fwd_tc(Dims dm, const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
               const bf16* __restrict__ Q, float* __restrict__ o_loc, float* __restrict__ lse_loc, int* __restrict__ status) {
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ uint64_t barS[2], barK[2], barV, barPV;
  __shared__ uint32_t tbase_s;
  __shared__ float mx_s[2][kTcM];
  constexpr int HD = D / 2, kKB = kTcN * D * 2;
  constexpr uint32_t cO = 2 * kTcN;                        // TMEM: S0 | S1 | O
  const int tid = threadIdx.x, warp = tid >> 5, row = tid & 127, wg = tid >> 7;
  unsigned char* sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);
  unsigned char *Qs = sm + LfSmem<D>::q, *Ks = sm + LfSmem<D>::k, *Vs = sm + LfSmem<D>::v, *Ps = sm + LfSmem<D>::p;
  if (warp == 0) tc::tmem_alloc(&tbase_s, 256);
  if (tid == 0) {
    tc::mbar_init(&barS[0], 1); tc::mbar_init(&barS[1], 1); tc::mbar_init(&barK[0], 1); tc::mbar_init(&barK[1], 1);
    tc::mbar_init(&barV, 1); tc::mbar_init(&barPV, 1); tc::mbar_init_fence();
  }
  const int tpb = cdiv(dm.Bs, kTcM);
  // heaviest tiles (latest in a block) first
  const int lin = blockIdx.x, qt = tpb - 1 - lin / dm.S, blk = lin % dm.S, pq = blockIdx.y;
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int bstart = blk * dm.Bs, bend = bstart + dm.Bs;
  const int q0 = bstart + qt * kTcM, nq = min(kTcM, bend - q0);
  const bf16* Qb = Q + (size_t)pq * dm.N * D;
  const int k_lo = bstart, k_hi = q0 + nq;                  // causal: keys up to the tile's last row
  const int T = (k_hi - k_lo + kTcN - 1) / kTcN;
  const int krow0 = pk * dm.N + k_lo;                       // row of the first key in the [B*Hkv*N][D] tensors
  for (int e = tid; e < kTcM * (D / 8); e += kLfThreads) {
    const int r = e / (D / 8), ck = e % (D / 8);
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (r < nq) v = reinterpret_cast<const uint4*>(Qb + (size_t)(q0 + r) * D)[ck];
    *reinterpret_cast<uint4*>(Qs + (ck >> 3) * kTcM * 128 + tc::sw128_off(r, ck & 7)) = v;
  }
  tc::fence_async_smem();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tbase = tbase_s, tl = tbase + ((uint32_t)((warp & 3) * 32) << 16);
  const uint32_t qa = tc::smem_u32(Qs), ka = tc::smem_u32(Ks), va = tc::smem_u32(Vs), pa = tc::smem_u32(Ps);
  bool ok = true;
  // Thread 0 issues the MMAs, thread 32 the tile loads: a bulk-tensor instruction holds its thread for some
  // 270 clocks per 16 KB box, and every row of the tile waits for thread 0 at the next barrier.
  // Rows past the block's visible keys are loaded too (they are masked).
  auto load_k = [&](int t) {
    tc::mbar_expect_tx(&barK[t & 1], kKB);
    for (int g = 0; g < D / 64; ++g) tc::tma_load_2d(Ks + (t & 1) * kKB + g * kTcN * 128, &tm_k, 64 * g, krow0 + t * kTcN, &barK[t & 1]);
  };
  auto load_v = [&](int t) {
    tc::mbar_expect_tx(&barV, kKB);
    for (int g = 0; g < D / 64; ++g) tc::tma_load_2d(Vs + g * kTcN * 128, &tm_v, 64 * g, krow0 + t * kTcN, &barV);
  };
  auto issue_s = [&](int t) {                               // S(t) = Q K_t^T into S buffer t & 1
    if (!tc::mbar_wait(&barK[t & 1], (t >> 1) & 1)) ok = false;
    tc::fence_after_sync();
    const uint32_t idesc = tc::idesc_bf16(kTcM, kTcN, 0, 0);
    const uint32_t kat = ka + (t & 1) * kKB;
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks)
      tc::mma_bf16_ss(tbase + (t & 1) * kTcN, tc::smem_desc_sw128(qa + (ks / 4) * kTcM * 128 + (ks % 4) * 32, 16, 1024),
                      tc::smem_desc_sw128(kat + (ks / 4) * kTcN * 128 + (ks % 4) * 32, 16, 1024), idesc, ks > 0);
    tc::mma_commit(&barS[t & 1]);
  };
  if (tid == 32) {
    load_k(0);
    if (T > 1) load_k(1);
  }
  if (tid == 0) issue_s(0);
  const float scale2 = dm.sigma * 1.4426950408889634f;
  const int my_limit = q0 + row;                            // last visible key of this row
  // The output accumulates in TMEM over all key tiles.  m2 is the exponent base in use for this row (log2
  // units): it follows the running maximum lazily, only when that has grown by more than kLazy (probabilities
  // then stay below 2^kLazy), and only then is the accumulator rescaled, for every row of the tile at once.
  constexpr float kLazy = 8.f;
  float m2 = -INFINITY, l = 0.f;                            // l: this warpgroup's share of the row sum
  for (int t = 0; t < T && ok; ++t) {
    const int c0 = k_lo + t * kTcN, nk = min(kTcN, k_hi - c0);
    if (!tc::mbar_wait(&barS[t & 1], (t >> 1) & 1)) { ok = false; break; }
    tc::fence_after_sync();
    if (tid == 0 && t + 1 < T) issue_s(t + 1);              // runs during this tile's softmax
    __syncwarp();
    if (t > 0) {                                            // O(t-1) has landed: P and V are free (thread 0 has seen it too)
      if (!tc::mbar_wait(&barPV, (t - 1) & 1)) ok = false;
      tc::fence_after_sync();
    }
    if (tid == 32) {
      load_v(t);
      if (t + 2 < T) load_k(t + 2);                         // over K_t, which S(t) has consumed
    }
    float s[32];
    tc::tmem_ld32(tl + (t & 1) * kTcN + 32 * wg, s);
    const int vis = min(nk, my_limit - c0 + 1) - 32 * wg;  // visible columns among this thread's 32
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < 32; ++i) { s[i] = i < vis ? s[i] * scale2 : -INFINITY; mx = fmaxf(mx, s[i]); }
    mx_s[wg][row] = mx;
    // (the first tile gives every row a finite maximum: it holds the block's first key)
    const int grow = __syncthreads_or(t > 0 && mx > m2 + kLazy);
    const float mt = fmaxf(mx_s[0][row], mx_s[1][row]);
    if (t == 0) {
      m2 = mt;
    } else if (grow) {
      const float mn = mt > m2 + kLazy ? mt : m2;           // rows that did not grow keep their base (factor 1)
      const float resc = tc::fast_exp2(m2 - mn);
#pragma unroll
      for (int d0 = 0; d0 < HD; d0 += 32) {
        float v[32];
        tc::tmem_ld32(tl + cO + wg * HD + d0, v);
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] *= resc;
        tc::tmem_st32(tl + cO + wg * HD + d0, v);
      }
      l *= resc;
      m2 = mn;
    }
    const float base = m2 == -INFINITY ? 0.f : m2;
    float rs = 0.f;
#pragma unroll
    for (int ch = 0; ch < 4; ++ch) {
      uint32_t pk[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        __nv_bfloat162 b = __floats2bfloat162_rn(tc::fast_exp2(s[8 * ch + 2 * e] - base), tc::fast_exp2(s[8 * ch + 2 * e + 1] - base));
        rs += __low2float(b) + __high2float(b);             // the rounded values, as the P V product sees them
        pk[e] = *reinterpret_cast<uint32_t*>(&b);
      }
      *reinterpret_cast<uint4*>(Ps + tc::sw128_off(row, 4 * wg + ch)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
    }
    l += rs;
    tc::fence_async_smem();
    tc::fence_before_sync();
    __syncthreads();
    if (tid == 0) {
      if (!tc::mbar_wait(&barV, t & 1)) ok = false;
      tc::fence_after_sync();
      const uint32_t idesc = tc::idesc_bf16(kTcM, D, 0, 1);
#pragma unroll
      for (int ks = 0; ks < kTcN / 16; ++ks)
        tc::mma_bf16_ss(tbase + cO, tc::smem_desc_sw128(pa + ks * 32, 16, 1024),
                        tc::smem_desc_sw128(va + ks * 16 * 128, kTcN * 128, 1024), idesc, t > 0 || ks > 0);
      tc::mma_commit(&barPV);
    }
    __syncwarp();
  }
  if (ok && T > 0) {
    if (!tc::mbar_wait(&barPV, (T - 1) & 1)) ok = false;
    tc::fence_after_sync();
  }
  // the two halves of the row sum meet
  __syncthreads();
  mx_s[wg][row] = l;
  __syncthreads();
  const float lt = mx_s[0][row] + mx_s[1][row];
  if (ok && T > 0) {
    const size_t t = (size_t)pq * dm.N + q0 + row;
    const float inv = 1.f / lt;
    float4* dst = reinterpret_cast<float4*>(o_loc + t * D + wg * HD);
#pragma unroll
    for (int d0 = 0; d0 < HD; d0 += 32) {
      float v[32];
      tc::tmem_ld32(tl + cO + wg * HD + d0, v);
      if (row < nq) {
#pragma unroll
        for (int i = 0; i < 8; ++i) dst[d0 / 4 + i] = make_float4(v[4 * i] * inv, v[4 * i + 1] * inv, v[4 * i + 2] * inv, v[4 * i + 3] * inv);
      }
    }
    if (wg == 0 && row < nq) lse_loc[t] = (m2 + log2f(lt)) * 0.6931471805599453f;
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tbase, 256);
  if (!ok && tid == 0) report_status(status, 1);
}

// ---- exact retrieval ---------------------------------------------------------------------------------
// A popular cluster is retrieved by thousands of queries of a block: its 128-pair tiles are
// spread over kRetFwdSplit CTAs.
constexpr int kRetFwdSplit = 4;

template <int D>
__global__ void __launch_bounds__(128)
k_ret_fwd_tc(Dims dm, const bf16* __restrict__ Q, const bf16* __restrict__ Kp, const bf16* __restrict__ Vp,
             const int32_t* __restrict__ off_k, const int32_t* __restrict__ goff, const int32_t* __restrict__ pairs,
             bf16* __restrict__ o_part, float* __restrict__ l_part, int min_cluster_keys, int* __restrict__ status) {
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ uint64_t bar[2];
  __shared__ uint32_t tbase_s;
  __shared__ int32_t pid_s[kTcM];
  const int tid = threadIdx.x;
  const int j = blockIdx.x, pl = blockIdx.y / kRetFwdSplit, sub = blockIdx.y % kRetFwdSplit, pq = blockIdx.z;
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int nkeys = dm.SB * dm.Ck;
  const int32_t* go = goff + (size_t)pq * (nkeys + 1) + (size_t)j * dm.SB + pl;
  const int g0 = go[0], g1 = go[1];
  if (g0 + sub * kTcM >= g1) return;                     // no pair tile for this split (before any TMEM allocation)
  const int32_t* ok = off_k + (size_t)pk * (dm.Ck * dm.S + 1) + (size_t)j * dm.S;
  const int k0 = ok[0], k1 = ok[pl + 1];
  if (ok[dm.SB] - k0 < min_cluster_keys) return;         // short clusters are handled by the cluster-resident kernel
  TcCtx c;
  tc_setup<D>(c, sm_raw, bar, &tbase_s, tid);
  const bf16* Qb = Q + (size_t)pq * dm.N * D;
  const bf16* Kb = Kp + (size_t)pk * dm.N * D;
  const bf16* Vb = Vp + (size_t)pk * dm.N * D;
  const int32_t* pr = pairs + (size_t)pq * dm.N * dm.m;
  const float scale2 = dm.sigma * 1.4426950408889634f;
  for (int t0 = g0 + sub * kTcM; t0 < g1 && c.ok; t0 += kRetFwdSplit * kTcM) {
    const int nq = min(kTcM, g1 - t0);
    __syncthreads();
    pid_s[tid] = tid < nq ? pr[t0 + tid] : 0;
    __syncthreads();
    fill_kmajor<D, kTcM>(c.Qs, nq, [&](int r) { return Qb + (size_t)(pid_s[r] / dm.m) * D; }, tid);
    float o[D], m2 = -INFINITY, l = 0.f;
#pragma unroll
    for (int i = 0; i < D; ++i) o[i] = 0.f;
    attend_tc<D>(c, Kb, Vb, k0, k1, [&](int) { return k1 - 1; }, scale2, o, m2, l, tid);
    if (c.ok && tid < nq) {
      const size_t pid = (size_t)pq * dm.N * dm.m + pid_s[tid];
      const float inv = l > 0.f ? 1.f / l : 0.f;
      uint4* dst = reinterpret_cast<uint4*>(o_part + pid * D);          // normalised partial output, bf16 row
#pragma unroll
      for (int i = 0; i < D / 8; ++i) {
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          __nv_bfloat162 b2 = __floats2bfloat162_rn(o[8 * i + 2 * e] * inv, o[8 * i + 2 * e + 1] * inv);
          w[e] = *reinterpret_cast<uint32_t*>(&b2);
        }
        dst[i] = make_uint4(w[0], w[1], w[2], w[3]);
      }
      l_part[pid] = l > 0.f ? (m2 + log2f(l)) * 0.6931471805599453f : -INFINITY;
    }
  }
  tc_teardown<D>(c, tid, status);
}

int make_tmap_bf16_rows(void* out_map, const void* base, uint64_t rows, uint32_t cols, uint32_t box_rows);

int local_fwd_tc(const Dims& d, const void* Q, const void* K, const void* V, float* o_loc, float* lse_loc, int* status,
                 cudaStream_t st) {
  const int pq = d.B * d.Hq;
  CUtensorMap tk, tv;
  int rc = make_tmap_bf16_rows(&tk, K, (uint64_t)d.B * d.Hkv * d.N, (uint32_t)d.D, kTcN);
  if (rc == MUSE_OK) rc = make_tmap_bf16_rows(&tv, V, (uint64_t)d.B * d.Hkv * d.N, (uint32_t)d.D, kTcN);
  if (rc != MUSE_OK) return rc;
  dim3 grid(d.S * cdiv(d.Bs, kTcM), pq);
  prof_mark("k_local_fwd_tc", st);
  if (d.D == 128) {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_local_fwd_tc<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, LfSmem<128>::total));
    k_local_fwd_tc<128><<<grid, kLfThreads, LfSmem<128>::total, st>>>(d, tk, tv, (const bf16*)Q, o_loc, lse_loc, status);
  } else {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_local_fwd_tc<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, LfSmem<64>::total));
    k_local_fwd_tc<64><<<grid, kLfThreads, LfSmem<64>::total, st>>>(d, tk, tv, (const bf16*)Q, o_loc, lse_loc, status);
  }
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

int ret_fwd_pairs_tc(const Dims& d, const void* Q, const void* Kp, const void* Vp, const int32_t* off_k, const int32_t* goff,
                     const int32_t* pairs, void* o_part, float* l_part, int* status, cudaStream_t st);

int ret_fwd_tc(const Dims& d, const void* Q, const void* Kp, const void* Vp, const int32_t* off_k, const int32_t* goff,
               const int32_t* pairs, void* o_part, float* l_part, int* status, cudaStream_t st) {
  dim3 grid(d.Ck, d.SB * kRetFwdSplit, d.B * d.Hq);
  const int min_keys = 0;
  if (!path_forced(kForceRetFwdStream) || d.k2 > 0)           // (block selection exists in the pair kernel only)
    return ret_fwd_pairs_tc(d, Q, Kp, Vp, off_k, goff, pairs, o_part, l_part, status, st);
  prof_mark("k_ret_fwd_tc", st);
  if (d.D == 128) {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_ret_fwd_tc<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdTcSmem<128>::total));
    k_ret_fwd_tc<128><<<grid, 128, FwdTcSmem<128>::total, st>>>(d, (const bf16*)Q, (const bf16*)Kp, (const bf16*)Vp, off_k, goff, pairs, (bf16*)o_part, l_part, min_keys, status);
  } else {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_ret_fwd_tc<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdTcSmem<64>::total));
    k_ret_fwd_tc<64><<<grid, 128, FwdTcSmem<64>::total, st>>>(d, (const bf16*)Q, (const bf16*)Kp, (const bf16*)Vp, off_k, goff, pairs, (bf16*)o_part, l_part, min_keys, status);
  }
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

}  // namespace muse
