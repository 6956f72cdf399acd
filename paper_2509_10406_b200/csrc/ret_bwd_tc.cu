// Exact retrieval, backward (Section "Exact Retrieval and Local Attention"; gradients with the selections
// held constant, Appendix "Centroid Gradient Flow"), D = 64 or 128.  With L the merged log-sum-exp and
// delta = dO.O:   P = exp(sigma q.k - L),  G = sigma P (dO.v - delta),
//                 dQ = G K  (one bf16 partial row per (query, slot) pair),  dV = P^T dO,  dK = G^T Q.
// Organised by the inverse index like the forward pass: a CTA owns one key cluster of one head (or a share
// of it), keeps 64 of its keys and values in shared memory, and walks the retrieving pairs in tiles of 128
// (pairs on the MMA M side), ordered by plane:
//   S = Q K^T, dP = dO V^T            tcgen05.mma into tensor memory
//   P, G                               one thread per pair row, written as bf16 tiles to shared memory
//   dQ = G K                           over the tensor-memory columns that S and dP have vacated
//   dV^T += dO^T P,  dK^T += Q^T G     [D][keys], accumulated in tensor memory over all of the CTA's tiles
// The tiles of Q, dO, P and G fill shared memory, so only one CTA fits an SM; to keep the tensor cores, the
// load/store unit and the arithmetic warps busy at the same time, the CTA runs TWO independent pipelines
// ("halves") that share the key / value tiles and take alternate pair tiles.  Each half has four row warps,
// an MMA-issuing warp and four gather warps (the Q and dO rows arrive by 16-byte asynchronous copies, whose rate
// grows with the number of threads that issue them; no arithmetic warp spends its time on them), its own 256 tensor-memory columns, its own
// barriers and its own dV^T / dK^T accumulators, added to global memory with float atomics at the end of a sweep.
// A cluster with more than 64 visible keys takes further sweeps over the tiles that see them; later sweeps
// add to the stored dQ rows.
#include <cuda.h>
#include "common.cuh"
#include "tc05.cuh"

namespace muse {

typedef __nv_bfloat16 bf16;

namespace rb {
constexpr int kPairs = 128, kKeys = 64;
constexpr int kRowWarps = 4, kIssuerWarp0 = 8, kGatherWarp0 = 10, kGather = 128, kThreads = (kGatherWarp0 + 2 * kGather / 32) * 32;
constexpr int kSplit = 4, kTilesPerCta = 16;                // a cluster with many pair tiles is shared by up to 4 CTAs
constexpr int kOkCache = 72;
constexpr float kLog2e = 1.4426950408889634f;
template <int D> struct Lay {
  static constexpr int kTile = kPairs * D * 2, kKV = kKeys * D * 2, kPG = kPairs * kKeys * 2;
  static constexpr int oK = 0, oV = kKV, oHalf = 2 * kKV, kHalf = 2 * kTile + 2 * kPG;   // per half: Q | dO | P | G
  static constexpr int kSmem = oHalf + 2 * kHalf;           // 224 KB at D = 128: no slack, the kernel checks the alignment of its base
};
constexpr uint32_t cS = 0, cDP = 64, cDQ = 0, cDV = 128, cDK = 192, kCols = 256;   // per half; dQ reuses the columns of S and dP

struct Bars { uint64_t q_full, q_empty, s_done, pg_ready, m2_done, dq_free; };

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* src, bool valid) {
  const int n = valid ? 16 : 0;                             // 0 source bytes: the 16 bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(tc::smem_u32(smem_dst)), "l"(src), "r"(n) : "memory");
}
// K-major view of a [ROWS][D] tile at k-step ks (16 elements of D) / MN-major view at k-step ks (16 rows)
template <int ROWS> __device__ __forceinline__ uint64_t desc_k(uint32_t base, int ks) {
  return tc::smem_desc_sw128(base + (ks / 4) * ROWS * 128 + (ks % 4) * 32, 16, 1024);
}
template <int ROWS> __device__ __forceinline__ uint64_t desc_mn(uint32_t base, int ks) {
  return tc::smem_desc_sw128(base + ks * 16 * 128, ROWS * 128, 1024);
}
}  // namespace rb

template <int D>
__global__ void __launch_bounds__(rb::kThreads, 1)
k_ret_bwd_pairs_tc(Dims dm, const bf16* __restrict__ Q, const bf16* __restrict__ dO, const bf16* __restrict__ Kp,
                   const bf16* __restrict__ Vp, const float* __restrict__ LSE, const float* __restrict__ delta,
                   const int32_t* __restrict__ off_k, const int32_t* __restrict__ goff, const int32_t* __restrict__ pairs,
                   bf16* __restrict__ dq_part, float* __restrict__ dK_perm, float* __restrict__ dV_perm, int* __restrict__ status) {
  using namespace rb;
  typedef Lay<D> LY;
  constexpr int kTile = LY::kTile, kPG = LY::kPG, oK = LY::oK, oV = LY::oV, oHalf = LY::oHalf, kHalf = LY::kHalf;
  extern __shared__ __align__(1024) unsigned char sm[];
  __shared__ Bars bars[2];
  __shared__ uint32_t tbase_s;
  __shared__ int32_t ok_s[kOkCache];
  __shared__ int32_t tok_s[2][kPairs];                      // tokens of the tile each half is gathering
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // With spatial block selection (k2 > 0) the CTA owns one BUCKET (cluster j, block bb): its pairs are the (query, slot,
  // chosen block) triples that chose the block, and every one of them sees the whole bucket (as in the forward kernel).
  const bool bucket = dm.k2 > 0;
  const int j = bucket ? blockIdx.x / dm.SB : blockIdx.x, bb = bucket ? blockIdx.x % dm.SB : 0, sub = blockIdx.y, pq = blockIdx.z;
  const int mk = dm.m * (bucket ? dm.k2 : 1);               // partial dQ rows per query
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int ngroups = dm.SB * dm.Ck;
  const int32_t* go = goff + (size_t)pq * (ngroups + 1) + (size_t)j * dm.SB + bb;   // the group's pairs: plane pl is [go[pl], go[pl + 1])
  const int g0 = go[0], g1 = go[bucket ? 1 : dm.SB];
  const int ntiles = (g1 - g0 + kPairs - 1) / kPairs;
  const int nsub = min(kSplit, max(1, ntiles / kTilesPerCta));            // tiles are dealt round-robin to nsub CTAs
  const int32_t* okg = off_k + (size_t)pk * (dm.Ck * dm.S + 1) + (size_t)j * dm.S;   // okg[b]: first key of bucket (j, b)
  const int k0 = okg[bb], kall = (bucket ? okg[bb + 1] : okg[dm.SB]) - k0;   // keys that some pair of the group sees
  if (ntiles == 0 || sub >= nsub) return;
  if (tc::smem_u32(sm) & 1023u) {                           // the tiles fill the whole dynamic allocation: no room to realign
    if (tid == 0) report_status(status, MUSE_STATUS_BWD_TIMEOUT);
    return;
  }
  const int32_t* ok = dm.S + 1 <= kOkCache ? ok_s : okg;
  if (dm.S + 1 <= kOkCache)
    for (int b = tid; b <= dm.S; b += kThreads) ok_s[b] = okg[b];
  if (warp == 0) tc::tmem_alloc(&tbase_s, 2 * kCols);
  if (tid == 0) {
    for (int v = 0; v < 2; ++v) {
      tc::mbar_init(&bars[v].q_full, kGather); tc::mbar_init(&bars[v].q_empty, 1); tc::mbar_init(&bars[v].s_done, 1);
      tc::mbar_init(&bars[v].pg_ready, kRowWarps * 32); tc::mbar_init(&bars[v].m2_done, 1); tc::mbar_init(&bars[v].dq_free, kRowWarps * 32);
    }
    tc::mbar_init_fence();
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const bf16* Qb = Q + (size_t)pq * dm.N * D;
  const bf16* dOb = dO + (size_t)pq * dm.N * D;
  const bf16* Kb = Kp + ((size_t)pk * dm.N + k0) * D;
  const bf16* Vb = Vp + ((size_t)pk * dm.N + k0) * D;
  const int32_t* pr = pairs + (size_t)pq * dm.N * mk;
  const size_t pbase = (size_t)pq * dm.N * mk;
  // role of this warp: half v, and row / issuing / gather warp
  const bool roww = warp < 2 * kRowWarps, issw = warp >= kIssuerWarp0 && warp < kIssuerWarp0 + 2, gatw = warp >= kGatherWarp0;
  const int v = roww ? warp / kRowWarps : issw ? warp - kIssuerWarp0 : (warp - kGatherWarp0) / (kGather / 32);
  Bars& B = bars[v];
  unsigned char* hb = sm + oHalf + v * kHalf;               // this half's Q | dO | P | G tiles
  const uint32_t tbase = tbase_s + v * kCols;
  bool ok_ = true;                                          // false once a bounded wait ran out (every role still walks all its tiles)
  auto wait = [&](uint64_t* bar, uint32_t parity) { if (ok_ && !tc::mbar_wait(bar, parity)) ok_ = false; };
  // keys of sweep `kc` that the query of pair `pid` sees (its block's prefix of the cluster)
  auto visible = [&](int pid, int kc) {
    if (bucket) return min(kKeys, max(0, kall - kc));
    const int tok = pid / dm.m;
    return min(kKeys, max(0, ok[dm.causal ? tok / dm.Bs : 1] - k0 - kc));
  };

  uint32_t np = 0;                                          // tiles this half has processed: the phase count of its barriers
#ifdef MUSE_PHASE_CLOCKS
  long long pc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  const long long t_in_ = clock64();
  long long z_ = t_in_;
#define RBCLK(k) { long long n_ = clock64(); pc[k] += n_ - z_; z_ = n_; }
#else
#define RBCLK(k)
#endif
  // (a cluster none of whose keys is visible, possible with forced selections, still takes one sweep: its dQ rows are zeros)
  for (int kc = 0; kc == 0 || kc < kall; kc += kKeys) {
    const bool first = kc == 0;
    const int nkc = max(0, min(kKeys, kall - kc));
    // later sweeps pass over the tiles of planes that see none of the sweep's keys (a prefix of the cluster's tiles)
    int tile_lo = 0;
    if (!first && !bucket) {
      int pl = 0;
      while (pl + 1 < dm.SB && ok[pl + 1] - k0 <= kc) ++pl;
      tile_lo = (go[pl] - g0) / kPairs;
    }
    const int tile0 = tile_lo + ((sub - tile_lo % nsub) + nsub) % nsub + v * nsub;   // this half's first tile; it takes every second of the CTA's
    const int tstep = 2 * nsub;
    __syncthreads();                                        // the previous sweep's products are complete, its accumulators read
    // the sweep's keys and values as [2][64 rows][128 B] swizzled tiles (K-major and MN-major operands); rows past the cluster are zeros
    for (int e = tid; e < kKeys * (D / 8); e += kThreads) {
      const int r = e / (D / 8), ck = e % (D / 8);
      uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;
      if (r < nkc && MUSE_IN_RANGE(k0 + kc + r, dm.N)) {
        a = reinterpret_cast<const uint4*>(Kb + (size_t)(kc + r) * D)[ck];
        b = reinterpret_cast<const uint4*>(Vb + (size_t)(kc + r) * D)[ck];
      }
      const uint32_t off = (ck >> 3) * kKeys * 128 + tc::sw128_off(r, ck & 7);
      if (!MUSE_IN_RANGE(off, kKeys * D * 2 - 15)) continue;
      *reinterpret_cast<uint4*>(sm + oK + off) = a;
      *reinterpret_cast<uint4*>(sm + oV + off) = b;
    }
    tc::fence_async_smem();                                 // the tensor cores read the tiles through the async proxy
    __syncthreads();

    if (roww) {
      // ================= P, G and the dQ rows: thread = pair row =================
      const int row = tid & 127;
      const uint32_t tl = tbase + ((uint32_t)((warp & 3) * 32) << 16);
      const float scale2 = dm.sigma * kLog2e;
      // pair ids two tiles ahead and the rows' L, delta one tile ahead: no dependent global load at the top of a tile
      auto ld_pid = [&](int t) {
        const int t0 = g0 + t * kPairs;
        const int id = (t < ntiles && t0 + row < g1) ? __ldg(pr + t0 + row) : -1;
        return id >= 0 && !MUSE_IN_RANGE(id, (long long)dm.N * mk) ? -1 : id;
      };
      int pid = ld_pid(tile0), pid_n = ld_pid(tile0 + tstep);
      float L2 = 0.f, dl = 0.f, L2_n = 0.f, dl_n = 0.f;
      auto ld_scalars = [&](int p, float& l2, float& d_) {
        const size_t tt = (size_t)pq * dm.N + max(p, 0) / mk;
        l2 = p >= 0 ? LSE[tt] * kLog2e : 0.f;
        d_ = p >= 0 ? delta[tt] : 0.f;
      };
      ld_scalars(pid, L2, dl);
      bool started = false;
      for (int tile = tile0; tile < ntiles; tile += tstep, ++np) {
        const int pid_nn = ld_pid(tile + 2 * tstep);
        ld_scalars(pid_n, L2_n, dl_n);
        if (!first && pid_n >= 0) {                         // a later sweep adds to the stored dQ row: have the next tile's row on its way
          const char* pf = reinterpret_cast<const char*>(dq_part + (pbase + pid_n) * D);
#pragma unroll
          for (int o = 0; o < D * 2; o += 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(pf + o));
        }
        const int vis = pid >= 0 ? visible(pid, kc) : 0;
        const uint32_t ph = np & 1;
        RBCLK(0)
        wait(&B.s_done, ph);
        tc::fence_after_sync();
        RBCLK(1)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {                    // 32 key columns at a time
          float sv[32], dp[32];
          tc::tmem_ld32(tl + cS + 32 * hf, sv);
          tc::tmem_ld32(tl + cDP + 32 * hf, dp);
          uint32_t pw[16], gw[16];
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const float e0 = 32 * hf + i < vis ? tc::fast_exp2(fmaf(sv[i], scale2, -L2)) : 0.f;
            const float e1 = 32 * hf + i + 1 < vis ? tc::fast_exp2(fmaf(sv[i + 1], scale2, -L2)) : 0.f;
            __nv_bfloat162 pb = __floats2bfloat162_rn(e0, e1);
            __nv_bfloat162 gb = __floats2bfloat162_rn(e0 * (dp[i] - dl) * dm.sigma, e1 * (dp[i + 1] - dl) * dm.sigma);   // (sigma rides on G: dQ and dK come out scaled)
            pw[i / 2] = *reinterpret_cast<uint32_t*>(&pb);
            gw[i / 2] = *reinterpret_cast<uint32_t*>(&gb);
          }
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4) {
            const uint32_t off = tc::sw128_off(row, 4 * hf + c4);
            *reinterpret_cast<uint4*>(hb + 2 * kTile + off) = make_uint4(pw[4 * c4], pw[4 * c4 + 1], pw[4 * c4 + 2], pw[4 * c4 + 3]);
            *reinterpret_cast<uint4*>(hb + 2 * kTile + kPG + off) = make_uint4(gw[4 * c4], gw[4 * c4 + 1], gw[4 * c4 + 2], gw[4 * c4 + 3]);
          }
        }
        tc::fence_async_smem();                             // P and G are read by the tensor cores
        tc::fence_before_sync();
        tc::mbar_arrive(&B.pg_ready);
        RBCLK(2)
        wait(&B.m2_done, ph);
        tc::fence_after_sync();
        RBCLK(3)
        started = true;
        const bool live = pid >= 0 && ok_;
        bf16* drow = dq_part + (pbase + max(pid, 0)) * D;
#pragma unroll
        for (int d0 = 0; d0 < D; d0 += 32) {
          float x[32];
          tc::tmem_ld32(tl + cDQ + d0, x);                  // (warp-wide: every thread takes part, rows past the tile's end do not store)
          if (d0 + 32 == D) {                               // the columns may be overwritten by the next tile's S and dP
            tc::fence_before_sync();
            tc::mbar_arrive(&B.dq_free);
          }
          if (live) {
#pragma unroll
            for (int c = 0; c < 2; ++c) {                   // 16 columns = 32 bytes per store
              uint32_t w[8];
              if (!first) {
                tc::ld_global_32B(drow + d0 + 16 * c, w);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                  const __nv_bfloat162 o2 = *reinterpret_cast<const __nv_bfloat162*>(&w[e]);
                  __nv_bfloat162 b2 = __floats2bfloat162_rn(x[16 * c + 2 * e] + __low2float(o2), x[16 * c + 2 * e + 1] + __high2float(o2));
                  w[e] = *reinterpret_cast<uint32_t*>(&b2);
                }
              } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                  __nv_bfloat162 b2 = __floats2bfloat162_rn(x[16 * c + 2 * e], x[16 * c + 2 * e + 1]);
                  w[e] = *reinterpret_cast<uint32_t*>(&b2);
                }
              }
              tc::st_global_32B(drow + d0 + 16 * c, w);
            }
          }
        }
        pid = pid_n; pid_n = pid_nn; L2 = L2_n; dl = dl_n;
        RBCLK(4)
#ifdef MUSE_PHASE_CLOCKS
        pc[7] += 1;
#endif
      }
      // dV^T and dK^T of this sweep's keys: thread = output dim, one key per column; the other half of the CTA
      // (and other CTAs that share the cluster) add theirs to the same rows
      if (started && (warp & 3) * 32 < D) {                  // (warp-uniform: the lanes of a warp hold 32 consecutive dims)
        const int dd = (warp & 3) * 32 + lane;
#pragma unroll
        for (int w2 = 0; w2 < 2; ++w2) {
          float* dst = (w2 == 0 ? dV_perm : dK_perm) + ((size_t)pq * dm.N + k0 + kc) * D + dd;
#pragma unroll
          for (int u0 = 0; u0 < kKeys; u0 += 32) {
            float x[32];
            tc::tmem_ld32(tl + (w2 == 0 ? cDV : cDK) + u0, x);
            if (ok_) {
#pragma unroll
              for (int u = 0; u < 32; ++u)
                if (u0 + u < nkc && MUSE_IN_RANGE(k0 + kc + u0 + u, dm.N)) atomicAdd(dst + (size_t)(u0 + u) * D, x[u]);      // (result unused: no round trip)
            }
          }
        }
      }
    } else if (issw) {
      // ================= MMA issue =================
      const uint32_t qa = tc::smem_u32(hb), da = qa + kTile, pa = da + kTile, ga = pa + kPG;
      const uint32_t ka = tc::smem_u32(sm + oK), va = tc::smem_u32(sm + oV);
      const uint32_t np0 = np;
      for (int tile = tile0; tile < ntiles; tile += tstep, ++np) {
        if (lane == 0) {
          const uint32_t ph = np & 1;
          RBCLK(0)
          wait(&B.q_full, ph);                               // the tile's Q and dO rows are in shared memory
          RBCLK(1)
          if (np > 0) wait(&B.dq_free, ph ^ 1);              // the previous dQ rows have been read out of the columns S and dP go to
          tc::fence_after_sync();
          RBCLK(2)
          const uint32_t id1 = tc::idesc_bf16(kPairs, kKeys, 0, 0);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) tc::mma_bf16_ss(tbase + cS, desc_k<kPairs>(qa, ks), desc_k<kKeys>(ka, ks), id1, ks > 0);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) tc::mma_bf16_ss(tbase + cDP, desc_k<kPairs>(da, ks), desc_k<kKeys>(va, ks), id1, ks > 0);
          tc::mma_commit(&B.s_done);
          RBCLK(3)
          wait(&B.pg_ready, ph);                             // P and G are in shared memory, S and dP consumed
          tc::fence_after_sync();
          RBCLK(4)
          const uint32_t id_dq = tc::idesc_bf16(kPairs, D, 0, 1);        // A = G (contraction over keys), B = key rows MN-major
          // A = dO / Q tile and B = P / G tile, both contracted over pairs.  M = 128 output dims even when D = 64: the second
          // 64-dim group of the A operand is then the tile that follows in shared memory, and lanes 64..127 hold numbers nobody reads
          const uint32_t id_t = tc::idesc_bf16(128, kKeys, 1, 1);
          const bool acc = np > np0;                                     // the accumulators start at zero in every sweep
#pragma unroll
          for (int ks = 0; ks < kKeys / 16; ++ks)
            tc::mma_bf16_ss(tbase + cDQ, tc::smem_desc_sw128(ga + ks * 32, 16, 1024), desc_mn<kKeys>(ka, ks), id_dq, ks > 0);
#pragma unroll
          for (int ks = 0; ks < kPairs / 16; ++ks)
            tc::mma_bf16_ss(tbase + cDV, desc_mn<kPairs>(da, ks), tc::smem_desc_sw128(pa + ks * 16 * 128, kPairs * 128, 1024), id_t, acc || ks > 0);
#pragma unroll
          for (int ks = 0; ks < kPairs / 16; ++ks)
            tc::mma_bf16_ss(tbase + cDK, desc_mn<kPairs>(qa, ks), tc::smem_desc_sw128(ga + ks * 16 * 128, kPairs * 128, 1024), id_t, acc || ks > 0);
          tc::mma_commit(&B.m2_done);
          tc::mma_commit(&B.q_empty);                        // ... and the Q / dO tiles refilled
          RBCLK(5)
#ifdef MUSE_PHASE_CLOCKS
          pc[7] += 1;
#endif
        }
        __syncwarp();
      }
      if (lane == 0 && np > np0) {                           // all products done before the key tiles are replaced or the CTA ends
        wait(&B.m2_done, (np - 1) & 1);
        tc::fence_after_sync();
      }
    } else if (gatw) {
      // ================= gather of the Q and dO rows =================
      const int g = tid - (kGatherWarp0 + (kGather / 32) * v) * 32, ck = g % (D / 8);
      constexpr int RPP = kGather / (D / 8);                // rows per pass
      static_assert(kGather == kPairs, "one gather thread per pair row looks up its token");
      unsigned char* qd = hb + (ck >> 3) * kPairs * 128;
      unsigned char* od = hb + kTile + (ck >> 3) * kPairs * 128;
      auto ld1 = [&](int t) {                                // id of row g
        const int t0 = g0 + t * kPairs;
        return (t < ntiles && t0 + g < g1) ? __ldg(pr + t0 + g) : -1;
      };
      int pa_ = ld1(tile0);
      for (int tile = tile0; tile < ntiles; tile += tstep, ++np) {
        const int pa_n = ld1(tile + tstep);
        RBCLK(0)
        if (np > 0) wait(&B.q_empty, (np - 1) & 1);          // the previous tile's products have read the buffers
        RBCLK(1)
        tok_s[v][g] = pa_ >= 0 ? pa_ / mk : -1;
        tc::named_bar_sync(1 + v, kGather);
#pragma unroll 4
        for (int r = g / (D / 8); r < kPairs; r += RPP) {
          const int tok = tok_s[v][r];
          const size_t at = (size_t)max(tok, 0) * D + ck * 8;
          if (!MUSE_IN_RANGE(tok + 1, dm.N + 1) || !MUSE_IN_RANGE((ck >> 3) * kPairs * 128 + tc::sw128_off(r, ck & 7), kPairs * D * 2 - 15)) continue;
          cp_async16(qd + tc::sw128_off(r, ck & 7), Qb + at, tok >= 0);
          cp_async16(od + tc::sw128_off(r, ck & 7), dOb + at, tok >= 0);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        RBCLK(2)
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        tc::fence_async_smem();                              // the tensor cores read the rows through the async proxy
        tc::mbar_arrive(&B.q_full);
        RBCLK(3)
        tc::named_bar_sync(1 + v, kGather);                  // tok_s may be rewritten
        pa_ = pa_n;
#ifdef MUSE_PHASE_CLOCKS
        pc[7] += 1;
#endif
      }
    }
    tc::fence_before_sync();
  }
#ifdef MUSE_PHASE_CLOCKS
  // (instrumented builds only: words 8..22 of the status block, five per role, in units of 16 clocks)
  if (pc[7] >= 20 && lane == 0 && v == 0 && (warp == 0 || warp == kIssuerWarp0 || warp == kGatherWarp0)) {
    const int slot = warp == 0 ? 0 : warp == kIssuerWarp0 ? 1 : 2;
    if (atomicCAS(status + 5 + slot, 0, 1) == 0) {
      int* o = status + 8 + 5 * slot;
      if (slot == 0) { o[0] = (int)(pc[1] / 16); o[1] = (int)(pc[2] / 16); o[2] = (int)(pc[3] / 16); o[3] = (int)(pc[4] / 16); o[4] = (int)pc[7]; }
      if (slot == 1) { o[0] = (int)(pc[1] / 16); o[1] = (int)(pc[2] / 16); o[2] = (int)(pc[4] / 16); o[3] = (int)(pc[5] / 16); o[4] = (int)((clock64() - t_in_) / 16); }
      if (slot == 2) { o[0] = (int)(pc[1] / 16); o[1] = (int)(pc[2] / 16); o[2] = (int)(pc[3] / 16); o[3] = (int)pc[7]; o[4] = kall; }
    }
  }
#endif
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tbase_s, 2 * kCols);
  if (!ok_ && lane == 0) report_status(status, MUSE_STATUS_BWD_TIMEOUT);
}

int ret_bwd_pairs_tc(const Dims& d, const void* Q, const void* dO, const void* Kp, const void* Vp, const float* LSE,
                     const float* delta, const int32_t* off_k, const int32_t* goff, const int32_t* pairs, void* dq_part,
                     float* dK_perm, float* dV_perm, int* status, cudaStream_t st) {
  prof_mark("k_ret_bwd_pairs_tc", st);
  const dim3 grid(d.k2 > 0 ? d.Ck * d.SB : d.Ck, rb::kSplit, d.B * d.Hq);      // one CTA (or a few) per key cluster, or per bucket
  if (d.D == 128) {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_ret_bwd_pairs_tc<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, rb::Lay<128>::kSmem));
    k_ret_bwd_pairs_tc<128><<<grid, rb::kThreads, rb::Lay<128>::kSmem, st>>>(
        d, (const bf16*)Q, (const bf16*)dO, (const bf16*)Kp, (const bf16*)Vp, LSE, delta, off_k, goff, pairs, (bf16*)dq_part, dK_perm, dV_perm, status);
  } else {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_ret_bwd_pairs_tc<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, rb::Lay<64>::kSmem));
    k_ret_bwd_pairs_tc<64><<<grid, rb::kThreads, rb::Lay<64>::kSmem, st>>>(
        d, (const bf16*)Q, (const bf16*)dO, (const bf16*)Kp, (const bf16*)Vp, LSE, delta, off_k, goff, pairs, (bf16*)dq_part, dK_perm, dV_perm, status);
  }
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

}  // namespace muse
