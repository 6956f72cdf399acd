// Exact retrieval, forward (Section "Exact Retrieval and Local Attention"): every query attends, with
// its full query vector, the keys of its selected clusters that lie in earlier blocks.  The work is
// organised by the inverse index: a CTA owns one key cluster of one head (or a share of it), keeps up
// to 128 of the cluster's keys and values in shared memory, and walks the (query, slot) pairs that
// retrieve the cluster in tiles of 128 pairs, ordered by the plane (block) of the query:
//   S = Q_tile K^T          tcgen05.mma, pairs on M, only as many key columns as the tile can see
//   P = exp(sigma S - max)  one thread per pair row, straight out of tensor memory, written back to
//                           tensor memory as packed bf16 over the logits it has consumed
//   O = P V                 tcgen05.mma with P as the tensor-memory operand; the result is read out,
//                           normalised and stored as a bf16 partial row with its log-sum-exp (the
//                           merge kernel combines a query's slots)
// Warp roles: warps 0-3 softmax and read-out (thread = pair row), lane 0 of warp 4 issues the MMAs,
// warps 5-6 gather the Q rows of the next tile as soon as the first product has released the single Q
// buffer (16-byte asynchronous copies; an SM's load/store unit moves such scattered 256-byte rows at
// about 25 bytes per clock at best, so no arithmetic warp should spend its time issuing them; more
// gather warps were slower: their copies crowd out the row warps' stores).  The CTA is deliberately
// small (96 KB of shared memory, 256 TMEM columns, 224 threads) so that two of them share an SM and
// fill each other's waits.
// Clusters with more than 128 visible keys take further sweeps over the tiles that see them; a later
// sweep merges its partial result into the stored row by log-sum-exp weights.
#include <cuda.h>
#include "common.cuh"
#include "tc05.cuh"

namespace muse {

typedef __nv_bfloat16 bf16;

namespace rf {
constexpr int kRowThreads = 128, kIssuerWarp = 4, kGather0 = 160, kGather = 64, kThreads = kGather0 + kGather;
constexpr int kPairs = 128, kKeys = 128;
constexpr int kSplit = 4, kTilesPerCta = 8;                // a cluster with many pair tiles is shared by up to 4 CTAs
constexpr int kOkCache = 72;                               // bucket offsets of the cluster kept in shared memory (S + 1 <= 72)

template <int D> struct Smem {
  static constexpr int kv = kKeys * D * 2;                 // the K tile, and the V tile
  static constexpr int k = 0, v = kv, q = 2 * kv, total = q + kPairs * D * 2 + 1024;
  static constexpr uint32_t cS = 0, cO = kKeys, cols = 256;      // TMEM: logits, then P (packed bf16) over them | output
};

struct Bars { uint64_t q_full, q_empty, s_done, p_ready, o_done, o_free; };

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* src, bool valid) {
  const int n = valid ? 16 : 0;                            // 0 source bytes: the 16 bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(tc::smem_u32(smem_dst)), "l"(src), "r"(n) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]: A is a 128-row bf16 matrix in tensor memory, two K-elements per 32-bit column
__device__ __forceinline__ void mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// registers -> TMEM, 32 lanes x 16 columns; complete when the call returns
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      :: "r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
         "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]) : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
}  // namespace rf

template <int D>
__global__ void __launch_bounds__(rf::kThreads, 2)
k_ret_fwd_pairs_tc(Dims dm, const bf16* __restrict__ Q, const bf16* __restrict__ Kp, const bf16* __restrict__ Vp,
                   const int32_t* __restrict__ off_k, const int32_t* __restrict__ goff, const int32_t* __restrict__ pairs,
                   bf16* __restrict__ o_part, float* __restrict__ l_part, int* __restrict__ status) {
  using namespace rf;
  typedef Smem<D> SM;
  constexpr int CPR = D / 8;                               // 16-byte chunks per row
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ Bars bars;
  __shared__ uint32_t tbase_s;
  __shared__ int32_t ok_s[kOkCache];
  __shared__ int32_t tok_s[kPairs];                        // tokens of the tile being gathered
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // Without spatial block selection the CTA owns a key cluster and its pairs of every plane (a query sees the cluster's
  // keys of the earlier blocks).  With it (k2 > 0) the CTA owns one BUCKET (cluster, block bb): its pairs are the
  // (query, slot, chosen block) triples that chose this block, and every one of them sees the whole bucket.
  const bool bucket = dm.k2 > 0;
  const int j = bucket ? blockIdx.x / dm.SB : blockIdx.x, bb = bucket ? blockIdx.x % dm.SB : 0, sub = blockIdx.y, pq = blockIdx.z;
  const int mk = dm.m * (bucket ? dm.k2 : 1);              // partial results per query
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int ngroups = dm.SB * dm.Ck;
  const int32_t* go = goff + (size_t)pq * (ngroups + 1) + (size_t)j * dm.SB + bb;   // the group's pairs: plane pl is [go[pl], go[pl + 1])
  const int g0 = go[0], g1 = go[bucket ? 1 : dm.SB];
  const int ntiles = (g1 - g0 + kPairs - 1) / kPairs;
  const int nsub = min(kSplit, max(1, ntiles / kTilesPerCta));           // tiles are dealt round-robin to nsub CTAs
  if (ntiles == 0 || sub >= nsub) return;
  const int32_t* okg = off_k + (size_t)pk * (dm.Ck * dm.S + 1) + (size_t)j * dm.S;   // okg[b]: first key of bucket (j, b)
  const int k0 = okg[bb], kall = (bucket ? okg[bb + 1] : okg[dm.SB]) - k0;   // keys that some pair of the group sees
  const int32_t* ok = dm.S + 1 <= kOkCache ? ok_s : okg;
  if (dm.S + 1 <= kOkCache)
    for (int b = tid; b <= dm.S; b += kThreads) ok_s[b] = okg[b];

  unsigned char* sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);
  if (warp == 0) tc::tmem_alloc(&tbase_s, SM::cols);
  if (tid == 0) {
    tc::mbar_init(&bars.q_full, kGather); tc::mbar_init(&bars.q_empty, 1); tc::mbar_init(&bars.s_done, 1);
    tc::mbar_init(&bars.p_ready, kRowThreads); tc::mbar_init(&bars.o_done, 1); tc::mbar_init(&bars.o_free, kRowThreads);
    tc::mbar_init_fence();
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tbase = tbase_s;
  const bf16* Qb = Q + (size_t)pq * dm.N * D;
  const bf16* Kb = Kp + ((size_t)pk * dm.N + k0) * D;
  const bf16* Vb = Vp + ((size_t)pk * dm.N + k0) * D;
  const int32_t* pr = pairs + (size_t)pq * dm.N * mk;
  const size_t pbase = (size_t)pq * dm.N * mk;
  bool ok_ = true;                                         // false once a bounded wait ran out (every role still walks all its tiles)
  auto wait = [&](uint64_t* bar, uint32_t parity) { if (ok_ && !tc::mbar_wait(bar, parity)) ok_ = false; };
  // keys of sweep `kc` that the query of pair `pid` sees (its block's prefix of the cluster)
  auto visible = [&](int pid, int kc) {
    if (bucket) return min(kKeys, max(0, kall - kc));
    const int tok = pid / dm.m;
    return min(kKeys, max(0, ok[dm.causal ? tok / dm.Bs : 1] - k0 - kc));
  };
#ifdef MUSE_PHASE_CLOCKS
  long long pc[10] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
  const long long t_in_ = clock64();
  long long z_ = t_in_;
#define RFCLK(k) { long long n_ = clock64(); pc[k] += n_ - z_; z_ = n_; }
#else
#define RFCLK(k)
#endif

  // Number of completed phases of each barrier, the same on every role: a tile with visible keys completes each once.
  uint32_t nproc = 0;
  for (int kc = 0; kc == 0 || kc < kall; kc += kKeys) {
    const bool first = kc == 0;
    // later sweeps pass over the tiles of planes that see none of the sweep's keys (a prefix of the cluster's tiles)
    int tile_lo = 0;
    if (!first && !bucket) {
      int pl = 0;
      while (pl + 1 < dm.SB && ok[pl + 1] - k0 <= kc) ++pl;
      tile_lo = (go[pl] - g0) / kPairs;
    }
    int tile = tile_lo + ((sub - tile_lo % nsub) + nsub) % nsub;
    __syncthreads();                                        // the previous sweep's products are complete (every role waited for them)
    // the sweep's keys (K-major for S = Q K^T) and values (MN-major for O = P V); rows past the cluster are zeros
    for (int e = tid; e < kKeys * CPR; e += kThreads) {
      const int r = e / CPR, ck = e % CPR;
      uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;
      if (kc + r < kall && MUSE_IN_RANGE(k0 + kc + r, dm.N)) {
        a = reinterpret_cast<const uint4*>(Kb + (size_t)(kc + r) * D)[ck];
        b = reinterpret_cast<const uint4*>(Vb + (size_t)(kc + r) * D)[ck];
      }
      const uint32_t off = (ck >> 3) * kKeys * 128 + tc::sw128_off(r, ck & 7);
      if (!MUSE_IN_RANGE(off, kKeys * D * 2 - 15)) continue;
      *reinterpret_cast<uint4*>(sm + SM::k + off) = a;
      *reinterpret_cast<uint4*>(sm + SM::v + off) = b;
    }
    tc::fence_async_smem();                                 // the tensor cores read the tiles through the async proxy
    __syncthreads();
    RFCLK(0)

    if (warp < kIssuerWarp) {
      // ================= softmax and read-out: thread = pair row =================
      const int row = tid;
      const uint32_t tl = tbase + ((uint32_t)(warp * 32) << 16);
      const float scale2 = dm.sigma * 1.4426950408889634f;
      // ids one tile ahead, so that no global-memory latency sits at the top of a tile
      auto tile_ids = [&](int t, int& pid, int& last) {
        const int t0 = g0 + t * kPairs, nq = min(kPairs, g1 - t0);
        pid = (t < ntiles && row < nq) ? __ldg(pr + t0 + row) : -1;
        if (pid >= 0 && !MUSE_IN_RANGE(pid, (long long)dm.N * mk)) pid = -1;
        last = t < ntiles ? __ldg(pr + t0 + nq - 1) : 0;
      };
      int pid, last;
      tile_ids(tile, pid, last);
      for (; tile < ntiles; tile += nsub) {
        int pid_n, last_n;
        tile_ids(tile + nsub, pid_n, last_n);
        if (!first && pid_n >= 0) {                         // a later sweep merges into the stored row: have the next tile's row on its way
          const char* pf = reinterpret_cast<const char*>(o_part + (pbase + pid_n) * D);
#pragma unroll
          for (int o = 0; o < D * 2; o += 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(pf + o));
          asm volatile("prefetch.global.L2 [%0];" ::"l"(l_part + pbase + pid_n));
        }
        const int nk = visible(last, kc), nk16 = (nk + 15) & ~15;      // the tile's last pair has the latest plane: it sees the most keys
        // which of the sweep's 128 key columns this row sees (a prefix: the cluster's keys of the earlier blocks, or the bucket)
        uint32_t vm[4] = {0u, 0u, 0u, 0u};
        auto set_range = [&](int lo, int hi) {               // columns [lo, hi) of the sweep
          lo = max(lo, 0); hi = min(hi, kKeys);
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const int a = max(lo - 32 * g, 0), z = min(hi - 32 * g, 32);
            if (z > a) vm[g] |= (z - a >= 32 ? 0xffffffffu : ((1u << (z - a)) - 1u) << a);
          }
        };
        if (pid >= 0) set_range(0, visible(pid, kc));
        const float lse_old = (!first && pid >= 0) ? l_part[pbase + pid] : -INFINITY;
        float M = -INFINITY, l = 0.f;
        RFCLK(1)
        if (nk16 > 0) {
          const uint32_t ph = nproc & 1;
          wait(&bars.s_done, ph);
          tc::fence_after_sync();
          RFCLK(2)
          // the logits are read twice (row maximum, then probabilities) rather than kept in registers
          float mx = -INFINITY;
          for (int g = 0; 32 * g < nk16; ++g) {
            float sv[32];
            tc::tmem_ld32(tl + SM::cS + 32 * g, sv);
            const uint32_t w = vm[g];
#pragma unroll
            for (int i = 0; i < 32; ++i) mx = fmaxf(mx, (w >> i) & 1u ? sv[i] : -INFINITY);
          }
          M = mx * scale2;                                 // (scale2 > 0)
          const float base = M == -INFINITY ? 0.f : M;
          RFCLK(3)
          for (int g = 0; 32 * g < nk16; ++g) {
            float sv[32];
            tc::tmem_ld32(tl + SM::cS + 32 * g, sv);
            const uint32_t w = vm[g];
            uint32_t pk2[16];
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              const float e0 = (w >> i) & 1u ? tc::fast_exp2(fmaf(sv[i], scale2, -base)) : 0.f;
              const float e1 = (w >> (i + 1)) & 1u ? tc::fast_exp2(fmaf(sv[i + 1], scale2, -base)) : 0.f;
              l += e0 + e1;
              __nv_bfloat162 b2 = __floats2bfloat162_rn(e0, e1);
              pk2[i / 2] = *reinterpret_cast<uint32_t*>(&b2);
            }
            // P over the logits already consumed: keys [32 g, 32 g + 32) -> columns [16 g, 16 g + 16)
            tmem_st16(tl + SM::cS + 16 * g, pk2);
          }
          tc::fence_before_sync();
          tc::mbar_arrive(&bars.p_ready);
          RFCLK(4)
          wait(&bars.o_done, ph);
          tc::fence_after_sync();
          RFCLK(5)
        }
        const bool live = pid >= 0 && ok_;
        const float inv = l > 0.f ? 1.f / l : 0.f;
        float lse_new = l > 0.f ? (M + log2f(l)) * 0.6931471805599453f : -INFINITY;
        float wn = inv, wo = 0.f;
        if (!first) {
          // merge with what earlier sweeps stored: weights e^(L_old - L), e^(L_new - L), L = log(e^L_old + e^L_new)
          const float mxl = fmaxf(lse_old, lse_new);
          const float eo = lse_old == -INFINITY ? 0.f : __expf(lse_old - mxl), en = lse_new == -INFINITY ? 0.f : __expf(lse_new - mxl);
          const float tot = eo + en;
          wo = tot > 0.f ? eo / tot : 0.f;
          wn = tot > 0.f ? en / tot * inv : 0.f;
          lse_new = tot > 0.f ? mxl + __logf(tot) : -INFINITY;
        }
        bf16* orow = o_part + (pbase + (pid >= 0 ? pid : 0)) * D;
#pragma unroll
        for (int d0 = 0; d0 < D; d0 += 32) {
          float v[32];
          if (nk16 > 0) tc::tmem_ld32(tl + SM::cO + d0, v);          // (warp-wide: every thread takes part, rows past the tile's end do not store)
          else {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = 0.f;
          }
          if (d0 + 32 == D && nk16 > 0) {                            // the output accumulator may be overwritten
            tc::fence_before_sync();
            tc::mbar_arrive(&bars.o_free);
          }
          if (live) {
#pragma unroll
            for (int c = 0; c < 2; ++c) {                            // 16 columns = 32 bytes per store
              uint32_t w[8];
              if (!first) {
                tc::ld_global_32B(orow + d0 + 16 * c, w);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                  const __nv_bfloat162 o2 = *reinterpret_cast<const __nv_bfloat162*>(&w[e]);
                  __nv_bfloat162 b2 = __floats2bfloat162_rn(fmaf(wn, v[16 * c + 2 * e], wo * __low2float(o2)),
                                                            fmaf(wn, v[16 * c + 2 * e + 1], wo * __high2float(o2)));
                  w[e] = *reinterpret_cast<uint32_t*>(&b2);
                }
              } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                  __nv_bfloat162 b2 = __floats2bfloat162_rn(v[16 * c + 2 * e] * wn, v[16 * c + 2 * e + 1] * wn);
                  w[e] = *reinterpret_cast<uint32_t*>(&b2);
                }
              }
              tc::st_global_32B(orow + d0 + 16 * c, w);
            }
          }
        }
        if (live) l_part[pbase + pid] = lse_new;
        if (nk16 > 0) ++nproc;
        pid = pid_n; last = last_n;
        RFCLK(6)
#ifdef MUSE_PHASE_CLOCKS
        pc[9] += 1;
#endif
      }
    } else if (warp == kIssuerWarp) {
      // ================= MMA issue =================
      const uint32_t qa = tc::smem_u32(sm + SM::q), ka = tc::smem_u32(sm + SM::k), va = tc::smem_u32(sm + SM::v);
      int last = tile < ntiles ? __ldg(pr + g0 + tile * kPairs + min(kPairs, g1 - g0 - tile * kPairs) - 1) : 0;
      for (; tile < ntiles; tile += nsub) {
        const int tn = tile + nsub;
        const int last_n = tn < ntiles ? __ldg(pr + g0 + tn * kPairs + min(kPairs, g1 - g0 - tn * kPairs) - 1) : 0;
        const int nk = visible(last, kc), nk16 = (nk + 15) & ~15;
        last = last_n;
        if (nk16 == 0) continue;
        const uint32_t ph = nproc & 1;
        if (lane == 0) {
          wait(&bars.q_full, ph);                            // the tile's Q rows are in shared memory
          if (nproc > 0) wait(&bars.o_done, ph ^ 1);         // the previous product has read P: the logits may be overwritten
          tc::fence_after_sync();
          const uint32_t idesc = tc::idesc_bf16(kPairs, nk16, 0, 0);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            tc::mma_bf16_ss(tbase + SM::cS, tc::smem_desc_sw128(qa + (ks / 4) * kPairs * 128 + (ks % 4) * 32, 16, 1024),
                            tc::smem_desc_sw128(ka + (ks / 4) * kKeys * 128 + (ks % 4) * 32, 16, 1024), idesc, ks > 0);
          tc::mma_commit(&bars.s_done);
          tc::mma_commit(&bars.q_empty);                     // ... and the Q buffer refilled, once these products are done
          wait(&bars.p_ready, ph);                           // P is in tensor memory
          if (nproc > 0) wait(&bars.o_free, ph ^ 1);         // the previous output has been read out
          tc::fence_after_sync();
          const uint32_t idesc2 = tc::idesc_bf16(kPairs, D, 0, 1);
          for (int ks = 0; ks < nk16 / 16; ++ks)
            mma_bf16_ts(tbase + SM::cO, tbase + SM::cS + 8 * ks, tc::smem_desc_sw128(va + ks * 16 * 128, kKeys * 128, 1024), idesc2, ks > 0);
          tc::mma_commit(&bars.o_done);
        }
        __syncwarp();
        ++nproc;
      }
      if (lane == 0 && nproc > 0) {                          // all products done before the tiles are replaced or the CTA ends
        wait(&bars.o_done, (nproc - 1) & 1);
        tc::fence_after_sync();
      }
    } else if (warp >= kGather0 / 32) {
      // ================= gather of the Q rows =================
      const int g = tid - kGather0, ck = g % CPR;
      constexpr int RPP = kGather / CPR;                   // rows per pass
      unsigned char* qd = sm + SM::q + (ck >> 3) * kPairs * 128;
      constexpr int RPT = kPairs / kGather;                // rows whose token this thread looks up
      auto tile_pids = [&](int t, int (&a)[RPT], int& last) {       // ids of rows g, g + kGather, ..., and of the tile's last row
        const int t0 = g0 + t * kPairs, nq = min(kPairs, g1 - t0);
#pragma unroll
        for (int u = 0; u < RPT; ++u) a[u] = (t < ntiles && g + u * kGather < nq) ? __ldg(pr + t0 + g + u * kGather) : -1;
        last = t < ntiles ? __ldg(pr + t0 + nq - 1) : 0;
      };
      int pa[RPT], last;
      tile_pids(tile, pa, last);
      for (; tile < ntiles; tile += nsub) {
        int pa_n[RPT], last_n;
        tile_pids(tile + nsub, pa_n, last_n);
        const int nk = visible(last, kc);
        if (nk > 0) {
          if (nproc > 0) wait(&bars.q_empty, (nproc - 1) & 1);   // the previous tile's first product has read the buffer
#pragma unroll
          for (int u = 0; u < RPT; ++u) tok_s[g + u * kGather] = pa[u] >= 0 ? pa[u] / mk : -1;
          tc::named_bar_sync(1, kGather);
#pragma unroll 4
          for (int r = g / CPR; r < kPairs; r += RPP) {
            const int tok = tok_s[r];
            if (!MUSE_IN_RANGE(tok + 1, dm.N + 1) || !MUSE_IN_RANGE((ck >> 3) * kPairs * 128 + tc::sw128_off(r, ck & 7), kPairs * D * 2 - 15)) continue;
            cp_async16(qd + tc::sw128_off(r, ck & 7), Qb + (size_t)max(tok, 0) * D + ck * 8, tok >= 0);
          }
          asm volatile("cp.async.commit_group;" ::: "memory");
          asm volatile("cp.async.wait_group 0;" ::: "memory");
          tc::fence_async_smem();                            // the tensor cores read the rows through the async proxy
          tc::mbar_arrive(&bars.q_full);
          tc::named_bar_sync(1, kGather);                    // tok_s may be rewritten
          ++nproc;
        }
#pragma unroll
        for (int u = 0; u < RPT; ++u) pa[u] = pa_n[u];
        last = last_n;
      }
    }
  }
#ifdef MUSE_PHASE_CLOCKS
  if (tid == 0 && pc[9] >= 6 && atomicCAS(status + 40, 0, 1) == 0) {
    for (int k = 0; k < 10; ++k) status[41 + k] = (int)pc[k];
    status[51] = (int)(clock64() - t_in_); status[52] = ntiles; status[53] = nsub; status[54] = kall; status[55] = g1 - g0;
  }
#endif
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tbase, SM::cols);
  if (!ok_ && lane == 0) report_status(status, MUSE_STATUS_FWD_TIMEOUT);
}

int ret_fwd_pairs_tc(const Dims& d, const void* Q, const void* Kp, const void* Vp, const int32_t* off_k, const int32_t* goff,
                     const int32_t* pairs, void* o_part, float* l_part, int* status, cudaStream_t st) {
  const dim3 grid(d.k2 > 0 ? d.Ck * d.SB : d.Ck, rf::kSplit, d.B * d.Hq);     // one CTA (or a few) per key cluster, or per bucket
  prof_mark("k_ret_fwd_pairs_tc", st);
  if (d.D == 128) {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_ret_fwd_pairs_tc<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, rf::Smem<128>::total));
    k_ret_fwd_pairs_tc<128><<<grid, rf::kThreads, rf::Smem<128>::total, st>>>(d, (const bf16*)Q, (const bf16*)Kp, (const bf16*)Vp, off_k, goff, pairs,
                                                                          (bf16*)o_part, l_part, status);
  } else {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_ret_fwd_pairs_tc<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, rf::Smem<64>::total));
    k_ret_fwd_pairs_tc<64><<<grid, rf::kThreads, rf::Smem<64>::total, st>>>(d, (const bf16*)Q, (const bf16*)Kp, (const bf16*)Vp, off_k, goff, pairs,
                                                                        (bf16*)o_part, l_part, status);
  }
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

}  // namespace muse
