// Spatial block selection inside the selected clusters (Section "Two-Level Retrieval", second level) and the
// near-field component of the merge (Section "Output merging", component 2).  For a query t of query
// cluster i in block b and each of its selected key clusters j, the earlier blocks b' < b of the cluster are
// scored with the PER-BLOCK (pre-accumulation) summaries of (i, j, b'):
//     logit(b') = sigma q . kappa_b' + beta_b',   beta_b' = mu_b' - sigma qbar_i . kappa_b'   (Eq. 6 at block level)
// the k2 best blocks (ties to the lower block) are retrieved exactly, every other non-empty earlier block of
// the cluster stands in through its summary: a virtual key with that logit and value nu_b'.  The kernel
// writes the chosen blocks and the softmax (o, lse) over the query's virtual keys.
// One warp per query; a lane owns D / 32 consecutive dims.  The warps of a CTA take consecutive queries of the
// (block, query cluster) ordering, i.e. of one segment as a rule: those read the same per-block summary rows
// whenever they selected the same clusters, so that most of the row traffic is served by the L1 / L2 caches.
#include "common.cuh"

namespace muse {

constexpr int kBsMaxBlocks = 32;     // S - 1 <= 32 block logits per (query, slot) are kept in registers of lane b'

template <class T, int D>
__global__ void __launch_bounds__(256)
k_block_select(Dims dm, const T* __restrict__ Q, const int32_t* __restrict__ assign_q, const int32_t* __restrict__ perm_q,
               const int32_t* __restrict__ sel, SummPtrs sp, const int32_t* __restrict__ bsel_in, int32_t* __restrict__ bsel_out,
               float* __restrict__ o_near, float* __restrict__ lse_near) {
  constexpr int EPL = D / 32;
  const int pq = blockIdx.y, lane = threadIdx.x & 31;
  const int pos = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (pos >= dm.N) return;
  const int t = perm_q[(size_t)pq * dm.N + pos];          // position in (block, query cluster) order -> query
  if (!MUSE_IN_RANGE(t, dm.N)) return;
  const size_t row = (size_t)pq * dm.N + t;
  const int b = t / dm.Bs, m = dm.m, k2 = dm.k2;
  int32_t* bo = bsel_out + row * m * k2;
  if (b == 0) {                                          // nothing earlier: no block, no near field
    for (int e = lane; e < m * k2; e += 32) bo[e] = -1;
    if (lane == 0) lse_near[row] = -INFINITY;
    float z[EPL];
#pragma unroll
    for (int k = 0; k < EPL; ++k) z[k] = 0.f;
    stv<EPL>(o_near + row * D + lane * EPL, z);
    return;
  }
  const int i = min(max(assign_q[row], 0), dm.Cq - 1);
  float q[EPL];
  ldv<EPL>(Q + row * D + lane * EPL, q);
#pragma unroll
  for (int k = 0; k < EPL; ++k) q[k] *= dm.sigma;
  float mN = -INFINITY, sN = 0.f, acc[EPL];              // online softmax over the query's virtual keys
#pragma unroll
  for (int k = 0; k < EPL; ++k) acc[k] = 0.f;
  const int jl0 = lane < m ? sel[row * m + lane] : -1, jl1 = lane + 32 < m ? sel[row * m + lane + 32] : -1;   // m <= 64 selections
  for (int s = 0; s < m; ++s) {
    const int j = __shfl_sync(0xffffffffu, s < 32 ? jl0 : jl1, s & 31);
    if (j < 0 || j >= dm.Ck) {                           // (uniform over the warp)
      for (int e = lane; e < k2; e += 32) bo[s * k2 + e] = -1;
      continue;
    }
    // block logits: lane b' ends up holding logit(b').  Lane b' fetches beta_b'; the rows are fetched four blocks at a
    // time so that their loads (and the four warp sums) are in flight together.
    const size_t e0 = ((size_t)pq * dm.SB * dm.Cq + i) * dm.Ck + j, estep = (size_t)dm.Cq * dm.Ck;   // entry of block 0, stride per block
    if (!MUSE_IN_RANGE(e0 + (size_t)(b - 1) * estep, (size_t)gridDim.y * dm.SB * estep)) continue;
    const float be = lane < b ? sp.beta[e0 + lane * estep] : -INFINITY;
    const uint32_t live = __ballot_sync(0xffffffffu, be != -INFINITY);       // non-empty earlier blocks of the cluster
    float mine = -INFINITY;
    for (int bp0 = 0; bp0 < b; bp0 += 4) {
      float kh[4][EPL], kl[4][EPL], part[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const bool on = (live >> (bp0 + u)) & 1u;            // (uniform over the warp; bits from b up are clear)
        const size_t e = e0 + (size_t)(bp0 + u) * estep;
#pragma unroll
        for (int k = 0; k < EPL; ++k) kh[u][k] = kl[u][k] = 0.f;
        if (on) {
          ldv<EPL>((const T*)sp.khi + e * D + lane * EPL, kh[u]);
          if (sizeof(T) == 2) ldv<EPL>((const T*)sp.klo + e * D + lane * EPL, kl[u]);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        part[u] = 0.f;
#pragma unroll
        for (int k = 0; k < EPL; ++k) part[u] = fmaf(q[k], kh[u][k] + kl[u][k], part[u]);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
        for (int u = 0; u < 4; ++u) part[u] += __shfl_xor_sync(0xffffffffu, part[u], o);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (lane == bp0 + u && be != -INFINITY) mine = part[u] + be;
    }
    // the k2 best blocks: largest logit first, ties to the lower block; fewer candidates -> all of them
    uint32_t chosen = 0u;
    if (bsel_in != nullptr) {
      for (int e = 0; e < k2; ++e) {
        const int c = bsel_in[(row * m + s) * k2 + e];
        const bool take = c >= 0 && c < b && !((chosen >> c) & 1u);     // a block named twice is retrieved once
        if (take) chosen |= 1u << c;
        if (lane == 0) bo[s * k2 + e] = take ? c : -1;
      }
    } else {
      float v = mine;
      for (int e = 0; e < k2; ++e) {
        float bv = v; int bi = lane;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float ov = __shfl_xor_sync(0xffffffffu, bv, o); const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
          if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        const bool any = bv != -INFINITY;
        if (lane == 0) bo[s * k2 + e] = any ? bi : -1;
        if (any) { chosen |= 1u << bi; if (lane == bi) v = -INFINITY; }
      }
    }
    // near field: every other non-empty earlier block of the cluster is a virtual key (logit(b'), nu_b'); four rows in flight
    const uint32_t rest = live & ~chosen;
    for (int bp0 = 0; bp0 < b; bp0 += 4) {
      if (((rest >> bp0) & 15u) == 0u) continue;
      float nv[4][EPL];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if ((rest >> (bp0 + u)) & 1u) ldv<EPL>((const T*)sp.nu + (e0 + (size_t)(bp0 + u) * estep) * D + lane * EPL, nv[u]);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (!((rest >> (bp0 + u)) & 1u)) continue;                     // (uniform over the warp)
        const float lg = __shfl_sync(0xffffffffu, mine, bp0 + u);
        const float mn = fmaxf(mN, lg);
        const float sc = __expf(mN - mn), p = __expf(lg - mn);         // exp(-inf) = 0 on the first virtual key
        sN = sN * sc + p;
#pragma unroll
        for (int k = 0; k < EPL; ++k) acc[k] = fmaf(acc[k], sc, p * nv[u][k]);
        mN = mn;
      }
    }
  }
  const float inv = sN > 0.f ? 1.f / sN : 0.f;
#pragma unroll
  for (int k = 0; k < EPL; ++k) acc[k] *= inv;
  stv<EPL>(o_near + row * D + lane * EPL, acc);
  if (lane == 0) lse_near[row] = sN > 0.f ? mN + __logf(sN) : -INFINITY;
}

bool block_select_supported(const Dims& d) { return d.causal && d.S - 1 <= kBsMaxBlocks && d.k2 <= 8; }

int block_select(const Dims& d, int dtype, const void* Q, const int32_t* assign_q, const int32_t* perm_q, const int32_t* sel,
                 const SummPtrs& sp, const int32_t* bsel_in, int32_t* bsel_out, float* o_near, float* lse_near, cudaStream_t st) {
  const dim3 grid(cdiv(d.N, 8), d.B * d.Hq);
  prof_mark("k_block_select", st);
  typedef __nv_bfloat16 bf;
  if (dtype == MUSE_F32) {
    if (d.D == 64) k_block_select<float, 64><<<grid, 256, 0, st>>>(d, (const float*)Q, assign_q, perm_q, sel, sp, bsel_in, bsel_out, o_near, lse_near);
    else k_block_select<float, 128><<<grid, 256, 0, st>>>(d, (const float*)Q, assign_q, perm_q, sel, sp, bsel_in, bsel_out, o_near, lse_near);
  } else {
    if (d.D == 64) k_block_select<bf, 64><<<grid, 256, 0, st>>>(d, (const bf*)Q, assign_q, perm_q, sel, sp, bsel_in, bsel_out, o_near, lse_near);
    else k_block_select<bf, 128><<<grid, 256, 0, st>>>(d, (const bf*)Q, assign_q, perm_q, sel, sp, bsel_in, bsel_out, o_near, lse_near);
  }
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

}  // namespace muse
