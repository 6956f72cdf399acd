// Spatial block selection inside the selected clusters (Section "Two-Level Retrieval", second level) and the
// near-field component of the merge (Section "Output merging", component 2).  For a query t of query
// cluster i in block b and each of its selected key clusters j, the earlier blocks b' < b of the cluster are
// scored with the PER-BLOCK (pre-accumulation) summaries of (i, j, b'):
//     logit(b') = sigma q . kappa_b' + beta_b',   beta_b' = mu_b' - sigma qbar_i . kappa_b'   (Eq. 6 at block level)
// the k2 best blocks (ties to the lower block) are retrieved exactly, every other non-empty earlier block of
// the cluster stands in through its summary: a virtual key with that logit and value nu_b'.  The kernel
// writes the chosen blocks and the softmax (o, lse) over the query's virtual keys.
//
// Organisation: the summary rows a query needs depend only on (i, b, j), so the queries of one segment (block b,
// query cluster i) that selected the same cluster j need the same rows.  A CTA owns a segment and takes its queries
// 32 at a time (a warp owns four of them, their q in registers); it forms the set of clusters those queries selected
// and walks it in ascending j, staging the rows of (i, j, b' < b) in shared memory ONCE (asynchronous copies, the next
// cluster's rows in flight while the current one is used); each warp then serves its queries that selected j.  A
// query's virtual keys are accumulated by an online softmax in the owning warp's registers, in cluster order, so the
// result does not depend on scheduling.
#include <algorithm>
#include "common.cuh"

namespace muse {

constexpr int kBsMaxBlocks = 32;     // S - 1 <= 32 block logits per (query, slot) are kept in registers of lane b'
constexpr int kBsThreads = 256, kBsWarps = kBsThreads / 32, kBsQPW = 4, kBsChunk = kBsWarps * kBsQPW;   // 32 queries per pass

__device__ __forceinline__ void bs_cp_async16(void* smem_dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void bs_cp_async4(void* smem_dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(src) : "memory");
}

// per staged cluster: for each earlier block the rows kappa_hi | kappa_lo (bf16 mode only) | nu, then the betas
template <class T> __host__ __device__ constexpr int bs_rows() { return sizeof(T) == 2 ? 3 : 2; }
template <class T> __host__ __device__ inline size_t bs_stage_bytes(int SB, int D) {
  return (size_t)SB * bs_rows<T>() * D * sizeof(T) + (size_t)kBsMaxBlocks * sizeof(float);
}

template <class T, int D>
__global__ void __launch_bounds__(kBsThreads)
k_block_select(Dims dm, const T* __restrict__ Q, const int32_t* __restrict__ off_q, const int32_t* __restrict__ perm_q,
               const int32_t* __restrict__ sel, SummPtrs sp, const int32_t* __restrict__ bsel_in, int32_t* __restrict__ bsel_out,
               float* __restrict__ o_near, float* __restrict__ lse_near) {
  constexpr int EPL = D / 32, ROWS = bs_rows<T>();
  extern __shared__ __align__(16) unsigned char bs_smem[];
  const int m = dm.m, k2 = dm.k2, SB = dm.SB, Ck = dm.Ck;
  const size_t stage_bytes = bs_stage_bytes<T>(SB, D);
  unsigned char* stage0 = bs_smem;
  int* sel_s = reinterpret_cast<int*>(bs_smem + 2 * stage_bytes);   // [32][m + 1] the chunk's selections (-1 = none)
  uint32_t* bitmap = reinterpret_cast<uint32_t*>(sel_s + kBsChunk * (m + 1));   // clusters selected by the chunk, one bit each
  int* ulist = reinterpret_cast<int*>(bitmap + ((Ck + 31) >> 5));  // those clusters, ascending
  __shared__ int nU_s;
  const int seg = blockIdx.x, pq = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = seg / dm.Cq, i = seg % dm.Cq;                        // segments are (block, query cluster), block-major
  const int32_t* oq = off_q + (size_t)pq * (dm.S * dm.Cq + 1) + seg;
  const int p0 = oq[0], p1 = oq[1];
  const int32_t* pm = perm_q + (size_t)pq * dm.N;
  const size_t estep = (size_t)dm.Cq * Ck;                           // entries per block plane
  const size_t ebase = ((size_t)pq * SB * dm.Cq + i) * Ck;           // entry (block 0, i, cluster 0)
  const int nwords = (Ck + 31) >> 5;

  for (int c0 = p0; c0 < p1; c0 += kBsChunk) {
    const int nq = min(kBsChunk, p1 - c0);
    // ---- the chunk's queries, selections and the set of clusters they name
    int tq[kBsQPW];
    float q[kBsQPW][EPL];
#pragma unroll
    for (int k = 0; k < kBsQPW; ++k) {
      const int r = warp * kBsQPW + k;
      tq[k] = r < nq ? pm[c0 + r] : -1;
      if (tq[k] >= 0 && !MUSE_IN_RANGE(tq[k], dm.N)) tq[k] = -1;
#pragma unroll
      for (int e = 0; e < EPL; ++e) q[k][e] = 0.f;
      if (tq[k] >= 0) {
        ldv<EPL>(Q + ((size_t)pq * dm.N + tq[k]) * D + lane * EPL, q[k]);
#pragma unroll
        for (int e = 0; e < EPL; ++e) q[k][e] *= dm.sigma;
      }
    }
    for (int w = tid; w < nwords; w += kBsThreads) bitmap[w] = 0u;
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kBsQPW; ++k) {
      const int r = warp * kBsQPW + k;
      for (int s = lane; s < m; s += 32) {
        int j = -1;
        if (tq[k] >= 0 && b > 0) {
          j = sel[((size_t)pq * dm.N + tq[k]) * m + s];
          if (j < 0 || j >= Ck) j = -1;
        }
        sel_s[r * (m + 1) + s] = j;
        if (j >= 0) atomicOr(&bitmap[j >> 5], 1u << (j & 31));
      }
      if (tq[k] >= 0) {                                              // default: no block chosen (valid slots are overwritten below)
        int32_t* bo = bsel_out + ((size_t)pq * dm.N + tq[k]) * m * k2;
        for (int e = lane; e < m * k2; e += 32) bo[e] = -1;
      }
    }
    __syncthreads();
    if (warp == 0) {                                                 // ascending list of the named clusters
      int n = 0;
      for (int w0 = 0; w0 < nwords; w0 += 32) {
        const uint32_t bits = w0 + lane < nwords ? bitmap[w0 + lane] : 0u;
        const int cnt = __popc(bits);
        int pre = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, pre, o); if (lane >= o) pre += v; }
        int at = n + pre - cnt;
        for (uint32_t rest = bits; rest; rest &= rest - 1) ulist[at++] = (w0 + lane) * 32 + __ffs(rest) - 1;
        n += __shfl_sync(0xffffffffu, pre, 31);
      }
      if (lane == 0) nU_s = n;
    }
    __syncthreads();
    const int nU = nU_s;
    // ---- rows of cluster ulist[u] for the earlier blocks -> stage u & 1 (asynchronous; one commit group per cluster)
    auto stage_rows = [&](int u) {
      unsigned char* st = stage0 + (u & 1) * stage_bytes;
      const int j = ulist[u];
      constexpr int CPR = D * (int)sizeof(T) / 16;                   // 16-byte pieces per row
      for (int e = tid; e < b * ROWS * CPR; e += kBsThreads) {
        const int bp = e / (ROWS * CPR), rw = (e / CPR) % ROWS, c = e % CPR;
        const size_t ent = ebase + (size_t)bp * estep + j;
        const T* src = rw == 0 ? (const T*)sp.khi : (rw == ROWS - 1 ? (const T*)sp.nu : (const T*)sp.klo);
        bs_cp_async16(st + ((size_t)(bp * ROWS + rw) * D) * sizeof(T) + c * 16, reinterpret_cast<const unsigned char*>(src + ent * D) + c * 16);
      }
      if (tid < b) bs_cp_async4(st + (size_t)SB * ROWS * D * sizeof(T) + tid * 4, sp.beta + ebase + (size_t)tid * estep + j);
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    float mN[kBsQPW], sN[kBsQPW], acc[kBsQPW][EPL];                  // online softmax over each query's virtual keys
#pragma unroll
    for (int k = 0; k < kBsQPW; ++k) {
      mN[k] = -INFINITY; sN[k] = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[k][e] = 0.f;
    }
    if (nU > 0) stage_rows(0);
    for (int u = 0; u < nU; ++u) {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      __syncthreads();                                               // cluster u's rows are in place; everyone is done with cluster u - 1
      if (u + 1 < nU) stage_rows(u + 1);
      const unsigned char* st = stage0 + (u & 1) * stage_bytes;
      const T* rows = reinterpret_cast<const T*>(st);
      const float* betas = reinterpret_cast<const float*>(st + (size_t)SB * ROWS * D * sizeof(T));
      const int j = ulist[u];
      const float be = lane < b ? betas[lane] : -INFINITY;
      const uint32_t live = __ballot_sync(0xffffffffu, be != -INFINITY);     // non-empty earlier blocks of the cluster
#pragma unroll
      for (int k = 0; k < kBsQPW; ++k) {
        if (tq[k] < 0) continue;                                     // (warp-uniform)
        const int r = warp * kBsQPW + k;
        // the slots of this query that name cluster j (one, unless a forced selection repeats a cluster)
        unsigned long long hit = (unsigned long long)__ballot_sync(0xffffffffu, lane < m && sel_s[r * (m + 1) + min(lane, m - 1)] == j);
        if (m > 32) hit |= (unsigned long long)__ballot_sync(0xffffffffu, lane + 32 < m && sel_s[r * (m + 1) + min(lane + 32, m - 1)] == j) << 32;
        for (; hit != 0ull; hit &= hit - 1ull) {
          const int s = __ffsll((long long)hit) - 1;
          const size_t row = (size_t)pq * dm.N + tq[k];
          // block logits: lane b' ends up holding logit(b'); four blocks at a time
          float mine = -INFINITY;
          for (int bp0 = 0; bp0 < b; bp0 += 4) {
            float part[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
              part[x] = 0.f;
              if ((live >> (bp0 + x)) & 1u) {                        // (uniform over the warp; bits from b up are clear)
                float kh[EPL], kl[EPL];
                ldv<EPL>(rows + (size_t)((bp0 + x) * ROWS) * D + lane * EPL, kh);
                if (ROWS == 3) ldv<EPL>(rows + (size_t)((bp0 + x) * ROWS + 1) * D + lane * EPL, kl);
                else {
#pragma unroll
                  for (int e = 0; e < EPL; ++e) kl[e] = 0.f;
                }
#pragma unroll
                for (int e = 0; e < EPL; ++e) part[x] = fmaf(q[k][e], kh[e] + kl[e], part[x]);
              }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
              for (int x = 0; x < 4; ++x) part[x] += __shfl_xor_sync(0xffffffffu, part[x], o);
            }
#pragma unroll
            for (int x = 0; x < 4; ++x)
              if (lane == bp0 + x && be != -INFINITY) mine = part[x] + be;
          }
          // the k2 best blocks: largest logit first, ties to the lower block; fewer candidates -> all of them
          int32_t* bo = bsel_out + (row * m + s) * k2;
          uint32_t chosen = 0u;
          if (bsel_in != nullptr) {
            for (int e = 0; e < k2; ++e) {
              const int c = bsel_in[(row * m + s) * k2 + e];
              const bool take = c >= 0 && c < b && !((chosen >> c) & 1u);     // a block named twice is retrieved once
              if (take) chosen |= 1u << c;
              if (lane == 0) bo[e] = take ? c : -1;
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
              if (lane == 0) bo[e] = any ? bi : -1;
              if (any) { chosen |= 1u << bi; if (lane == bi) v = -INFINITY; }
            }
          }
          // near field: every other non-empty earlier block of the cluster is a virtual key (logit(b'), nu_b')
          for (uint32_t rest = live & ~chosen; rest != 0u; rest &= rest - 1u) {
            const int bp = __ffs(rest) - 1;
            const float lg = __shfl_sync(0xffffffffu, mine, bp);
            float nv[EPL];
            ldv<EPL>(rows + (size_t)(bp * ROWS + ROWS - 1) * D + lane * EPL, nv);
            const float mn = fmaxf(mN[k], lg);
            const float sc = __expf(mN[k] - mn), p = __expf(lg - mn);         // exp(-inf) = 0 on the first virtual key
            sN[k] = sN[k] * sc + p;
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[k][e] = fmaf(acc[k][e], sc, p * nv[e]);
            mN[k] = mn;
          }
        }
      }
    }
    // ---- the chunk's near-field results
#pragma unroll
    for (int k = 0; k < kBsQPW; ++k) {
      if (tq[k] < 0) continue;
      const size_t row = (size_t)pq * dm.N + tq[k];
      const float inv = sN[k] > 0.f ? 1.f / sN[k] : 0.f;
      float o[EPL];
#pragma unroll
      for (int e = 0; e < EPL; ++e) o[e] = acc[k][e] * inv;
      stv<EPL>(o_near + row * D + lane * EPL, o);
      if (lane == 0) lse_near[row] = sN[k] > 0.f ? mN[k] + __logf(sN[k]) : -INFINITY;
    }
    __syncthreads();                                                 // sel_s, bitmap and the stages are reused by the next chunk
  }
}

bool block_select_supported(const Dims& d) { return d.causal && d.S - 1 <= kBsMaxBlocks && d.k2 <= 8; }

template <class T, int D>
static int block_select_t(const Dims& d, const T* Q, const int32_t* off_q, const int32_t* perm_q, const int32_t* sel, const SummPtrs& sp,
                          const int32_t* bsel_in, int32_t* bsel_out, float* o_near, float* lse_near, cudaStream_t st) {
  const size_t smem = 2 * bs_stage_bytes<T>(d.SB, D) + (size_t)kBsChunk * (d.m + 1) * sizeof(int) + (size_t)((d.Ck + 31) >> 5) * sizeof(uint32_t) +
                      (size_t)std::min(d.Ck, kBsChunk * d.m) * sizeof(int);
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_block_select<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  prof_mark("k_block_select", st);
  k_block_select<T, D><<<dim3(d.S * d.Cq, d.B * d.Hq), kBsThreads, smem, st>>>(d, Q, off_q, perm_q, sel, sp, bsel_in, bsel_out, o_near, lse_near);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

int block_select(const Dims& d, int dtype, const void* Q, const int32_t* off_q, const int32_t* perm_q, const int32_t* sel,
                 const SummPtrs& sp, const int32_t* bsel_in, int32_t* bsel_out, float* o_near, float* lse_near, cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  if (dtype == MUSE_F32) {
    if (d.D == 64) return block_select_t<float, 64>(d, (const float*)Q, off_q, perm_q, sel, sp, bsel_in, bsel_out, o_near, lse_near, st);
    return block_select_t<float, 128>(d, (const float*)Q, off_q, perm_q, sel, sp, bsel_in, bsel_out, o_near, lse_near, st);
  }
  if (d.D == 64) return block_select_t<bf, 64>(d, (const bf*)Q, off_q, perm_q, sel, sp, bsel_in, bsel_out, o_near, lse_near, st);
  return block_select_t<bf, 128>(d, (const bf*)Q, off_q, perm_q, sel, sp, bsel_in, bsel_out, o_near, lse_near, st);
}

}  // namespace muse
