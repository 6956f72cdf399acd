// Backward of the near field of the two-level retrieval (Section "Two-Level Retrieval", second level; Section
// "Output merging", component 2; gradients with the chosen clusters and blocks held constant, Appendix "Centroid
// Gradient Flow").  A stand-in key (i, j, b') - the per-block summary of a non-retrieved earlier block b' of a
// selected cluster j, seen by a query t of query cluster i - has
//     logit = sigma q . kappa + beta,  beta = mu - sigma qbar_i . kappa,   value nu            (kappa, mu, nu of (i, j, b'))
// With L the merged log-sum-exp and delta = dO . O of the query:
//     p = exp(logit - L),  g = p (dO . nu - delta),
//     dq += g sigma kappa,   d nu += p dO,   d kappa += g sigma (q - qbar_i),   d mu += g.
// The sums over queries of d nu, d kappa and of the scalar dS = d mu - d kappa . kappa - d nu . nu (the form in which
// the key-side pass takes the log-mass gradient) are the gradients of the per-block summaries, which that pass then
// carries to the keys and values of bucket (j, b').
//
// Organisation: entries (i, j, b') receive contributions from the queries of cluster i in every later block, so one
// CTA owns a query cluster i of one head and walks its segments (block b, i) in turn: it is the only writer of the
// gradient entries of i, which it updates with plain read-modify-writes.  Within a segment it works like the block
// selection kernel of the forward pass: 32 queries at a time (a warp owns four), the clusters they selected in
// ascending order, each cluster's per-block rows staged once in shared memory; the warps add their queries'
// contributions for the staged cluster into shared-memory accumulators, which are flushed before the next cluster.
#include <algorithm>
#include "common.cuh"

namespace muse {

constexpr int kNbMaxBlocks = 32;
constexpr int kNbThreads = 256, kNbWarps = kNbThreads / 32, kNbQPW = 4, kNbChunk = kNbWarps * kNbQPW;

__device__ __forceinline__ void nb_cp_async16(void* smem_dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void nb_cp_async4(void* smem_dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(src) : "memory");
}
template <class T> __host__ __device__ constexpr int nb_rows() { return sizeof(T) == 2 ? 3 : 2; }   // kappa_hi | kappa_lo (bf16) | nu
template <class T> __host__ __device__ inline size_t nb_stage_bytes(int SB, int D) {
  return (size_t)SB * nb_rows<T>() * D * sizeof(T) + (size_t)kNbMaxBlocks * sizeof(float);
}

template <class T, int D>
__global__ void __launch_bounds__(kNbThreads)
k_near_bwd(Dims dm, const T* __restrict__ Q, const T* __restrict__ dO, const float* __restrict__ qbar, const float* __restrict__ LSE,
           const float* __restrict__ delta, const int32_t* __restrict__ off_q, const int32_t* __restrict__ perm_q,
           const int32_t* __restrict__ sel, const int32_t* __restrict__ bsel, SummPtrs sp, float* __restrict__ dQacc,
           float* __restrict__ dkappa_b, float* __restrict__ dnu_b, float* __restrict__ dS_b, int grad_ji) {
  // grad_ji: the gradient entries are laid out [plane][j][i] (what the tensor-core key-side kernel reads) instead of [plane][i][j]
  constexpr int EPL = D / 32, ROWS = nb_rows<T>();
  extern __shared__ __align__(16) unsigned char nb_smem[];
  const int m = dm.m, k2 = dm.k2, SB = dm.SB, Ck = dm.Ck;
  const size_t stage_bytes = nb_stage_bytes<T>(SB, D);
  unsigned char* stage0 = nb_smem;
  float* gka = reinterpret_cast<float*>(nb_smem + 2 * stage_bytes);   // [SB][D] sum over queries of g sigma (q - qbar_i), staged cluster
  float* gnu = gka + (size_t)SB * D;                                   // [SB][D] sum of p dO
  float* gmu = gnu + (size_t)SB * D;                                   // [SB]    sum of g (1 - sigma (q - qbar_i) . kappa) - p dO . nu
  int* sel_s = reinterpret_cast<int*>(gmu + kNbMaxBlocks);             // [32][m + 1]
  uint32_t* bitmap = reinterpret_cast<uint32_t*>(sel_s + kNbChunk * (m + 1));
  int* ulist = reinterpret_cast<int*>(bitmap + ((Ck + 31) >> 5));
  __shared__ int nU_s, touched_s;
  const int i = blockIdx.x, pq = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int32_t* pm = perm_q + (size_t)pq * dm.N;
  const size_t estep = (size_t)dm.Cq * Ck;
  const size_t ebase = ((size_t)pq * SB * dm.Cq + i) * Ck;             // entry (block 0, i, cluster 0)
  const int nwords = (Ck + 31) >> 5;
  float qb[EPL];                                                       // sigma qbar_i, this lane's dims
  ldv<EPL>(qbar + ((size_t)pq * dm.Cq + i) * D + lane * EPL, qb);
#pragma unroll
  for (int e = 0; e < EPL; ++e) qb[e] *= dm.sigma;
  for (int e = tid; e < SB * D; e += kNbThreads) { gka[e] = 0.f; gnu[e] = 0.f; }
  if (tid < kNbMaxBlocks) gmu[tid] = 0.f;
  if (tid == 0) touched_s = 0;
  __syncthreads();

  for (int b = 1; b < dm.S; ++b) {
    const int32_t* oq = off_q + (size_t)pq * (dm.S * dm.Cq + 1) + (size_t)b * dm.Cq + i;
    const int p0 = oq[0], p1 = oq[1];
    for (int c0 = p0; c0 < p1; c0 += kNbChunk) {
      const int nq = min(kNbChunk, p1 - c0);
      int tq[kNbQPW];
      float q[kNbQPW][EPL], go[kNbQPW][EPL], dqa[kNbQPW][EPL], Lq[kNbQPW], dl[kNbQPW];
#pragma unroll
      for (int k = 0; k < kNbQPW; ++k) {
        const int r = warp * kNbQPW + k;
        tq[k] = r < nq ? pm[c0 + r] : -1;
        if (tq[k] >= 0 && !MUSE_IN_RANGE(tq[k], dm.N)) tq[k] = -1;
        Lq[k] = 0.f; dl[k] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) { q[k][e] = 0.f; go[k][e] = 0.f; dqa[k][e] = 0.f; }
        if (tq[k] >= 0) {
          const size_t row = (size_t)pq * dm.N + tq[k];
          ldv<EPL>(Q + row * D + lane * EPL, q[k]);
          ldv<EPL>(dO + row * D + lane * EPL, go[k]);
#pragma unroll
          for (int e = 0; e < EPL; ++e) q[k][e] *= dm.sigma;
          Lq[k] = LSE[row]; dl[k] = delta[row];
        }
      }
      for (int w = tid; w < nwords; w += kNbThreads) bitmap[w] = 0u;
      __syncthreads();
#pragma unroll
      for (int k = 0; k < kNbQPW; ++k) {
        const int r = warp * kNbQPW + k;
        for (int s = lane; s < m; s += 32) {
          int j = -1;
          if (tq[k] >= 0) {
            j = sel[((size_t)pq * dm.N + tq[k]) * m + s];
            if (j < 0 || j >= Ck) j = -1;
          }
          sel_s[r * (m + 1) + s] = j;
          if (j >= 0) atomicOr(&bitmap[j >> 5], 1u << (j & 31));
        }
      }
      __syncthreads();
      if (warp == 0) {
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
      auto stage_rows = [&](int u) {
        unsigned char* st = stage0 + (u & 1) * stage_bytes;
        const int j = ulist[u];
        constexpr int CPR = D * (int)sizeof(T) / 16;
        for (int e = tid; e < b * ROWS * CPR; e += kNbThreads) {
          const int bp = e / (ROWS * CPR), rw = (e / CPR) % ROWS, c = e % CPR;
          const size_t ent = ebase + (size_t)bp * estep + j;
          const T* src = rw == 0 ? (const T*)sp.khi : (rw == ROWS - 1 ? (const T*)sp.nu : (const T*)sp.klo);
          nb_cp_async16(st + ((size_t)(bp * ROWS + rw) * D) * sizeof(T) + c * 16, reinterpret_cast<const unsigned char*>(src + ent * D) + c * 16);
        }
        if (tid < b) nb_cp_async4(st + (size_t)SB * ROWS * D * sizeof(T) + tid * 4, sp.beta + ebase + (size_t)tid * estep + j);
        asm volatile("cp.async.commit_group;" ::: "memory");
      };
      if (nU > 0) stage_rows(0);
      for (int u = 0; u < nU; ++u) {
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();                                               // cluster u's rows are in place; the accumulators are clear
        if (u + 1 < nU) stage_rows(u + 1);
        const unsigned char* st = stage0 + (u & 1) * stage_bytes;
        const T* rows = reinterpret_cast<const T*>(st);
        const float* betas = reinterpret_cast<const float*>(st + (size_t)SB * ROWS * D * sizeof(T));
        const int j = ulist[u];
        const float be = lane < b ? betas[lane] : -INFINITY;
        const uint32_t live = __ballot_sync(0xffffffffu, be != -INFINITY);
#pragma unroll
        for (int k = 0; k < kNbQPW; ++k) {
          if (tq[k] < 0) continue;                                     // (warp-uniform)
          const int r = warp * kNbQPW + k;
          unsigned long long hit = (unsigned long long)__ballot_sync(0xffffffffu, lane < m && sel_s[r * (m + 1) + min(lane, m - 1)] == j);
          if (m > 32) hit |= (unsigned long long)__ballot_sync(0xffffffffu, lane + 32 < m && sel_s[r * (m + 1) + min(lane + 32, m - 1)] == j) << 32;
          for (; hit != 0ull; hit &= hit - 1ull) {
            const int s = __ffsll((long long)hit) - 1;
            const size_t row = (size_t)pq * dm.N + tq[k];
            // the blocks this (query, slot) retrieved exactly are not stand-in keys
            uint32_t chosen = 0u;
            for (int e = 0; e < k2; ++e) {
              const int c = bsel[(row * m + s) * k2 + e];
              if (c >= 0 && c < b) chosen |= 1u << c;
            }
            for (uint32_t rest = live & ~chosen; rest != 0u; rest &= rest - 1u) {
              const int bp = __ffs(rest) - 1;
              float kh[EPL], kl[EPL], nv[EPL];
              ldv<EPL>(rows + (size_t)(bp * ROWS) * D + lane * EPL, kh);
              if (ROWS == 3) ldv<EPL>(rows + (size_t)(bp * ROWS + 1) * D + lane * EPL, kl);
              else {
#pragma unroll
                for (int e = 0; e < EPL; ++e) kl[e] = 0.f;
              }
              ldv<EPL>(rows + (size_t)(bp * ROWS + ROWS - 1) * D + lane * EPL, nv);
              float s1 = 0.f, s2 = 0.f, s3 = 0.f;                      // sigma q . kappa,  dO . nu,  sigma qbar_i . kappa
#pragma unroll
              for (int e = 0; e < EPL; ++e) {
                kh[e] += kl[e];
                s1 = fmaf(q[k][e], kh[e], s1); s2 = fmaf(go[k][e], nv[e], s2); s3 = fmaf(qb[e], kh[e], s3);
              }
#pragma unroll
              for (int o = 16; o > 0; o >>= 1) {
                s1 += __shfl_xor_sync(0xffffffffu, s1, o); s2 += __shfl_xor_sync(0xffffffffu, s2, o); s3 += __shfl_xor_sync(0xffffffffu, s3, o);
              }
              const float p = __expf(s1 + __shfl_sync(0xffffffffu, be, bp) - Lq[k]);
              const float g = p * (s2 - dl[k]);
#pragma unroll
              for (int e = 0; e < EPL; ++e) {
                dqa[k][e] = fmaf(g, kh[e], dqa[k][e]);
                atomicAdd(&gka[bp * D + lane * EPL + e], g * (q[k][e] - qb[e]));
                atomicAdd(&gnu[bp * D + lane * EPL + e], p * go[k][e]);
              }
              // the scalar the key-side pass wants per entry: d mu - d kappa . kappa - d nu . nu  (this query's share)
              if (lane == 0) { atomicAdd(&gmu[bp], g * (1.f - (s1 - s3)) - p * s2); touched_s = 1; }
            }
          }
        }
        __syncthreads();                                               // every warp has added its queries' share for cluster j
        if (touched_s) {                                               // (block-uniform) flush into the gradient entries (b', i, j), which this CTA owns
          for (int e = tid; e < b * D; e += kNbThreads) {
            const int bp = e / D, d0 = e % D;
            const size_t ent = grad_ji ? (((size_t)pq * SB + bp) * Ck + j) * dm.Cq + i : ebase + (size_t)bp * estep + j;
            const float a = gka[e], c = gnu[e];
            if (a != 0.f) dkappa_b[ent * D + d0] += a;
            if (c != 0.f) dnu_b[ent * D + d0] += c;
            gka[e] = 0.f; gnu[e] = 0.f;
          }
          if (tid < b) {
            const float a = gmu[tid];
            if (a != 0.f) dS_b[grad_ji ? (((size_t)pq * SB + tid) * Ck + j) * dm.Cq + i : ebase + (size_t)tid * estep + j] += a;
            gmu[tid] = 0.f;
          }
        }
        __syncthreads();
        if (tid == 0) touched_s = 0;
      }
      // the chunk's contribution to dQ (the far-field and local parts are already in the accumulator)
#pragma unroll
      for (int k = 0; k < kNbQPW; ++k) {
        if (tq[k] < 0) continue;
        float* dst = dQacc + ((size_t)pq * dm.N + tq[k]) * D + lane * EPL;
        float cur[EPL];
        ldv<EPL>(dst, cur);
#pragma unroll
        for (int e = 0; e < EPL; ++e) cur[e] = fmaf(dm.sigma, dqa[k][e], cur[e]);
        stv<EPL>(dst, cur);
      }
      __syncthreads();
    }
  }
}

// fp32 gradient rows -> bf16 (the operand type of the tensor-core key-side kernel), same layout
__global__ void k_grad_to_bf16(const float* __restrict__ in, long long n4, __nv_bfloat16* __restrict__ out) {
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= n4) return;
  st4(out + 4 * e, ld4(in + 4 * e));
}

int grad_to_bf16(const float* in, size_t n, void* out, cudaStream_t st) {
  const long long n4 = (long long)(n / 4);
  prof_mark("k_grad_to_bf16", st);
  k_grad_to_bf16<<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(in, n4, (__nv_bfloat16*)out);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

size_t near_bwd_smem_bytes(const Dims& d, int elem_bytes) {
  const size_t stage = (size_t)d.SB * (elem_bytes == 2 ? 3 : 2) * d.D * elem_bytes + (size_t)kNbMaxBlocks * sizeof(float);
  return 2 * stage + (size_t)(2 * d.SB * d.D + kNbMaxBlocks) * sizeof(float) + (size_t)kNbChunk * (d.m + 1) * sizeof(int) +
         (size_t)((d.Ck + 31) >> 5) * sizeof(uint32_t) + (size_t)std::min(d.Ck, kNbChunk * d.m) * sizeof(int);
}

template <class T, int D>
static int near_bwd_t(const Dims& d, const T* Q, const T* dO, const float* qbar, const float* LSE, const float* delta,
                      const int32_t* off_q, const int32_t* perm_q, const int32_t* sel, const int32_t* bsel, const SummPtrs& sp,
                      float* dQacc, float* dkappa_b, float* dnu_b, float* dS_b, int grad_ji, cudaStream_t st) {
  const size_t smem = near_bwd_smem_bytes(d, (int)sizeof(T));
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_near_bwd<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  prof_mark("k_near_bwd", st);
  k_near_bwd<T, D><<<dim3(d.Cq, d.B * d.Hq), kNbThreads, smem, st>>>(d, Q, dO, qbar, LSE, delta, off_q, perm_q, sel, bsel, sp, dQacc,
                                                                   dkappa_b, dnu_b, dS_b, grad_ji);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

int near_bwd(const Dims& d, int dtype, const void* Q, const void* dO, const float* qbar, const float* LSE, const float* delta,
             const int32_t* off_q, const int32_t* perm_q, const int32_t* sel, const int32_t* bsel, const SummPtrs& sp, float* dQacc,
             float* dkappa_b, float* dnu_b, float* dS_b, int grad_ji, cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  if (dtype == MUSE_F32) {
    if (d.D == 64) return near_bwd_t<float, 64>(d, (const float*)Q, (const float*)dO, qbar, LSE, delta, off_q, perm_q, sel, bsel, sp, dQacc, dkappa_b, dnu_b, dS_b, grad_ji, st);
    return near_bwd_t<float, 128>(d, (const float*)Q, (const float*)dO, qbar, LSE, delta, off_q, perm_q, sel, bsel, sp, dQacc, dkappa_b, dnu_b, dS_b, grad_ji, st);
  }
  if (d.D == 64) return near_bwd_t<bf, 64>(d, (const bf*)Q, (const bf*)dO, qbar, LSE, delta, off_q, perm_q, sel, bsel, sp, dQacc, dkappa_b, dnu_b, dS_b, grad_ji, st);
  return near_bwd_t<bf, 128>(d, (const bf*)Q, (const bf*)dO, qbar, LSE, delta, off_q, perm_q, sel, bsel, sp, dQacc, dkappa_b, dnu_b, dS_b, grad_ji, st);
}

}  // namespace muse
