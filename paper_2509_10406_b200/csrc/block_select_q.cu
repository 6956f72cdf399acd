// Spatial block selection and near field of the two-level retrieval (Section "Two-Level Retrieval", second level;
// Section "Output merging", component 2), the kernel for bf16 mode with at most 8 earlier blocks (S <= 9); the
// definitions are those at the head of block_select.cu, which serves the other shapes.
//
// A dot product of a query with a summary row costs a warp ~40 instructions when the lanes share the D dimensions
// (shuffle reduction per product).  Here a LANE owns a QUERY instead: the 32 queries of a chunk of one segment
// (block b, query cluster i) sit in shared memory as padded fp32 rows, a warp takes one of the clusters the chunk
// selected, converts that cluster's per-block rows kappa_hi + kappa_lo to fp32 once (lanes sharing D), and then every
// lane whose query selected the cluster runs down D with 16-byte loads: its own q row (conflict-free thanks to the
// padding) against the broadcast kappa rows, all earlier blocks at once.  The block logits of a (query, slot) end up in
// the registers of one lane, so the top-k2 choice is lane-local.  The near-field softmax needs a query's logits from all
// its clusters, which different warps handled: the logits go to shared memory, a second phase takes each query's maximum
// and weights, a third (a warp per query, lanes sharing D again) adds up the weighted nu rows.
#include <algorithm>
#include "common.cuh"

namespace muse {

typedef __nv_bfloat16 bf16;

constexpr int kBqThreads = 256, kBqWarps = kBqThreads / 32, kBqChunk = 32, kBqMaxSB = 8;

size_t block_select_q_smem(const Dims& d) {
  const int LDQ = d.D + 4;
  return (size_t)kBqChunk * LDQ * 4 + (size_t)kBqWarps * d.SB * d.D * 4 + (size_t)d.m * d.SB * kBqChunk * 4 + (size_t)2 * kBqWarps * kBqChunk * 4 +
         (size_t)kBqChunk * (d.m + 1) * 4 + (size_t)((d.Ck + 31) >> 5) * 4 + (size_t)std::min(d.Ck, kBqChunk * d.m) * 4;
}

bool block_select_q_supported(const Dims& d, int dtype) {
  return dtype == MUSE_BF16 && d.causal && d.SB <= kBqMaxSB && d.k2 <= 8 && block_select_q_smem(d) <= 200 * 1024;
}

template <int D>
__global__ void __launch_bounds__(kBqThreads)
k_block_select_q(Dims dm, const bf16* __restrict__ Q, const int32_t* __restrict__ off_q, const int32_t* __restrict__ perm_q,
                 const int32_t* __restrict__ sel, SummPtrs sp, const int32_t* __restrict__ bsel_in, int32_t* __restrict__ bsel_out,
                 float* __restrict__ o_near, float* __restrict__ lse_near, int* __restrict__ status) {
  constexpr int EPL = D / 32, LDQ = D + 4;
#ifdef MUSE_PHASE_CLOCKS
  long long pc[4] = {0, 0, 0, 0}, z_ = clock64();
#define BQCLK(k) { long long n_ = clock64(); pc[k] += n_ - z_; z_ = n_; }
#else
#define BQCLK(k)
#endif
  extern __shared__ __align__(16) unsigned char bq_smem[];
  const int m = dm.m, k2 = dm.k2, SB = dm.SB, Ck = dm.Ck;
  float* q_s = reinterpret_cast<float*>(bq_smem);                    // [32][LDQ] sigma q of the chunk's queries
  float* kf = q_s + kBqChunk * LDQ;                                  // [warp][SB][D] kappa rows of the cluster a warp has in hand
  float* lgs = kf + (size_t)kBqWarps * SB * D;                       // [m][SB][32] stand-in logits per (slot, block, query); later weights
  float* red = lgs + (size_t)m * SB * kBqChunk;                      // [2][8][32] partial maxima / sums
  int* sel_s = reinterpret_cast<int*>(red + 2 * kBqWarps * kBqChunk);   // [32][m + 1]
  uint32_t* bitmap = reinterpret_cast<uint32_t*>(sel_s + kBqChunk * (m + 1));
  int* ulist = reinterpret_cast<int*>(bitmap + ((Ck + 31) >> 5));
  __shared__ int nU_s;
  const int seg = blockIdx.x, pq = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = seg / dm.Cq, i = seg % dm.Cq;
  const int32_t* oq = off_q + (size_t)pq * (dm.S * dm.Cq + 1) + seg;
  const int p0 = oq[0], p1 = oq[1];
  const int32_t* pm = perm_q + (size_t)pq * dm.N;
  const size_t estep = (size_t)dm.Cq * Ck;
  const size_t ebase = ((size_t)pq * SB * dm.Cq + i) * Ck;
  const int nwords = (Ck + 31) >> 5;
  float* kw = kf + (size_t)warp * SB * D;

  for (int c0 = p0; c0 < p1; c0 += kBqChunk) {
    const int nq = min(kBqChunk, p1 - c0);
    // ---- phase 0: the chunk's queries (rows of q_s), selections, set of selected clusters, defaults
    int tq4[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int r = warp * 4 + k;
      int t = r < nq ? pm[c0 + r] : -1;
      if (t >= 0 && !MUSE_IN_RANGE(t, dm.N)) t = -1;
      tq4[k] = t;
      float x[EPL];
#pragma unroll
      for (int e = 0; e < EPL; ++e) x[e] = 0.f;
      if (t >= 0) {
        ldv<EPL>(Q + ((size_t)pq * dm.N + t) * D + lane * EPL, x);
#pragma unroll
        for (int e = 0; e < EPL; ++e) x[e] *= dm.sigma;
      }
      stv<EPL>(q_s + r * LDQ + lane * EPL, x);
      for (int s = lane; s < m; s += 32) {
        int j = -1;
        if (t >= 0 && b > 0) {
          j = sel[((size_t)pq * dm.N + t) * m + s];
          if (j < 0 || j >= Ck) j = -1;
        }
        sel_s[r * (m + 1) + s] = j;
      }
      if (t >= 0) {
        int32_t* bo = bsel_out + ((size_t)pq * dm.N + t) * m * k2;
        for (int e = lane; e < m * k2; e += 32) bo[e] = -1;
      }
    }
    for (int w = tid; w < nwords; w += kBqThreads) bitmap[w] = 0u;
    for (int e = tid; e < m * SB * kBqChunk; e += kBqThreads) lgs[e] = -INFINITY;
    __syncthreads();
    for (int e = tid; e < kBqChunk * m; e += kBqThreads) {
      const int j = sel_s[(e / m) * (m + 1) + e % m];
      if (j >= 0) atomicOr(&bitmap[j >> 5], 1u << (j & 31));
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
    BQCLK(0)
    const int tq = lane < nq ? pm[c0 + lane] : -1;                   // lane = query from here on
    const size_t row = (size_t)pq * dm.N + max(tq, 0);

    // ---- phase 1: a warp per selected cluster; lane = query
    for (int u = warp; u < nU; u += kBqWarps) {
      const int j = ulist[u];
      __syncwarp();                                                  // the previous cluster's rows have been used
      for (int bp = 0; bp < b; ++bp) {                               // kappa_hi + kappa_lo -> fp32 rows in shared memory (lanes share D)
        const size_t ent = ebase + (size_t)bp * estep + j;
        float kh[EPL], kl[EPL];
        ldv<EPL>((const bf16*)sp.khi + ent * D + lane * EPL, kh);
        ldv<EPL>((const bf16*)sp.klo + ent * D + lane * EPL, kl);
#pragma unroll
        for (int e = 0; e < EPL; ++e) kh[e] += kl[e];
        stv<EPL>(kw + bp * D + lane * EPL, kh);
      }
      const float be = lane < b ? sp.beta[ebase + (size_t)lane * estep + j] : -INFINITY;
      const uint32_t live = __ballot_sync(0xffffffffu, be != -INFINITY);
      __syncwarp();
      int s_r = -1;                                                  // the slot in which this lane's query names cluster j
      if (tq >= 0)
        for (int s = 0; s < m; ++s)
          if (s_r < 0 && sel_s[lane * (m + 1) + s] == j) s_r = s;
      if (__ballot_sync(0xffffffffu, s_r >= 0) == 0u) continue;
      float lg[kBqMaxSB];
#pragma unroll
      for (int bp = 0; bp < kBqMaxSB; ++bp) lg[bp] = 0.f;
      const float* qr = q_s + lane * LDQ;
#pragma unroll 4
      for (int d4 = 0; d4 < D; d4 += 4) {
        const float4 x = *reinterpret_cast<const float4*>(qr + d4);
#pragma unroll
        for (int bp = 0; bp < kBqMaxSB; ++bp) {
          if (bp < b) {                                              // (uniform)
            const float4 c = *reinterpret_cast<const float4*>(kw + bp * D + d4);
            lg[bp] = fmaf(x.x, c.x, fmaf(x.y, c.y, fmaf(x.z, c.z, fmaf(x.w, c.w, lg[bp]))));
          }
        }
      }
#pragma unroll
      for (int bp = 0; bp < kBqMaxSB; ++bp) {
        const float bb = __shfl_sync(0xffffffffu, be, bp);
        lg[bp] = (bp < b && ((live >> bp) & 1u)) ? lg[bp] + bb : -INFINITY;
      }
      if (s_r >= 0) {
        // the k2 best blocks: largest logit first, ties to the lower block; fewer candidates -> all of them
        int32_t* bo = bsel_out + (row * m + s_r) * k2;
        uint32_t chosen = 0u;
        if (bsel_in != nullptr) {
          for (int e = 0; e < k2; ++e) {
            const int c = bsel_in[(row * m + s_r) * k2 + e];
            const bool take = c >= 0 && c < b && !((chosen >> c) & 1u);   // a block named twice is retrieved once
            if (take) chosen |= 1u << c;
            bo[e] = take ? c : -1;
          }
        } else {
          for (int e = 0; e < k2; ++e) {
            float bv = -INFINITY;
            int bi = -1;
#pragma unroll
            for (int bp = 0; bp < kBqMaxSB; ++bp)
              if (!((chosen >> bp) & 1u) && lg[bp] > bv) { bv = lg[bp]; bi = bp; }
            bo[e] = bi;
            if (bi >= 0) chosen |= 1u << bi;
          }
        }
        // every other non-empty earlier block of the cluster is a stand-in key of this query
#pragma unroll
        for (int bp = 0; bp < kBqMaxSB; ++bp)
          if (bp < b && !((chosen >> bp) & 1u)) lgs[(s_r * SB + bp) * kBqChunk + lane] = lg[bp];
      }
    }
    __syncthreads();
    BQCLK(1)

    // ---- phase 2: per query the maximum of its stand-in logits, the weights exp(logit - max) in place, their sum
    {
      const int r = lane, part = warp, ne = m * SB;
      float mx = -INFINITY;
      for (int e = part; e < ne; e += kBqWarps) mx = fmaxf(mx, lgs[e * kBqChunk + r]);
      red[part * kBqChunk + r] = mx;
      __syncthreads();
      float M = -INFINITY;
#pragma unroll
      for (int w = 0; w < kBqWarps; ++w) M = fmaxf(M, red[w * kBqChunk + r]);
      float sum = 0.f;
      for (int e = part; e < ne; e += kBqWarps) {
        const float v = lgs[e * kBqChunk + r];
        const float p = v == -INFINITY ? 0.f : __expf(v - M);
        lgs[e * kBqChunk + r] = p;
        sum += p;
      }
      red[(kBqWarps + part) * kBqChunk + r] = sum;
      __syncthreads();
    }

    BQCLK(2)
    // ---- phase 3: a warp per query, lanes share D: the weighted nu rows
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int r = warp * 4 + k;
      if (tq4[k] < 0) continue;                                      // (warp-uniform)
      float M = -INFINITY, sN = 0.f;
#pragma unroll
      for (int w = 0; w < kBqWarps; ++w) { M = fmaxf(M, red[w * kBqChunk + r]); sN += red[(kBqWarps + w) * kBqChunk + r]; }
      float acc[EPL];
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
      if (sN > 0.f) {
        for (int s = 0; s < m; ++s) {
          const int j = sel_s[r * (m + 1) + s];
          if (j < 0) continue;
          for (int bp = 0; bp < b; ++bp) {
            const float p = lgs[(s * SB + bp) * kBqChunk + r];
            if (p > 0.f) {                                           // (warp-uniform)
              float nv[EPL];
              ldv<EPL>((const bf16*)sp.nu + (ebase + (size_t)bp * estep + j) * D + lane * EPL, nv);
#pragma unroll
              for (int e = 0; e < EPL; ++e) acc[e] = fmaf(p, nv[e], acc[e]);
            }
          }
        }
      }
      const size_t orow = (size_t)pq * dm.N + tq4[k];
      const float inv = sN > 0.f ? 1.f / sN : 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[e] *= inv;
      stv<EPL>(o_near + orow * D + lane * EPL, acc);
      if (lane == 0) lse_near[orow] = sN > 0.f ? M + __logf(sN) : -INFINITY;
    }
    __syncthreads();                                                 // the chunk's shared arrays are reused by the next chunk
    BQCLK(3)
  }
#ifdef MUSE_PHASE_CLOCKS
  if (tid == 0 && blockIdx.x == (unsigned)(3 * dm.Cq + 1) && blockIdx.y == 0)
    for (int k = 0; k < 4; ++k) status[8 + k] = (int)pc[k];
#endif
}

int block_select_q(const Dims& d, const void* Q, const int32_t* off_q, const int32_t* perm_q, const int32_t* sel, const SummPtrs& sp,
                   const int32_t* bsel_in, int32_t* bsel_out, float* o_near, float* lse_near, int* status, cudaStream_t st) {
  const size_t smem = block_select_q_smem(d);
  prof_mark("k_block_select_q", st);
  const dim3 grid(d.S * d.Cq, d.B * d.Hq);
  if (d.D == 128) {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_block_select_q<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_block_select_q<128><<<grid, kBqThreads, smem, st>>>(d, (const bf16*)Q, off_q, perm_q, sel, sp, bsel_in, bsel_out, o_near, lse_near, status);
  } else {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_block_select_q<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_block_select_q<64><<<grid, kBqThreads, smem, st>>>(d, (const bf16*)Q, off_q, perm_q, sel, sp, bsel_in, bsel_out, o_near, lse_near, status);
  }
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

}  // namespace muse
