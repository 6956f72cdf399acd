// k-means assignment on the tensor cores (bf16 inputs): argmin_c |c|^2 - 2 x.c with the dot
// products from tcgen05 MMAs.  The centres are fp32; they enter the MMA as a bf16 hi + lo pair
// (two accumulating products), which keeps ~16 mantissa bits so that the discrete assignment
// agrees with an fp64 evaluation except at genuine near-ties (Appendix "Balanced Assignment":
// the |x|^2 term cancels between centres).  One CTA = 128 points, one thread per point scans
// the distance row chunk by chunk straight out of tensor memory.
#include "common.cuh"
#include "tc05.cuh"

namespace muse {

typedef __nv_bfloat16 bf16;
constexpr int kAtRows = 128, kAtCols = 128;

// fp32 centres -> bf16 hi and lo planes
__global__ void k_split_centres(const float* __restrict__ c, long long n, bf16* __restrict__ hi, bf16* __restrict__ lo) {
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= n) return;
  const float x = c[e];
  const bf16 h = __float2bfloat16_rn(x);
  hi[e] = h;
  lo[e] = __float2bfloat16_rn(x - __bfloat162float(h));
}

template <int D>
__global__ void __launch_bounds__(128)
k_assign_tc(const bf16* __restrict__ X, int N, int C, const bf16* __restrict__ chi, const bf16* __restrict__ clo,
            const float* __restrict__ cnorm, int32_t* __restrict__ assign, int* __restrict__ status) {
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  __shared__ uint64_t bar;
  __shared__ uint32_t tbase_s;
  __shared__ float cn[kAtCols];
  constexpr int kX = kAtRows * D * 2, kC = kAtCols * D * 2;
  unsigned char* sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);
  unsigned char *Xs = sm, *Hs = sm + kX, *Ls = Hs + kC;
  const int tid = threadIdx.x, warp = tid >> 5, prob = blockIdx.y, row0 = blockIdx.x * kAtRows;
  if (warp == 0) tc::tmem_alloc(&tbase_s, kAtCols);
  if (tid == 0) { tc::mbar_init(&bar, 1); tc::mbar_init_fence(); }
  const bf16* Xp = X + (size_t)prob * N * D;
  const bf16* hp = chi + (size_t)prob * C * D;
  const bf16* lp = clo + (size_t)prob * C * D;
  const float* cnp = cnorm + (size_t)prob * C;
  constexpr int CPR = D / 8;
  for (int e = tid; e < kAtRows * CPR; e += 128) {
    const int r = e / CPR, ck = e % CPR;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row0 + r < N) v = reinterpret_cast<const uint4*>(Xp + (size_t)(row0 + r) * D)[ck];
    *reinterpret_cast<uint4*>(Xs + (ck >> 3) * kAtRows * 128 + tc::sw128_off(r, ck & 7)) = v;
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tbase = tbase_s, tlane = tbase + ((uint32_t)(warp * 32) << 16);
  uint32_t ph = 0;
  bool ok = true;
  float best = INFINITY;
  int bidx = 0x7fffffff;
  for (int c0 = 0; c0 < C && ok; c0 += kAtCols) {
    for (int e = tid; e < kAtCols * CPR; e += 128) {
      const int r = e / CPR, ck = e % CPR;
      uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;
      if (c0 + r < C) {
        a = reinterpret_cast<const uint4*>(hp + (size_t)(c0 + r) * D)[ck];
        b = reinterpret_cast<const uint4*>(lp + (size_t)(c0 + r) * D)[ck];
      }
      const uint32_t off = (ck >> 3) * kAtCols * 128 + tc::sw128_off(r, ck & 7);
      *reinterpret_cast<uint4*>(Hs + off) = a;
      *reinterpret_cast<uint4*>(Ls + off) = b;
    }
    cn[tid] = c0 + tid < C ? cnp[c0 + tid] : INFINITY;
    tc::fence_async_smem();
    tc::fence_before_sync();
    __syncthreads();
    if (tid == 0) {
      tc::fence_after_sync();
      const uint32_t idesc = tc::idesc_bf16(kAtRows, kAtCols, 0, 0);
      const uint32_t xa = tc::smem_u32(Xs), ha = tc::smem_u32(Hs), la = tc::smem_u32(Ls);
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks)
        tc::mma_bf16_ss(tbase, tc::smem_desc_sw128(xa + (ks / 4) * kAtRows * 128 + (ks % 4) * 32, 16, 1024),
                        tc::smem_desc_sw128(ha + (ks / 4) * kAtCols * 128 + (ks % 4) * 32, 16, 1024), idesc, ks > 0);
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks)
        tc::mma_bf16_ss(tbase, tc::smem_desc_sw128(xa + (ks / 4) * kAtRows * 128 + (ks % 4) * 32, 16, 1024),
                        tc::smem_desc_sw128(la + (ks / 4) * kAtCols * 128 + (ks % 4) * 32, 16, 1024), idesc, 1);
      tc::mma_commit(&bar);
    }
    if (!tc::mbar_wait(&bar, ph)) ok = false;
    ph ^= 1;
    tc::fence_after_sync();
#pragma unroll
    for (int q = 0; q < kAtCols / 32; ++q) {
      float v[32];
      tc::tmem_ld32(tlane + 32 * q, v);
#pragma unroll
      for (int k = 0; k < 32; ++k) {
        const float dist = fmaf(-2.f, v[k], cn[32 * q + k]);
        if (dist < best) { best = dist; bidx = c0 + 32 * q + k; }     // ascending index: ties keep the lower
      }
    }
    tc::fence_before_sync();
    __syncthreads();
  }
  if (ok && row0 + tid < N) assign[(size_t)prob * N + row0 + tid] = bidx;
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tbase, kAtCols);
  if (!ok && tid == 0) atomicExch(status, 6);
}

int assign_tc(const void* X, int problems, int N, int D, int C, const float* centres, const float* cnorm, void* chi,
              void* clo, int32_t* assign, int* status, cudaStream_t st) {
  const long long n = (long long)problems * C * D;
  prof_mark("k_split_centres", st);
  k_split_centres<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(centres, n, (bf16*)chi, (bf16*)clo);
  MUSE_LAUNCH_OK();
  const size_t smem = (size_t)(kAtRows + 2 * kAtCols) * D * 2 + 1024;
  dim3 grid(cdiv(N, kAtRows), problems);
  prof_mark("k_assign_tc", st);
  if (D == 128) {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_assign_tc<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_assign_tc<128><<<grid, 128, smem, st>>>((const bf16*)X, N, C, (const bf16*)chi, (const bf16*)clo, cnorm, assign, status);
  } else {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_assign_tc<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_assign_tc<64><<<grid, 128, smem, st>>>((const bf16*)X, N, C, (const bf16*)chi, (const bf16*)clo, cnorm, assign, status);
  }
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

}  // namespace muse
