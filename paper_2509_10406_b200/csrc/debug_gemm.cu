// Diagnostic GEMM on the tcgen05 path: checks the shared-memory layouts and descriptors that
// the attention kernels rely on against a host reference.  Not part of the public header.
#include "common.cuh"
#include "tc05.cuh"

namespace muse {

// mode 0: C = A[M,K] * B[N,K]^T   (A, B K-major)
// mode 1: C = A[M,K] * B[K,N]     (B MN-major)
// mode 2: C = A[K,M]^T * B[N,K]^T (A MN-major)
// MN-major operands: leading-dimension offset = distance between 64-wide column groups,
// stride offset = distance between groups of 8 k-rows (1024 bytes).  (`variant` is unused.)
__global__ void __launch_bounds__(128)
k_debug_gemm(int mode, int variant, const __nv_bfloat16* __restrict__ A, const __nv_bfloat16* __restrict__ B,
             float* __restrict__ C, int M, int N, int K, int* __restrict__ status) {
  extern __shared__ __align__(1024) unsigned char sm_raw[];
  unsigned char* sm = sm_raw + ((1024u - (tc::smem_u32(sm_raw) & 1023u)) & 1023u);   // 1024-byte aligned in the shared window
  __shared__ uint64_t bar;
  __shared__ uint32_t tbase_s;
  const int tid = threadIdx.x, warp = tid >> 5, row0 = blockIdx.x * 128;
  unsigned char* As = sm;                            // K/64 blocks of [128][128 B]  (or MN-major: 2 groups of [K][128 B])
  unsigned char* Bs = sm + (size_t)128 * K * 2;      // K/64 blocks of [N][128 B]    (or MN-major: N/64 groups of [K][128 B])
  uint32_t ncols = 32;
  while ((int)ncols < N) ncols <<= 1;
  if (warp == 0) tc::tmem_alloc(&tbase_s, ncols);
  if (tid == 0) { tc::mbar_init(&bar, 1); tc::mbar_init_fence(); }
  // ---- fill A
  if (mode != 2) {
    for (int e = tid; e < 128 * (K / 8); e += 128) {
      int r = e / (K / 8), ck = e % (K / 8), kb = ck / 8, c = ck % 8;
      uint4 v = *reinterpret_cast<const uint4*>(A + (size_t)(row0 + r) * K + ck * 8);
      *reinterpret_cast<uint4*>(As + (size_t)kb * 128 * 128 + tc::sw128_off(r, c)) = v;
    }
  } else {
    for (int e = tid; e < K * (128 / 8); e += 128) {
      int k = e / 16, cm = e % 16, g = cm / 8, c = cm % 8;
      uint4 v = *reinterpret_cast<const uint4*>(A + (size_t)k * M + row0 + cm * 8);
      *reinterpret_cast<uint4*>(As + (size_t)g * K * 128 + tc::sw128_off(k, c)) = v;
    }
  }
  // ---- fill B
  if (mode != 1) {
    for (int e = tid; e < N * (K / 8); e += 128) {
      int r = e / (K / 8), ck = e % (K / 8), kb = ck / 8, c = ck % 8;
      uint4 v = *reinterpret_cast<const uint4*>(B + (size_t)r * K + ck * 8);
      *reinterpret_cast<uint4*>(Bs + (size_t)kb * N * 128 + tc::sw128_off(r, c)) = v;
    }
  } else {
    for (int e = tid; e < K * (N / 8); e += 128) {
      int k = e / (N / 8), cn = e % (N / 8), g = cn / 8, c = cn % 8;
      uint4 v = *reinterpret_cast<const uint4*>(B + (size_t)k * N + cn * 8);
      *reinterpret_cast<uint4*>(Bs + (size_t)g * K * 128 + tc::sw128_off(k, c)) = v;
    }
  }
  tc::fence_async_smem();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tbase = tbase_s;
  if (tid == 0) {
    const uint32_t idesc = tc::idesc_bf16(128, N, mode == 2, mode == 1);
    const uint32_t a0 = tc::smem_u32(As), b0 = tc::smem_u32(Bs);
    for (int ks = 0; ks < K / 16; ++ks) {
      uint64_t ad, bd;
      if (mode != 2) ad = tc::smem_desc_sw128(a0 + (ks / 4) * 128 * 128 + (ks % 4) * 32, 16, 1024);
      else ad = tc::smem_desc_sw128(a0 + ks * 16 * 128, K * 128, 1024);
      if (mode != 1) bd = tc::smem_desc_sw128(b0 + (ks / 4) * N * 128 + (ks % 4) * 32, 16, 1024);
      else bd = tc::smem_desc_sw128(b0 + ks * 16 * 128, K * 128, 1024);
      tc::mma_bf16_ss(tbase, ad, bd, idesc, ks > 0);
    }
    tc::mma_commit(&bar);
  }
  const bool ok = tc::mbar_wait(&bar, 0);
  tc::fence_after_sync();
  if (ok) {
    for (int c0 = 0; c0 < N; c0 += 32) {
      float v[32];
      tc::tmem_ld32(tbase + ((uint32_t)(warp * 32) << 16) + c0, v);
      float* dst = C + (size_t)(row0 + tid) * N + c0;
#pragma unroll
      for (int i = 0; i < 32; ++i) if (c0 + i < N) dst[i] = v[i];
    }
  } else if (tid == 0) {
    atomicExch(status, 1);
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tbase, ncols);
}

}  // namespace muse

extern "C" __attribute__((visibility("default")))
int muse_debug_gemm(int mode, int variant, const void* A, const void* B, float* C, int M, int N, int K, int* status,
                    cudaStream_t st) {
  using namespace muse;
  if (M % 128 || K % 64 || K > 256 || N % 16 || N > 256 || N < 16) return MUSE_ERR_INVALID_ARG;
  if (mode == 1 && N % 64) return MUSE_ERR_INVALID_ARG;
  const size_t smem = (size_t)128 * K * 2 + (size_t)N * K * 2 + 1024;
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_debug_gemm, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  k_debug_gemm<<<M / 128, 128, smem, st>>>(mode, variant, (const __nv_bfloat16*)A, (const __nv_bfloat16*)B, C, M, N, K, status);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}
