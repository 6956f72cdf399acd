// Shared declarations of the MuSe CUDA library (internal; the public C ABI is include/muse.h).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include <math.h>
#include "../../include/muse.h"

namespace muse {

constexpr int kMaxHeads = 128;
constexpr int kMaxM = 64;
constexpr int kMaxC = 4096;

struct HeadMap { int16_t g[kMaxHeads]; };

// Resolved problem description passed by value to kernels.
struct Dims {
  int B, Hq, Hkv, N, D, Cq, Ck, m;
  int S;        // spatial blocks (1 when non-causal)
  int SB;       // stored summary planes: S-1 (causal) or 1
  int Bs;       // block size N / S
  int causal, sel_mode, agg_grad;
  int dipole;   // 1: untilted dipole correction of the far field; with m > 0 restricted to the clusters a query did not retrieve;
                // 2: the same with the shared covariance tilted at one point per query head (kept in the summaries buffer)
  int k2;       // spatial selection: 0 = every earlier block of a selected cluster is retrieved; > 0 = only the k2 best (causal only)
  float sigma;
  HeadMap hm;
};

#define MUSE_CUDA_OK(expr) do { cudaError_t e_ = (expr); if (e_ != cudaSuccess) return MUSE_ERR_CUDA; } while (0)
#define MUSE_LAUNCH_OK() do { if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return MUSE_ERR_CUDA; } } while (0)

// Bump allocator over the caller's workspace (256-byte granularity); with base == nullptr it
// only measures.
struct Arena {
  char* base; size_t used;
  explicit Arena(void* b) : base(static_cast<char*>(b)), used(0) {}
  template <class T> T* take(size_t count) {
    size_t bytes = (count * sizeof(T) + 255) & ~size_t(255);
    T* p = base ? reinterpret_cast<T*>(base + used) : nullptr;
    used += bytes;
    return p;
  }
};

__host__ __device__ inline int cdiv(int a, int b) { return (a + b - 1) / b; }

// ---- element access -----------------------------------------------------------------------
__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }
template <class T> __device__ __forceinline__ T from_f(float x);
template <> __device__ __forceinline__ float from_f<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Load 4 consecutive elements (16-byte aligned for float, 8-byte for bf16) as floats.
__device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 ld4(const __nv_bfloat16* p) {
  uint2 u = *reinterpret_cast<const uint2*>(p);
  float4 r;
  r.x = __uint_as_float(u.x << 16); r.y = __uint_as_float(u.x & 0xffff0000u);
  r.z = __uint_as_float(u.y << 16); r.w = __uint_as_float(u.y & 0xffff0000u);
  return r;
}
__device__ __forceinline__ void st4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void st4(__nv_bfloat16* p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 u; u.x = *reinterpret_cast<uint32_t*>(&a); u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}

// EPL (2 or 4) consecutive elements as floats / back, one vector access
template <int EPL> __device__ __forceinline__ void ldv(const float* p, float (&x)[EPL]) {
  if (EPL == 4) { const float4 v = *reinterpret_cast<const float4*>(p); x[0] = v.x; x[1] = v.y; x[EPL - 2] = v.z; x[EPL - 1] = v.w; }
  else { const float2 v = *reinterpret_cast<const float2*>(p); x[0] = v.x; x[1] = v.y; }
}
template <int EPL> __device__ __forceinline__ void ldv(const __nv_bfloat16* p, float (&x)[EPL]) {
  if (EPL == 4) { const float4 v = ld4(p); x[0] = v.x; x[1] = v.y; x[EPL - 2] = v.z; x[EPL - 1] = v.w; }
  else { const uint32_t u = *reinterpret_cast<const uint32_t*>(p); x[0] = __uint_as_float(u << 16); x[1] = __uint_as_float(u & 0xffff0000u); }
}
template <int EPL> __device__ __forceinline__ void stv(float* p, const float (&x)[EPL]) {
  if (EPL == 4) *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[EPL - 2], x[EPL - 1]);
  else *reinterpret_cast<float2*>(p) = make_float2(x[0], x[1]);
}
template <int EPL> __device__ __forceinline__ void stv(__nv_bfloat16* p, const float (&x)[EPL]) {
  if (EPL == 4) st4(p, make_float4(x[0], x[1], x[EPL - 2], x[EPL - 1]));
  else { __nv_bfloat162 b = __floats2bfloat162_rn(x[0], x[1]); *reinterpret_cast<uint32_t*>(p) = *reinterpret_cast<uint32_t*>(&b); }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// per-kernel timing hook (no-op unless muse_profile(1) was called); name = nullptr ends a call
void prof_mark(const char* name, cudaStream_t st);

// Status words: the first kStatusWords int32 of every stage's workspace.  Word 0 holds the first
// MUSE_STATUS_* code a kernel reported (0 = none); the entry points clear the words once per call.
// Words from 8 up carry diagnostics of instrumented builds only.
constexpr int kStatusWords = 64;
__device__ __forceinline__ void report_status(int* status, int code) { atomicCAS(status, 0, code); }

// Bounds-checked build (compiled with -DMUSE_DEBUG into a second library): every index that a kernel derives from data
// (assignments, selections, pair ids, bucket offsets, permutations) and the hand-computed shared-memory offsets of the
// gathers pass through MUSE_IN_RANGE(index, bound).  A value outside [0, bound) is recorded (source line, value, bound,
// count) in a per-source-file device record that muse_debug_report reads, and the caller skips the access: nothing
// traps, the kernel runs to its end.  In the product build the macro is the constant `true` and the checks vanish.
#ifdef MUSE_DEBUG
static __device__ int g_dbg_rec[4];                      // {line, value, bound, violations} of this source file
typedef void (*dbg_reader_t)(int out[4], int reset);
void dbg_register(const char* file, dbg_reader_t fn);    // api.cu
static void dbg_read_tu(int out[4], int reset) {
  if (cudaMemcpyFromSymbol(out, g_dbg_rec, 16) != cudaSuccess) { out[0] = out[1] = out[2] = 0; out[3] = -1; cudaGetLastError(); }
  if (reset) { const int z[4] = {0, 0, 0, 0}; if (cudaMemcpyToSymbol(g_dbg_rec, z, 16) != cudaSuccess) cudaGetLastError(); }
}
struct DbgReg { DbgReg() { dbg_register(__BASE_FILE__, &dbg_read_tu); } };
static const DbgReg g_dbg_reg;
__device__ __forceinline__ bool dbg_in_range(long long v, long long n, int line) {
  if (v >= 0 && v < n) return true;
  if (atomicAdd(&g_dbg_rec[3], 1) == 0) { g_dbg_rec[0] = line; g_dbg_rec[1] = (int)v; g_dbg_rec[2] = (int)n; }
  return false;
}
#define MUSE_IN_RANGE(v, n) muse::dbg_in_range((long long)(v), (long long)(n), __LINE__)
#else
#define MUSE_IN_RANGE(v, n) true
#endif

// Test hook: bit set = take the library's other kernel for that step at shapes where the default is
// the tensor-core kernel (muse_test_force_paths; never set in production).
enum ForcePath : unsigned {
  kForceSummFwdSimt = 1u, kForceFarSimt = 2u, kForceSummBwdSimt = 4u, kForceRetFwdStream = 8u,
  kForceRetBwdSplit = 16u, kForceDipoleSimt = 32u, kForceBlockSelectWarp = 64u
};
bool path_forced(unsigned bit);

// ---- stage launchers (each enqueues on `st`, returns MUSE_OK or MUSE_ERR_CUDA) ---------------
// clustering side: kind 0 = queries (key = block*C + cluster), kind 1 = keys (key = cluster*S + block)
size_t sort_ws_elems(int N, int nkeys);   // int32 scratch elements per problem for bucket_sort
int bucket_sort(int dtype_unused, const int32_t* assign, int problems, int N, int C, int S, int Bs,
                int kind, int32_t* off, int32_t* perm, int32_t* scratch, cudaStream_t st);

int lloyd(const Dims& d, int dtype, const void* X, int problems, int C, int kind,
          const int32_t* init_idx, int init_mode, uint64_t seed, int T,
          int32_t* assign, float* centres, void* ws, cudaStream_t st, float* dist_out = nullptr);   // dist_out: [problems, N, C]
                                                                                               // |c|^2 - 2 x.c of the final assignment (optional)
size_t lloyd_ws_bytes(const Dims& d, int problems, int C, int kind);

// the paper's own clustering: one streaming pass (state = totals, counts; n_batches < 0: to the end) and the
// per-block assignment under a bucket-size cap (factor <= 0: plain nearest centroid)
int kmeanspp(int dtype, const void* X, int problems, int N, int D, int C, int kind, uint64_t seed, float* mind2,
             int32_t* idx_out, int* status, cudaStream_t st);
int stream_kmeans(const Dims& d, int dtype, const void* X, int problems, int C, int kind, uint64_t seed, float beta,
                  int first_batch, int n_batches, float* totals, float* counts, float* centres, int32_t* assign_stream,
                  int32_t* status, cudaStream_t st);
int balanced_assign(const Dims& d, int dtype, const void* X, int problems, int C, int kind, const float* centres, float factor,
                    int32_t* assign, void* ws, cudaStream_t st);
size_t balanced_ws_bytes(const Dims& d, int problems, int C);

// assign_k == nullptr: the keys are already bucketed (off_k, perm_k are inputs) and `status` names the
// caller's status words; counts / ksum / vsum (untilted per-bucket statistics) may be nullptr
int summarize(const Dims& d, int dtype, const void* K, const void* V, const int32_t* assign_k,
              const float* qbar, int32_t* off_k, int32_t* perm_k, int32_t* counts, float* ksum, float* vsum,
              void* summaries, void* ws, int32_t* status, cudaStream_t st);
size_t summarize_ws_bytes(const Dims& d, int dtype);

// sigma * qbar as two bf16 planes (hi + lo keeps ~16 mantissa bits), [B*Hq*Cq][D] each: the tensor-core
// summary kernels load their centroid tiles from these by TMA instead of converting them per CTA
int split_qbar(const Dims& d, const float* qbar, void* qhi, void* qlo, cudaStream_t st);


// Byte offsets inside the caller's summaries buffer.  Per entry (b, h, plane, i, j):
//   mu   fp32  accumulated log-mass            beta fp32  mu - sigma qbar_i . kappa  (so that the
//   Eq. 6 score is sigma q . kappa + beta with the full query)
//   fp32 mode: kappa, nu fp32 [D]   (klo unused)
//   bf16 mode: kappa = khi + klo, two bf16 planes [D] (tensor-core operands that keep ~16 bits
//              of mantissa, so discrete top-m decisions match fp64); nu one bf16 plane [D]
//   cbar (dipole only): merged dipole matrices [B,Hq,SB,Cq][D value dims][D key dims], fp32 or bf16
//   blk (k2 > 0 only): a second set mu | beta | kappa (hi, lo) | nu with the same shapes holding the PER-BLOCK
//              (pre-accumulation) summaries: plane s = the summary of the keys of block s alone
struct SummLayout { size_t mu, beta, khi, klo, nu, Kp, Vp, cbar, cov, pw, zall, qstar, blk, blk_beta, blk_khi, blk_klo, blk_nu, total; };
SummLayout summ_layout(const Dims& d, int dtype);

struct SummPtrs { float* mu; float* beta; void* khi; void* klo; void* nu; };
inline SummPtrs summ_ptrs(const SummLayout& L, const void* base_) {
  char* b = (char*)base_;
  return SummPtrs{(float*)(b + L.mu), (float*)(b + L.beta), b + L.khi, b + L.klo, b + L.nu};
}
// dipole part of the summaries buffer: merged matrices, shared covariances, centroid weights and their sums
struct DipolePtrs { void* cbar; void* cov; void* pw; float* zall; float* qstar; };
inline DipolePtrs dipole_ptrs(const SummLayout& L, const void* base_) {
  char* b = (char*)base_;
  return DipolePtrs{b + L.cbar, b + L.cov, b + L.pw, (float*)(b + L.zall), (float*)(b + L.qstar)};
}
inline SummPtrs summ_ptrs_blk(const SummLayout& L, const void* base_) {      // the per-block set (k2 > 0)
  char* b = (char*)base_;
  return SummPtrs{(float*)(b + L.blk), (float*)(b + L.blk_beta), b + L.blk_khi, b + L.blk_klo, b + L.blk_nu};
}
// dipole correction (dipole.cu): construction at summary time, consumption after the far field
size_t dipole_fwd_ws_bytes(const Dims& d);
// its backward (dipole_bwd.cu); scratch carved from the backward workspace
struct DipoleBwdWs { int32_t* sel_tmp; float *lse_far, *zq, *dz, *delta_far, *xq, *corr, *csub, *dcbar, *dcov, *dpw, *dzs; void* dcbar_bf; };
DipoleBwdWs dipole_bwd_ws(const Dims& d, Arena& ar);       // sized for either kind of contraction kernel
bool dipole_bwd_supported(const Dims& d);
bool dipole_bwd_tc_supported(const Dims& d, int dtype);
bool dipole_bwd_pairs_tc_supported(const Dims& d, int dtype);
int dipole_bwd_pairs_tc(const Dims& d, const void* Q, const float* qbar, const int32_t* assign_q, const int32_t* goff,
                        const int32_t* pairs, const void* cov, const void* pw, const float* xq, const float* dz, float* dQacc,
                        float* dcov, float* dpw, int fill_empty, int* status, cudaStream_t st);
int dipole_bwd_tc(const Dims& d, const void* P, const void* cov, const float* dcbar, void* dcbar_bf, const float* dzs, float* dcov,
                  float* dpw, int with_dpw, const int32_t* goff, int* status, cudaStream_t st);
int dipole_tilt_point(const Dims& d, const int32_t* assign_q, const float* qbar, float* qstar, cudaStream_t st);
int far_fwd_again(const Dims& d, int dtype, const void* Q, const float* qbar, const int32_t* off_q, const int32_t* perm_q,
                  const SummPtrs& sp, const int32_t* sel_in, int32_t* sel_tmp, float* o_far, float* lse_far, int* status,
                  cudaStream_t st);
int dipole_bwd_pre(const Dims& d, int dtype, const void* Q, const void* dO, const float* qbar, const float* LSE, const float* delta,
                   const int32_t* assign_q, const int32_t* off_q, const int32_t* perm_q, const DipolePtrs& dp, const int32_t* goff,
                   const int32_t* pairs, const DipoleBwdWs& w, float* dQacc, int* status, cudaStream_t st);
int dipole_bwd_dmu(const Dims& d, int dtype, const DipolePtrs& dp, const DipoleBwdWs& w, float* dS, int grad_by_key_cluster,
                   cudaStream_t st);
int dipole_bwd_keys(const Dims& d, int dtype, const void* Kp, const void* Vp, const int32_t* off_k, const DipolePtrs& dp,
                    const DipoleBwdWs& w, float* dK_perm, float* dV_perm, cudaStream_t st);
int dipole_build(const Dims& d, int dtype, const void* Kp, const void* Vp, const int32_t* off_k, const float* mu,
                 const DipolePtrs& dp, int* status, cudaStream_t st);
int dipole_apply(const Dims& d, int dtype, const void* Q, const float* qbar, const int32_t* assign_q, const int32_t* off_q,
                 const int32_t* perm_q, const DipolePtrs& dp, const float* lse_far, const int32_t* sel, const int32_t* goff,
                 const int32_t* pairs, float* csub, float* o_far, float* corr, float* zq, int* status, cudaStream_t st);
// ST = storage element type of kappa / nu (float or bf16); idx = element index (entry * D + d), d % 4 == 0
template <class ST> __device__ __forceinline__ float4 ld_kappa4(const SummPtrs& s, size_t idx);
template <> __device__ __forceinline__ float4 ld_kappa4<float>(const SummPtrs& s, size_t idx) { return ld4((const float*)s.khi + idx); }
template <> __device__ __forceinline__ float4 ld_kappa4<__nv_bfloat16>(const SummPtrs& s, size_t idx) {
  float4 a = ld4((const __nv_bfloat16*)s.khi + idx), b = ld4((const __nv_bfloat16*)s.klo + idx);
  return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
}
// value that the stored kappa represents: x itself (fp32) or hi + lo (two bf16)
template <class ST> __device__ __forceinline__ float kappa_repr(float x);
template <> __device__ __forceinline__ float kappa_repr<float>(float x) { return x; }
template <> __device__ __forceinline__ float kappa_repr<__nv_bfloat16>(float x) {
  const float h = __bfloat162float(__float2bfloat16_rn(x));
  return h + __bfloat162float(__float2bfloat16_rn(x - h));
}
template <class ST> __device__ __forceinline__ float4 ld_nu4(const SummPtrs& s, size_t idx) { return ld4((const ST*)s.nu + idx); }
template <class ST> __device__ __forceinline__ void st_kappa4(const SummPtrs& s, size_t idx, float4 v);
template <> __device__ __forceinline__ void st_kappa4<float>(const SummPtrs& s, size_t idx, float4 v) { st4((float*)s.khi + idx, v); }
template <> __device__ __forceinline__ void st_kappa4<__nv_bfloat16>(const SummPtrs& s, size_t idx, float4 v) {
  const float hx = __bfloat162float(__float2bfloat16_rn(v.x)), hy = __bfloat162float(__float2bfloat16_rn(v.y)),
              hz = __bfloat162float(__float2bfloat16_rn(v.z)), hw = __bfloat162float(__float2bfloat16_rn(v.w));
  st4((__nv_bfloat16*)s.khi + idx, make_float4(hx, hy, hz, hw));
  st4((__nv_bfloat16*)s.klo + idx, make_float4(v.x - hx, v.y - hy, v.z - hz, v.w - hw));
}
template <class ST> __device__ __forceinline__ void st_nu4(const SummPtrs& s, size_t idx, float4 v) { st4((ST*)s.nu + idx, v); }

int attn_fwd(const Dims& d, int dtype, const void* Q, const void* K, const void* V,
             const int32_t* assign_q, const float* qbar, const int32_t* off_k, const int32_t* perm_k,
             const void* summaries, const int32_t* sel_in, const int32_t* bsel_in, void* O, float* LSE, int32_t* sel_out,
             int32_t* bsel_out, void* ws, cudaStream_t st);
size_t attn_fwd_ws_bytes(const Dims& d, int dtype);

int attn_bwd(const Dims& d, int dtype, const void* Q, const void* K, const void* V, const void* O,
             const float* LSE, const void* dO, const int32_t* assign_q, const float* qbar,
             const int32_t* off_k, const int32_t* perm_k, const void* summaries, const int32_t* sel, const int32_t* bsel,
             void* dQ, void* dK, void* dV, void* ws, cudaStream_t st);
size_t attn_bwd_ws_bytes(const Dims& d, int dtype);

// retrieval inverse index, shared by forward and backward: groups the (query, slot) pairs by
// (query block - 1, key cluster).  pair id = t * m + slot.
struct RetIndex { int32_t* goff; int32_t* pairs; int32_t* cursor; };
size_t ret_index_elems(const Dims& d);     // int32 elements per query head
// bsel != nullptr (k2 > 0): groups are the (cluster, chosen block) buckets, pair id = (t * m + slot) * k2 + e
int build_ret_index(const Dims& d, const int32_t* sel, const int32_t* bsel, int32_t* scratch, RetIndex* out, cudaStream_t st);

}  // namespace muse
