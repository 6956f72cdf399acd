// C-ABI entry points: argument validation on the host, then the stage launchers.
#include <stdio.h>
#include <algorithm>
#include "common.cuh"
#include "tc05.cuh"

using namespace muse;

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

unsigned g_forced_paths = 0;

// The status words are cleared once per public call (every kernel of the call reports into them).
int clear_status(void* ws, cudaStream_t st) {
  return cudaMemsetAsync(ws, 0, kStatusWords * sizeof(int32_t), st) == cudaSuccess ? MUSE_OK : MUSE_ERR_CUDA;
}

// A deliberately unreachable wait: nothing ever arrives at the barrier, so the bounded wait runs out
// after `limit_clocks` and the kernel reports through the status word like any production kernel.
__global__ void k_selftest_wait(int* status, unsigned limit_clocks) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) { tc::mbar_init(&bar, 1); tc::mbar_init_fence(); }
  __syncthreads();
  if (threadIdx.x == 0 && !tc::mbar_wait(&bar, 0, limit_clocks)) report_status(status, MUSE_STATUS_SELFTEST_TIMEOUT);
}

// Validates the parameter block and resolves defaults.  Returns MUSE_OK or an error code.
int resolve(const muse_params_t* p, Dims* d) {
  if (p == nullptr) return MUSE_ERR_INVALID_ARG;
  if (p->B < 1 || p->Hq < 1 || p->Hkv < 1 || p->N < 1) return MUSE_ERR_INVALID_ARG;
  if (p->Cq < 1 || p->Ck < 1 || p->m < 0 || p->m > p->Ck) return MUSE_ERR_INVALID_ARG;
  if (p->Cq > p->N || p->Ck > p->N) return MUSE_ERR_INVALID_ARG;
  if (p->dtype != MUSE_BF16 && p->dtype != MUSE_F32) return MUSE_ERR_INVALID_ARG;
  if (p->kmeans_iters < 0 || p->init_mode < 0 || p->init_mode > 3) return MUSE_ERR_INVALID_ARG;
  if (p->sel_mode != MUSE_SEL_PER_QUERY && p->sel_mode != MUSE_SEL_PER_QCLUSTER) return MUSE_ERR_INVALID_ARG;
  if (p->n_blocks < 0 || p->k2 < 0) return MUSE_ERR_INVALID_ARG;
  if (p->D != 64 && p->D != 128) return MUSE_ERR_UNSUPPORTED;
  if (p->Hq > kMaxHeads || p->m > kMaxM || p->Cq > kMaxC || p->Ck > kMaxC) return MUSE_ERR_UNSUPPORTED;
  if (p->dipole < 0 || p->dipole > 2) return MUSE_ERR_INVALID_ARG;
  if (p->k2 > 8 || (p->k2 > 0 && p->dipole != 0)) return MUSE_ERR_UNSUPPORTED;
  int S = p->causal ? (p->n_blocks == 0 ? 8 : p->n_blocks) : 1;
  if (p->N % S != 0) return MUSE_ERR_INVALID_ARG;
  if ((long long)S * p->Cq > 32768 || (long long)S * p->Ck > 32768) return MUSE_ERR_UNSUPPORTED;
  if ((long long)p->N * (p->m > 0 ? p->m : 1) > 0x7fffffffLL) return MUSE_ERR_UNSUPPORTED;
  d->B = p->B; d->Hq = p->Hq; d->Hkv = p->Hkv; d->N = p->N; d->D = p->D;
  d->Cq = p->Cq; d->Ck = p->Ck; d->m = p->m;
  d->S = S; d->SB = p->causal ? S - 1 : 1; d->Bs = p->N / S;
  d->causal = p->causal ? 1 : 0; d->sel_mode = p->sel_mode; d->agg_grad = p->agg_grad ? 1 : 0;
  d->dipole = p->dipole;
  d->k2 = p->causal ? p->k2 : 0;                          // spatial selection needs spatial blocks
  if (d->k2 > 0 && S - 1 > 32) return MUSE_ERR_UNSUPPORTED;
  if (d->k2 > 0 && p->dtype != MUSE_BF16) return MUSE_ERR_UNSUPPORTED;   // built on the bf16 retrieval kernel
  if (d->k2 > 0 && p->m * d->k2 > kMaxM) return MUSE_ERR_UNSUPPORTED;    // at most 64 retrieved buckets per query
  d->sigma = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->D);
  for (int h = 0; h < kMaxHeads; ++h) d->hm.g[h] = 0;
  for (int h = 0; h < p->Hq; ++h) {
    int g;
    if (p->head_map) g = p->head_map[h];
    else { if (p->Hq % p->Hkv != 0) return MUSE_ERR_INVALID_ARG; g = (int)((long long)h * p->Hkv / p->Hq); }
    if (g < 0 || g >= p->Hkv) return MUSE_ERR_INVALID_ARG;
    d->hm.g[h] = (int16_t)g;
  }
  return MUSE_OK;
}

}  // namespace

namespace muse { bool path_forced(unsigned bit) { return (g_forced_paths & bit) != 0; } }

#ifdef MUSE_DEBUG
namespace muse {
struct DbgEntry { const char* file; dbg_reader_t fn; };
static DbgEntry g_dbg_tus[64];
static int g_dbg_ntus = 0;
void dbg_register(const char* file, dbg_reader_t fn) { if (g_dbg_ntus < 64) g_dbg_tus[g_dbg_ntus++] = DbgEntry{file, fn}; }
}  // namespace muse
#endif

extern "C" {

int muse_debug_report(char* text, size_t text_bytes, int reset) {
  if (text != nullptr && text_bytes > 0) text[0] = 0;
#ifdef MUSE_DEBUG
  if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return MUSE_ERR_CUDA; }
  int bad = 0;
  size_t used = 0;
  for (int t = 0; t < muse::g_dbg_ntus; ++t) {
    int rec[4];
    muse::g_dbg_tus[t].fn(rec, reset);
    if (rec[3] == 0) continue;
    ++bad;
    if (text != nullptr && used + 1 < text_bytes) {
      const char* f = muse::g_dbg_tus[t].file;
      for (const char* c = f; *c; ++c) if (*c == '/') f = c + 1;
      const int w = snprintf(text + used, text_bytes - used, "%s:%d value %d outside [0, %d), %d violation(s); ", f, rec[0], rec[1], rec[2], rec[3]);
      if (w > 0) used = used + (size_t)w < text_bytes ? used + (size_t)w : text_bytes - 1;
    }
  }
  return bad;
#else
  (void)reset;
  return MUSE_ERR_UNSUPPORTED;
#endif
}

int muse_test_force_paths(unsigned mask) { g_forced_paths = mask; return MUSE_OK; }

int muse_status_copy(const void* ws, int32_t* dst, cudaStream_t stream) {
  if (ws == nullptr || dst == nullptr) return MUSE_ERR_INVALID_ARG;
  MUSE_CUDA_OK(cudaMemcpyAsync(dst, ws, sizeof(int32_t), cudaMemcpyDefault, stream));
  return MUSE_OK;
}

int muse_test_wait_timeout(void* ws, unsigned limit_clocks, cudaStream_t stream) {
  if (ws == nullptr) return MUSE_ERR_INVALID_ARG;
  if (clear_status(ws, stream) != MUSE_OK) return MUSE_ERR_CUDA;
  k_selftest_wait<<<1, 32, 0, stream>>>((int*)ws, limit_clocks);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

const char* muse_strerror(int code) {
  switch (code) {
    case MUSE_OK: return "ok";
    case MUSE_ERR_INVALID_ARG: return "invalid argument";
    case MUSE_ERR_UNSUPPORTED: return "unsupported configuration";
    case MUSE_ERR_WORKSPACE: return "workspace too small";
    case MUSE_ERR_CUDA: return "CUDA runtime error";
    default: return "unknown error";
  }
}

int muse_workspace_bytes(const muse_params_t* p, size_t out[6]) {
  Dims d;
  int rc = resolve(p, &d);
  if (rc != MUSE_OK) return rc;
  if (out == nullptr) return MUSE_ERR_INVALID_ARG;
  size_t cq = lloyd_ws_bytes(d, d.B * d.Hq, d.Cq, 0), ck = lloyd_ws_bytes(d, d.B * d.Hkv, d.Ck, 1);
  out[0] = cq > ck ? cq : ck;
  out[1] = summarize_ws_bytes(d, p->dtype);
  out[2] = attn_fwd_ws_bytes(d, p->dtype);
  out[3] = attn_bwd_ws_bytes(d, p->dtype);
  out[4] = summ_layout(d, p->dtype).total;
  for (int k = 0; k < 4; ++k) if (out[k] < 256) out[k] = 256;
  // backward without stored summaries: its scratch, then a summaries buffer, then the summaries stage's scratch
  out[5] = out[3] + out[4] + out[1];
  return MUSE_OK;
}

int muse_summaries_layout(const muse_params_t* p, size_t off[9]) {
  Dims d;
  int rc = resolve(p, &d);
  if (rc != MUSE_OK) return rc;
  if (off == nullptr) return MUSE_ERR_INVALID_ARG;
  SummLayout L = summ_layout(d, p->dtype);
  off[0] = L.mu; off[1] = L.beta; off[2] = L.khi; off[3] = L.klo; off[4] = L.nu; off[5] = L.Kp; off[6] = L.Vp; off[7] = L.cbar; off[8] = L.blk;
  return MUSE_OK;
}

int muse_dipole_layout(const muse_params_t* p, size_t off[5]) {
  Dims d;
  int rc = resolve(p, &d);
  if (rc != MUSE_OK) return rc;
  if (off == nullptr) return MUSE_ERR_INVALID_ARG;
  SummLayout L = summ_layout(d, p->dtype);
  off[0] = L.cbar; off[1] = L.cov; off[2] = L.pw; off[3] = L.zall; off[4] = L.qstar;
  return MUSE_OK;
}

int muse_dipole_tilt_point(const muse_params_t* p, const int32_t* assign_q, const float* qbar, void* summaries,
                           cudaStream_t stream) {
  Dims d;
  int rc = resolve(p, &d);
  if (rc != MUSE_OK) return rc;
  if (!assign_q || !qbar || !summaries || !aligned16(qbar) || !aligned16(summaries)) return MUSE_ERR_INVALID_ARG;
  if (d.dipole != 2) return MUSE_ERR_INVALID_ARG;
  rc = dipole_tilt_point(d, assign_q, qbar, dipole_ptrs(summ_layout(d, p->dtype), summaries).qstar, stream);
  prof_mark(nullptr, stream);
  return rc;
}

int muse_cluster(const muse_params_t* p, const void* Q, const void* K, const int32_t* init_q,
                 const int32_t* init_k, int32_t* assign_q, int32_t* assign_k, float* qbar, float* kcent,
                 void* ws, size_t ws_bytes, cudaStream_t stream) {
  Dims d;
  int rc = resolve(p, &d);
  if (rc != MUSE_OK) return rc;
  if (ws == nullptr || !aligned16(ws)) return MUSE_ERR_INVALID_ARG;
  if (Q == nullptr && K == nullptr) return MUSE_ERR_INVALID_ARG;
  size_t need[6];
  muse_workspace_bytes(p, need);
  if (ws_bytes < need[0]) return MUSE_ERR_WORKSPACE;
  if (clear_status(ws, stream) != MUSE_OK) return MUSE_ERR_CUDA;
  if (Q != nullptr) {
    if (assign_q == nullptr || qbar == nullptr || !aligned16(Q) || !aligned16(qbar)) return MUSE_ERR_INVALID_ARG;
    if (p->init_mode == MUSE_INIT_INDICES && init_q == nullptr) return MUSE_ERR_INVALID_ARG;
    rc = lloyd(d, p->dtype, Q, d.B * d.Hq, d.Cq, 0, init_q, p->init_mode, p->seed, p->kmeans_iters, assign_q, qbar, ws, stream);
    if (rc != MUSE_OK) return rc;
  }
  if (K != nullptr) {
    if (assign_k == nullptr || kcent == nullptr || !aligned16(K) || !aligned16(kcent)) return MUSE_ERR_INVALID_ARG;
    if (p->init_mode == MUSE_INIT_INDICES && init_k == nullptr) return MUSE_ERR_INVALID_ARG;
    rc = lloyd(d, p->dtype, K, d.B * d.Hkv, d.Ck, 1, init_k, p->init_mode, p->seed, p->kmeans_iters, assign_k, kcent, ws, stream);
    if (rc != MUSE_OK) return rc;
  }
  prof_mark(nullptr, stream);
  return MUSE_OK;
}

static size_t up256(size_t x) { return (x + 255) & ~size_t(255); }

int muse_stream_workspace_bytes(const muse_params_t* p, size_t* bytes) {
  Dims d;
  int rc = resolve(p, &d);
  if (rc != MUSE_OK) return rc;
  if (bytes == nullptr) return MUSE_ERR_INVALID_ARG;
  const size_t pq = (size_t)d.B * d.Hq, pk = (size_t)d.B * d.Hkv;
  const size_t bal = std::max(balanced_ws_bytes(d, (int)pq, d.Cq), balanced_ws_bytes(d, (int)pk, d.Ck));
  const size_t tot = std::max(pq * d.Cq, pk * d.Ck);
  *bytes = up256(bal) + up256(tot * d.D * sizeof(float)) + up256(tot * sizeof(float));
  return MUSE_OK;
}

int muse_kmeanspp_init(const muse_params_t* p, const void* X, int side, int32_t* idx_out, void* ws, size_t ws_bytes,
                       cudaStream_t stream) {
  Dims d;
  int rc = resolve(p, &d);
  if (rc != MUSE_OK) return rc;
  if (!X || !idx_out || !ws || (side != 0 && side != 1)) return MUSE_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(ws)) return MUSE_ERR_INVALID_ARG;
  const int problems = side == 0 ? d.B * d.Hq : d.B * d.Hkv, C = side == 0 ? d.Cq : d.Ck;
  if (ws_bytes < up256(kStatusWords * sizeof(int32_t)) + up256((size_t)problems * d.N * sizeof(float))) return MUSE_ERR_WORKSPACE;
  if (clear_status(ws, stream) != MUSE_OK) return MUSE_ERR_CUDA;
  Arena ar(ws);
  ar.take<int32_t>(kStatusWords);
  float* mind2 = ar.take<float>((size_t)problems * d.N);
  rc = kmeanspp(p->dtype, X, problems, d.N, d.D, C, side, p->seed, mind2, idx_out, (int*)ws, stream);
  prof_mark(nullptr, stream);
  return rc;
}

int muse_stream_kmeans(const muse_params_t* p, const void* X, int side, float beta, int first_batch, int n_batches,
                       float* totals, float* counts, float* centres, int32_t* assign_stream, void* ws, size_t ws_bytes,
                       cudaStream_t stream) {
  Dims d;
  int rc = resolve(p, &d);
  if (rc != MUSE_OK) return rc;
  if (!X || !totals || !counts || !centres || !ws || (side != 0 && side != 1)) return MUSE_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(totals) || !aligned16(centres) || !aligned16(ws)) return MUSE_ERR_INVALID_ARG;
  if (!(beta > 0.f) || beta > 1.f) return MUSE_ERR_INVALID_ARG;
  if (ws_bytes < 256) return MUSE_ERR_WORKSPACE;
  if (clear_status(ws, stream) != MUSE_OK) return MUSE_ERR_CUDA;
  rc = stream_kmeans(d, p->dtype, X, side == 0 ? d.B * d.Hq : d.B * d.Hkv, side == 0 ? d.Cq : d.Ck, side, p->seed, beta,
                     first_batch, n_batches, totals, counts, centres, assign_stream, (int32_t*)ws, stream);
  prof_mark(nullptr, stream);
  return rc;
}

int muse_balanced_assign(const muse_params_t* p, const void* X, int side, const float* centres, float cap_factor,
                         int32_t* assign, void* ws, size_t ws_bytes, cudaStream_t stream) {
  Dims d;
  int rc = resolve(p, &d);
  if (rc != MUSE_OK) return rc;
  if (!X || !centres || !assign || !ws || (side != 0 && side != 1)) return MUSE_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(centres) || !aligned16(ws)) return MUSE_ERR_INVALID_ARG;
  const int problems = side == 0 ? d.B * d.Hq : d.B * d.Hkv, C = side == 0 ? d.Cq : d.Ck;
  if (ws_bytes < balanced_ws_bytes(d, problems, C)) return MUSE_ERR_WORKSPACE;
  if (clear_status(ws, stream) != MUSE_OK) return MUSE_ERR_CUDA;
  rc = balanced_assign(d, p->dtype, X, problems, C, side, centres, cap_factor, assign, ws, stream);
  prof_mark(nullptr, stream);
  return rc;
}

int muse_cluster_streaming(const muse_params_t* p, const void* Q, const void* K, float beta, float cap_factor,
                           int32_t* assign_q, int32_t* assign_k, float* qbar, float* kcent, void* ws, size_t ws_bytes,
                           cudaStream_t stream) {
  Dims d;
  int rc = resolve(p, &d);
  if (rc != MUSE_OK) return rc;
  if (ws == nullptr || !aligned16(ws) || (Q == nullptr && K == nullptr)) return MUSE_ERR_INVALID_ARG;
  if (!(beta > 0.f) || beta > 1.f) return MUSE_ERR_INVALID_ARG;
  size_t need = 0;
  muse_stream_workspace_bytes(p, &need);
  if (ws_bytes < need) return MUSE_ERR_WORKSPACE;
  if (clear_status(ws, stream) != MUSE_OK) return MUSE_ERR_CUDA;
  const size_t pq = (size_t)d.B * d.Hq, pk = (size_t)d.B * d.Hkv;
  const size_t bal = up256(std::max(balanced_ws_bytes(d, (int)pq, d.Cq), balanced_ws_bytes(d, (int)pk, d.Ck)));
  const size_t tot = std::max(pq * d.Cq, pk * d.Ck);
  float* totals = reinterpret_cast<float*>((char*)ws + bal);
  float* counts = reinterpret_cast<float*>((char*)ws + bal + up256(tot * d.D * sizeof(float)));
  for (int side = 0; side < 2; ++side) {
    const void* X = side == 0 ? Q : K;
    if (X == nullptr) continue;
    int32_t* assign = side == 0 ? assign_q : assign_k;
    float* cen = side == 0 ? qbar : kcent;
    if (assign == nullptr || cen == nullptr || !aligned16(X) || !aligned16(cen)) return MUSE_ERR_INVALID_ARG;
    const int problems = side == 0 ? (int)pq : (int)pk, C = side == 0 ? d.Cq : d.Ck;
    rc = stream_kmeans(d, p->dtype, X, problems, C, side, p->seed, beta, 0, -1, totals, counts, cen, nullptr, (int32_t*)ws, stream);
    if (rc != MUSE_OK) return rc;
    rc = balanced_assign(d, p->dtype, X, problems, C, side, cen, cap_factor, assign, ws, stream);
    if (rc != MUSE_OK) return rc;
  }
  prof_mark(nullptr, stream);
  return MUSE_OK;
}

int muse_summarize(const muse_params_t* p, const void* K, const void* V, const int32_t* assign_k,
                   const float* qbar, int32_t* off_k, int32_t* perm_k, int32_t* counts, float* ksum, float* vsum,
                   void* summaries, void* ws, size_t ws_bytes, cudaStream_t stream) {
  Dims d;
  int rc = resolve(p, &d);
  if (rc != MUSE_OK) return rc;
  if (!K || !V || !assign_k || !qbar || !off_k || !perm_k || !summaries || !ws) return MUSE_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(qbar) || !aligned16(summaries) || !aligned16(ws)) return MUSE_ERR_INVALID_ARG;
  const int nstat = (counts != nullptr) + (ksum != nullptr) + (vsum != nullptr);
  if (nstat != 0 && nstat != 3) return MUSE_ERR_INVALID_ARG;            // the three untilted outputs come together
  if (nstat == 3 && (!aligned16(ksum) || !aligned16(vsum))) return MUSE_ERR_INVALID_ARG;
  size_t need[6];
  muse_workspace_bytes(p, need);
  if (ws_bytes < need[1]) return MUSE_ERR_WORKSPACE;
  if (clear_status(ws, stream) != MUSE_OK) return MUSE_ERR_CUDA;
  rc = summarize(d, p->dtype, K, V, assign_k, qbar, off_k, perm_k, counts, ksum, vsum, summaries, ws, nullptr, stream);
  prof_mark(nullptr, stream);
  return rc;
}

int muse_attn_fwd(const muse_params_t* p, const void* Q, const void* K, const void* V,
                  const int32_t* assign_q, const float* qbar, const int32_t* off_k, const int32_t* perm_k,
                  const void* summaries, const int32_t* sel_in, const int32_t* bsel_in, void* O, float* LSE, int32_t* sel_out,
                  int32_t* bsel_out, void* ws, size_t ws_bytes, cudaStream_t stream) {
  Dims d;
  int rc = resolve(p, &d);
  if (rc != MUSE_OK) return rc;
  if (!Q || !K || !V || !assign_q || !qbar || !off_k || !perm_k || !summaries || !O || !LSE || !ws) return MUSE_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(qbar) || !aligned16(summaries) || !aligned16(O) || !aligned16(ws)) return MUSE_ERR_INVALID_ARG;
  size_t need[6];
  muse_workspace_bytes(p, need);
  if (ws_bytes < need[2]) return MUSE_ERR_WORKSPACE;
  if (clear_status(ws, stream) != MUSE_OK) return MUSE_ERR_CUDA;
  rc = attn_fwd(d, p->dtype, Q, K, V, assign_q, qbar, off_k, perm_k, summaries, sel_in, bsel_in, O, LSE, sel_out, bsel_out, ws, stream);
  prof_mark(nullptr, stream);
  return rc;
}

int muse_attn_bwd(const muse_params_t* p, const void* Q, const void* K, const void* V, const void* O,
                  const float* LSE, const void* dO, const int32_t* assign_q, const float* qbar,
                  const int32_t* off_k, const int32_t* perm_k, const void* summaries, const int32_t* sel,
                  const int32_t* bsel, void* dQ, void* dK, void* dV, void* ws, size_t ws_bytes, cudaStream_t stream) {
  Dims d;
  int rc = resolve(p, &d);
  if (rc != MUSE_OK) return rc;
  if (!Q || !K || !V || !O || !LSE || !dO || !assign_q || !qbar || !off_k || !perm_k || !dQ || !dK || !dV || !ws) return MUSE_ERR_INVALID_ARG;
  if (d.dipole && !dipole_bwd_supported(d)) return MUSE_ERR_UNSUPPORTED;
  if (d.m > 0 && d.SB > 0 && sel == nullptr) return MUSE_ERR_INVALID_ARG;
  if (d.k2 > 0 && d.m > 0 && d.SB > 0 && bsel == nullptr) return MUSE_ERR_INVALID_ARG;   // the forward pass's chosen blocks
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(dO) || !aligned16(qbar) ||
      !aligned16(summaries) || !aligned16(dQ) || !aligned16(dK) || !aligned16(dV) || !aligned16(ws)) return MUSE_ERR_INVALID_ARG;
  size_t need[6];
  muse_workspace_bytes(p, need);
  if (ws_bytes < (summaries ? need[3] : need[5])) return MUSE_ERR_WORKSPACE;
  if (clear_status(ws, stream) != MUSE_OK) return MUSE_ERR_CUDA;
  if (summaries == nullptr) {
    // Rebuild the summaries from the bucketed keys in the tail of the workspace (the keys keep the
    // bucketing that off_k / perm_k describe, so no sort is needed).
    char* tail = (char*)ws + need[3];
    if (d.dipole == 2) {                                  // the rebuilt buffer needs its tilt point first
      rc = dipole_tilt_point(d, assign_q, qbar, dipole_ptrs(summ_layout(d, p->dtype), tail).qstar, stream);
      if (rc != MUSE_OK) return rc;
    }
    rc = summarize(d, p->dtype, K, V, nullptr, qbar, const_cast<int32_t*>(off_k), const_cast<int32_t*>(perm_k), nullptr, nullptr,
                   nullptr, tail, tail + need[4], (int32_t*)ws, stream);
    if (rc != MUSE_OK) return rc;
    summaries = tail;
  }
  rc = attn_bwd(d, p->dtype, Q, K, V, O, LSE, dO, assign_q, qbar, off_k, perm_k, summaries, sel, bsel, dQ, dK, dV, ws, stream);
  prof_mark(nullptr, stream);
  return rc;
}

}  // extern "C"
