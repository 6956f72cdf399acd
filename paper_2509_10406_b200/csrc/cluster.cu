// Clustering stage: Lloyd k-means (Appendix "Clustering Details") and the stable
// (cluster, block) bucketing used by every later stage (Section "Exact retrieval": keys and
// values are bucketed by (cluster, block)).
#include "common.cuh"
#include "feistel.cuh"

namespace muse {

// ---------------------------------------------------------------------------------------------
// Stable counting sort of tokens by an integer key.
//   kind 0 (queries): key = block * C + cluster   -> segments (block, cluster) contiguous
//   kind 1 (keys)   : key = cluster * S + block   -> a cluster's blocks are one contiguous run
// Three kernels: per-chunk histogram, one scan per problem, stable scatter.
// ---------------------------------------------------------------------------------------------
constexpr int kSortChunk = 4096;
constexpr int kSortThreads = 256;

__device__ __forceinline__ int sort_key(int t, int a, int C, int S, int Bs, int kind) {
  int b = t / Bs;
  a = min(max(a, 0), C - 1);             // a caller-provided assignment outside [0, C) is pinned, never used as an index
  return kind == 0 ? b * C + a : a * S + b;
}

__global__ void __launch_bounds__(kSortThreads)
k_sort_hist(const int32_t* __restrict__ assign, int N, int C, int S, int Bs, int kind, int nkeys,
            int nchunks, int32_t* __restrict__ cnt) {
  extern __shared__ int32_t sh[];
  const int chunk = blockIdx.x, prob = blockIdx.y;
  for (int k = threadIdx.x; k < nkeys; k += kSortThreads) sh[k] = 0;
  __syncthreads();
  const int32_t* a = assign + (size_t)prob * N;
  const int t0 = chunk * kSortChunk, t1 = min(N, t0 + kSortChunk);
  for (int t = t0 + threadIdx.x; t < t1; t += kSortThreads)
    atomicAdd(&sh[sort_key(t, a[t], C, S, Bs, kind)], 1);
  __syncthreads();
  int32_t* c = cnt + (size_t)prob * nkeys * nchunks;
  for (int k = threadIdx.x; k < nkeys; k += kSortThreads) c[(size_t)k * nchunks + chunk] = sh[k];
}

// Exclusive scan of cnt[key][chunk] in (key, chunk) order; off[key] = start of the key's run.
__global__ void __launch_bounds__(1024)
k_sort_scan(int32_t* __restrict__ cnt, int nkeys, int nchunks, int32_t* __restrict__ off) {
  __shared__ int32_t part[1024];
  const int prob = blockIdx.x, tid = threadIdx.x;
  const int L = nkeys * nchunks;
  int32_t* c = cnt + (size_t)prob * L;
  int32_t* o = off + (size_t)prob * (nkeys + 1);
  const int per = cdiv(L, 1024);
  const int e0 = min(L, tid * per), e1 = min(L, e0 + per);
  int s = 0;
  for (int e = e0; e < e1; ++e) s += c[e];
  part[tid] = s;
  __syncthreads();
  for (int ofs = 1; ofs < 1024; ofs <<= 1) {       // Hillis-Steele inclusive scan
    int v = tid >= ofs ? part[tid - ofs] : 0;
    __syncthreads();
    part[tid] += v;
    __syncthreads();
  }
  int run = part[tid] - s;
  for (int e = e0; e < e1; ++e) {
    int v = c[e];
    c[e] = run;
    if (e % nchunks == 0) o[e / nchunks] = run;
    run += v;
  }
  if (tid == 1023) o[nkeys] = run;     // the last thread ends on the grand total
}

// Same scan for the large [key][chunk] arrays of the bucket sorts: a problem's array is cut into
// kScanParts contiguous parts, one CTA each.  The CTA first adds up everything in front of its part
// (coalesced), then scans its part; the result goes to a second array because other CTAs still
// read the counts.
constexpr int kScanParts = 8;

__global__ void __launch_bounds__(1024)
k_sort_scan_parts(const int32_t* __restrict__ cnt, int32_t* __restrict__ pre, int nkeys, int nchunks, int32_t* __restrict__ off) {
  __shared__ int32_t part[1024];
  __shared__ int32_t base_s;
  const int prob = blockIdx.x, g = blockIdx.y, tid = threadIdx.x;
  const int L = nkeys * nchunks;
  const int32_t* c = cnt + (size_t)prob * L;
  int32_t* out = pre + (size_t)prob * L;
  int32_t* o = off + (size_t)prob * (nkeys + 1);
  const int plen = cdiv(L, kScanParts), p0 = min(L, g * plen), p1 = min(L, p0 + plen);
  int s0 = 0;
  for (int e = tid; e < p0; e += 1024) s0 += c[e];
  part[tid] = s0;
  __syncthreads();
  for (int ofs = 512; ofs > 0; ofs >>= 1) {
    if (tid < ofs) part[tid] += part[tid + ofs];
    __syncthreads();
  }
  if (tid == 0) base_s = part[0];
  __syncthreads();
  const int base = base_s;
  const int per = cdiv(p1 - p0, 1024);
  const int e0 = min(p1, p0 + tid * per), e1 = min(p1, e0 + per);
  int s = 0;
  for (int e = e0; e < e1; ++e) s += c[e];
  part[tid] = s;
  __syncthreads();
  for (int ofs = 1; ofs < 1024; ofs <<= 1) {       // Hillis-Steele inclusive scan
    int v = tid >= ofs ? part[tid - ofs] : 0;
    __syncthreads();
    part[tid] += v;
    __syncthreads();
  }
  int run = base + part[tid] - s;
  for (int e = e0; e < e1; ++e) {
    int v = c[e];
    out[e] = run;
    if (e % nchunks == 0) o[e / nchunks] = run;
    run += v;
  }
  if (g == kScanParts - 1 && tid == 1023) o[nkeys] = run;     // the last thread of the last part ends on the grand total
}

int launch_scan(int32_t* cnt, int problems, int nkeys, int nchunks, int32_t* off, cudaStream_t st) {
  prof_mark("k_sort_scan", st);
  k_sort_scan<<<problems, 1024, 0, st>>>(cnt, nkeys, nchunks, off);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

__global__ void __launch_bounds__(kSortThreads)
k_sort_scatter(const int32_t* __restrict__ assign, int N, int C, int S, int Bs, int kind, int nkeys,
               int nchunks, const int32_t* __restrict__ cnt, int32_t* __restrict__ perm) {
  extern __shared__ int32_t cur[];
  const int chunk = blockIdx.x, prob = blockIdx.y;
  const int32_t* c = cnt + (size_t)prob * nkeys * nchunks;
  for (int k = threadIdx.x; k < nkeys; k += kSortThreads) cur[k] = c[(size_t)k * nchunks + chunk];
  __syncthreads();
  const int32_t* a = assign + (size_t)prob * N;
  int32_t* pm = perm + (size_t)prob * N;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t0 = chunk * kSortChunk, t1 = min(N, t0 + kSortChunk);
  for (int base = t0; base < t1; base += kSortThreads) {
    const int t = base + threadIdx.x;
    const bool live = t < t1;
    const int key = live ? sort_key(t, a[t], C, S, Bs, kind) : -1 - lane;
    // warps take turns in token order so equal keys keep ascending positions (stable)
    for (int w = 0; w < kSortThreads / 32; ++w) {
      if (warp == w) {
        unsigned peers = __match_any_sync(0xffffffffu, key);
        int rank = __popc(peers & ((1u << lane) - 1u));
        int start = live ? cur[key] : 0;
        __syncwarp();
        if (live && MUSE_IN_RANGE(start + rank, N)) {
          pm[start + rank] = t;
          if (rank == __popc(peers) - 1) cur[key] = start + rank + 1;
        }
      }
      __syncthreads();
    }
  }
}

// counts [key][chunk] and their exclusive scan
size_t sort_ws_elems(int N, int nkeys) { return 2 * (size_t)nkeys * cdiv(N, kSortChunk); }

int bucket_sort(int, const int32_t* assign, int problems, int N, int C, int S, int Bs, int kind,
                int32_t* off, int32_t* perm, int32_t* scratch, cudaStream_t st) {
  const int nkeys = C * S, nchunks = cdiv(N, kSortChunk);
  const size_t smem = (size_t)nkeys * sizeof(int32_t);
  if (smem > 48 * 1024) {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_sort_hist, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_sort_scatter, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  }
  prof_mark("k_sort_hist", st);
  k_sort_hist<<<dim3(nchunks, problems), kSortThreads, smem, st>>>(assign, N, C, S, Bs, kind, nkeys, nchunks, scratch);
  MUSE_LAUNCH_OK();
  int32_t* pre = scratch + (size_t)problems * nkeys * nchunks;
  prof_mark("k_sort_scan", st);
  k_sort_scan_parts<<<dim3(problems, kScanParts), 1024, 0, st>>>(scratch, pre, nkeys, nchunks, off);
  MUSE_LAUNCH_OK();
  prof_mark("k_sort_scatter", st);
  k_sort_scatter<<<dim3(nchunks, problems), kSortThreads, smem, st>>>(assign, N, C, S, Bs, kind, nkeys, nchunks, pre, perm);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

// ---------------------------------------------------------------------------------------------
// Lloyd iterations
// ---------------------------------------------------------------------------------------------
int assign_tc(const void* X, int problems, int N, int D, int C, const float* centres, const float* cnorm, void* chi,
              void* clo, int32_t* assign, float* dist_out, int* status, cudaStream_t st);

template <class T>
__global__ void k_init_centres(const T* __restrict__ X, int N, int D, int C, const int32_t* __restrict__ init_idx,
                               int init_mode, uint64_t seed, int kind, float* __restrict__ centres) {
  const int c = blockIdx.x, prob = blockIdx.y;
  int idx;
  if (init_mode == MUSE_INIT_INDICES) idx = init_idx[(size_t)prob * C + c];
  else idx = feistel_permute(c * (N / C), N, seed, (uint64_t)prob * 2 + kind);
  idx = min(max(idx, 0), N - 1);
  const T* x = X + ((size_t)prob * N + idx) * D;
  float* o = centres + ((size_t)prob * C + c) * D;
  for (int d = threadIdx.x; d < D; d += blockDim.x) o[d] = to_f(x[d]);
}

__global__ void k_centre_norms(const float* __restrict__ centres, int total, int D, float* __restrict__ cnorm) {
  const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (w >= total) return;
  const float* c = centres + (size_t)w * D;
  float s = 0.f;
  for (int d = lane; d < D; d += 32) s = fmaf(c[d], c[d], s);
  s = warp_sum(s);
  if (lane == 0) cnorm[w] = s;
}

// Assignment: argmin_c |c|^2 - 2 x.c, fp32 FFMA, 128 points x 64 centres per tile, 8x4 per thread.
constexpr int kAsgRows = 128, kAsgCols = 64, kAsgThreads = 256;

template <class T, int D>
__global__ void __launch_bounds__(kAsgThreads)
k_assign(const T* __restrict__ X, int N, int C, const float* __restrict__ centres,
         const float* __restrict__ cnorm, int32_t* __restrict__ assign, float* __restrict__ dist_out) {
  constexpr int LD = D + 4;
  extern __shared__ float smf[];
  float* Xs = smf;                       // [128][LD]
  float* Cs = Xs + kAsgRows * LD;        // [64][LD]
  float* cn = Cs + kAsgCols * LD;        // [64]
  const int prob = blockIdx.y, row0 = blockIdx.x * kAsgRows;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const T* Xp = X + (size_t)prob * N * D;
  const float* Cp = centres + (size_t)prob * C * D;
  const float* cnp = cnorm + (size_t)prob * C;
  for (int e = tid; e < kAsgRows * (D / 4); e += kAsgThreads) {
    int r = e / (D / 4), q = e % (D / 4);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (row0 + r < N) v = ld4(Xp + (size_t)(row0 + r) * D + q * 4);
    st4(Xs + r * LD + q * 4, v);
  }
  float best[8]; int bidx[8];
#pragma unroll
  for (int r = 0; r < 8; ++r) { best[r] = INFINITY; bidx[r] = 0x7fffffff; }
  for (int c0 = 0; c0 < C; c0 += kAsgCols) {
    __syncthreads();
    for (int e = tid; e < kAsgCols * (D / 4); e += kAsgThreads) {
      int r = e / (D / 4), q = e % (D / 4);
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (c0 + r < C) v = ld4(Cp + (size_t)(c0 + r) * D + q * 4);
      st4(Cs + r * LD + q * 4, v);
    }
    if (tid < kAsgCols) cn[tid] = (c0 + tid < C) ? cnp[c0 + tid] : INFINITY;
    __syncthreads();
    float acc[8][4];
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
      for (int k = 0; k < 4; ++k) acc[r][k] = 0.f;
#pragma unroll 4
    for (int d = 0; d < D; d += 4) {
      float4 cv[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) cv[k] = ld4(Cs + (tx * 4 + k) * LD + d);
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        float4 xv = ld4(Xs + (ty * 8 + r) * LD + d);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          acc[r][k] = fmaf(xv.x, cv[k].x, acc[r][k]);
          acc[r][k] = fmaf(xv.y, cv[k].y, acc[r][k]);
          acc[r][k] = fmaf(xv.z, cv[k].z, acc[r][k]);
          acc[r][k] = fmaf(xv.w, cv[k].w, acc[r][k]);
        }
      }
    }
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float dist = fmaf(-2.f, acc[r][k], cn[tx * 4 + k]);
        int c = c0 + tx * 4 + k;
        if (dist < best[r]) { best[r] = dist; bidx[r] = c; }   // ascending c: ties keep the lower
        // (optional output: the whole matrix |c|^2 - 2 x.c, for the balanced assignment's second step)
        if (dist_out != nullptr && c < C && row0 + ty * 8 + r < N) dist_out[((size_t)prob * N + row0 + ty * 8 + r) * C + c] = dist;
      }
  }
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    float b = best[r]; int i = bidx[r];
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) {
      float ob = __shfl_xor_sync(0xffffffffu, b, o);
      int oi = __shfl_xor_sync(0xffffffffu, i, o);
      if (ob < b || (ob == b && oi < i)) { b = ob; i = oi; }
    }
    int row = row0 + ty * 8 + r;
    // a row of NaN or infinities never compares below the running minimum: it goes to cluster 0
    if (tx == 0 && row < N) assign[(size_t)prob * N + row] = (unsigned)i < (unsigned)C ? i : 0;
  }
}

// Centre update: mean of the members, summed with a fixed reduction tree (slot s of the CTA adds members
// s, s + SLOTS, ... in bucket order, then the slots are added in order), so the result does not depend
// on scheduling.  An empty cluster keeps its centre.  One 256-thread CTA per cluster; a lane owns 16 bytes
// of a row, and every slot keeps four row loads in flight (the member list is an indirection, so a
// single load per slot leaves the kernel waiting on memory latency).
constexpr int kUpdThreads = 256;

__device__ __forceinline__ void ld16f(const float* p, float (&x)[4]) { const float4 v = *reinterpret_cast<const float4*>(p); x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w; }
__device__ __forceinline__ void ld16f(const __nv_bfloat16* p, float (&x)[8]) {
  const uint4 u = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int k = 0; k < 4; ++k) { x[2 * k] = __uint_as_float(w[k] << 16); x[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u); }
}

template <class T, int D>
__global__ void __launch_bounds__(kUpdThreads)
k_update(const T* __restrict__ X, int N, int C, int S, int kind, const int32_t* __restrict__ off,
         const int32_t* __restrict__ perm, float* __restrict__ centres, float* __restrict__ cnorm) {
  constexpr int VEC = 16 / (int)sizeof(T);     // elements per lane
  constexpr int LPR = D / VEC;                 // lanes per row
  constexpr int RPW = 32 / LPR;                // rows per warp step
  constexpr int SLOTS = (kUpdThreads / 32) * RPW;
  __shared__ float part[SLOTS][D];
  __shared__ float n2_s[kUpdThreads / 32];
  const int c = blockIdx.x, prob = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane / LPR, q = lane % LPR;
  const int slot = warp * RPW + sub;
  const T* Xp = X + (size_t)prob * N * D + q * VEC;
  const int32_t* o = off + (size_t)prob * (C * S + 1);
  const int32_t* pm = perm + (size_t)prob * N;
  float s[VEC];
#pragma unroll
  for (int k = 0; k < VEC; ++k) s[k] = 0.f;
  int count = 0;
  const int nranges = kind == 0 ? S : 1;
  for (int r = 0; r < nranges; ++r) {
    const int p0 = kind == 0 ? o[r * C + c] : o[c * S];
    const int p1 = kind == 0 ? o[r * C + c + 1] : o[(c + 1) * S];
    count += p1 - p0;
    for (int p = p0 + slot; p < p1; p += 4 * SLOTS) {
      int idx[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        idx[u] = p + u * SLOTS < p1 && MUSE_IN_RANGE(p + u * SLOTS, N) ? pm[p + u * SLOTS] : -1;
        if (idx[u] >= 0 && !MUSE_IN_RANGE(idx[u], N)) idx[u] = -1;
      }
      float v[4][VEC];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (idx[u] >= 0) ld16f(Xp + (size_t)idx[u] * D, v[u]);
        else {
#pragma unroll
          for (int k = 0; k < VEC; ++k) v[u][k] = 0.f;
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int k = 0; k < VEC; ++k) s[k] += v[u][k];
    }
  }
#pragma unroll
  for (int k = 0; k < VEC; ++k) part[slot][q * VEC + k] = s[k];
  __syncthreads();
  float n2 = 0.f;
  if (threadIdx.x < D) {
    const int d = threadIdx.x;
    float tot = 0.f;
    float* dst = centres + ((size_t)prob * C + c) * D + d;
#pragma unroll
    for (int k = 0; k < SLOTS; ++k) tot += part[k][d];
    if (count > 0) { tot *= 1.f / (float)count; *dst = tot; }
    else tot = *dst;
    n2 = tot * tot;
  }
  n2 = warp_sum(n2);
  if (lane == 0) n2_s[warp] = n2;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
#pragma unroll
    for (int k = 0; k < D / 32; ++k) t += n2_s[k];
    cnorm[(size_t)prob * C + c] = t;
  }
}

template <class T, int D>
static int lloyd_t(const Dims& d, const T* X, int problems, int C, int kind, const int32_t* init_idx,
                   int init_mode, uint64_t seed, int T_iters, int32_t* assign, float* centres, void* ws,
                   float* dist_out, cudaStream_t st) {
  Arena ar(ws);
  int32_t* status = ar.take<int32_t>(kStatusWords);     // cleared by the entry point, shared by both sides
  float* cnorm = ar.take<float>((size_t)problems * C);
  int32_t* off = ar.take<int32_t>((size_t)problems * (C * d.S + 1));
  int32_t* perm = ar.take<int32_t>((size_t)problems * d.N);
  int32_t* scratch = ar.take<int32_t>((size_t)problems * sort_ws_elems(d.N, C * d.S));
  __nv_bfloat16* chi = ar.take<__nv_bfloat16>((size_t)problems * C * D);
  __nv_bfloat16* clo = ar.take<__nv_bfloat16>((size_t)problems * C * D);
  constexpr bool kTensor = sizeof(T) == 2;     // bf16 inputs: distances on the tensor cores
  if (init_mode == MUSE_INIT_KMEANSPP) {
    // the draws borrow two arrays that the iterations only fill later: perm as the running minimum distance
    // [problems, N] fp32, off (at least C + 1 words per problem) as the drawn indices [problems, C]
    int rc = kmeanspp(sizeof(T) == 2 ? MUSE_BF16 : MUSE_F32, X, problems, d.N, D, C, kind, seed, reinterpret_cast<float*>(perm),
                      off, status, st);
    if (rc != MUSE_OK) return rc;
    init_idx = off;
    init_mode = MUSE_INIT_INDICES;
  }
  if (init_mode != MUSE_INIT_CENTRES) {
    prof_mark("k_init_centres", st);
    k_init_centres<T><<<dim3(C, problems), 32, 0, st>>>(X, d.N, D, C, init_idx, init_mode, seed, kind, centres);
    MUSE_LAUNCH_OK();
  }
  const int total = problems * C;
  prof_mark("k_centre_norms", st);
  k_centre_norms<<<cdiv(total * 32, 256), 256, 0, st>>>(centres, total, D, cnorm);
  MUSE_LAUNCH_OK();
  const size_t smem = (size_t)((kAsgRows + kAsgCols) * (D + 4) + kAsgCols) * sizeof(float);
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_assign<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  for (int it = 0; it <= T_iters; ++it) {
    if (kTensor) {
      int rc = assign_tc(X, problems, d.N, D, C, centres, cnorm, chi, clo, assign, it == T_iters ? dist_out : nullptr, status, st);
      if (rc != MUSE_OK) return rc;
    } else {
      prof_mark("k_assign", st);
      k_assign<T, D><<<dim3(cdiv(d.N, kAsgRows), problems), kAsgThreads, smem, st>>>(X, d.N, C, centres, cnorm, assign,
                                                                                          it == T_iters ? dist_out : nullptr);
      MUSE_LAUNCH_OK();
    }
    if (it == T_iters) break;
    int rc = bucket_sort(0, assign, problems, d.N, C, d.S, d.Bs, kind, off, perm, scratch, st);
    if (rc != MUSE_OK) return rc;
    prof_mark("k_update", st);
    k_update<T, D><<<dim3(C, problems), kUpdThreads, 0, st>>>(X, d.N, C, d.S, kind, off, perm, centres, cnorm);
    MUSE_LAUNCH_OK();
  }
  return MUSE_OK;
}

size_t lloyd_ws_bytes(const Dims& d, int problems, int C, int) {
  Arena ar(nullptr);
  ar.take<int32_t>(64);
  ar.take<float>((size_t)problems * C);
  ar.take<int32_t>((size_t)problems * (C * d.S + 1));
  ar.take<int32_t>((size_t)problems * d.N);
  ar.take<int32_t>((size_t)problems * sort_ws_elems(d.N, C * d.S));
  ar.take<__nv_bfloat16>((size_t)problems * C * d.D);
  ar.take<__nv_bfloat16>((size_t)problems * C * d.D);
  return ar.used;
}

int lloyd(const Dims& d, int dtype, const void* X, int problems, int C, int kind, const int32_t* init_idx,
          int init_mode, uint64_t seed, int T, int32_t* assign, float* centres, void* ws, cudaStream_t st, float* dist_out) {
  if (dtype == MUSE_F32) {
    if (d.D == 64) return lloyd_t<float, 64>(d, (const float*)X, problems, C, kind, init_idx, init_mode, seed, T, assign, centres, ws, dist_out, st);
    return lloyd_t<float, 128>(d, (const float*)X, problems, C, kind, init_idx, init_mode, seed, T, assign, centres, ws, dist_out, st);
  }
  if (d.D == 64) return lloyd_t<__nv_bfloat16, 64>(d, (const __nv_bfloat16*)X, problems, C, kind, init_idx, init_mode, seed, T, assign, centres, ws, dist_out, st);
  return lloyd_t<__nv_bfloat16, 128>(d, (const __nv_bfloat16*)X, problems, C, kind, init_idx, init_mode, seed, T, assign, centres, ws, dist_out, st);
}

}  // namespace muse
