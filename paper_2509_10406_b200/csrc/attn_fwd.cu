// Forward attention stage (Algorithm 1, "Two-level retrieval + attention (per query)"):
// far-field scoring / top-m selection / approximate attention (Eq. 6), exact attention over the
// retrieved clusters via an inverse index, exact causal attention inside each spatial block,
// and the log-sum-exp merge ("Output merging").
#include "common.cuh"
#include "flash_core.cuh"

namespace muse {

int launch_scan(int32_t* cnt, int problems, int nkeys, int nchunks, int32_t* off, cudaStream_t st);
int local_fwd_tc(const Dims& d, const void* Q, const void* K, const void* V, float* o_loc, float* lse_loc, int* status,
                 cudaStream_t st);
bool far_fwd_tc_supported(const Dims& d, int dtype);
int far_fwd_tc(const Dims& d, const SummPtrs& sp, const void* Q, const int32_t* off_q, const int32_t* perm_q,
               const int32_t* sel_in, int32_t* sel_out, float* o_far, float* lse_far, int* status, cudaStream_t st);
int ret_fwd_tc(const Dims& d, const void* Q, const void* Kp, const void* Vp, const int32_t* off_k, const int32_t* goff,
               const int32_t* pairs, void* o_part, float* l_part, int* status, cudaStream_t st);
bool block_select_q_supported(const Dims& d, int dtype);
int block_select_q(const Dims& d, const void* Q, const int32_t* off_q, const int32_t* perm_q, const int32_t* sel, const SummPtrs& sp,
                   const int32_t* bsel_in, int32_t* bsel_out, float* o_near, float* lse_near, int* status, cudaStream_t st);
int block_select(const Dims& d, int dtype, const void* Q, const int32_t* off_q, const int32_t* perm_q, const int32_t* sel,
                 const SummPtrs& sp, const int32_t* bsel_in, int32_t* bsel_out, float* o_near, float* lse_near, cudaStream_t st);

// plane of a query = index of the accumulated-summary plane it reads: block - 1 when causal
// (block 0 sees no far field), 0 when non-causal.
__device__ __forceinline__ int query_plane(const Dims& d, int t) { return d.causal ? t / d.Bs - 1 : 0; }

// ---------------------------------------------------------------------------------------------
// Inverse index for retrieval (Section "Exact Retrieval and Local Attention"): for every
// (key cluster, plane) the list of (query, slot) pairs that retrieve it.  Group key = cluster * SB + plane,
// so that the pairs of one cluster over all planes form one run, ordered by plane.
// ---------------------------------------------------------------------------------------------
// Thread e handles (slot = e / N, query = e % N): the lanes of a warp are consecutive queries,
// which often retrieve the same cluster in the same slot, so equal keys are combined with a warp
// match and only one atomic per distinct key and warp reaches memory.
// With spatial block selection (bsel != nullptr, k2 > 0) a pair is (query, slot, chosen block e2), its group the
// BUCKET (cluster, chosen block) and its id (query * m + slot) * k2 + e2: the retrieval kernel then keeps one bucket
// resident and every pair of the group sees all of it.
__device__ __forceinline__ void ret_pair_key(const Dims& d, const int32_t* sel, const int32_t* bsel, int pq, long long e, int e2,
                                             int& key, int& pid) {
  key = -1; pid = 0;
  if (e >= (long long)d.N * d.m) return;
  const int t = (int)(e % d.N), k = (int)(e / d.N);
  const size_t slot = ((size_t)pq * d.N + t) * d.m + k;
  const int c = sel[slot];
  const int pl = query_plane(d, t);
  if (c < 0 || c >= d.Ck || pl < 0) return;                // entries outside [0, Ck) count as "none"
  if (bsel == nullptr) { key = c * d.SB + pl; pid = t * d.m + k; return; }
  const int bb = bsel[slot * d.k2 + e2];
  if (bb < 0 || bb > pl) return;                           // (block bb is earlier than the query's block pl + 1)
  key = c * d.SB + bb; pid = (t * d.m + k) * d.k2 + e2;
}

__global__ void k_ret_count(Dims d, const int32_t* __restrict__ sel, const int32_t* __restrict__ bsel, int32_t* __restrict__ cnt) {
  const int pq = blockIdx.y;
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int lane = threadIdx.x & 31;
  for (int e2 = 0; e2 < (bsel ? d.k2 : 1); ++e2) {
    int key, pid;
    ret_pair_key(d, sel, bsel, pq, e, e2, key, pid);
    const unsigned peers = __match_any_sync(0xffffffffu, key);
    if (key >= 0 && lane == __ffs(peers) - 1) atomicAdd(&cnt[(size_t)pq * d.SB * d.Ck + key], __popc(peers));
  }
}

__global__ void k_ret_fill(Dims d, const int32_t* __restrict__ sel, const int32_t* __restrict__ bsel, int32_t* __restrict__ cursor,
                           int32_t* __restrict__ pairs) {
  const int pq = blockIdx.y;
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int lane = threadIdx.x & 31;
  const size_t npairs = (size_t)d.N * d.m * (bsel ? d.k2 : 1);
  for (int e2 = 0; e2 < (bsel ? d.k2 : 1); ++e2) {
    int key, pid;
    ret_pair_key(d, sel, bsel, pq, e, e2, key, pid);
    const unsigned peers = __match_any_sync(0xffffffffu, key);
    const int leader = __ffs(peers) - 1;
    int base = 0;
    if (key >= 0 && lane == leader) base = atomicAdd(&cursor[(size_t)pq * d.SB * d.Ck + key], __popc(peers));
    base = __shfl_sync(0xffffffffu, base, leader);
    if (key >= 0 && MUSE_IN_RANGE(base + __popc(peers & ((1u << lane) - 1u)), npairs))
      pairs[(size_t)pq * npairs + base + __popc(peers & ((1u << lane) - 1u))] = pid;
  }
}

size_t ret_index_elems(const Dims& d) {
  // cursor [SB*Ck] + goff [SB*Ck+1] + pairs [N*m*max(k2,1)], each rounded up to 64 ints
  auto up = [](size_t x) { return (x + 63) & ~size_t(63); };
  return up((size_t)d.SB * d.Ck) + up((size_t)d.SB * d.Ck + 1) + up((size_t)d.N * d.m * (d.k2 > 0 ? d.k2 : 1));
}

int build_ret_index(const Dims& d, const int32_t* sel, const int32_t* bsel, int32_t* scratch, RetIndex* out, cudaStream_t st) {
  auto up = [](size_t x) { return (x + 63) & ~size_t(63); };
  const int pq = d.B * d.Hq, nkeys = d.SB * d.Ck;
  out->cursor = scratch;
  out->goff = scratch + (size_t)pq * up(nkeys);
  out->pairs = out->goff + (size_t)pq * up((size_t)nkeys + 1);
  // note: cursor / goff are indexed with their natural strides (nkeys, nkeys + 1); the padded
  // region sizes above only reserve space
  if (d.m == 0 || nkeys == 0) return MUSE_OK;
  prof_mark("memset", st);
  MUSE_CUDA_OK(cudaMemsetAsync(out->cursor, 0, (size_t)pq * nkeys * sizeof(int32_t), st));
  dim3 grid(cdiv((long long)d.N * d.m > 0 ? d.N * d.m : 1, 256), pq);
  prof_mark("k_ret_count", st);
  k_ret_count<<<grid, 256, 0, st>>>(d, sel, bsel, out->cursor);
  MUSE_LAUNCH_OK();
  int rc = launch_scan(out->cursor, pq, nkeys, 1, out->goff, st);
  if (rc != MUSE_OK) return rc;
  prof_mark("k_ret_fill", st);
  k_ret_fill<<<grid, 256, 0, st>>>(d, sel, bsel, out->cursor, out->pairs);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

// ---------------------------------------------------------------------------------------------
// Far field: scores against all accumulated cluster summaries, top-m, approximate attention
// over the rest.  One CTA per (query cluster i, plane, head) segment.
// ---------------------------------------------------------------------------------------------
constexpr int kFarThreads = 512, kFarJC = 64;

__host__ __device__ inline int far_rows(int Ck) { return Ck <= 1024 ? 32 : Ck <= 2048 ? 16 : 8; }

template <class T, int D>
__global__ void __launch_bounds__(kFarThreads)
k_far_fwd(Dims dm, const T* __restrict__ Q, const float* __restrict__ qbar, const int32_t* __restrict__ off_q,
          const int32_t* __restrict__ perm_q, SummPtrs sp, const int32_t* __restrict__ sel_in, int32_t* __restrict__ sel_out,
          float* __restrict__ o_far, float* __restrict__ lse_far) {
  constexpr int LD = D + 4;
  const int RT = far_rows(dm.Ck), Ck = dm.Ck, LDS_ = Ck + 4;
  extern __shared__ float smf[];
  float* sc = smf;                           // [RT][LDS_] scores, then probabilities
  float* ch = sc + RT * LDS_;                // [64][LD]  chunk of kappa / nu rows
  float* qr = ch + kFarJC * LD;              // [RT][LD]  residual queries (scaled)
  float* rinv = qr + RT * LD;                // [RT] 1 / far normaliser
  int32_t* rows = (int32_t*)(rinv + RT);     // [RT] token index of each row
  int32_t* selq = rows + RT;                 // [kMaxM] per-query-cluster selection
  const int i = blockIdx.x, pl = blockIdx.y, pq = blockIdx.z;
  const int blk = dm.causal ? pl + 1 : 0;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int32_t* oq = off_q + (size_t)pq * (dm.S * dm.Cq + 1) + (size_t)blk * dm.Cq + i;
  const int p0 = oq[0], p1 = oq[1];
  if (p0 >= p1) return;
  const size_t ent0 = (((size_t)pq * dm.SB + pl) * dm.Cq + i) * Ck;
  const float* mup = sp.mu + ent0;
  const T* Qp = Q + (size_t)pq * dm.N * D;
  const float* qb = qbar + ((size_t)pq * dm.Cq + i) * D;
  const int32_t* pm = perm_q + (size_t)pq * dm.N;
  const int m = dm.m;

  if (dm.sel_mode == MUSE_SEL_PER_QCLUSTER && sel_in == nullptr && m > 0) {
    // one selection for the whole segment: rank clusters by accumulated log-mass alone
    if (warp == 0) {
      float* tmp = sc;                        // scratch [Ck]
      for (int j = lane; j < Ck; j += 32) tmp[j] = mup[j];
      __syncwarp();
      for (int k = 0; k < m; ++k) {
        float bv = -INFINITY; int bi = 0x7fffffff;
        for (int j = lane; j < Ck; j += 32) { float v = tmp[j]; if (v > bv) { bv = v; bi = j; } }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          float ov = __shfl_xor_sync(0xffffffffu, bv, o); int oi = __shfl_xor_sync(0xffffffffu, bi, o);
          if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        if (lane == 0) selq[k] = bv == -INFINITY ? -1 : bi;
        if (bv != -INFINITY && (bi & 31) == lane) tmp[bi] = -INFINITY;
        __syncwarp();
      }
    }
    __syncthreads();
  }

  for (int r0 = p0; r0 < p1; r0 += RT) {
    const int n = min(RT, p1 - r0);
    __syncthreads();
    if (tid < RT) rows[tid] = tid < n ? pm[r0 + tid] : -1;
    for (int e = tid; e < RT * (D / 4); e += kFarThreads) {
      int r = e / (D / 4), q = e % (D / 4);
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (r < n) {
        float4 x = ld4(Qp + (size_t)pm[r0 + r] * D + q * 4), c = ld4(qb + q * 4);
        v = make_float4(dm.sigma * (x.x - c.x), dm.sigma * (x.y - c.y), dm.sigma * (x.z - c.z), dm.sigma * (x.w - c.w));
      }
      st4(qr + r * LD + q * 4, v);
    }
    // ---- A: score[r][j] = qres_r . kappa_j + mu_j  (Eq. 6)
    for (int j0 = 0; j0 < Ck; j0 += kFarJC) {
      __syncthreads();
      for (int e = tid; e < kFarJC * (D / 4); e += kFarThreads) {
        int r = e / (D / 4), q = e % (D / 4);
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (j0 + r < Ck) v = ld_kappa4<T>(sp, (ent0 + j0 + r) * D + q * 4);
        st4(ch + r * LD + q * 4, v);
      }
      __syncthreads();
      const int jj = tid & 63, rg = tid >> 6;           // 8 row groups
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
      for (int dd = 0; dd < D; dd += 4) {
        float4 kv = ld4(ch + jj * LD + dd);
#pragma unroll
        for (int a = 0; a < 4; ++a) {
          int r = rg + 8 * a;
          if (r < RT) {
            float4 qv = ld4(qr + r * LD + dd);
            acc[a] = fmaf(qv.x, kv.x, acc[a]); acc[a] = fmaf(qv.y, kv.y, acc[a]);
            acc[a] = fmaf(qv.z, kv.z, acc[a]); acc[a] = fmaf(qv.w, kv.w, acc[a]);
          }
        }
      }
      if (j0 + jj < Ck) {
        const float mj = mup[j0 + jj];
#pragma unroll
        for (int a = 0; a < 4; ++a) {
          int r = rg + 8 * a;
          if (r < RT) sc[r * LDS_ + j0 + jj] = mj == -INFINITY ? -INFINITY : acc[a] + mj;
        }
      }
    }
    __syncthreads();
    // ---- B: selection (one warp per row), C: softmax statistics of the remaining clusters
    for (int r = warp; r < n; r += kFarThreads / 32) {
      float* s = sc + r * LDS_;
      const int t = rows[r];
      int32_t* so = sel_out + ((size_t)pq * dm.N + t) * m;
      if (sel_in != nullptr) {
        const int32_t* si = sel_in + ((size_t)pq * dm.N + t) * m;
        for (int k = lane; k < m; k += 32) { int c = si[k]; c = (c >= 0 && c < Ck) ? c : -1; so[k] = c; if (c >= 0) s[c] = -INFINITY; }
      } else if (dm.sel_mode == MUSE_SEL_PER_QCLUSTER) {
        for (int k = lane; k < m; k += 32) { int c = selq[k]; so[k] = c; if (c >= 0) s[c] = -INFINITY; }
      } else {
        float lv = -INFINITY; int li = 0x7fffffff;
        for (int j = lane; j < Ck; j += 32) { float v = s[j]; if (v > lv) { lv = v; li = j; } }
        for (int k = 0; k < m; ++k) {
          float bv = lv; int bi = li;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, bv, o); int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
          }
          const bool any = bv != -INFINITY;
          if (lane == 0) so[k] = any ? bi : -1;
          if (any && (bi & 31) == lane) {
            s[bi] = -INFINITY;
            lv = -INFINITY; li = 0x7fffffff;
            for (int j = lane; j < Ck; j += 32) { float v = s[j]; if (v > lv) { lv = v; li = j; } }
          }
        }
      }
      __syncwarp();
      float mx = -INFINITY;
      for (int j = lane; j < Ck; j += 32) mx = fmaxf(mx, s[j]);
      mx = warp_max(mx);
      float sum = 0.f;
      if (mx != -INFINITY) {
        for (int j = lane; j < Ck; j += 32) { float p = expf(s[j] - mx); s[j] = p; sum += p; }
      } else {
        for (int j = lane; j < Ck; j += 32) s[j] = 0.f;
      }
      sum = warp_sum(sum);
      if (lane == 0) {
        rinv[r] = sum > 0.f ? 1.f / sum : 0.f;
        lse_far[(size_t)pq * dm.N + t] = sum > 0.f ? mx + logf(sum) : -INFINITY;
      }
    }
    for (int r = n + warp; r < RT; r += kFarThreads / 32)
      for (int j = lane; j < Ck; j += 32) sc[r * LDS_ + j] = 0.f;
    // ---- D: o_far = P . nu
    constexpr int NSL = D / 4, NRG = kFarThreads / NSL;      // dim slices, row groups
    const int slc = tid % NSL, rgd = tid / NSL;
    float4 oacc[2];
    oacc[0] = make_float4(0.f, 0.f, 0.f, 0.f); oacc[1] = oacc[0];
    for (int j0 = 0; j0 < Ck; j0 += kFarJC) {
      __syncthreads();
      for (int e = tid; e < kFarJC * (D / 4); e += kFarThreads) {
        int r = e / (D / 4), q = e % (D / 4);
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (j0 + r < Ck) v = ld_nu4<T>(sp, (ent0 + j0 + r) * D + q * 4);
        st4(ch + r * LD + q * 4, v);
      }
      __syncthreads();
      const int jn = min(kFarJC, Ck - j0);
#pragma unroll
      for (int a = 0; a < 2; ++a) {
        const int r = rgd + NRG * a;
        if (r < RT) {
          for (int j = 0; j < jn; ++j) {
            const float p = sc[r * LDS_ + j0 + j];
            float4 v = ld4(ch + j * LD + slc * 4);
            oacc[a].x = fmaf(p, v.x, oacc[a].x); oacc[a].y = fmaf(p, v.y, oacc[a].y);
            oacc[a].z = fmaf(p, v.z, oacc[a].z); oacc[a].w = fmaf(p, v.w, oacc[a].w);
          }
        }
      }
    }
#pragma unroll
    for (int a = 0; a < 2; ++a) {
      const int r = rgd + NRG * a;
      if (r < n) {
        const float iv = rinv[r];
        st4(o_far + ((size_t)pq * dm.N + rows[r]) * D + slc * 4,
            make_float4(oacc[a].x * iv, oacc[a].y * iv, oacc[a].z * iv, oacc[a].w * iv));
      }
    }
  }
}

static size_t far_smem(int Ck, int D) {
  const int RT = far_rows(Ck);
  return (size_t)(RT * (Ck + 4) + kFarJC * (D + 4) + RT * (D + 4) + RT) * sizeof(float) + (RT + kMaxM) * sizeof(int32_t);
}

// Queries that see no far field (block 0 when causal, or m > 0 rows never visited): defaults.
__global__ void k_far_defaults(Dims d, float* __restrict__ lse_far, int32_t* __restrict__ sel_out) {
  const int pq = blockIdx.y;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= d.N) return;
  if (query_plane(d, t) >= 0) return;
  lse_far[(size_t)pq * d.N + t] = -INFINITY;
  for (int k = 0; k < d.m; ++k) sel_out[((size_t)pq * d.N + t) * d.m + k] = -1;
}

// ---------------------------------------------------------------------------------------------
// Exact retrieval: one CTA per (key cluster j, plane, head) group; the group's queries attend
// the contiguous run of the cluster's keys in earlier blocks.  Each (query, slot) pair yields a
// normalised partial output and its log-sum-exp.
// ---------------------------------------------------------------------------------------------
template <class T, int D>
__global__ void __launch_bounds__(kFlashThreads)
k_ret_fwd(Dims dm, const T* __restrict__ Q, const T* __restrict__ Kp, const T* __restrict__ Vp,
          const int32_t* __restrict__ off_k, const int32_t* __restrict__ goff, const int32_t* __restrict__ pairs,
          float* __restrict__ o_part, float* __restrict__ l_part) {
  constexpr int LD = D + Pad<T>::v;
  extern __shared__ __align__(16) unsigned char smraw[];
  T* Qs = (T*)smraw; T* Ks = Qs + kTile * LD; T* Vs = Ks + kTile * LD;
  float* Ps = (float*)(Vs + kTile * LD);
  __shared__ int32_t pid_s[kTile];
  const int j = blockIdx.x, pl = blockIdx.y, pq = blockIdx.z;
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int nkeys = dm.SB * dm.Ck;
  const int32_t* go = goff + (size_t)pq * (nkeys + 1) + (size_t)j * dm.SB + pl;
  const int g0 = go[0], g1 = go[1];
  if (g0 >= g1) return;
  const int32_t* ok = off_k + (size_t)pk * (dm.Ck * dm.S + 1) + (size_t)j * dm.S;
  const int k0 = ok[0], k1 = ok[pl + 1];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const T* Qb = Q + (size_t)pq * dm.N * D;
  const T* Kb = Kp + (size_t)pk * dm.N * D;
  const T* Vb = Vp + (size_t)pk * dm.N * D;
  const int32_t* pr = pairs + (size_t)pq * dm.N * dm.m;
  for (int t0 = g0; t0 < g1; t0 += kTile) {
    const int nq = min(kTile, g1 - t0);
    __syncthreads();
    if (tid < kTile) pid_s[tid] = tid < nq ? pr[t0 + tid] : 0;
    __syncthreads();
    load_tile<T, D>(Qs, Qb, nq, [&](int r) { return pid_s[r] / dm.m; }, tid);
    float m_run[4], l_run[4], o[4][D / 64][4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      m_run[r] = -INFINITY; l_run[r] = 0.f;
#pragma unroll
      for (int k = 0; k < D / 64; ++k)
#pragma unroll
        for (int c = 0; c < 4; ++c) o[r][k][c] = 0.f;
    }
    for (int c0 = k0; c0 < k1; c0 += kTile) {
      const int nk = min(kTile, k1 - c0);
      __syncthreads();
      load_tile<T, D>(Ks, Kb, nk, [&](int r) { return c0 + r; }, tid);
      load_tile<T, D>(Vs, Vb, nk, [&](int r) { return c0 + r; }, tid);
      __syncthreads();
      float s[4][4];
      mm_nt<T, D>(Qs, Ks, s, ty, tx);
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) s[r][c] = (tx * 4 + c < nk) ? s[r][c] * dm.sigma : -INFINITY;
      online_softmax_step<D>(s, m_run, l_run, o, Ps, ty, tx);
      __syncthreads();
      mm_pn<T, D>(Ps, Vs, o, ty, tx);
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int row = ty * 4 + r;
      if (row < nq) {
        const size_t pid = (size_t)pq * dm.N * dm.m + pid_s[row];
        const float inv = l_run[r] > 0.f ? 1.f / l_run[r] : 0.f;
#pragma unroll
        for (int k = 0; k < D / 64; ++k)
          st4(o_part + pid * D + tx * 4 + 64 * k, make_float4(o[r][k][0] * inv, o[r][k][1] * inv, o[r][k][2] * inv, o[r][k][3] * inv));
        if (tx == 0) l_part[pid] = l_run[r] > 0.f ? m_run[r] + logf(l_run[r]) : -INFINITY;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Local attention: exact causal attention inside each spatial block ("Local attention").
// ---------------------------------------------------------------------------------------------
template <class T, int D>
__global__ void __launch_bounds__(kFlashThreads)
k_local_fwd(Dims dm, const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
            float* __restrict__ o_loc, float* __restrict__ lse_loc) {
  constexpr int LD = D + Pad<T>::v;
  extern __shared__ __align__(16) unsigned char smraw[];
  T* Qs = (T*)smraw; T* Ks = Qs + kTile * LD; T* Vs = Ks + kTile * LD;
  float* Ps = (float*)(Vs + kTile * LD);
  const int tiles_per_block = cdiv(dm.Bs, kTile);
  const int blk = blockIdx.x / tiles_per_block, qt = blockIdx.x % tiles_per_block, pq = blockIdx.y;
  const int b_ = pq / dm.Hq, h = pq % dm.Hq, pk = b_ * dm.Hkv + dm.hm.g[h];
  const int bstart = blk * dm.Bs, bend = bstart + dm.Bs;
  const int q0 = bstart + qt * kTile, nq = min(kTile, bend - q0);
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const T* Qb = Q + (size_t)pq * dm.N * D;
  const T* Kb = K + (size_t)pk * dm.N * D;
  const T* Vb = V + (size_t)pk * dm.N * D;
  load_tile<T, D>(Qs, Qb, nq, [&](int r) { return q0 + r; }, tid);
  float m_run[4], l_run[4], o[4][D / 64][4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    m_run[r] = -INFINITY; l_run[r] = 0.f;
#pragma unroll
    for (int k = 0; k < D / 64; ++k)
#pragma unroll
      for (int c = 0; c < 4; ++c) o[r][k][c] = 0.f;
  }
  const int kend = q0 + nq;                         // keys u <= t < kend
  for (int c0 = bstart; c0 < kend; c0 += kTile) {
    const int nk = min(kTile, kend - c0);
    __syncthreads();
    load_tile<T, D>(Ks, Kb, nk, [&](int r) { return c0 + r; }, tid);
    load_tile<T, D>(Vs, Vb, nk, [&](int r) { return c0 + r; }, tid);
    __syncthreads();
    float s[4][4];
    mm_nt<T, D>(Qs, Ks, s, ty, tx);
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int t = q0 + ty * 4 + r, u = c0 + tx * 4 + c;
        s[r][c] = (u <= t && u < kend) ? s[r][c] * dm.sigma : -INFINITY;
      }
    online_softmax_step<D>(s, m_run, l_run, o, Ps, ty, tx);
    __syncthreads();
    mm_pn<T, D>(Ps, Vs, o, ty, tx);
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int row = ty * 4 + r;
    if (row < nq) {
      const size_t t = (size_t)pq * dm.N + q0 + row;
      const float inv = 1.f / l_run[r];
#pragma unroll
      for (int k = 0; k < D / 64; ++k)
        st4(o_loc + t * D + tx * 4 + 64 * k, make_float4(o[r][k][0] * inv, o[r][k][1] * inv, o[r][k][2] * inv, o[r][k][3] * inv));
      if (tx == 0) lse_loc[t] = m_run[r] + logf(l_run[r]);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Merge: L = LSE over components, O = sum_c exp(lse_c - L) o_c.  One warp per query.
// ---------------------------------------------------------------------------------------------
template <class T, int D, class PT>      // PT: element type of the retrieval partial outputs
__global__ void k_merge(Dims dm, const float* __restrict__ o_far, const float* __restrict__ lse_far,
                        const float* __restrict__ o_loc, const float* __restrict__ lse_loc,
                        const PT* __restrict__ o_part, const float* __restrict__ l_part,
                        const float* __restrict__ o_near, const float* __restrict__ lse_near,
                        const int32_t* __restrict__ sel, const int32_t* __restrict__ bsel, T* __restrict__ O, float* __restrict__ LSE) {
  const int pq = blockIdx.y;
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (t >= dm.N) return;
  const size_t row = (size_t)pq * dm.N + t;
  const int pl = query_plane(dm, t);
  const bool far_ok = pl >= 0 && dm.SB > 0;
  const float lf = far_ok ? lse_far[row] : -INFINITY;
  const float ll = dm.causal ? lse_loc[row] : -INFINITY;
  // near field (component 2 of the merge): non-retrieved earlier blocks of the selected clusters; empty unless k2 > 0
  const float ln = (far_ok && lse_near != nullptr) ? lse_near[row] : -INFINITY;
  float mx = fmaxf(fmaxf(lf, ll), ln);
  // retrieved partial results of this query: one per slot, or one per (slot, chosen block) with spatial block selection
  const int kk = bsel != nullptr ? dm.k2 : 1, m = dm.m * kk;
  float lp_mine[2] = {-INFINITY, -INFINITY};        // partials lane, lane + 32
  if (far_ok) {
#pragma unroll
    for (int a = 0; a < 2; ++a) {
      const int s = lane + 32 * a;
      if (s < m && sel[row * dm.m + s / kk] >= 0 && (bsel == nullptr || bsel[row * m + s] >= 0)) lp_mine[a] = l_part[row * m + s];
      mx = fmaxf(mx, lp_mine[a]);
    }
  }
  mx = warp_max(mx);
  float tot = 0.f;
#pragma unroll
  for (int a = 0; a < 2; ++a) tot += lp_mine[a] == -INFINITY ? 0.f : expf(lp_mine[a] - mx);
  tot = warp_sum(tot);
  const float wf = lf == -INFINITY ? 0.f : expf(lf - mx), wl = ll == -INFINITY ? 0.f : expf(ll - mx);
  const float wn = ln == -INFINITY ? 0.f : expf(ln - mx);
  tot += wf + wl + wn;
  const float inv = 1.f / tot;
  // lane owns EPL consecutive output dims: one vector load per input row and lane
  constexpr int EPL = D / 32;
  const int dd = lane * EPL;
  float acc[EPL];
#pragma unroll
  for (int k = 0; k < EPL; ++k) acc[k] = 0.f;
  if (wf > 0.f) {
    float x[EPL];
    ldv<EPL>(o_far + row * D + dd, x);
#pragma unroll
    for (int k = 0; k < EPL; ++k) acc[k] = fmaf(wf, x[k], acc[k]);
  }
  if (wl > 0.f) {
    float x[EPL];
    ldv<EPL>(o_loc + row * D + dd, x);
#pragma unroll
    for (int k = 0; k < EPL; ++k) acc[k] = fmaf(wl, x[k], acc[k]);
  }
  if (wn > 0.f) {
    float x[EPL];
    ldv<EPL>(o_near + row * D + dd, x);
#pragma unroll
    for (int k = 0; k < EPL; ++k) acc[k] = fmaf(wn, x[k], acc[k]);
  }
  // retrieved slots four at a time, so that four independent row loads are in flight
  for (int s0 = 0; s0 < m; s0 += 4) {
    float w[4], x[4][EPL];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int s = s0 + u;
      const float lp = s < m ? __shfl_sync(0xffffffffu, lp_mine[s >> 5], s & 31) : -INFINITY;
      w[u] = lp == -INFINITY ? 0.f : expf(lp - mx);
      if (w[u] > 0.f) ldv<EPL>(o_part + (row * m + s) * D + dd, x[u]);
      else {
#pragma unroll
        for (int k = 0; k < EPL; ++k) x[u][k] = 0.f;
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int k = 0; k < EPL; ++k) acc[k] = fmaf(w[u], x[u][k], acc[k]);
  }
#pragma unroll
  for (int k = 0; k < EPL; ++k) acc[k] *= inv;
  stv<EPL>(O + row * D + dd, acc);
  if (lane == 0) LSE[row] = mx + logf(tot);
}

// ---------------------------------------------------------------------------------------------
template <class T> constexpr bool kTensorT() { return sizeof(T) == 2; }

struct FwdWs { int32_t *status, *off_q, *perm_q, *sort_scratch, *ret_scratch, *sel_tmp, *bsel_tmp; float *o_far, *lse_far, *o_loc, *lse_loc, *o_part, *l_part, *o_near, *lse_near, *csub; };

static FwdWs fwd_ws(const Dims& d, Arena& ar) {
  FwdWs w;
  const size_t pq = (size_t)d.B * d.Hq;
  w.status = ar.take<int32_t>(64);          // ws[0]: non-zero if a bounded device-side wait gave up
  w.off_q = ar.take<int32_t>(pq * (d.S * d.Cq + 1));
  w.perm_q = ar.take<int32_t>(pq * d.N);
  w.sort_scratch = ar.take<int32_t>(pq * sort_ws_elems(d.N, d.Cq * d.S));
  w.ret_scratch = ar.take<int32_t>(pq * ret_index_elems(d));
  w.sel_tmp = ar.take<int32_t>(pq * d.N * (d.m > 0 ? d.m : 1));
  w.o_far = ar.take<float>(pq * d.N * d.D);
  w.lse_far = ar.take<float>(pq * d.N);
  w.o_loc = ar.take<float>(pq * d.N * d.D);
  w.lse_loc = ar.take<float>(pq * d.N);
  const size_t mk = (size_t)d.m * (d.k2 > 0 ? d.k2 : 1);      // partial results per query
  w.o_part = ar.take<float>(pq * d.N * mk * d.D);
  w.l_part = ar.take<float>(pq * d.N * mk);
  const bool two_level = d.k2 > 0 && d.causal;
  w.bsel_tmp = ar.take<int32_t>(two_level ? pq * d.N * d.m * d.k2 : 0);
  w.o_near = ar.take<float>(two_level ? pq * d.N * d.D : 0);
  w.lse_near = ar.take<float>(two_level ? pq * d.N : 0);
  w.csub = ar.take<float>(d.dipole && d.m > 0 && d.SB > 0 ? pq * d.N * d.D : 0);
  return w;
}

size_t attn_fwd_ws_bytes(const Dims& d, int) { Arena ar(nullptr); fwd_ws(d, ar); return ar.used; }

template <class T, int D>
static int attn_fwd_t(const Dims& d, const T* Q, const T* K, const T* V, const int32_t* assign_q,
                      const float* qbar, const int32_t* off_k, const int32_t* perm_k, const void* summaries,
                      const int32_t* sel_in, const int32_t* bsel_in, T* O, float* LSE, int32_t* sel_out, int32_t* bsel_out, void* ws,
                      int dtype, cudaStream_t st) {
  Arena ar(ws);
  FwdWs w = fwd_ws(d, ar);
  const int pq = d.B * d.Hq;
  SummLayout L = summ_layout(d, dtype);
  const char* base = (const char*)summaries;
  const T* Kp = (const T*)(base + L.Kp); const T* Vp = (const T*)(base + L.Vp);
  int32_t* sel = sel_out ? sel_out : w.sel_tmp;
  const bool two_level = d.k2 > 0 && d.causal && d.m > 0;
  int32_t* bsel = two_level ? (bsel_out ? bsel_out : w.bsel_tmp) : nullptr;
  if (two_level && !kTensorT<T>()) return MUSE_ERR_UNSUPPORTED;   // spatial block selection is built on the bf16 retrieval kernel
  const size_t fl_smem = 3 * tile_bytes<T, D>() + ptile_bytes();
  constexpr bool kTensor = sizeof(T) == 2;      // bf16 mode runs the exact-attention parts on tcgen05
  // local attention
  if (d.causal && kTensor) {
    int rc = local_fwd_tc(d, Q, K, V, w.o_loc, w.lse_loc, w.status, st);
    if (rc != MUSE_OK) return rc;
  } else if (d.causal) {
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_local_fwd<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fl_smem));
    prof_mark("k_local_fwd", st);
    k_local_fwd<T, D><<<dim3(d.S * cdiv(d.Bs, kTile), pq), kFlashThreads, fl_smem, st>>>(d, Q, K, V, w.o_loc, w.lse_loc);
    MUSE_LAUNCH_OK();
  }
  prof_mark("k_far_defaults", st);
  k_far_defaults<<<dim3(cdiv(d.N, 256), pq), 256, 0, st>>>(d, w.lse_far, sel);
  MUSE_LAUNCH_OK();
  if (d.SB > 0) {
    int rc = bucket_sort(0, assign_q, pq, d.N, d.Cq, d.S, d.Bs, 0, w.off_q, w.perm_q, w.sort_scratch, st);
    if (rc != MUSE_OK) return rc;
    if (far_fwd_tc_supported(d, dtype) && !path_forced(kForceFarSimt)) {
      rc = far_fwd_tc(d, summ_ptrs(L, base), Q, w.off_q, w.perm_q, sel_in, sel, w.o_far, w.lse_far, w.status, st);
      if (rc != MUSE_OK) return rc;
    } else {
      const size_t fs = far_smem(d.Ck, D);
      MUSE_CUDA_OK(cudaFuncSetAttribute(k_far_fwd<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fs));
      prof_mark("k_far_fwd", st);
      k_far_fwd<T, D><<<dim3(d.Cq, d.SB, pq), kFarThreads, fs, st>>>(
          d, Q, qbar, w.off_q, w.perm_q, summ_ptrs(L, base), sel_in, sel, w.o_far, w.lse_far);
      MUSE_LAUNCH_OK();
    }
    if (two_level) {
      // second level: the k2 best earlier blocks of every selected cluster, and the near field of the others
      if (block_select_q_supported(d, dtype) && !path_forced(kForceBlockSelectWarp))
        rc = block_select_q(d, Q, w.off_q, w.perm_q, sel, summ_ptrs_blk(L, base), bsel_in, bsel, w.o_near, w.lse_near, w.status, st);
      else
      rc = block_select(d, dtype, Q, w.off_q, w.perm_q, sel, summ_ptrs_blk(L, base), bsel_in, bsel, w.o_near, w.lse_near, st);
      if (rc != MUSE_OK) return rc;
    }
    if (d.dipole && d.m == 0) {
      rc = dipole_apply(d, dtype, Q, qbar, assign_q, w.off_q, w.perm_q, dipole_ptrs(L, base), w.lse_far, nullptr, nullptr, nullptr,
                        nullptr, w.o_far, nullptr, nullptr, w.status, st);
      if (rc != MUSE_OK) return rc;
    }
    if (d.m > 0) {
      RetIndex ri;
      rc = build_ret_index(d, sel, bsel, w.ret_scratch, &ri, st);
      if (rc != MUSE_OK) return rc;
      if (d.dipole) {
        rc = dipole_apply(d, dtype, Q, qbar, assign_q, w.off_q, w.perm_q, dipole_ptrs(L, base), w.lse_far, sel, ri.goff, ri.pairs,
                          w.csub, w.o_far, nullptr, nullptr, w.status, st);
        if (rc != MUSE_OK) return rc;
      }
      if (kTensor) {
        rc = ret_fwd_tc(d, Q, Kp, Vp, off_k, ri.goff, ri.pairs, w.o_part, w.l_part, w.status, st);
        if (rc != MUSE_OK) return rc;
      } else {
        MUSE_CUDA_OK(cudaFuncSetAttribute(k_ret_fwd<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fl_smem));
        prof_mark("k_ret_fwd", st);
        k_ret_fwd<T, D><<<dim3(d.Ck, d.SB, pq), kFlashThreads, fl_smem, st>>>(d, Q, Kp, Vp, off_k, ri.goff, ri.pairs, w.o_part, w.l_part);
        MUSE_LAUNCH_OK();
      }
    }
  }
  prof_mark("k_merge", st);
  if (kTensor)
    k_merge<T, D, __nv_bfloat16><<<dim3(cdiv(d.N, 8), pq), 256, 0, st>>>(d, w.o_far, w.lse_far, w.o_loc, w.lse_loc,
                                                                       (const __nv_bfloat16*)w.o_part, w.l_part, two_level ? w.o_near : nullptr,
                                                                       two_level ? w.lse_near : nullptr, sel, bsel, O, LSE);
  else
    k_merge<T, D, float><<<dim3(cdiv(d.N, 8), pq), 256, 0, st>>>(d, w.o_far, w.lse_far, w.o_loc, w.lse_loc, w.o_part, w.l_part, nullptr, nullptr,
                                                               sel, nullptr, O, LSE);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

// The far field alone, with the selection given (the backward of the dipole correction needs each query's far
// log-sum-exp again, which the forward does not hand over): lse_far [B*Hq*N], o_far [B*Hq*N*D] fp32, sel_tmp
// [B*Hq*N*m] scratch that receives a copy of the selection.
template <class T, int D>
static int far_fwd_again_t(const Dims& d, int dtype, const T* Q, const float* qbar, const int32_t* off_q, const int32_t* perm_q,
                           const SummPtrs& sp, const int32_t* sel_in, int32_t* sel_tmp, float* o_far, float* lse_far, int* status,
                           cudaStream_t st) {
  const int pq = d.B * d.Hq;
  prof_mark("k_far_defaults", st);
  k_far_defaults<<<dim3(cdiv(d.N, 256), pq), 256, 0, st>>>(d, lse_far, sel_tmp);
  MUSE_LAUNCH_OK();
  if (d.SB == 0) return MUSE_OK;
  if (far_fwd_tc_supported(d, dtype) && !path_forced(kForceFarSimt))
    return far_fwd_tc(d, sp, Q, off_q, perm_q, sel_in, sel_tmp, o_far, lse_far, status, st);
  const size_t fs = far_smem(d.Ck, D);
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_far_fwd<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fs));
  prof_mark("k_far_fwd", st);
  k_far_fwd<T, D><<<dim3(d.Cq, d.SB, pq), kFarThreads, fs, st>>>(d, Q, qbar, off_q, perm_q, sp, sel_in, sel_tmp, o_far, lse_far);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

int far_fwd_again(const Dims& d, int dtype, const void* Q, const float* qbar, const int32_t* off_q, const int32_t* perm_q,
                  const SummPtrs& sp, const int32_t* sel_in, int32_t* sel_tmp, float* o_far, float* lse_far, int* status,
                  cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  if (dtype == MUSE_F32) {
    if (d.D == 64) return far_fwd_again_t<float, 64>(d, dtype, (const float*)Q, qbar, off_q, perm_q, sp, sel_in, sel_tmp, o_far, lse_far, status, st);
    return far_fwd_again_t<float, 128>(d, dtype, (const float*)Q, qbar, off_q, perm_q, sp, sel_in, sel_tmp, o_far, lse_far, status, st);
  }
  if (d.D == 64) return far_fwd_again_t<bf, 64>(d, dtype, (const bf*)Q, qbar, off_q, perm_q, sp, sel_in, sel_tmp, o_far, lse_far, status, st);
  return far_fwd_again_t<bf, 128>(d, dtype, (const bf*)Q, qbar, off_q, perm_q, sp, sel_in, sel_tmp, o_far, lse_far, status, st);
}

int attn_fwd(const Dims& d, int dtype, const void* Q, const void* K, const void* V, const int32_t* assign_q,
             const float* qbar, const int32_t* off_k, const int32_t* perm_k, const void* summaries,
             const int32_t* sel_in, const int32_t* bsel_in, void* O, float* LSE, int32_t* sel_out, int32_t* bsel_out, void* ws,
             cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  if (dtype == MUSE_F32) {
    if (d.D == 64) return attn_fwd_t<float, 64>(d, (const float*)Q, (const float*)K, (const float*)V, assign_q, qbar, off_k, perm_k, summaries, sel_in, bsel_in, (float*)O, LSE, sel_out, bsel_out, ws, dtype, st);
    return attn_fwd_t<float, 128>(d, (const float*)Q, (const float*)K, (const float*)V, assign_q, qbar, off_k, perm_k, summaries, sel_in, bsel_in, (float*)O, LSE, sel_out, bsel_out, ws, dtype, st);
  }
  if (d.D == 64) return attn_fwd_t<bf, 64>(d, (const bf*)Q, (const bf*)K, (const bf*)V, assign_q, qbar, off_k, perm_k, summaries, sel_in, bsel_in, (bf*)O, LSE, sel_out, bsel_out, ws, dtype, st);
  return attn_fwd_t<bf, 128>(d, (const bf*)Q, (const bf*)K, (const bf*)V, assign_q, qbar, off_k, perm_k, summaries, sel_in, bsel_in, (bf*)O, LSE, sel_out, bsel_out, ws, dtype, st);
}

}  // namespace muse
