// The paper's own clustering (Appendix "Clustering Details").
//
// "Centroid Computation": one pass of streaming mini-batch k-means.  The N vectors of a problem (one head,
// queries or keys) are visited in the order of the seeded shuffle, 64 at a time; a minibatch is assigned to
// the nearest current centroids t_j / c_j, then its vectors update their centroids one after the other,
// t_j <- beta t_j + x, c_j <- beta c_j + 1.  Centroid r starts as the r-th strided sample of the shuffled
// sequence with t = x, c = 1.  The pass is a chain of N / 64 dependent steps, so a problem is owned by one
// thread-block cluster (its CTAs split the centroids) and the problems run side by side; a step is a
// 64 x C x D distance product (fp32 FFMA on shared-memory tiles of 64 vectors x 64 centroids, 4 x 2 results
// per thread), an arg-min with ties to the lower index, and the update, in which one warp per touched centroid
// replays that centroid's vectors of the minibatch in stream order - exactly the sequential recurrence,
// parallel over centroids.  The next minibatch's rows are fetched while the current one is worked on.
//
// "Balanced Assignment": independently in each spatial block every vector goes to its nearest centroid
// subject to a bucket size of at most cap = ceil(factor * B / K).  Step 1 (data parallel): the nearest
// centroid of every vector (the assignment kernels of the Lloyd path), a stable (block, cluster) counting
// sort, and each vector's rank inside its bucket in position order; the first cap of a bucket keep it.
// Step 2: one CTA per (problem, block) walks the displaced vectors in position order and gives each the
// nearest centroid whose bucket still has room: a masked arg-min over one row of the distance matrix that the
// step-1 assignment wrote.  Where the cap rarely binds (the paper's regime: 128 clusters, cap 256 per block)
// step 2 is short; where it binds for most vectors the sequential walk dominates the stage.
#include <cooperative_groups.h>
#include "common.cuh"
#include "feistel.cuh"
#include "tc05.cuh"

namespace cg = cooperative_groups;

namespace muse {

constexpr int kSkThreads = 512, kSkBatch = 64, kSkChunk = 64, kSkMaxCluster = 8;

template <int D> constexpr size_t stream_smem_bytes(int C) {
  return (size_t)(2 * kSkBatch * (D + 4) + 2 * C + kSkBatch * 32 + 2 * kSkMaxCluster * kSkBatch) * sizeof(float) +
         (size_t)(kSkBatch * 32 + 2 * kSkMaxCluster * kSkBatch + kSkBatch) * sizeof(int);
}

// One problem = one thread-block cluster of CS CTAs (CS = 1, 2, 4 or 8).  Every CTA holds the whole minibatch but
// only its own slice of the centroids: it computes the distances to that slice, the CTAs exchange their 64 best
// (distance, centroid) pairs through distributed shared memory, every CTA takes the overall arg-min, and each
// updates the centroids it owns.  A centroid row is only ever read and written by its owner, so the only traffic
// between the CTAs is the exchange, ordered by one hardware cluster barrier per minibatch.
template <class T, int D>
__global__ void __launch_bounds__(kSkThreads)
k_stream_kmeans(const T* __restrict__ X, int N, int C, uint64_t seed, int kind, float beta, int first_batch, int n_batches,
                float* __restrict__ totals, float* __restrict__ counts, float* __restrict__ centres,
                int32_t* __restrict__ assign_stream) {
  constexpr int LD = D + 4, EPL = D / 32, NW = kSkThreads / 32, PPW = kSkBatch / NW;
  constexpr int RV = D / 32;                   // 16-byte-of-fp32 groups of a row per loading thread (8 threads per row)
  cg::cluster_group cluster = cg::this_cluster();
  const int CS = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  extern __shared__ __align__(16) float sk_smem[];
  float* Xs = sk_smem;                         // [64][LD]  the minibatch
  float* Ct = Xs + kSkBatch * LD;              // [64][LD]  a chunk of centroids
  float* cn = Ct + kSkChunk * LD;              // [C] squared norms of the current centroids (own slice in use)
  float* cc = cn + C;                          // [C] counts c_j (own slice in use)
  float* bd = cc + C;                          // [64][32] per-thread best distances
  float* exd = bd + kSkBatch * 32;             // [2][CS max][64] exchanged best distances, double-buffered by step parity
  int* bi = reinterpret_cast<int*>(exd + 2 * kSkMaxCluster * kSkBatch);   // [64][32] centroids of bd
  int* exi = bi + kSkBatch * 32;               // [2][CS max][64] exchanged best centroids
  int* as = exi + 2 * kSkMaxCluster * kSkBatch;   // [64] the minibatch's assignments
  const int prob = blockIdx.x / CS, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const T* Xp = X + (size_t)prob * N * D;
  float* Tp = totals + (size_t)prob * C * D;
  float* Cp = centres + (size_t)prob * C * D;
  float* cntp = counts + (size_t)prob * C;
  const uint64_t strm = (uint64_t)prob * 2 + kind;
  const int per = ((C + CS - 1) / CS + 1) & ~1;                     // centroids per CTA (even: a thread takes two)
  const int j0 = min(C, rank * per), j1 = min(C, j0 + per);

  // state before the first minibatch of this call: the strided start (t = x, c = 1), or the caller's (t, c)
  for (int j = j0 + warp; j < j1; j += NW) {
    float t[EPL], c;
    if (first_batch == 0) {
      const int u = feistel_permute(j * (N / C), N, seed, strm);
      ldv<EPL>(Xp + (size_t)u * D + lane * EPL, t);
      c = 1.f;
      stv<EPL>(Tp + (size_t)j * D + lane * EPL, t);
    } else {
      ldv<EPL>(Tp + (size_t)j * D + lane * EPL, t);
      c = cntp[j];
    }
    float n2 = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) { t[e] = t[e] / c; n2 = fmaf(t[e], t[e], n2); }
    stv<EPL>(Cp + (size_t)j * D + lane * EPL, t);
    n2 = warp_sum(n2);
    if (lane == 0) { cn[j] = n2; cc[j] = c; }
  }

  // rows of the next minibatch travel in registers while the current one is worked on: thread = (row, eighth of the row)
  const int lr = tid >> 3, lq = tid & 7;
  float4 xr[RV];
  auto fetch = [&](int s) {
    const int pos = s * kSkBatch + lr;
    const int u = pos < N ? feistel_permute(pos, N, seed, strm) : -1;
#pragma unroll
    for (int v = 0; v < RV; ++v)
      xr[v] = (u >= 0 && MUSE_IN_RANGE(u, N)) ? ld4(Xp + (size_t)u * D + (lq * RV + v) * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
  };
  if (n_batches > 0) fetch(first_batch);
  cluster.sync();                              // every CTA of the problem is running before any of them writes into another's shared memory

  // Thread tile: 4 vectors x 2 centroids of a 64 x 64 chunk.  A warp covers 8 vector rows x 4 centroid pairs at a
  // time, so that a shared-memory load of the warp touches 8 (vectors) or 4 (centroids) distinct rows: one wavefront each.
  const int pi = (warp & 1) * 32 + (lane & 7), ci = (warp >> 1) * 4 + (lane >> 3);   // vectors pi + 8 i; centroids 2 ci, 2 ci + 1
  for (int s = first_batch; s < first_batch + n_batches; ++s) {
    const int nb = min(kSkBatch, N - s * kSkBatch), par = s & 1;
#pragma unroll
    for (int v = 0; v < RV; ++v) *reinterpret_cast<float4*>(Xs + lr * LD + (lq * RV + v) * 4) = xr[v];
    if (s + 1 < first_batch + n_batches) fetch(s + 1);
    float best[4];
    int bidx[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) { best[i] = INFINITY; bidx[i] = 0x7fffffff; }
    for (int c0 = j0; c0 < j1; c0 += kSkChunk) {
      __syncthreads();                         // the minibatch is in place / the previous chunk has been used
      for (int e = tid; e < kSkChunk * (D / 4); e += kSkThreads) {
        const int r = e / (D / 4), q = e % (D / 4);
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c0 + r < j1) v = *reinterpret_cast<const float4*>(Cp + (size_t)(c0 + r) * D + q * 4);
        *reinterpret_cast<float4*>(Ct + r * LD + q * 4) = v;
      }
      __syncthreads();
      float acc[4][2];
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[i][0] = acc[i][1] = 0.f;
#pragma unroll 4
      for (int d4 = 0; d4 < D; d4 += 4) {
        const float4 a0 = *reinterpret_cast<const float4*>(Ct + (2 * ci) * LD + d4);
        const float4 a1 = *reinterpret_cast<const float4*>(Ct + (2 * ci + 1) * LD + d4);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float4 x = *reinterpret_cast<const float4*>(Xs + (pi + 8 * i) * LD + d4);
          acc[i][0] = fmaf(x.x, a0.x, fmaf(x.y, a0.y, fmaf(x.z, a0.z, fmaf(x.w, a0.w, acc[i][0]))));
          acc[i][1] = fmaf(x.x, a1.x, fmaf(x.y, a1.y, fmaf(x.z, a1.z, fmaf(x.w, a1.w, acc[i][1]))));
        }
      }
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const int j = c0 + 2 * ci + k;
        if (j < j1) {
          const float n2 = cn[j];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float dist = fmaf(-2.f, acc[i][k], n2);           // |c|^2 - 2 x.c: |x|^2 is the same for every centroid
            if (dist < best[i]) { best[i] = dist; bidx[i] = j; }    // (ascending j: ties stay with the lower index)
          }
        }
      }
    }
    if (j0 >= j1) __syncthreads();             // (a CTA without centroids still has to have the minibatch in place)
#pragma unroll
    for (int i = 0; i < 4; ++i) { bd[(pi + 8 * i) * 32 + ci] = best[i]; bi[(pi + 8 * i) * 32 + ci] = bidx[i]; }
    __syncthreads();
    for (int k = 0; k < PPW; ++k) {            // a warp reduces four vectors' 32 candidates and posts the result to every CTA
      const int p = warp * PPW + k;
      float dv = bd[p * 32 + lane];
      int iv = bi[p * 32 + lane];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float od = __shfl_xor_sync(0xffffffffu, dv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, iv, o);
        if (od < dv || (od == dv && oi < iv)) { dv = od; iv = oi; }
      }
      if (lane < CS) {
        *cluster.map_shared_rank(exd + (par * kSkMaxCluster + rank) * kSkBatch + p, lane) = dv;
        *cluster.map_shared_rank(exi + (par * kSkMaxCluster + rank) * kSkBatch + p, lane) = iv;
      }
    }
    cluster.sync();                            // every CTA's candidates have arrived (and the previous step's have been read)
    if (tid < kSkBatch) {
      float dv = exd[(par * kSkMaxCluster) * kSkBatch + tid];
      int iv = exi[(par * kSkMaxCluster) * kSkBatch + tid];
      for (int r = 1; r < CS; ++r) {
        const float od = exd[(par * kSkMaxCluster + r) * kSkBatch + tid];
        const int oi = exi[(par * kSkMaxCluster + r) * kSkBatch + tid];
        if (od < dv || (od == dv && oi < iv)) { dv = od; iv = oi; }
      }
      as[tid] = (tid < nb && (unsigned)iv < (unsigned)C) ? iv : (tid < nb ? 0 : -1);   // (a NaN row goes to centroid 0)
    }
    __syncthreads();
    // update: the first vector of the minibatch on a centroid ("leader") replays all of that centroid's vectors in order
    const int a_lo = as[lane], a_hi = as[lane + 32];                // the minibatch's assignments, two per lane
    for (int k = 0; k < PPW; ++k) {
      const int p = warp + NW * k;
      const int j = as[p];
      if (j < j0 || j >= j1) continue;                              // (warp-uniform: shared-memory values) not this CTA's centroid
      // the vectors of the minibatch on centroid j, as a 64-bit mask in stream order
      const unsigned long long mem = (unsigned long long)__ballot_sync(0xffffffffu, a_lo == j) |
                                     ((unsigned long long)__ballot_sync(0xffffffffu, a_hi == j) << 32);
      if (__ffsll((long long)mem) - 1 != p) continue;               // not the centroid's first vector
      float t[EPL], c = cc[j];
      ldv<EPL>(Tp + (size_t)j * D + lane * EPL, t);
      for (unsigned long long rest = mem; rest != 0ull; rest &= rest - 1ull) {
        const int q = __ffsll((long long)rest) - 1;
#pragma unroll
        for (int e = 0; e < EPL; ++e) t[e] = fmaf(beta, t[e], Xs[q * LD + lane * EPL + e]);
        c = fmaf(beta, c, 1.f);
      }
      stv<EPL>(Tp + (size_t)j * D + lane * EPL, t);
      float n2 = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) { t[e] = t[e] / c; n2 = fmaf(t[e], t[e], n2); }
      stv<EPL>(Cp + (size_t)j * D + lane * EPL, t);
      n2 = warp_sum(n2);
      if (lane == 0) { cn[j] = n2; cc[j] = c; }
    }
    if (rank == 0 && assign_stream != nullptr && tid < nb) assign_stream[(size_t)prob * N + (size_t)s * kSkBatch + tid] = as[tid];
    __syncthreads();                           // the centroid rows written above are read by every thread in the next step
  }
  for (int j = j0 + tid; j < j1; j += kSkThreads) cntp[j] = cc[j];
  cluster.sync();                              // no CTA leaves while another may still write into its shared memory
}

// ---------------------------------------------------------------------------------------------
// The same pass with the distance product on the tensor cores (bf16 inputs, C <= 256 centroids per CTA).
// A CTA keeps ITS centroids resident in shared memory as bf16 hi + lo tiles ([128 centroids][D], 128-byte
// swizzle, K-major) and rewrites the rows it updates in place; the minibatch is the A operand ([128][D] with
// rows 64..127 zero), the product x.c for 64 vectors x 128 centroids per tile lands in tensor memory
// (tcgen05.mma, M = 128, N = 128, hi then lo accumulated), four warps read it back and take the arg-min of
// |c|^2 - 2 x.c.  Exchange between the CTAs of a problem and the update are as in the kernel above.
// ---------------------------------------------------------------------------------------------
constexpr int kStThreads = 256;

template <int D> constexpr size_t stream_tc_smem_bytes(int NT) { return 1024 + (size_t)(1 + 2 * NT) * 128 * D * 2 + (size_t)2 * NT * 128 * sizeof(float); }

template <int D>
__global__ void __launch_bounds__(kStThreads, 1)
k_stream_kmeans_tc(const __nv_bfloat16* __restrict__ X, int N, int C, uint64_t seed, int kind, float beta, int first_batch,
                   int n_batches, float* __restrict__ totals, float* __restrict__ counts, float* __restrict__ centres,
                   int32_t* __restrict__ assign_stream, int NT, int* __restrict__ status) {
  typedef __nv_bfloat16 bf16;
  constexpr int EPL = D / 32, NW = kStThreads / 32, PPW = kSkBatch / NW, CPR = D / 8, RV = CPR / 4, kTile = 128 * D * 2;
  cg::cluster_group cluster = cg::this_cluster();
  const int CS = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  extern __shared__ __align__(1024) unsigned char st_raw[];
  __shared__ uint64_t sdone;
  __shared__ uint32_t tbase_s;
  __shared__ float exd[2][kSkMaxCluster][kSkBatch], rd[kSkBatch];
  __shared__ int exi[2][kSkMaxCluster][kSkBatch], ri[kSkBatch], as[kSkBatch];
  unsigned char* sm = st_raw + ((1024u - (tc::smem_u32(st_raw) & 1023u)) & 1023u);
  unsigned char* Xs = sm;                                    // [128][D] bf16: the minibatch in rows 0..63
  unsigned char* Chi = Xs + kTile;                           // NT tiles [128][D] bf16: high parts of this CTA's centroids
  unsigned char* Clo = Chi + (size_t)NT * kTile;             // ... and low parts
  float* cn = reinterpret_cast<float*>(Clo + (size_t)NT * kTile);   // [NT * 128] |c|^2 (infinity past the slice)
  float* cc = cn + NT * 128;                                 // [NT * 128] counts
  const int prob = blockIdx.x / CS, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bf16* Xp = X + (size_t)prob * N * D;
  float* Tp = totals + (size_t)prob * C * D;
  float* Cp = centres + (size_t)prob * C * D;
  float* cntp = counts + (size_t)prob * C;
  const uint64_t strm = (uint64_t)prob * 2 + kind;
  const int per = ((C + CS - 1) / CS + 1) & ~1;
  const int j0 = min(C, rank * per), j1 = min(C, j0 + per);
  // byte offset of elements [lane * EPL, lane * EPL + EPL) of row r inside a swizzled [128][D] tile
  const int e0 = lane * EPL;
  auto row_off = [&](int r) { return (uint32_t)((e0 >> 6) * 128 * 128) + tc::sw128_off(r, (e0 >> 3) & 7) + (uint32_t)((e0 & 7) * 2); };

  if (warp == 0) tc::tmem_alloc(&tbase_s, NT * 128);
  if (tid == 0) { tc::mbar_init(&sdone, 1); tc::mbar_init_fence(); }
  for (int e = tid; e < (1 + 2 * NT) * kTile / 16; e += kStThreads) reinterpret_cast<uint4*>(sm)[e] = make_uint4(0u, 0u, 0u, 0u);
  for (int e = tid; e < NT * 128; e += kStThreads) { cn[e] = INFINITY; cc[e] = 0.f; }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tbase = tbase_s;

  // a centroid row: totals -> mean (global fp32), bf16 hi / lo into the resident tiles, |c|^2 and count
  auto put_centroid = [&](int j, float (&t)[EPL], float c) {
    const int jl = j - j0;
    float n2 = 0.f;
    uint32_t hw[EPL / 2], lw[EPL / 2];
#pragma unroll
    for (int e = 0; e < EPL; ++e) { t[e] = t[e] / c; n2 = fmaf(t[e], t[e], n2); }
    stv<EPL>(Cp + (size_t)j * D + e0, t);
#pragma unroll
    for (int e = 0; e < EPL; e += 2) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(t[e], t[e + 1]);
      const __nv_bfloat162 l = __floats2bfloat162_rn(t[e] - __low2float(h), t[e + 1] - __high2float(h));
      hw[e / 2] = *reinterpret_cast<const uint32_t*>(&h);
      lw[e / 2] = *reinterpret_cast<const uint32_t*>(&l);
    }
    const uint32_t off = (uint32_t)(jl >> 7) * kTile + row_off(jl & 127);
    if (EPL == 4) {
      *reinterpret_cast<uint2*>(Chi + off) = make_uint2(hw[0], hw[EPL / 2 - 1]);
      *reinterpret_cast<uint2*>(Clo + off) = make_uint2(lw[0], lw[EPL / 2 - 1]);
    } else {
      *reinterpret_cast<uint32_t*>(Chi + off) = hw[0];
      *reinterpret_cast<uint32_t*>(Clo + off) = lw[0];
    }
    n2 = warp_sum(n2);
    if (lane == 0) { cn[jl] = n2; cc[jl] = c; }
  };

  for (int j = j0 + warp; j < j1; j += NW) {
    float t[EPL], c;
    if (first_batch == 0) {
      const int u = feistel_permute(j * (N / C), N, seed, strm);
      ldv<EPL>(Xp + (size_t)u * D + e0, t);
      c = 1.f;
      stv<EPL>(Tp + (size_t)j * D + e0, t);
    } else {
      ldv<EPL>(Tp + (size_t)j * D + e0, t);
      c = cntp[j];
    }
    put_centroid(j, t, c);
  }

  // rows of the next minibatch travel in registers: thread = (row, quarter of the row), 16-byte pieces as stored
  const int lr = tid >> 2, lq = tid & 3;
  uint4 xr[RV];
  auto fetch = [&](int s) {
    const int pos = s * kSkBatch + lr;
    const int u = pos < N ? feistel_permute(pos, N, seed, strm) : -1;
#pragma unroll
    for (int v = 0; v < RV; ++v)
      xr[v] = (u >= 0 && MUSE_IN_RANGE(u, N)) ? reinterpret_cast<const uint4*>(Xp + (size_t)u * D)[lq * RV + v] : make_uint4(0u, 0u, 0u, 0u);
  };
  if (n_batches > 0) fetch(first_batch);
  cluster.sync();                                            // every CTA of the problem is running before any of them writes into another's shared memory
  bool ok = true;
  const bool reader = (warp & 3) < 2;                        // warps 0, 1, 4, 5 own the tensor-memory lanes of rows 0..63
  const int half = warp >> 2;                                // ... and one half of every tile's 128 columns

  for (int s = first_batch, it = 0; s < first_batch + n_batches; ++s, ++it) {
    const int nb = min(kSkBatch, N - s * kSkBatch), par = s & 1;
#pragma unroll
    for (int v = 0; v < RV; ++v) {
      const int c = lq * RV + v;
      *reinterpret_cast<uint4*>(Xs + (c >> 3) * 128 * 128 + tc::sw128_off(lr, c & 7)) = xr[v];
    }
    if (s + 1 < first_batch + n_batches) fetch(s + 1);
    tc::fence_async_smem();                                  // the minibatch and the rewritten centroid rows are read by the tensor cores
    tc::fence_before_sync();
    __syncthreads();
    if (tid == 6 * 32) {                                     // ---- one thread issues the products
      tc::fence_after_sync();
      const uint32_t idesc = tc::idesc_bf16(128, 128, 0, 0);
      const uint64_t dx0 = tc::smem_desc_sw128(tc::smem_u32(Xs), 16, 1024);
      for (int t = 0; t < NT; ++t) {
        const uint64_t dh = tc::smem_desc_sw128(tc::smem_u32(Chi + (size_t)t * kTile), 16, 1024);
        const uint64_t dl = tc::smem_desc_sw128(tc::smem_u32(Clo + (size_t)t * kTile), 16, 1024);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc::mma_bf16_ss(tbase + t * 128, tc::desc_step(dx0, (ks / 4) * 128 * 128 + (ks % 4) * 32),
                          tc::desc_step(dh, (ks / 4) * 128 * 128 + (ks % 4) * 32), idesc, ks > 0);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc::mma_bf16_ss(tbase + t * 128, tc::desc_step(dx0, (ks / 4) * 128 * 128 + (ks % 4) * 32),
                          tc::desc_step(dl, (ks / 4) * 128 * 128 + (ks % 4) * 32), idesc, 1);
      }
      tc::mma_commit(&sdone);
    }
    if (reader) {                                            // ---- arg-min over this CTA's centroids: thread = (vector, column half)
      if (ok && !tc::mbar_wait(&sdone, it & 1)) ok = false;
      tc::fence_after_sync();
      const uint32_t tl = tbase + ((uint32_t)((warp & 3) * 32) << 16);
      float best = INFINITY;
      int bidx = 0x7fffffff;
      for (int t = 0; t < NT; ++t) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          float v[32];
          tc::tmem_ld32(tl + t * 128 + half * 64 + 32 * q, v);
          const int c0 = t * 128 + half * 64 + 32 * q;
#pragma unroll
          for (int k = 0; k < 32; ++k) {
            const float dist = fmaf(-2.f, v[k], cn[c0 + k]);
            if (dist < best) { best = dist; bidx = j0 + c0 + k; }      // ascending index: ties keep the lower
          }
        }
      }
      tc::fence_before_sync();
      const int p = (warp & 3) * 32 + lane;
      if (half == 1) { rd[p] = best; ri[p] = bidx; }
      tc::named_bar_sync(1, 128);
      if (half == 0) {
        const float ob = rd[p];
        const int oi = ri[p];
        if (ob < best || (ob == best && oi < bidx)) { best = ob; bidx = oi; }
        for (int r = 0; r < CS; ++r) {                       // post this CTA's candidate to every CTA of the problem
          *cluster.map_shared_rank(&exd[par][rank][p], r) = best;
          *cluster.map_shared_rank(&exi[par][rank][p], r) = bidx;
        }
      }
    }
    cluster.sync();                                          // every CTA's candidates have arrived (and the previous step's have been read)
    if (tid < kSkBatch) {
      float dv = exd[par][0][tid];
      int iv = exi[par][0][tid];
      for (int r = 1; r < CS; ++r) {
        const float od = exd[par][r][tid];
        const int oi = exi[par][r][tid];
        if (od < dv || (od == dv && oi < iv)) { dv = od; iv = oi; }
      }
      as[tid] = (tid < nb && (unsigned)iv < (unsigned)C) ? iv : (tid < nb ? 0 : -1);   // (a NaN row goes to centroid 0)
    }
    __syncthreads();
    // update: the first vector of the minibatch on a centroid replays all of that centroid's vectors in stream order
    const int a_lo = as[lane], a_hi = as[lane + 32];
    // (the rows of totals of all of this warp's centroids are requested before any of them is used)
    unsigned long long mems[PPW];
    float tt[PPW][EPL];
#pragma unroll
    for (int k = 0; k < PPW; ++k) {
      const int p = warp + NW * k;
      const int j = as[p];
      mems[k] = 0ull;
      if (j < j0 || j >= j1) continue;                       // (warp-uniform) not this CTA's centroid
      const unsigned long long mem = (unsigned long long)__ballot_sync(0xffffffffu, a_lo == j) |
                                     ((unsigned long long)__ballot_sync(0xffffffffu, a_hi == j) << 32);
      if (__ffsll((long long)mem) - 1 != p) continue;
      mems[k] = mem;
      ldv<EPL>(Tp + (size_t)j * D + e0, tt[k]);
    }
#pragma unroll
    for (int k = 0; k < PPW; ++k) {
      const unsigned long long mem = mems[k];
      if (mem == 0ull) continue;
      const int j = as[warp + NW * k];
      float t[EPL], c = cc[j - j0];
#pragma unroll
      for (int e = 0; e < EPL; ++e) t[e] = tt[k][e];
      for (unsigned long long rest = mem; rest != 0ull; rest &= rest - 1ull) {
        const int q = __ffsll((long long)rest) - 1;
        float x[EPL];
        ldv<EPL>(reinterpret_cast<const bf16*>(Xs + row_off(q)), x);
#pragma unroll
        for (int e = 0; e < EPL; ++e) t[e] = fmaf(beta, t[e], x[e]);
        c = fmaf(beta, c, 1.f);
      }
      stv<EPL>(Tp + (size_t)j * D + e0, t);
      put_centroid(j, t, c);
    }
    if (rank == 0 && assign_stream != nullptr && tid < nb) assign_stream[(size_t)prob * N + (size_t)s * kSkBatch + tid] = as[tid];
    __syncthreads();                                         // the minibatch rows have been read: the next step may overwrite them
  }
  for (int j = j0 + tid; j < j1; j += kStThreads) cntp[j] = cc[j - j0];
  if (!ok && tid == 0) report_status(status, MUSE_STATUS_ASSIGN_TIMEOUT);
  tc::fence_before_sync();
  cluster.sync();                                            // no CTA leaves while another may still write into its shared memory
  if (warp == 0) tc::tmem_dealloc(tbase, NT * 128);
}

template <class T, int D>
static int stream_kmeans_t(const Dims& d, const T* X, int problems, int C, int kind, uint64_t seed, float beta,
                           int first_batch, int n_batches, float* totals, float* counts, float* centres,
                           int32_t* assign_stream, int* status, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cfg.stream = st;
  if (sizeof(T) == 2 && C <= 256 * kSkMaxCluster) {
    // tensor-core kernel: at most 256 centroids (two tiles) per CTA, 128 where the GPU has room for twice the CTAs
    int cs = 1;
    while (cs < kSkMaxCluster && (C > 256 * cs || (C > 128 * cs && (long long)problems * cs * 2 <= 148))) cs *= 2;
    const int per = ((C + cs - 1) / cs + 1) & ~1, NT = (per + 127) / 128;
    const size_t smem = stream_tc_smem_bytes<D>(NT);
    MUSE_CUDA_OK(cudaFuncSetAttribute(k_stream_kmeans_tc<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    cfg.gridDim = dim3(problems * cs);
    cfg.blockDim = dim3(kStThreads);
    cfg.dynamicSmemBytes = smem;
    attr[0].val.clusterDim.x = cs;
    prof_mark("k_stream_kmeans_tc", st);
    MUSE_CUDA_OK(cudaLaunchKernelEx(&cfg, k_stream_kmeans_tc<D>, (const __nv_bfloat16*)X, d.N, C, seed, kind, beta, first_batch, n_batches,
                                    totals, counts, centres, assign_stream, NT, status));
    return MUSE_OK;
  }
  const size_t smem = stream_smem_bytes<D>(C);
  MUSE_CUDA_OK(cudaFuncSetAttribute(k_stream_kmeans<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  // CTAs per problem: enough that a CTA owns at most two chunks of 64 centroids, as long as the GPU has room for them
  int cs = 1;
  while (cs < kSkMaxCluster && C > 2 * kSkChunk * cs && (long long)problems * cs * 2 <= 2 * 148) cs *= 2;
  cfg.gridDim = dim3(problems * cs);
  cfg.blockDim = dim3(kSkThreads);
  cfg.dynamicSmemBytes = smem;
  attr[0].val.clusterDim.x = cs;
  prof_mark("k_stream_kmeans", st);
  MUSE_CUDA_OK(cudaLaunchKernelEx(&cfg, k_stream_kmeans<T, D>, X, d.N, C, seed, kind, beta, first_batch, n_batches, totals, counts,
                                  centres, assign_stream));
  return MUSE_OK;
}

int stream_kmeans(const Dims& d, int dtype, const void* X, int problems, int C, int kind, uint64_t seed, float beta,
                  int first_batch, int n_batches, float* totals, float* counts, float* centres, int32_t* assign_stream,
                  int32_t* status, cudaStream_t st) {
  const int all = cdiv(d.N, kSkBatch);
  if (first_batch < 0 || first_batch > all) return MUSE_ERR_INVALID_ARG;
  if (n_batches < 0) n_batches = all - first_batch;
  if (first_batch + n_batches > all) return MUSE_ERR_INVALID_ARG;
  typedef __nv_bfloat16 bf;
  if (dtype == MUSE_F32) {
    if (d.D == 64) return stream_kmeans_t<float, 64>(d, (const float*)X, problems, C, kind, seed, beta, first_batch, n_batches, totals, counts, centres, assign_stream, status, st);
    return stream_kmeans_t<float, 128>(d, (const float*)X, problems, C, kind, seed, beta, first_batch, n_batches, totals, counts, centres, assign_stream, status, st);
  }
  if (d.D == 64) return stream_kmeans_t<bf, 64>(d, (const bf*)X, problems, C, kind, seed, beta, first_batch, n_batches, totals, counts, centres, assign_stream, status, st);
  return stream_kmeans_t<bf, 128>(d, (const bf*)X, problems, C, kind, seed, beta, first_batch, n_batches, totals, counts, centres, assign_stream, status, st);
}

// ---------------------------------------------------------------------------------------------
// Balanced assignment
// ---------------------------------------------------------------------------------------------

// rank of every vector inside its (block, cluster) bucket in position order (the sort is stable)
__global__ void k_bucket_rank(const int32_t* __restrict__ assign, const int32_t* __restrict__ off, const int32_t* __restrict__ perm,
                              int N, int C, int S, int Bs, int32_t* __restrict__ rank) {
  const int prob = blockIdx.y, pos = blockIdx.x * blockDim.x + threadIdx.x;
  if (pos >= N) return;
  const int t = perm[(size_t)prob * N + pos];
  if (!MUSE_IN_RANGE(t, N)) return;
  const int a = min(max(assign[(size_t)prob * N + t], 0), C - 1);
  const int key = (t / Bs) * C + a;
  rank[(size_t)prob * N + t] = pos - off[(size_t)prob * (C * S + 1) + key];
}

constexpr int kCapThreads = 512;

// Step 2: the displaced vectors of one (problem, block), in position order; each takes the nearest centroid whose bucket
// still has room.  The distances of every vector to every centroid were written by the step-1 assignment, so a placement is
// a masked arg-min over one row of that matrix (ties to the lower index).
__global__ void __launch_bounds__(kCapThreads)
k_cap_overflow(int N, int C, int S, int Bs, int cap, const float* __restrict__ dist, const int32_t* __restrict__ off,
               const int32_t* __restrict__ rank, int32_t* __restrict__ assign) {
  constexpr int NW = kCapThreads / 32;
  extern __shared__ int cap_smem[];
  int* size = cap_smem;                        // [C] bucket sizes of this block
  __shared__ int lst[kCapThreads], wcnt[NW], ri[NW];
  __shared__ float rd[NW];
  const int b = blockIdx.x, prob = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int32_t* o = off + (size_t)prob * (C * S + 1) + (size_t)b * C;
  const int32_t* rk = rank + (size_t)prob * N;
  int32_t* as = assign + (size_t)prob * N;
  for (int j = tid; j < C; j += kCapThreads) size[j] = min(o[j + 1] - o[j], cap);     // step 1: the first cap of a bucket keep it
  __syncthreads();
  for (int base = b * Bs; base < (b + 1) * Bs; base += kCapThreads) {
    // the displaced vectors of this stretch, in position order
    const int t = base + tid;
    const bool over = t < (b + 1) * Bs && rk[t] >= cap;
    const unsigned bal = __ballot_sync(0xffffffffu, over);
    if (lane == 0) wcnt[warp] = __popc(bal);
    __syncthreads();
    int before = 0, total = 0;
    for (int w = 0; w < NW; ++w) { if (w < warp) before += wcnt[w]; total += wcnt[w]; }
    if (over) lst[before + __popc(bal & ((1u << lane) - 1u))] = t;
    __syncthreads();
    for (int e = 0; e < total; ++e) {
      const int u = lst[e];
      const float* dr = dist + ((size_t)prob * N + u) * C;
      float best = INFINITY;
      int bj = 0x7fffffff;
      for (int j = tid; j < C; j += kCapThreads) {
        if (size[j] >= cap) continue;
        const float dv = dr[j];
        if (dv < best) { best = dv; bj = j; }                          // (ascending j per thread)
      }
#pragma unroll
      for (int o2 = 16; o2 > 0; o2 >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, o2);
        const int oj = __shfl_xor_sync(0xffffffffu, bj, o2);
        if (ob < best || (ob == best && oj < bj)) { best = ob; bj = oj; }
      }
      if (lane == 0) { rd[warp] = best; ri[warp] = bj; }
      __syncthreads();
      if (tid == 0) {
        float bd = rd[0];
        int bi = ri[0];
        for (int w = 1; w < NW; ++w)
          if (rd[w] < bd || (rd[w] == bd && ri[w] < bi)) { bd = rd[w]; bi = ri[w]; }
        if ((unsigned)bi >= (unsigned)C)                               // every distance was NaN: first centroid with room
          for (bi = 0; bi < C - 1 && size[bi] >= cap; ++bi) {}
        as[u] = bi;
        size[bi] += 1;
      }
      __syncthreads();
    }
  }
}

size_t balanced_ws_bytes(const Dims& d, int problems, int C) {
  Arena ar(nullptr);
  ar.take<char>(lloyd_ws_bytes(d, problems, C, 0));
  ar.take<float>((size_t)problems * C);
  ar.take<int32_t>((size_t)problems * (C * d.S + 1));
  ar.take<int32_t>((size_t)problems * d.N);
  ar.take<int32_t>((size_t)problems * sort_ws_elems(d.N, C * d.S));
  ar.take<int32_t>((size_t)problems * d.N);
  ar.take<float>((size_t)problems * d.N * C);
  return ar.used;
}

int balanced_assign(const Dims& d, int dtype, const void* X, int problems, int C, int kind, const float* centres, float factor,
                    int32_t* assign, void* ws, cudaStream_t st) {
  const int cap = factor > 0.f ? (int)ceil((double)factor * d.Bs / C) : d.Bs;
  const bool binds = cap < d.Bs;               // otherwise the cap cannot bind: plain nearest centroid
  Arena ar(ws);
  ar.take<char>(lloyd_ws_bytes(d, problems, C, 0));
  ar.take<float>((size_t)problems * C);
  int32_t* off = ar.take<int32_t>((size_t)problems * (C * d.S + 1));
  int32_t* perm = ar.take<int32_t>((size_t)problems * d.N);
  int32_t* scratch = ar.take<int32_t>((size_t)problems * sort_ws_elems(d.N, C * d.S));
  int32_t* rank = ar.take<int32_t>((size_t)problems * d.N);
  float* dist = ar.take<float>((size_t)problems * d.N * C);      // |c|^2 - 2 x.c of every (vector, centroid), written by step 1
  // step 1a: nearest centroid of every vector (the Lloyd path's final assignment against given centres)
  int rc = lloyd(d, dtype, X, problems, C, kind, nullptr, MUSE_INIT_CENTRES, 0, 0, assign, const_cast<float*>(centres), ws, st,
                 binds ? dist : nullptr);
  if (rc != MUSE_OK || !binds) return rc;
  rc = bucket_sort(0, assign, problems, d.N, C, d.S, d.Bs, 0, off, perm, scratch, st);      // key = block * C + cluster
  if (rc != MUSE_OK) return rc;
  prof_mark("k_bucket_rank", st);
  k_bucket_rank<<<dim3(cdiv(d.N, 256), problems), 256, 0, st>>>(assign, off, perm, d.N, C, d.S, d.Bs, rank);
  MUSE_LAUNCH_OK();
  prof_mark("k_cap_overflow", st);
  k_cap_overflow<<<dim3(d.S, problems), kCapThreads, (size_t)C * sizeof(int), st>>>(d.N, C, d.S, d.Bs, cap, dist, off, rank, assign);
  MUSE_LAUNCH_OK();
  return MUSE_OK;
}

}  // namespace muse
