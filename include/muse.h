/*
 * muse.h — C ABI of the B200 (sm_100a) implementation of the Multipole Semantic Attention
 * (MuSe) layer: approximate causal softmax attention, forward and backward.
 *
 * The four stages follow the paper's Algorithm 1 ("MuSe Causal Attention"):
 *   muse_cluster    — lines "Cluster Q / Cluster K" (Section "Clustering", Appendix
 *                     "Clustering Details"), as Lloyd iterations;
 *   muse_summarize  — "Per-block summaries" and "Causal accumulation along spatial axis"
 *                     (Section "Summary Computation and Causal Accumulation", Eq. 3-5);
 *   muse_attn_fwd   — "Two-level retrieval + attention (per query)" and the log-sum-exp merge
 *                     (Sections "Two-Level Retrieval", Eq. 6, "Exact Retrieval and Local
 *                     Attention", "Output merging");
 *   muse_attn_bwd   — gradients with assignments, selections and query centroids held constant
 *                     (Appendix "Centroid Gradient Flow", "Aggregation Weight Gradient Flow").
 *
 * General conventions
 *   - Every tensor pointer is a DEVICE pointer to a contiguous row-major array unless marked
 *     HOST.  Q, O, dO, dQ are [B,Hq,N,D]; K, V, dK, dV are [B,Hkv,N,D]; D is innermost.
 *     Element type is given by muse_params_t.dtype (bf16 or fp32); centroids, LSE and
 *     summaries are always fp32; indices are int32.
 *   - The caller owns every buffer.  The library never allocates, frees or synchronises: all
 *     work is enqueued on `stream` and the call returns at once.  Scratch memory is passed as
 *     (ws, ws_bytes); sizes come from muse_workspace_bytes.  Workspaces may be reused between
 *     calls on the same stream.  Pointers must be 16-byte aligned.
 *   - Return value: MUSE_OK (0) or a negative MUSE_ERR_* code.  Arguments are checked on the
 *     host before anything is launched; nothing aborts or throws.
 *   - Device status.  Inside the kernels every wait on the hardware (a tensor-core or copy
 *     completion barrier) is bounded by elapsed SM clocks (about half a second); a wait that runs out
 *     makes its kernel stop early instead of hanging the GPU, and the outputs of that call are then
 *     undefined.  The first 64 int32 words of `ws` are status words: each entry point clears them
 *     when it starts, word 0 receives the first MUSE_STATUS_* code a kernel of the call reported
 *     (0 = the call ran to completion), the other words are reserved.  The word is written
 *     asynchronously: read it after synchronising the stream, directly from `ws` or through
 *     muse_status_copy.  Indices supplied by the caller are never trusted as addresses: an
 *     assignment outside [0, C) is treated as the nearest valid cluster index and a selection entry
 *     outside [0, Ck) as -1 (none); a row of Q or K that holds NaN or infinities is assigned to
 *     cluster 0.
 *   - Spatial blocks: block(t) = t / (N / n_blocks).  Keys are bucketed cluster-major,
 *     block-minor: bucket (j,b) occupies positions [off_k[j*S+b], off_k[j*S+b+1]) of the
 *     permutation perm_k (position -> original key index, stable, i.e. ascending inside a
 *     bucket).
 */
#ifndef MUSE_H_
#define MUSE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#ifndef __DRIVER_TYPES_H__
typedef struct CUstream_st* cudaStream_t;
#endif

#if defined(__GNUC__)
#define MUSE_API __attribute__((visibility("default")))
#else
#define MUSE_API
#endif

enum { MUSE_BF16 = 0, MUSE_F32 = 1 };
enum { MUSE_SEL_PER_QUERY = 0, MUSE_SEL_PER_QCLUSTER = 1 };
enum { MUSE_INIT_INDICES = 0, MUSE_INIT_STRIDED = 1, MUSE_INIT_CENTRES = 2, MUSE_INIT_KMEANSPP = 3 };
/* Device status word (see "Device status" below): first code reported by a kernel of the call. */
enum {
  MUSE_STATUS_OK = 0,
  MUSE_STATUS_FWD_TIMEOUT = 1,       /* exact-attention forward kernels (local, retrieval)         */
  MUSE_STATUS_BWD_TIMEOUT = 2,       /* exact-attention backward kernels                           */
  MUSE_STATUS_FAR_FWD_TIMEOUT = 3,   /* far-field forward (scores, top-m, approximate attention)   */
  MUSE_STATUS_FAR_BWD_TIMEOUT = 4,   /* far-field backward                                         */
  MUSE_STATUS_SUMM_BWD_TIMEOUT = 5,  /* key-side pass through the summaries                        */
  MUSE_STATUS_ASSIGN_TIMEOUT = 6,    /* k-means assignment                                         */
  MUSE_STATUS_SUMM_TIMEOUT = 7,      /* summaries / dipole construction                            */
  MUSE_STATUS_SELFTEST_TIMEOUT = 9   /* muse_test_wait_timeout                                     */
};
enum {
  MUSE_OK = 0,
  MUSE_ERR_INVALID_ARG = -1,   /* null pointer, bad size, misaligned pointer            */
  MUSE_ERR_UNSUPPORTED = -2,   /* legal request that this build does not implement       */
  MUSE_ERR_WORKSPACE = -3,     /* ws_bytes smaller than muse_workspace_bytes reports     */
  MUSE_ERR_CUDA = -4           /* a CUDA runtime call (launch, attribute) failed         */
};

typedef struct muse_params {
  int32_t B, Hq, Hkv, N, D;     /* D in {64,128}; Hq % Hkv == 0 unless head_map is given; Hq <= 128 */
  int32_t Cq, Ck, m;            /* 1 <= Cq <= 4096, 1 <= Ck <= 4096, 0 <= m <= min(Ck,64)          */
  int32_t causal;               /* 1: blocked causal handling of the paper; 0: one block, no local */
  int32_t n_blocks;             /* S, spatial blocks (0 -> 8); N % S == 0; forced to 1 if !causal  */
  int32_t k2;                   /* spatial selection inside the selected clusters (Section "Two-Level Retrieval"):
                                   0 = every earlier block is retrieved; 1..8 = only the k2 best-scoring earlier
                                   blocks, the others enter through their per-block summaries (bf16 mode, causal,
                                   m * k2 <= 64, S - 1 <= 32; ignored when !causal)                              */
  int32_t dtype;                /* MUSE_BF16 | MUSE_F32: type of Q,K,V,O,dO,dQ,dK,dV               */
  float   softmax_scale;        /* sigma; <= 0 -> 1/sqrt(D)                                        */
  int32_t kmeans_iters;         /* T Lloyd iterations before the final assignment (>= 0)           */
  int32_t init_mode;            /* MUSE_INIT_*                                                     */
  uint64_t seed;                /* used by MUSE_INIT_STRIDED and MUSE_INIT_KMEANSPP                */
  int32_t sel_mode;             /* MUSE_SEL_*: rank clusters by the Eq. 6 score per query, or by
                                   the accumulated log-mass per (query cluster, block)            */
  int32_t dipole;               /* 0 off; 1: untilted dipole correction of the far field (Appendix
                                   "Error Analysis", "Dipole Correction"): pre-merged with m == 0 as in
                                   the paper; with m > 0 each query's correction is the merge over the
                                   clusters it did not retrieve ("Compatibility with Retrieval"); 2: the
                                   same with the shared covariance tilted at one point per query head
                                   (muse_dipole_tilt_point).  Forward and backward; not with k2 > 0     */
  int32_t agg_grad;             /* 1: differentiate the tilted aggregation weights; 0: constants   */
  const int32_t* head_map;      /* HOST [Hq] -> kv head, or NULL for h * Hkv / Hq                  */
} muse_params_t;

/* Sizes in bytes of the scratch each stage needs and of the opaque summaries buffer.
 * out[0] cluster, out[1] summarize, out[2] attn_fwd, out[3] attn_bwd, out[4] summaries,
 * out[5] attn_bwd when it is called with summaries == NULL and rebuilds them in its scratch.
 * Appendix "Clustering Cost" / Section "Summary Computation": the summaries buffer holds the
 * S-1 accumulated (mu, beta, kappa, nu) planes over [B,Hq,S-1,Cq,Ck], followed by the bucketed
 * copies of K and V (see muse_summaries_layout). */
MUSE_API int muse_workspace_bytes(const muse_params_t* p, size_t out[6]);

/* Byte offsets inside the summaries buffer, per entry e = (b, h, plane, i, j) of
 * [B,Hq,SB,Cq,Ck], SB = S-1 (causal) or 1; plane s is the accumulated summary seen by queries
 * of block s+1 (Section "Causal accumulation": exclusive, block 0 sees nothing):
 *   off[0] mu    f32 [e]    accumulated log-mass, -inf for a cluster with no visible key
 *   off[1] beta  f32 [e]    mu - sigma qbar_i . kappa, so that the Eq. 6 score of a query q is
 *                           sigma q . kappa + beta
 *   off[2] kappa     [e][D] fp32 mode: fp32.  bf16 mode: the bf16 rounding of kappa ...
 *   off[3] kappa_lo  [e][D] ... and the bf16 rounding of the remainder (kappa = hi + lo);
 *                           fp32 mode: unused (same offset as off[4])
 *   off[4] nu        [e][D] fp32 (fp32 mode) or bf16 (bf16 mode)
 *   off[5], off[6]          K and V bucketed by (cluster, block), [B,Hkv,N,D] dtype
 *   off[7] cbar             dipole != 0 only: merged dipole matrices Cbar = sum_j p(j) Cov_j(v,k),
 *                           [B,Hq,SB,Cq][D value dims][D key dims], fp32 (fp32 mode, or m > 0) or bf16,
 *                           followed by the shared covariances, the centroid weights, their sums and the
 *                           tilt points (muse_dipole_layout); with dipole == 0 nothing is stored there
 *   off[8] per-block set    k2 > 0 only: a second mu | beta | kappa | kappa_lo | nu group of the same shapes
 *                           and spacing as off[0..4], holding the summaries of each block alone (plane s =
 *                           the keys of block s), which the spatial block selection scores; with k2 == 0
 *                           nothing is stored there (off[8] = end of the buffer) */
MUSE_API int muse_summaries_layout(const muse_params_t* p, size_t off[9]);

/* Lloyd k-means of the queries (per query head, Cq clusters) and keys (per kv head, Ck
 * clusters): T x (assign to argmin_c |c|^2 - 2 x.c, lowest index on ties; move each centre to
 * the mean of its members, empty clusters keep theirs), then a final assignment
 * (Appendix "Clustering Details"; distance identity of "Balanced Assignment").
 *   Q, K        in   inputs
 *   init_q/k    in   [B,Hq,Cq] / [B,Hkv,Ck] start indices (MUSE_INIT_INDICES), else NULL
 *   assign_q/k  out  [B,Hq,N] / [B,Hkv,N] cluster of every query / key
 *   qbar, kcent out  [B,Hq,Cq,D] / [B,Hkv,Ck,D] fp32 centres used by the final assignment;
 *                    with MUSE_INIT_CENTRES they are also the input start centres.
 *   MUSE_INIT_KMEANSPP: the start points are drawn on the GPU by muse_kmeanspp_init.
 * Either side may be skipped by passing its Q/K pointer as NULL. */
MUSE_API int muse_cluster(const muse_params_t* p, const void* Q, const void* K,
                 const int32_t* init_q, const int32_t* init_k,
                 int32_t* assign_q, int32_t* assign_k, float* qbar, float* kcent,
                 void* ws, size_t ws_bytes, cudaStream_t stream);

/* Clustering without a caller-provided workspace (the paper has no counterpart; this is a
 * deployment aid).  Same inputs, outputs and results as muse_cluster, but the scratch memory is
 * a fixed 32 MiB array built into the library's device image, so the call itself makes no
 * allocation request of any kind and needs no scratch pointer.  It is meant for callers that cannot
 * allocate or own no spare device memory: code running inside a serving loop where a device
 * allocation would stall every stream, plugins living under a framework whose pool already
 * owns the whole GPU, or hosts that must not fail with out-of-memory in mid-request.
 *   - Every GPU that loads the library carries the 32 MiB until the process exits.
 *   - Problems whose clustering scratch (muse_workspace_bytes out[0]) exceeds
 *     muse_cluster_noalloc_max_bytes() are rejected with MUSE_ERR_WORKSPACE; nothing is launched.
 *   - Every call looks up the array's device address for the current device.  The first lookup on
 *     a device loads the library's device image there, and that is when the driver reserves the
 *     32 MiB: this first call can therefore return MUSE_ERR_CUDA (no memory left for the image) and
 *     should be made before any stream capture.  Later calls only read a host-side table.
 *   - The status word of the call sits inside the built-in array: muse_cluster_noalloc_status_copy
 *     enqueues its copy to memory the caller owns.
 *   - All calls share the one array and find in it whatever the previous call left; the stage
 *     clears what it needs zeroed itself.  Two calls that overlap on the GPU (different streams,
 *     or different threads) race on it: serialise them. */
MUSE_API int muse_cluster_noalloc(const muse_params_t* p, const void* Q, const void* K,
                         const int32_t* init_q, const int32_t* init_k,
                         int32_t* assign_q, int32_t* assign_k, float* qbar, float* kcent,
                         cudaStream_t stream);
MUSE_API size_t muse_cluster_noalloc_max_bytes(void);
MUSE_API int muse_cluster_noalloc_status_copy(int32_t* dst, cudaStream_t stream);

/* Enqueues a copy of status word 0 of workspace `ws` to `dst` (HOST or device memory, 4 bytes)
 * on `stream`; see "Device status" above (no counterpart in the paper). */
MUSE_API int muse_status_copy(const void* ws, int32_t* dst, cudaStream_t stream);

/* Buckets the keys by (cluster, block) and builds the accumulated tilted summaries
 * mu_ijb = log sum exp(sigma qbar_i.k), kappa_ijb, nu_ijb = weighted means of k, v over the
 * keys of cluster j in blocks < b (Eq. 3-5 and "Causal accumulation").
 *   K, V, assign_k, qbar  in
 *   off_k     out [B,Hkv,Ck*S+1]   bucket offsets
 *   perm_k    out [B,Hkv,N]        bucketed position -> key index
 *   counts    out [B,Hkv,Ck,S]     keys per bucket (j, b)                 } the untilted
 *   ksum      out [B,Hkv,Ck,S,D]   fp32 sum of the keys of bucket (j, b)   } per-block statistics
 *   vsum      out [B,Hkv,Ck,S,D]   fp32 sum of its values                  } (Eq. 3-5 at zero tilt);
 *                                  pass all three or NULL for all three
 *   summaries out opaque, muse_workspace_bytes out[4] bytes (layout: muse_summaries_layout) */
MUSE_API int muse_summarize(const muse_params_t* p, const void* K, const void* V,
                   const int32_t* assign_k, const float* qbar,
                   int32_t* off_k, int32_t* perm_k,
                   int32_t* counts, float* ksum, float* vsum, void* summaries,
                   void* ws, size_t ws_bytes, cudaStream_t stream);

/* Forward: per query, score every key cluster (Eq. 6), retrieve the top-m for exact
 * attention, approximate the rest with the summaries, add exact causal attention inside the
 * query's block, merge by log-sum-exp.
 *   sel_in   in   [B,Hq,N,m] clusters to retrieve (-1 = none) or NULL to select here
 *   bsel_in  in   k2 > 0: [B,Hq,N,m,k2] blocks to retrieve inside each selected cluster (-1 = none), in
 *                 the slot order of sel_in, or NULL to select here; ignored when k2 == 0
 *   O        out  [B,Hq,N,D] dtype
 *   LSE      out  [B,Hq,N] fp32 log of the merged normaliser
 *   sel_out  out  [B,Hq,N,m] retrieved clusters in no particular order, padded with -1 (may be NULL)
 *   bsel_out out  k2 > 0: [B,Hq,N,m,k2] retrieved blocks of each slot of sel_out, best first, -1 padded
 *                 (may be NULL) */
MUSE_API int muse_attn_fwd(const muse_params_t* p, const void* Q, const void* K, const void* V,
                  const int32_t* assign_q, const float* qbar,
                  const int32_t* off_k, const int32_t* perm_k, const void* summaries,
                  const int32_t* sel_in, const int32_t* bsel_in, void* O, float* LSE, int32_t* sel_out,
                  int32_t* bsel_out, void* ws, size_t ws_bytes, cudaStream_t stream);

/* Backward of sum(O * dO) w.r.t. Q, K, V with assign_*, sel, bsel and qbar constant; dK, dV of a
 * kv head are summed over the query heads that share it.
 *   O, LSE, sel  in   as returned by muse_attn_fwd (sel must be the selection used there)
 *   bsel         in   k2 > 0: the chosen blocks [B,Hq,N,m,k2] as returned by muse_attn_fwd (required);
 *                     ignored (may be NULL) when k2 == 0.  With k2 > 0 the stand-in keys of the
 *                     non-retrieved blocks pass their gradient on through the per-block summaries
 *   summaries    in   as written by muse_summarize, or NULL: the summaries are then rebuilt from
 *                     K, V, off_k, perm_k, qbar inside the scratch, which must hold
 *                     muse_workspace_bytes out[5] bytes instead of out[3]
 *   dQ, dK, dV   out  dtype */
MUSE_API int muse_attn_bwd(const muse_params_t* p, const void* Q, const void* K, const void* V,
                  const void* O, const float* LSE, const void* dO,
                  const int32_t* assign_q, const float* qbar,
                  const int32_t* off_k, const int32_t* perm_k, const void* summaries,
                  const int32_t* sel, const int32_t* bsel, void* dQ, void* dK, void* dV,
                  void* ws, size_t ws_bytes, cudaStream_t stream);

/* Dipole correction, optional parts (Appendix "Error Analysis").
 * muse_dipole_tilt_point - dipole == 2 only ("Untilted (Partially Specialized) Covariances": the shared
 *   covariance tilted at ONE point per query head instead of at zero): writes that point, the mean of the
 *   head's query centroids weighted by the number of queries each holds (assign_q [B,Hq,N], qbar
 *   [B,Hq,Cq,D], DEVICE), into the summaries buffer at muse_dipole_layout off[4] ([B,Hq,D] fp32).  It is an
 *   INPUT of muse_summarize, which builds the covariances with the weights exp(sigma qstar . k) normalised
 *   inside each (cluster, plane) set; a caller may store any other tilt point there instead.  Call it (or
 *   fill the array) before muse_summarize; muse_attn_bwd with summaries == NULL calls it itself.
 * muse_dipole_layout - byte offsets inside the summaries buffer of: off[0] merged matrices Cbar
 *   [B,Hq,SB,Cq][D][D] (fp32 when m > 0 or in fp32 mode, else bf16), off[1] shared covariances Cov
 *   [B,H,SB,Ck][D value dims][D key dims] (H = Hkv for dipole == 1, Hq for dipole == 2; dtype), off[2]
 *   centroid weights p [B,Hq,SB,Cq,Ck] (dtype), off[3] the sums over j of the stored weights [B,Hq,SB,Cq]
 *   fp32, off[4] tilt points [B,Hq,D] fp32.  All outputs of muse_summarize except off[4]. */
MUSE_API int muse_dipole_layout(const muse_params_t* p, size_t off[5]);
MUSE_API int muse_dipole_tilt_point(const muse_params_t* p, const int32_t* assign_q, const float* qbar,
                                    void* summaries, cudaStream_t stream);

/* Seeded k-means++ start points, drawn on the GPU (the paper starts from a strided sample, Appendix
 * "Centroid Computation" step 1; this is the usual better-spread alternative for the Lloyd iterations).
 * Per head of side 0 (queries X = [B,Hq,N,D], C_q points) or 1 (keys [B,Hkv,N,D], C_k points): the first
 * start point is position 0 of the seeded shuffle; draw c = 1 .. C-1 takes vector t with probability
 * d2_t / sum d2, d2 = squared distance (fp32) to the nearest start point so far.  The draw is an exponential
 * race, reproducible from p->seed alone: u_t = ((h >> 41) + 1/2) / 2^23 with h = splitmix64(splitmix64(seed
 * ^ stream << 32 ^ 0xA5 << 56 ^ c) ^ t), stream = 2 * head + side; the largest d2_t / -log(u_t) wins, the
 * lower index on ties.  idx_out [problems, C] int32 (DEVICE, out).  ws: muse_workspace_bytes out[0].
 * Errors as for muse_cluster. */
MUSE_API int muse_kmeanspp_init(const muse_params_t* p, const void* X, int side, int32_t* idx_out,
                                void* ws, size_t ws_bytes, cudaStream_t stream);

/* The paper's own clustering (Appendix "Clustering Details").  An alternative to muse_cluster with the
 * same outputs; the rest of the path does not care which produced them.
 *
 * muse_stream_kmeans - "Centroid Computation": ONE pass of streaming mini-batch k-means over the vectors X
 *   (DEVICE, [B,Hq,N,D] for side 0 = queries with C_q centroids, [B,Hkv,N,D] for side 1 = keys with C_k) of
 *   every head.  The vectors are visited in the order of the seeded shuffle (p->seed; the same bijection as
 *   MUSE_INIT_STRIDED, position s of the stream = vector pi(s)), MUSE_STREAM_BATCH = 64 per minibatch; a
 *   minibatch is assigned to the nearest current centroids t_j / c_j (|c|^2 - 2 x.c, ties to the lower
 *   index), then its vectors update their centroids one after the other in stream order:
 *   t_j <- beta t_j + x, c_j <- beta c_j + 1 (the paper uses beta = 0.9).  Centroid r starts as the r-th
 *   strided sample of the shuffled sequence with t = x, c = 1.  The call runs minibatches
 *   [first_batch, first_batch + n_batches) (n_batches < 0: up to the last, which may be short):
 *   first_batch = 0 starts from the start state, otherwise from the state in totals / counts.
 *   totals [problems, C, D] fp32 and counts [problems, C] fp32 (DEVICE, in/out: the state t, c),
 *   centres [problems, C, D] fp32 (DEVICE, out: t_j / c_j), assign_stream [problems, N] int32 (DEVICE, out,
 *   may be NULL: the centroid each streamed vector was assigned to, by stream position; positions outside
 *   the call's minibatches are not written).  fp32 arithmetic.  ws: >= 256 bytes (status words only).
 * muse_balanced_assign - "Balanced Assignment": independently in each spatial block, every vector goes to
 *   its nearest centroid subject to a bucket size of at most cap = ceil(cap_factor * B / K) (the paper uses
 *   cap_factor = 4).  The paper gives no rule for a vector whose nearest centroid is full; the one taken:
 *   (1) every vector names its nearest centroid, and of the vectors of a block that name centroid j the
 *   first cap in position order keep it; (2) the others, in position order, take the nearest centroid
 *   whose bucket still has room (counting step-1 members and earlier step-2 placements).  cap_factor <= 0:
 *   no cap (plain nearest centroid).  centres [problems, C, D] fp32 (DEVICE, in), assign [problems, N]
 *   int32 (DEVICE, out).  ws: muse_stream_workspace_bytes.
 * muse_cluster_streaming - both steps for Q and/or K (either may be NULL with its outputs), with the
 *   streaming state kept in ws; outputs as muse_cluster.  ws: muse_stream_workspace_bytes.
 * Errors as for muse_cluster; beta outside (0, 1] is MUSE_ERR_INVALID_ARG. */
#define MUSE_STREAM_BATCH 64
MUSE_API int muse_stream_workspace_bytes(const muse_params_t* p, size_t* bytes);
MUSE_API int muse_stream_kmeans(const muse_params_t* p, const void* X, int side, float beta, int first_batch,
                                int n_batches, float* totals, float* counts, float* centres,
                                int32_t* assign_stream, void* ws, size_t ws_bytes, cudaStream_t stream);
MUSE_API int muse_balanced_assign(const muse_params_t* p, const void* X, int side, const float* centres,
                                  float cap_factor, int32_t* assign, void* ws, size_t ws_bytes,
                                  cudaStream_t stream);
MUSE_API int muse_cluster_streaming(const muse_params_t* p, const void* Q, const void* K, float beta,
                                    float cap_factor, int32_t* assign_q, int32_t* assign_k, float* qbar,
                                    float* kcent, void* ws, size_t ws_bytes, cudaStream_t stream);

/* Per-kernel timing for benchmarks (no counterpart in the paper).  muse_profile(1) clears the
 * record and makes every later library call record CUDA events on its stream around each
 * kernel launch (events are created on demand and reused); muse_profile(0) stops recording.
 * muse_profile_report waits for the last recorded event, then writes one text line per kernel
 * name, "name launches total_ms", into buf (HOST, cap bytes) and returns the byte count, or a
 * negative MUSE_ERR_* code.  Not thread-safe with respect to concurrent library calls. */
MUSE_API int muse_profile(int enable);
MUSE_API long muse_profile_report(char* buf, size_t cap);

/* Test hooks (no counterpart in the paper; not for production use).
 * muse_test_force_paths: bit mask; a set bit makes later calls take the library's other kernel
 *   for one step at shapes where the tensor-core kernel is the default (1 summaries, 2 far field
 *   forward and backward, 4 key-side summary backward, 8 retrieval forward per (cluster, plane)
 *   group, 16 retrieval backward as separate dQ and dK/dV kernels, 32 every tensor-core kernel of the
 *   dipole correction (merge, per-pair products, the dense contractions of its backward), 64 block
 *   selection of the two-level retrieval with a warp per query); 0 restores the default.
 *   Process-wide.
 * muse_test_wait_timeout: clears the status words of `ws` (>= 256 bytes) and launches a one-warp
 *   kernel whose bounded wait can never be satisfied, with a limit of `limit_clocks` SM clocks:
 *   word 0 ends up MUSE_STATUS_SELFTEST_TIMEOUT and the context stays usable. */
MUSE_API int muse_test_force_paths(unsigned mask);
MUSE_API int muse_test_wait_timeout(void* ws, unsigned limit_clocks, cudaStream_t stream);

/* Bounds-checked build (no counterpart in the paper).  The same sources compiled with
 * -DMUSE_DEBUG (python -m paper_2509_10406_b200.build --debug -> libmuse_debug.so) check every
 * index that a kernel derives from data (assignments, selections, pair ids, bucket offsets,
 * permutations) and the computed shared-memory offsets of its gathers against their bounds; an
 * index out of range is recorded and the access skipped, nothing traps.  muse_debug_report waits
 * for the device, writes one "file:line value v outside [0, n), c violation(s); " entry per source
 * file that recorded one into text (HOST, text_bytes; may be NULL) and returns the number of such
 * files, 0 when every check held; reset != 0 clears the records.  In the product build it
 * returns MUSE_ERR_UNSUPPORTED.  Not thread-safe with respect to concurrent library calls. */
MUSE_API int muse_debug_report(char* text, size_t text_bytes, int reset);

/* Human-readable text for a return code (static storage). */
MUSE_API const char* muse_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* MUSE_H_ */
