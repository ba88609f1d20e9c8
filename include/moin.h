/*
 * moin.h - C ABI of the MoIN serving hot path for NVIDIA B200 (sm_100a).
 *
 * MoIN ("Mixture of Introvert Experts") routes every request to ONE expert - a LoRA adapter
 * on a frozen dense base model - and runs the whole forward pass with that adapter.  This
 * library is the data-parallel hot path of serving such a model on one GPU:
 *
 *   moin_route            query embedding -> nearest topic embedding -> expert id
 *   moin_plan_build       group the tokens of a batch by expert (once per batch)
 *   moin_lora_linear      y = x W^T + s (x A_e^T) B_e^T with the expert e differing per token
 *   moin_decoder_forward  Llama-architecture decoder whose seven per-block projections are
 *                         that layer
 *
 * General conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller unless the comment says
 *     "host".  The library borrows it for the duration of the call's work on `stream`; it
 *     never frees it and never allocates device memory itself (scratch comes in through the
 *     `workspace` arguments, sized by the *_workspace_bytes queries).
 *   - Descriptor structs (moin_router, moin_pool, moin_plan, moin_model) are plain host
 *     structs filled by the caller; arrays of pointers inside moin_model are HOST arrays of
 *     device pointers.
 *   - Matrices are row-major, bf16 (IEEE bfloat16 bit patterns) unless stated; device
 *     pointers to bf16/fp32 tensors must be 16-byte aligned (MOIN_ERR_MISALIGNED otherwise).
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = the legacy
 *     default stream) except where a comment says the call synchronises.  Errors that the
 *     host can detect are returned at once and nothing is launched.  Conditions only the
 *     device can see (an expert id outside [0, E), a bounded wait that ran out) never trap or
 *     hang: an out-of-range id means "no adapter" and is counted, a wait that runs out sets a
 *     flag, the kernel returns; both are read back with moin_device_status.
 *   - Results are deterministic: identical inputs give bit-identical outputs run to run.
 *   - Devices and threads: the library keeps its host-side state (side streams, events, the address of the
 *     status block, kernel attributes) per device ordinal and sets it up on the first call made with that
 *     device current, so one process may drive several GPUs; calls that target the SAME device must come
 *     from one host thread at a time (the per-device record and the side streams are not locked).
 *   - Arithmetic: bf16 operands, fp32 accumulation, one rounding to bf16 at the output.
 */
#ifndef MOIN_H_
#define MOIN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t moin_status;
typedef void* moin_stream; /* cudaStream_t */

enum {
  MOIN_OK = 0,
  MOIN_ERR_INVALID_ARG = -1,      /* null pointer, negative size */
  MOIN_ERR_BAD_SHAPE = -2,        /* a dimension violates the documented divisibility rules */
  MOIN_ERR_MISALIGNED = -3,       /* a tensor pointer is not 16-byte aligned */
  MOIN_ERR_WORKSPACE = -4,        /* workspace too small or null */
  MOIN_ERR_UNSUPPORTED_RANK = -5, /* LoRA rank not a multiple of 8 in 8..128 */
  MOIN_ERR_CUDA = -6,             /* a CUDA runtime/driver call failed (see moin_last_cuda_error) */
  MOIN_ERR_TIMEOUT = -7,          /* a device-side bounded wait ran out (reported by moin_device_status) */
  MOIN_ERR_NO_DEVICE = -8         /* no sm_100 device is current */
};

/* Human-readable name of a status code (static string). */
const char* moin_status_string(moin_status s);
/* Library version, major*10000 + minor*100 + patch. */
int32_t moin_version(void);
/* cudaError_t value of the last failing CUDA call seen by this library on this thread (0 = none). */
int32_t moin_last_cuda_error(void);

/* Device-side condition counters, accumulated since the last moin_device_status_reset. */
typedef struct {
  int32_t timeout_flag;       /* != 0: some bounded wait ran out; results of that call are undefined */
  int32_t timeout_site;       /* small integer naming the wait that gave up (diagnostic) */
  int32_t invalid_expert_ids; /* token expert ids outside [-1, E) seen by moin_plan_build (treated as -1) */
  int32_t reserved[5];
} moin_device_status_t;
/* Copies the counters to *out (host).  SYNCHRONISES `stream`. */
moin_status moin_device_status(moin_device_status_t* out, moin_stream stream);
moin_status moin_device_status_reset(moin_stream stream);

/* Self-test of the bounded wait (no counterpart in the paper).  Every device-side wait of the library gives up
 * after a time limit instead of hanging; a healthy run never gets there.  This call launches one tiny kernel
 * whose wait can never be satisfied (a barrier that nothing arms, no copy or MMA in flight) with a limit of
 * limit_us microseconds (1..1 000 000), so that the expiry path runs: the wait returns, a second waiter leaves
 * through the CTA's abort flag, the kernel ends normally, and moin_device_status afterwards shows timeout_flag
 * != 0 with timeout_site = 99.  result (device, 3 x int32): [0] = 0 if the first wait gave up, [1] = 0 if the
 * second waiter left through the abort flag, [2] = microseconds the kernel spent waiting.  Asynchronous on
 * `stream`.  Call moin_device_status_reset afterwards. */
moin_status moin_selftest_bounded_wait(int32_t limit_us, int32_t* result, moin_stream stream);

/* Testing/tuning knobs (host-side path selection only; every path computes the same function).
 *   MOIN_OPT_GEMM_IMPL: 0 = automatic, 1 = force the warp-MMA kernels, 2 = force the tcgen05 kernels
 *                       (calls whose shapes the forced kernel cannot take fail with MOIN_ERR_BAD_SHAPE). */
/*   MOIN_OPT_NVTX: 1 = every kernel group the library launches is wrapped in an NVTX range named like
 *   moin_kernel_name() (for timelines of tools that read NVTX); 0 (default) = no ranges. */
enum { MOIN_OPT_GEMM_IMPL = 1, MOIN_OPT_NVTX = 3 };
moin_status moin_set_option(int32_t key, int32_t value);

/* Per-kernel timing for benchmarks (no counterpart in the paper).  While enabled, every kernel group the
 * library launches is bracketed by a pair of CUDA events on the call's stream (this adds launch gaps:
 * never leave it on for a throughput measurement).  moin_profile_enable(capacity > 0) pre-creates the
 * events; capacity == 0 disables and frees them.  moin_profile_read SYNCHRONISES the device, writes up to
 * `capacity` records in launch order, sets *n to the number recorded since the last read, and clears them. */
typedef struct {
  int32_t kernel;   /* MOIN_K_* */
  int32_t launches; /* kernel launches inside the bracket */
  float ms;         /* device time between the two events */
} moin_profile_record;
enum {
  MOIN_K_ROUTE_SIMPLE = 0, MOIN_K_ROUTE_TC = 1, MOIN_K_ROUTE_FINISH = 2, MOIN_K_PLAN = 3, MOIN_K_GEMM_WARP = 4,
  MOIN_K_GEMM_TC = 5, MOIN_K_SHRINK_STREAM = 6, MOIN_K_EXPAND_STREAM = 7, MOIN_K_SHRINK_TC = 8,
  MOIN_K_FUSED_TC = 9, MOIN_K_GLUE = 10, MOIN_K_ATTENTION = 11, MOIN_K_ROUTE_CLUSTER = 12, MOIN_K_KMEANS_UPDATE = 13, MOIN_K_COUNT = 14
};
moin_status moin_profile_enable(int32_t capacity);
moin_status moin_profile_read(moin_profile_record* out, int32_t capacity, int32_t* n);
const char* moin_kernel_name(int32_t kernel);

/* ---------------------------------------------------------------------------------------
 * Router.  Paper Sec. 3.3 (model inference): the query is embedded and a nearest-neighbour
 * search over the topic embeddings picks the expert; the metric used here is the cosine
 * similarity, lowest index on exact ties.
 *
 *   id_i = argmax_k <q_i, c_k> / (|q_i| |c_k|)
 *
 * |q_i| is a positive per-query constant and is not needed for the argmax; |c_k| is, because
 * bf16-rounded "unit" vectors are not unit.  A zero-norm centroid has similarity -inf.
 * Similarities are accumulated in fp32 and compared in fp32.
 * ------------------------------------------------------------------------------------- */
typedef struct {
  const void* centroids;             /* [K, D] bf16 topic embeddings */
  const float* inv_norm;             /* [K] fp32, 1/|c_k| (0 for a zero-norm row); see moin_router_prepare */
  const int32_t* centroid_to_expert; /* [K] int32 or NULL: expert id of each topic, -1 = topic has no adapter
                                        (paper Sec. 4: some clusters were not retained) */
  int32_t K;                         /* number of topic embeddings, >= 1 */
  int32_t D;                         /* embedding dimension, multiple of 8, 8 <= D <= 8192 */
} moin_router;

/* Fills inv_norm[K] (fp32, device) from centroids[K, D].  Once per centroid table. */
moin_status moin_router_prepare(const void* centroids, int32_t K, int32_t D, float* inv_norm, moin_stream stream);

size_t moin_route_workspace_bytes(int32_t Q, int32_t K, int32_t D);
/* queries [Q, D] bf16 -> out_expert[Q] (int32: centroid_to_expert[id] if the map is given, else id),
 * out_centroid[Q] (nullable, int32 id), out_best_sim[Q] (nullable, fp32 cosine of the winner).
 * Q == 0 is a no-op.  Workspace contents are scratch. */
moin_status moin_route(const moin_router* router, const void* queries, int32_t Q, int32_t* out_expert,
                       int32_t* out_centroid, float* out_best_sim, void* workspace, size_t workspace_bytes,
                       moin_stream stream);

/* Router with runner-up.  Paper Sec. 3.3 routes by nearest topic embedding; how far the nearest is ahead of the
 * second nearest tells how safe that choice was (a query whose two best cosines differ by less than ~1e-4 sits
 * between two topics: a different rounding order may route it to the other one).  Same arguments and rules as
 * moin_route, plus
 *   out_second  [Q] int32, nullable: centroid index of the second-best similarity, -1 if there is none
 *   out_margin  [Q] fp32,  nullable: cos(best) - cos(second), +inf if there is no second candidate
 * out_expert and out_centroid may be NULL here.  Workspace: moin_route_top2_workspace_bytes. */
size_t moin_route_top2_workspace_bytes(int32_t Q, int32_t K, int32_t D);
moin_status moin_route_top2(const moin_router* router, const void* queries, int32_t Q, int32_t* out_expert,
                            int32_t* out_centroid, int32_t* out_second, float* out_best_sim, float* out_margin,
                            void* workspace, size_t workspace_bytes, moin_stream stream);

/* Routing for callers that cannot hand the library a workspace.  (The paper has no counterpart: this is
 * a packaging variant of moin_route, added for processes that must not allocate device memory - e.g. a
 * serving worker whose memory pool was sized and frozen at start-up, or a plug-in that runs inside
 * someone else's CUDA context and is forbidden to call cudaMalloc.)
 *
 * It computes what moin_route computes - same arguments minus the workspace, same choice of kernel for the
 * shape and the options in force, hence the same ids and the same cosines.  The per-query scratch that the
 * tensor-core router needs lives in a fixed array inside the library image (MOIN_ROUTE_STATIC_MAX_Q * 8 bytes
 * = 512 KiB, held by every GPU that loads the library until the process exits); shapes that moin_route serves
 * without scratch do not touch it.  The call performs no cudaMalloc/cudaFree and calls no allocating routine.
 *   - Q > MOIN_ROUTE_STATIC_MAX_Q returns MOIN_ERR_WORKSPACE and launches nothing.
 *   - The first call on each device that needs the array looks up its device address (with that device
 *     current); make that first call outside any stream capture, and from one host thread at a time (the
 *     look-up is not guarded against two threads making their first call together).
 *   - All calls share the one array, which keeps the previous call's contents; the part a call uses is
 *     cleared on `stream` before use.  Two calls whose GPU work overlaps (different streams, no ordering
 *     between them) race on it: order them, or use moin_route with separate workspaces. */
enum { MOIN_ROUTE_STATIC_MAX_Q = 65536 };
moin_status moin_route_static(const moin_router* router, const void* queries, int32_t Q, int32_t* out_expert,
                              int32_t* out_centroid, float* out_best_sim, moin_stream stream);

/* ---------------------------------------------------------------------------------------
 * Adapter pool of ONE projection.  Paper Sec. 3.2: W_a in R^{r x d}, W_b in R^{k x r} per
 * expert and linear layer; Sec. 1: the adapters in use are kept in GPU memory.  The pool
 * stores the paper's matrices as written, stacked over slots:
 *   A[n_slots, r, d_in] = W_a,  B[n_slots, d_out, r] = W_b,
 * and slot_of_expert[E] maps an expert id to its slot, -1 = the expert has no adapter
 * (paper Sec. 4: then the base model alone is used).
 *
 * Two optional members cover variants from the paper's future-work list (Sec. 5); zero / NULL gives the paper's
 * layer.  A caller that fills the struct member by member should zero it first.
 *   slot_rank   "adaptive rank": a rank per topic.  slot_rank[s] (device, [n_slots] int32, a multiple of 8 in
 *               [0, r]) is the rank of slot s; r stays the STORED rank (row count of A[s], row pitch of B[s]).
 *               Only the first slot_rank[s] rows of A[s] and columns of B[s] enter the result, and the kernels
 *               that stream adapters read nothing beyond them, so a low-rank topic costs proportionally fewer
 *               bytes.  What is stored beyond a slot's rank must be finite (the tensor-core path may multiply
 *               it by zero).  NULL: every slot has rank r.
 *   activation  a function applied between the two matrices: y = W x + s W_b act(W_a x); MOIN_ACT_*.
 * ------------------------------------------------------------------------------------- */
enum { MOIN_ACT_NONE = 0, MOIN_ACT_RELU = 1, MOIN_ACT_SILU = 2, MOIN_ACT_GELU = 3 /* 0.5 v (1 + erf(v / sqrt 2)) */ };
typedef struct {
  const void* A;
  const void* B;
  const int32_t* slot_of_expert; /* [E] int32, values in [-1, n_slots) */
  int32_t E;
  int32_t n_slots;
  int32_t r;     /* LoRA rank: multiple of 8, 8..128 (128 is the rank of the paper's experts, Sec. 4) */
  int32_t d_in;  /* multiple of 64 */
  int32_t d_out; /* multiple of 8 */
  int32_t activation;            /* MOIN_ACT_*; 0 = none (the paper's formula) */
  const int32_t* slot_rank;      /* device [n_slots] or NULL */
} moin_pool;

/* ---------------------------------------------------------------------------------------
 * Two-tier adapter store.  Paper Sec. 1: the adapters are small enough to be stored in bulk and the ones in
 * use are kept in GPU memory; fetching a missing one costs latency.  Here every expert's adapters stay in
 * HOST memory (E stacked adapters per projection, same layout as a pool), the device pools hold n_slots of
 * them, and moin_cache_admit - called between the router and the forward pass with the batch's expert ids on
 * the host - makes every expert of the batch resident: a hit only refreshes its age, a miss takes a free slot
 * or else the least recently used slot that this batch does not need, and enqueues one host-to-device copy
 * per matrix and projection on `stream`.  It then uploads the expert -> slot table (-1 = not resident) that
 * all the pools of the store share as their slot_of_expert.  Kernels already enqueued on `stream` still see
 * the old contents; everything enqueued after the call sees the batch's experts in place.
 *
 *   host_A [E, r, d_in], host_B [E, d_out, r]   host bf16, pinned for truly asynchronous copies
 *   dev_A [n_slots, r, d_in], dev_B [n_slots, d_out, r]   device bf16: the A / B of the projection's moin_pool
 * The object is host state plus a few small pinned staging buffers; it allocates no device memory.  One
 * thread at a time.  Errors: INVALID_ARG; WORKSPACE when a batch names more distinct experts than there are
 * slots (nothing is copied then); ids outside [0, E) are skipped (they mean "no adapter").
 * ------------------------------------------------------------------------------------- */
typedef struct moin_cache moin_cache;
typedef struct {
  const void* host_A;
  const void* host_B;
  void* dev_A;
  void* dev_B;
  int32_t r, d_in, d_out;
} moin_cache_projection;
moin_status moin_cache_create(int32_t E, int32_t n_slots, const moin_cache_projection* projs, int32_t n_projs,
                              int32_t* dev_slot_of_expert /* [E] device */, moin_cache** out);
void moin_cache_destroy(moin_cache* cache);
/* expert_ids: HOST array of n ids (one per request or token, repeats allowed).  n_missed / bytes_copied
 * (nullable): experts brought in by this call and the bytes of their copies. */
moin_status moin_cache_admit(moin_cache* cache, const int32_t* expert_ids, int32_t n, moin_stream stream,
                             int32_t* n_missed, uint64_t* bytes_copied);
/* Slot an expert occupies after the last admit (-1 = not resident); host bookkeeping only. */
moin_status moin_cache_slot_of(const moin_cache* cache, int32_t expert, int32_t* slot);

/* ---------------------------------------------------------------------------------------
 * Batch plan = the grouping of a batch's tokens by expert.  Paper Sec. 1 names the need
 * (many adapters in one batch) and Sec. 3.3 fixes that the expert is per request, so the
 * plan is built once per batch and reused by every projection of every block.
 *
 * The plan lives in a caller-provided device buffer of moin_plan_bytes(T, E) bytes and holds
 *   - a stable permutation of token indices ordered by expert id, with one segment
 *     (expert, start, length) per distinct expert - used when segments are short (decode);
 *   - the list of row tiles: maximal runs of consecutive tokens with one expert, cut into
 *     pieces of at most 128 rows - used when runs are long (prefill).  A build with mode
 *     MOIN_PLAN_SEGMENTS leaves this list empty (nothing in that mode reads it): such a plan
 *     must be rebuilt, not relabelled, before it is used as MOIN_PLAN_TILES.
 * Token expert ids: -1 = no expert (base model only); ids outside [-1, E) are treated as -1
 * and counted in moin_device_status.
 * ------------------------------------------------------------------------------------- */
enum {
  MOIN_PLAN_AUTO = 0,     /* choose from the built plan; moin_plan_build then SYNCHRONISES the stream */
  MOIN_PLAN_SEGMENTS = 1, /* short segments: stream each distinct adapter once over sorted tokens */
  MOIN_PLAN_TILES = 2     /* long runs: adapter folded into the tensor-core GEMM tile by tile */
};
typedef struct {
  void* buffer;        /* device, moin_plan_bytes(T, E) bytes, 16-byte aligned */
  size_t buffer_bytes;
  int32_t T;           /* tokens in the batch */
  int32_t E;           /* expert ids are in [0, E) */
  int32_t mode;        /* in: MOIN_PLAN_AUTO/SEGMENTS/TILES; out (AUTO only): the mode chosen */
  /* host-visible summary, filled only by an AUTO build (which synchronises): */
  int32_t n_segments, n_tiles, n_lora_tokens, max_segment;
} moin_plan;

size_t moin_plan_bytes(int32_t T, int32_t E);
/* token_expert [T] int32 (device).  Fills plan->buffer.  T == 0 is a no-op. */
moin_status moin_plan_build(const int32_t* token_expert, moin_plan* plan, moin_stream stream);

/* Copies the plan's arrays to host memory for inspection (tests).  Any pointer may be NULL.
 * perm[T]; seg_expert[S], seg_start[S+1] with S = *n_segments; tile_row0/rows/expert[n_tiles].
 * Output arrays must have room for T + 1 entries.  SYNCHRONISES `stream`. */
moin_status moin_plan_read(const moin_plan* plan, int32_t* n_segments, int32_t* n_tiles, int32_t* perm,
                           int32_t* seg_expert, int32_t* seg_start, int32_t* tile_row0, int32_t* tile_rows,
                           int32_t* tile_expert, moin_stream stream);

/* ---------------------------------------------------------------------------------------
 * K-means update.  Paper Sec. 3.1 (second approach): the topics are a K-means clustering of the
 * document embeddings; Sec. 4: the cluster centroid is the topic embedding the router searches.
 * One Lloyd iteration over N points is moin_route (assignment: nearest centroid under the cosine
 * metric), moin_plan_build on the N assignments with E = K (grouping of the points by cluster),
 * then this call: centroid k <- arithmetic mean of its members, summed in increasing point order
 * in fp32 and rounded once to bf16.  A cluster without members keeps its previous centroid;
 * points whose assignment is outside [0, K) belong to no cluster.
 *
 *   plan           built from the assignments (plan->T = N points, plan->E = K clusters), any mode
 *   x              device, [N, D] bf16 row-major, 16-byte aligned; D a multiple of 8, 8..8192
 *   centroids_old  device, [K, D] bf16; centroids_new device, [K, D] bf16 (may be the same buffer)
 *   inv_norm_new   device, [K] fp32 or NULL: 1/|c_k| of the NEW (bf16-rounded) centroids, 0 for a zero
 *                  row, i.e. what moin_router_prepare would compute for them
 * Asynchronous on `stream`; borrows everything, allocates nothing.  Errors: INVALID_ARG, BAD_SHAPE,
 * MISALIGNED; launches nothing on error.  N = 0 only copies the centroids. */
moin_status moin_kmeans_update(const moin_plan* plan, const void* x, const void* centroids_old, void* centroids_new,
                               float* inv_norm_new, int32_t D, moin_stream stream);


/* ---------------------------------------------------------------------------------------
 * Routed LoRA linear layer.  Paper Sec. 3.2: y = W x + W_b (W_a x), W in R^{k x d}; the
 * expert is the request's (Sec. 3.3); no adapter => W x only (Sec. 4).  With a scale s on
 * the low-rank term (s = 1 is the paper's formula):
 *
 *   y[t, :] = x[t, :] W^T + s * (x[t, :] A_e^T) B_e^T,   e = expert of token t
 *
 *   x [T, d_in] bf16, W [d_out, d_in] bf16, y [T, d_out] bf16 (must not alias x).
 *   pool == NULL (or plan == NULL): base layer only; then T, d_in, d_out come from base_T,
 *   base_d_in, base_d_out (ignored otherwise: plan->T and the pool give them).
 *   fp32 accumulation of the base and the low-rank term, added in fp32, rounded once to bf16.
 *   T == 0 is a no-op.  Workspace contents are scratch.
 * ------------------------------------------------------------------------------------- */
size_t moin_lora_linear_workspace_bytes(int32_t T, int32_t d_in, int32_t d_out, int32_t r);
moin_status moin_lora_linear(const moin_plan* plan, const void* x, const void* W, const moin_pool* pool,
                             float scale, int32_t base_T, int32_t base_d_in, int32_t base_d_out, void* y,
                             void* workspace, size_t workspace_bytes, moin_stream stream);

/* Grouped form: up to MOIN_MAX_GROUP projections that share the batch plan and do not depend on one
 * another - in a decoder block {q, k, v} and {gate, up} (paper Sec. 3.2: the adapter sits on every linear
 * layer, so independent layers of a block can be served together).  The result of every job is exactly
 * that of moin_lora_linear on it; the group exists because in the short-segment (decode) regime the
 * kernels are bound by adapter streaming plus a fixed per-launch cost, and one merged shrink and one
 * merged expand launch pay that cost once per group.  Every job needs a pool; the jobs' x, W, y follow
 * the rules of moin_lora_linear.  Workspace: moin_lora_linear_group_workspace_bytes. */
enum { MOIN_MAX_GROUP = 4 };
typedef struct {
  const void* x;          /* [T, pool->d_in] bf16 */
  const void* W;          /* [pool->d_out, pool->d_in] bf16 */
  const moin_pool* pool;  /* adapters of this projection */
  void* y;                /* [T, pool->d_out] bf16 */
} moin_lora_job;
size_t moin_lora_linear_group_workspace_bytes(int32_t T, const moin_lora_job* jobs, int32_t n_jobs);
moin_status moin_lora_linear_group(const moin_plan* plan, const moin_lora_job* jobs, int32_t n_jobs, float scale,
                                   void* workspace, size_t workspace_bytes, moin_stream stream);

/* ---------------------------------------------------------------------------------------
 * Decoder forward.  Paper Sec. 4: the base model is TinyLlama-1.1B (Llama-2 architecture);
 * Sec. 3.2: an adapter on each linear layer; Sec. 3.3: the request's expert for the whole
 * forward pass.  Conventions (the paper fixes none): pre-norm blocks; RMSNorm with gain;
 * rotary embedding pairing (i, i + head_dim/2), angle pos * rope_base^(-2i/head_dim),
 * positions restart at 0 per request; causal softmax attention within each request, scale
 * 1/sqrt(head_dim); query head h reads kv head h / (n_heads / n_kv_heads);
 * down(silu(gate(v)) * up(v)); no biases; untied lm_head; no adapter on embedding / lm_head.
 * Storage: residual stream fp32; norm outputs, projection outputs, rotated q/k, attention
 * output, SwiGLU output and logits bf16; the un-normalised attention weights exp(s - max) enter the
 * P V product as bf16 tensor-core operands (their sum, the softmax normaliser, is taken before rounding).
 * head_dim must be 64.
 * ------------------------------------------------------------------------------------- */
typedef struct {
  int32_t n_layers, hidden, n_heads, n_kv_heads, head_dim, ffn, vocab;
  float rms_eps, rope_base, lora_scale;
  const void* embed;             /* [vocab, hidden] bf16 */
  const void* lm_head;           /* [vocab, hidden] bf16 */
  const void* final_norm;        /* [hidden] bf16 gain */
  const void* const* attn_norm;  /* host array [n_layers] of device [hidden] bf16 */
  const void* const* mlp_norm;   /* host array [n_layers] of device [hidden] bf16 */
  const void* const* W;          /* host array [n_layers*7] of device [d_out, d_in] bf16; order q,k,v,o,gate,up,down */
  const moin_pool* pools;        /* host array [n_layers*7] or NULL (base model) */
  int32_t E;                     /* expert ids in [0, E) */
  /* Optional quantised base (see moin_dequant_fp8): host arrays [n_layers*7], either both NULL or both set; where
   * W8[i] is non-NULL the projection's weight is the dequantised W8[i] / W_scale[i] and W[i] is not read. */
  const void* const* W8;         /* device [d_out, d_in] bytes */
  const float* const* W_scale;   /* device [d_out] fp32 */
} moin_model;

/* Optional taps for block-by-block checks.  hidden_in (nullable, [T, hidden] fp32): start from this
 * residual stream instead of the embedding lookup; blocks [layer_begin, layer_end) are applied;
 * hidden_out (nullable, [T, hidden] fp32) receives the residual stream after them. */
typedef struct {
  const float* hidden_in;
  float* hidden_out;
  int32_t layer_begin, layer_end;
} moin_decoder_taps;

enum { MOIN_LOGITS_ALL = 0, MOIN_LOGITS_LAST = 1, MOIN_LOGITS_NONE = 2 };

size_t moin_decoder_workspace_bytes(const moin_model* model, int32_t R, int32_t T);
/* tokens [T] int32 packed request-major; cu_seqlens [R+1] int32 (cu[0] = 0, cu[R] = T);
 * req_expert [R] int32 (-1 = base only).  max_seqlen: host upper bound on a request's length.
 * logits: [T, vocab] bf16 (MOIN_LOGITS_ALL - what a perplexity evaluation needs) or [R, vocab]
 * (MOIN_LOGITS_LAST: last token of each request) or unused (MOIN_LOGITS_NONE). */
moin_status moin_decoder_forward(const moin_model* model, const int32_t* tokens, const int32_t* cu_seqlens,
                                 const int32_t* req_expert, int32_t R, int32_t T, int32_t max_seqlen,
                                 void* logits, int32_t logits_mode, const moin_decoder_taps* taps,
                                 void* workspace, size_t workspace_bytes, moin_stream stream);

/* Integration of a new or retrained expert into a resident pool.  Paper Sec. 1 / Sec. 5: experts are trained
 * independently and can be added or replaced one at a time.  Copies A_src [r, d_in] and B_src [d_out, r] (bf16;
 * device memory, or pinned host memory for a truly asynchronous copy) into slot `slot` of the pool and then maps
 * `expert` to it (slot_of_expert[expert] = slot), all on `stream`: calls issued later on that stream see the new
 * adapter, earlier ones the old one.  slot = -1 with NULL sources only unmaps the expert (it then runs on the base
 * model alone, Sec. 4).  The pool's tensors are the caller's; this call is the one place where the library writes
 * to them.  Errors: MOIN_ERR_INVALID_ARG (null pool / pointers, expert outside [0, E), slot outside [-1, n_slots)). */
moin_status moin_pool_set_adapter(const moin_pool* pool, int32_t expert, int32_t slot, const void* A_src,
                                  const void* B_src, moin_stream stream);

/* Quantised frozen base weights with 16-bit adapters.  Paper Sec. 5 lists a quantised base model ("QLoRA-like") as
 * a variant and fixes no format; the one taken here: one byte per weight in the 8-bit floating-point format with 4
 * exponent and 3 mantissa bits (bias 7, no infinities, 0x7F / 0xFF = NaN, largest finite value 448) and one fp32
 * scale per output row.  The weight the layer uses is W[j][i] = bf16(fp32(value(codes[j][i]) * scale[j])): this call
 * writes it, and the ordinary entry points then run on it, so the adapters, the accumulation and the tolerance are
 * those of the bf16 layer.  The base model is then stored in half of its bf16 size; a decoder forward with
 * moin_model.W8 set dequantises one projection group at a time into its workspace (at most three matrices live).
 *   codes  device, [d_out, d_in] bytes, 16-byte aligned; d_in a multiple of 16
 *   scale  device, [d_out] fp32
 *   W      device, [d_out, d_in] bf16, 16-byte aligned (output)
 * Asynchronous on `stream`.  Errors: MOIN_ERR_INVALID_ARG (null pointer, negative size), MOIN_ERR_BAD_SHAPE,
 * MOIN_ERR_MISALIGNED. */
moin_status moin_dequant_fp8(const void* codes, const float* scale, int32_t d_out, int32_t d_in, void* W,
                             moin_stream stream);

/* The same forward with one expert id per TOKEN: token_expert [T] int32, device, -1 = base only for that token.
 * Paper Sec. 5 (future work: "per-token adapters"); Sec. 3.3 itself uses one expert per request, which is the case
 * token_expert[t] = req_expert[request of t] and gives bit-identical results to moin_decoder_forward.  Every
 * projection of every block applies, row by row, the adapter of that row's token; attention, norms and the MLP
 * are unchanged.  The run structure of the ids is not known to the host, so the call reads the batch plan's
 * header back once (it synchronises `stream` once, before the first block).  All other arguments, layouts and
 * errors as for moin_decoder_forward; token_expert == NULL is MOIN_ERR_INVALID_ARG. */
moin_status moin_decoder_forward_per_token(const moin_model* model, const int32_t* tokens, const int32_t* cu_seqlens,
                                           const int32_t* token_expert, int32_t R, int32_t T, int32_t max_seqlen,
                                           void* logits, int32_t logits_mode, const moin_decoder_taps* taps,
                                           void* workspace, size_t workspace_bytes, moin_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* MOIN_H_ */
