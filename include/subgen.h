/*
 * subgen.h - C ABI of the B200 (sm_100a) SubGen streaming-attention library.
 *
 * The library keeps, per (sequence, KV head) unit, the sublinear cache of "SubGen: Token
 * Generation in Sublinear Time and Memory" (Algorithm 1):
 *   D  - online threshold clustering of the keys: per cluster a representative (its first key),
 *        a member count and t uniformly sampled member keys (procedure UpdateSoftmaxNormalizer,
 *        Section 2.3, Lemma 2),
 *   M  - s (key, value) pairs sampled with probability proportional to ||v||^2, and the running
 *        mu = sum ||v||^2 (procedure UpdateMatrixProduct, Section 2.2, Lemma 1),
 *   a ring buffer with the most recent `window` tokens kept verbatim (the sliding window of
 *        Section 3.2),
 * and answers every stream step with the estimator z / tau of procedure QueryStreamAttn.
 *
 * Conventions
 *  - "device" pointers are CUDA device pointers owned by the caller; they must stay valid until
 *    the handle's stream has executed the call. "host" pointers are ordinary host memory.
 *  - Tensors are dense row-major; element type is the handle's dtype (fp32 or bf16), also for
 *    outputs.
 *  - Calls are asynchronous on the handle's stream unless stated otherwise. One handle is used by
 *    one host thread at a time.
 *  - Inputs are consumed in stream order: q, k, v, K, V may be written by earlier work on the same
 *    stream (the kernel that produced them), also when that work signals early completion to its
 *    successors (programmatic dependent launch). The first kernel of every call orders itself after
 *    everything earlier in the stream before it reads any input and before it touches anything that
 *    earlier work may still be using (what it does before that point reads only cache arrays that
 *    no kernel in flight writes). Inputs produced on ANOTHER
 *    stream need an event, as usual. One thing is asked of work that the caller enqueues on the
 *    handle's stream BETWEEN two calls: if it is itself launched with programmatic dependent launch, it
 *    must wait for its predecessors (cudaGridDependencySynchronize) before it completes, as ordinary
 *    kernels do implicitly; a call relies on "my predecessor has completed" implying "everything
 *    before it has completed".
 *  - Return value: 0 (SUBGEN_OK) or a negative SUBGEN_E* code for a host-side error;
 *    subgen_last_error() then gives a text. Problems found on the device (cluster capacity
 *    exhausted, non-finite or out-of-range input) never trap: they set sticky per-unit status
 *    bits, the unit's output becomes NaN, and subgen_status() reports the OR of all bits.
 *  - There is no CPU fallback. Every entry point fails if no CUDA device is usable.
 *
 * Arithmetic that decides an integer (which cluster a key joins, whether it opens one, every
 * sampling coin) is done in order-independent integer arithmetic so that the result is unique:
 *   D2(x,k) = sum_j floor(fl32(fl32(x_j-k_j)^2) * 2^32),  join <=> D2 <= floor(delta^2 * 2^32)
 *   W(v)    = sum_j floor(fl32(v_j*v_j) * 2^24),           mu = sum of W
 *   cluster coin (prob 1/n):      u * n        < 2^32
 *   value coin  (prob W/(mu+W)):  u * (mu + W) < W * 2^32
 * with u a 32-bit word of Philox4x32-10, key = seed, counter = (token index, unit index,
 * slot / 4, domain), word = slot % 4, domain 0 = cluster slots, 1 = value slots, unit index =
 * seq * Hkv + kvhead. Inputs must be finite with |x| <= 32768.
 */
#ifndef SUBGEN_H_
#define SUBGEN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SUBGEN_OK 0
#define SUBGEN_EINVAL (-1)  /* bad argument */
#define SUBGEN_ENOMEM (-2)  /* allocation failed or workspace too small */
#define SUBGEN_ESTATE (-3)  /* call not valid in the handle's state */
#define SUBGEN_ECUDA (-4)   /* a CUDA runtime call failed */

#define SUBGEN_DTYPE_FP32 0
#define SUBGEN_DTYPE_BF16 1

/* sticky per-unit status bits */
#define SUBGEN_ST_CAPACITY 1 /* a key had to open a cluster but m_max clusters exist; the key is dropped from D, the
                              * unit's outputs are NaN from then on and its M and mu are unspecified */
#define SUBGEN_ST_RANGE 2    /* non-finite input, or |x| > 32768 */
#define SUBGEN_ST_TIMEOUT 4  /* a bounded wait inside a kernel ran out (not expected; the state is unusable) */

typedef struct subgen subgen_t;
typedef struct subgen_exact subgen_exact_t;

typedef struct subgen_config {
    int B;          /* sequences */
    int H;          /* query heads per sequence */
    int Hkv;        /* KV heads per sequence; H % Hkv == 0, H / Hkv in {1,2,4,8}; 0 means Hkv = H */
    int d;          /* head dimension: 64 or 128 */
    float delta;    /* cluster radius (Algorithm 1 input delta), >= 0 */
    int t;          /* key samples per cluster (Algorithm 1 input t), 1..64 */
    int s;          /* value samples (Algorithm 1 input s), 1..65536 */
    int window;     /* recent tokens kept verbatim (Section 3.2), >= 0 */
    uint64_t seed;  /* Philox key */
    int dtype;      /* SUBGEN_DTYPE_* */
    int m_max;      /* cluster capacity per unit; 0 = 8192 */
    int splits;     /* thread blocks that share one unit in the step kernels; 0 = chosen from B*Hkv */
    void* workspace;        /* device, >= subgen_workspace_bytes(), 256-byte aligned, or NULL: the library allocates */
    size_t workspace_bytes;
    void* stream;           /* cudaStream_t, or NULL for the default stream */
    int nq_max;             /* most queries per head one subgen_query call may carry; 0 = 1; (H / Hkv) * nq_max <= 8 */
    int bounded;            /* 0: Algorithm 1 as printed, m_max is a capacity (exceeding it is an error);
                             * 1: m_max is a budget, see "Bounded-m variant" below */
    int step_mode;          /* how subgen_step runs on bf16 handles: SUBGEN_STEP_AUTO (0) picks by the number of
                             * units, SUBGEN_STEP_FUSED one kernel per step, SUBGEN_STEP_SPLIT three kernels
                             * (insertion, cluster scan, value scan). Same results either way. */
    int unit_stride;        /* Sharding: a handle that serves part of a larger job (some KV heads of every sequence, or */
    int unit_offset;        /* some sequences) should draw exactly the coins the whole job would. The Philox counter's
                             * unit index of this handle's (seq, kvhead) is seq * unit_stride + unit_offset + kvhead;
                             * unit_stride = 0 means Hkv (with unit_offset = 0: the plain numbering seq * Hkv + kvhead).
                             * A shard holding KV heads [h0, h1) of a job with HKV heads: unit_stride = HKV,
                             * unit_offset = h0; a shard holding sequences [b0, b1): unit_offset = b0 * Hkv. */
} subgen_config;

#define SUBGEN_STEP_AUTO 0
#define SUBGEN_STEP_FUSED 1
#define SUBGEN_STEP_SPLIT 2

/* Bounded-m variant (subgen_config.bounded = 1). Algorithm 1 keeps as many clusters as the keys need; the
 * paper bounds their number only through its clusterability assumption and names the incremental clustering of
 * Charikar et al. as the inspiration of its online clustering (Section 1.1). With bounded = 1 a key that would
 * need cluster number m_max + 1 makes the unit double its threshold instead (thr^2 <- max(4 thr^2, 1) in fixed
 * point, capped at 2^62) and sweep its clusters in index order: cluster i is kept if no kept representative lies
 * within the new threshold of x_i, else it is merged into the nearest kept one (ties: lowest kept index); kept
 * clusters are renumbered in order. A merge adds the counts and lets each sample slot q of the surviving cluster
 * take slot q of the merged one with probability n_i / (n_j + n_i), so that slots stay uniform over the union
 * (property 5 of Lemma 2): coin u * (n_j + n_i) < n_i * 2^32 with u = word q % 4 of Philox(counter = (token,
 * unit, q / 4 + 256 * i, 2 + 4 * doublings)), i the merged cluster's index before the sweep. The key is then
 * placed under the new threshold; if it still needs a new cluster and none is free, the threshold doubles again.
 * M, mu and the window are untouched. Such handles insert prompts token by token (the chunked prefill assumes
 * stable cluster indices within a chunk), and a sweep is done by one thread block, so the step that triggers
 * one takes milliseconds; thresholds double, so a unit sees few of them. */

/* Bytes of device memory a handle of this configuration needs (0 on invalid configuration). */
size_t subgen_workspace_bytes(const subgen_config* cfg);

/* Create a handle: bf16, Hkv = H, default capacity, library-owned memory, default stream.
 * Parameter names follow Algorithm 1 (delta, t, s) and Section 3.2 (window). NULL on error. */
subgen_t* subgen_create(int B, int H, int d, float delta, int t, int s, int window, uint64_t seed);
subgen_t* subgen_create_ex(const subgen_config* cfg);
void subgen_destroy(subgen_t* h);

/* Append n tokens per sequence to every unit's stream WITHOUT producing outputs. The resulting
 * state equals that of n update passes of the main loop of Algorithm 1 (UpdateSoftmaxNormalizer,
 * UpdateMatrixProduct, mu update) applied token by token to the tokens that leave the window.
 * K, V: device [B, Hkv, n, d]. May be called repeatedly. n = 0 is a no-op. */
int subgen_prefill(subgen_t* h, const void* K, const void* V, int n);

/* Same with one length per sequence. K, V: device [Hkv, total, d] with the sequences packed along
 * the token axis; cu_seqlens: HOST array of B+1 non-decreasing offsets, cu_seqlens[0] = 0,
 * cu_seqlens[B] = total. */
int subgen_prefill_varlen(subgen_t* h, const void* K, const void* V, const int* cu_seqlens);

/* One pass of the main loop of Algorithm 1 for every unit: the new token (k, v) enters the
 * window, the token it pushes out is inserted into D and M (old mu in the coin, then mu grows),
 * and the query q is answered from the updated state:
 *   z   = sum_{(k,v) in M} mu/(s ||v||^2) exp<q,k> v  +  sum_{window} exp<q,k> v
 *   tau = sum_{(x,S,n') in D} n'/t sum_{k in S} exp<q,k>  +  sum_{window} exp<q,k>
 *   out = z / tau                       (no 1/sqrt(d): Eq. 1 has none)
 * q, out: device [B, H, d]; k, v: device [B, Hkv, d]. Query head h uses KV head h / (H/Hkv). */
int subgen_step(subgen_t* h, const void* q, const void* k, const void* v, void* out);

/* Procedure QueryStreamAttn alone, for nq queries per head at once, against the state as it stands (all tokens
 * appended so far; nothing is inserted, nothing changes): out[b, h, j] = z / tau for query q[b, h, j]. The cache
 * is read once for all nq queries: they ride in the spare columns of the tensor-core tiles that otherwise carry
 * the H / Hkv heads of a KV head, so a call costs about what a step's query costs. Use: scoring several draft
 * continuations, or several heads' worth of probes, against one context. q, out: device [B, H, nq, d]; nq a
 * power of two, (H / Hkv) * nq <= 8 and nq <= the nq_max given at creation. Every sequence must hold a token. */
int subgen_query(subgen_t* h, const void* q, int nq, void* out);

/* subgen_step with HOST buffers, returning when out is filled. With page-locked (pinned, mapped) buffers the
 * step's kernels write out across the bus themselves and read q, k, v the same way (handles whose one-kernel step
 * runs many blocks per unit let one small kernel bring q, k, v over first): no copy engine, one wait. With pageable
 * buffers q, k, v are copied to the device first and out is copied back. Three-kernel handles leave one more kernel
 * on the stream when the call returns: the nearest-representative search for the token that the next step will take
 * out of the window, which that step then only applies (any other call on the handle discards it). */
int subgen_step_host(subgen_t* h, const void* q, const void* k, const void* v, void* out);

/* Waits for the stream, returns the OR of all units' status bits (>= 0) or a negative error. */
int subgen_status(subgen_t* h);

typedef struct subgen_state_view {
    int n;             /* tokens seen by this unit */
    int inserted;      /* tokens that have left the window = tokens represented by D and M */
    int m;             /* clusters */
    int status;        /* SUBGEN_ST_* bits */
    uint64_t mu;       /* fixed-point sum of W over inserted tokens */
    int last_cluster;  /* cluster joined or opened by the most recent insertion, -1 if none yet */
    int last_opened;   /* 1 if that insertion opened a cluster */
    uint64_t last_d2;  /* D2 to the representative it joined; not meaningful when it opened a cluster */
    /* caller-allocated HOST arrays, any may be NULL */
    int* counts;       /* [m_max]      n_i */
    int* centre_tok;   /* [m_max]      token index of representative x_i */
    int* slot_tok;     /* [m_max * t]  token index held by S_i(j) */
    int* m_tok;        /* [s]          token index held by M(j), -1 = null */
    uint64_t* m_w;     /* [s]          W of that token, 0 = null */
    /* outputs again */
    uint64_t threshold2; /* squared threshold in force, fixed point: floor(delta^2 2^32) * 4^doublings */
    int doublings;       /* threshold doublings so far (always 0 unless the handle is bounded) */
} subgen_state_view;

/* Synchronous copy of one unit's bookkeeping to the host (waits for the stream). */
int subgen_export_state(subgen_t* h, int seq, int kvhead, subgen_state_view* view);

/* Synchronous copy of one unit's stored vectors to the host. which: 0 representatives [m_max,d],
 * 1 cluster samples [m_max,t,d] (rows of a cluster with n_i = 1 are not materialised: such a
 * cluster's samples all equal its representative), 2 M keys [s,d], 3 M values [s,d],
 * 4 window keys [window,d], 5 window values [window,d] (token j sits in row j % window). */
int subgen_export_rows(subgen_t* h, int seq, int kvhead, int which, void* host, size_t bytes);

typedef struct subgen_stats {
    uint64_t units;
    uint64_t clusters;           /* sum of m */
    uint64_t singleton_clusters; /* clusters with n_i = 1 (read as one row, not t) */
    uint64_t m_filled;           /* non-null M slots */
    uint64_t window_rows;        /* tokens currently in the windows */
    uint64_t tokens;             /* sum of n */
    uint64_t prefill_pairs;      /* (key, representative) pairs the chunked prefill has scored: 2*d flops each */
    uint64_t insert_bytes;       /* bytes one step must read to place a key: bf16, the first 32 coordinates of every
                                  * representative and their norms (full rows follow only for those not ruled out
                                  * by that lower bound); fp32, the representatives */
    uint64_t query_bytes;        /* bytes one step must read to answer the queries: cluster_bytes + value_bytes */
    uint64_t cluster_bytes;      /* cluster samples (bf16: each distinct sampled row once, as the t reservoirs of a
                                  * cluster often hold the same token more than once; fp32: t rows; the
                                  * representative alone while n_i = 1) with counts and slot aliases */
    uint64_t value_bytes;        /* M keys and values with their weights, window keys and values */
    uint64_t distinct_sample_rows; /* over clusters with n_i > 1: slots that are the first to hold their token */
} subgen_stats;

/* Synchronous. Sums over all units, from the current state. */
int subgen_cache_stats(subgen_t* h, subgen_stats* out);

/* Kernel timing with CUDA events on the handle's stream. While enabled every subgen_step records
 * events around its kernels; subgen_profile_read waits, adds up the elapsed milliseconds since the last
 * read and resets. ms[0]: insertion kernel (window push, nearest representative, updates); ms[1]: scan
 * of the clusters (partition function); ms[2]: scan of M and the window plus the final merge. For fp32
 * handles the whole query is one kernel, reported in ms[1], and ms[2] is 0. */
int subgen_profile_enable(subgen_t* h, int on);
int subgen_profile_read(subgen_t* h, double ms[3], int* steps);
/* Phases of the most recent chunked prefill call made while profiling was enabled: ms[0] value phase (W, scan,
 * coins, gather), ms[1] sum over chunks of the score kernel, ms[2] sum over chunks of the resolve kernel. */
int subgen_profile_prefill_read(subgen_t* h, double ms[3]);

/* Number of kernels this handle has launched so far. */
uint64_t subgen_launch_count(const subgen_t* h);
/* Kernels one subgen_step launches on this handle: 1 (fused step: its whole duration is reported in ms[1] of
 * subgen_profile_read, ms[0] and ms[2] are 0), 2 (fp32) or 3. */
int subgen_step_kernels(const subgen_t* h);

/* Checkpoint and resume. The paper describes a stream that never stops; a serving process has to move a
 * conversation between GPUs or survive a restart, so the state between two calls (D with its samples and counts, M
 * with its weights, mu, the window ring, the per-unit counters and status bits) can be written to one host blob and
 * loaded into another handle. The blob stores cluster arrays only up to the largest cluster count of any unit.
 * Loading needs a handle created with the same B, H, Hkv, d, t, s, window, dtype, delta, seed and unit numbering (the Philox
 * draws of later tokens depend on the seed and on the token index, which the blob carries); m_max may differ as
 * long as it holds the stored clusters, which is also the way to continue a stream with a larger capacity.
 * Everything the handle held before is discarded. After a load the handle continues the stream exactly as the
 * saved one would have: the integer state stays identical token for token. All three calls are synchronous.
 * host: ordinary host memory (pinned memory makes the copies faster). */
int subgen_checkpoint_bytes(subgen_t* h, size_t* bytes);
int subgen_checkpoint_save(subgen_t* h, void* host, size_t bytes, size_t* written);
int subgen_checkpoint_load(subgen_t* h, const void* host, size_t bytes);

/* Growth of the cluster arrays. Algorithm 1 puts no bound on the number of clusters (Section 2.3: m depends on how
 * clusterable the keys are), while a handle's arrays hold m_max clusters per unit. subgen_grow re-lays the handle's
 * state out for a larger m_max on the device (one strided device copy per state array into a new workspace) and
 * leaves the stream exactly where it was: later steps and prefills give the integer state and the outputs that a
 * handle created with the larger m_max would give. Call it before a unit runs out of room (subgen_cache_stats and
 * subgen_export_state report the cluster counts); a SUBGEN_ST_CAPACITY bit that is already set stays set.
 * workspace: device memory owned by the caller for the new layout (subgen_workspace_bytes of the configuration
 * with the new m_max; 256-byte aligned, not overlapping the old one), or NULL: the library allocates it. The old
 * workspace is freed if the library had allocated it, else it is the caller's again once the call has returned.
 * Synchronous. m_max must exceed the current value (SUBGEN_EINVAL); bounded handles are refused (SUBGEN_ESTATE:
 * there m_max is the budget of the variant). Old and new workspace are both held until the copy is done. */
int subgen_grow(subgen_t* h, int m_max, void* workspace, size_t workspace_bytes);

/* Text of the calling thread's most recent error. */
const char* subgen_last_error(void);

/* ---- exact dense decode attention over a full KV cache: the comparison point (Eq. 1) ---------- */

/* Cache of up to n_max tokens per unit, K and V device [B*Hkv, n_max, d], owned by the library. */
subgen_exact_t* subgen_exact_create(int B, int H, int Hkv, int d, int n_max, int dtype, void* stream);
void subgen_exact_destroy(subgen_exact_t* h);
/* Append n tokens per sequence; K, V device [B, Hkv, n, d]. */
int subgen_exact_append(subgen_exact_t* h, const void* K, const void* V, int n);
/* Packed variant, layout and cu_seqlens as subgen_prefill_varlen. */
int subgen_exact_append_varlen(subgen_exact_t* h, const void* K, const void* V, const int* cu_seqlens);
/* Append (k, v), then out = softmax(K q)^T V over all cached tokens. Shapes as subgen_step. */
int subgen_exact_step(subgen_exact_t* h, const void* q, const void* k, const void* v, void* out);
/* Bytes one exact step must read (all cached keys and values), from the current lengths. Synchronous. */
int subgen_exact_bytes(subgen_exact_t* h, uint64_t* bytes);
uint64_t subgen_exact_launch_count(const subgen_exact_t* h);

/* Offline compression of the cache as in the paper's end-to-end experiment (Section 3.2): every unit keeps its r
 * most recent tokens and k centres chosen among the older ones by the greedy k-center algorithm (farthest-point
 * traversal: the first centre is the oldest token, each further centre is the token farthest from its nearest
 * chosen centre; fixed-point distances D2, ties to the lowest token index); with at most k older tokens all are
 * kept. Kept rows move to the front of the cache (centres in selection order, then the window) and later steps
 * attend them exactly and keep appending. Synchronous; allocates and frees its own scratch. */
int subgen_exact_kcenter_compress(subgen_exact_t* h, int k, int r);
/* Work done by the last compression, summed over units and passes: tokens_looked_at counts (token, pass) pairs
 * whose running distance was compared against a new centre; full_rows_read counts those for which the whole key
 * row had to be read because a lower bound from its first 16 coordinates did not settle the comparison. The
 * result never depends on which tokens were settled early. Either pointer may be NULL. */
int subgen_exact_kcenter_counters(const subgen_exact_t* h, uint64_t* tokens_looked_at, uint64_t* full_rows_read);
/* Stream positions of the tokens currently cached by one unit, in cache order. tok: host array of n_max ints
 * (may be NULL to query the count only). Synchronous. */
int subgen_exact_export_tokens(subgen_exact_t* h, int seq, int kvhead, int* n_out, int* tok);

/* ---- exact attention without any allocation -------------------------------------------------- */

/* The paper has no counterpart for this entry point; it exists for integration reasons only.
 *
 * Some callers must not call cudaMalloc, directly or through a library: a plugin running inside a
 * serving process whose own allocator claimed the device memory at start-up (a raw cudaMalloc
 * there fails or takes memory behind the allocator's back), or request-path code that cannot
 * afford the device-wide synchronisation an allocation or a free can cause. The handle-based
 * functions above allocate in their create call; this one needs no handle and allocates nothing,
 * neither with cudaMalloc/cudaFree nor through any allocating library routine.
 *
 * out = softmax(K q)^T V (Eq. 1, no scaling) for every head: q, out device [B, H, d]; K, V device
 * [B, Hkv, n, d], n >= 1; dtype, d and the H/Hkv rule as for subgen_exact_create; stream is a
 * cudaStream_t or NULL. The work of one (sequence, KV head) is split over several thread blocks;
 * their partial results and the arrival counters live in ONE fixed array of
 * SUBGEN_NOALLOC_SCRATCH_BYTES that is part of the library image: every GPU that loads the library
 * holds that much memory until the process exits. Shapes that need more than the array for a single
 * split, B*Hkv*(H/Hkv)*(d+2)*4 + 4*B*Hkv (rounded up to 256) bytes, are rejected with
 * SUBGEN_EINVAL and a message; larger split counts are reduced to fit.
 *
 * The first call on each device looks up the array's device address (the device must be current,
 * as for every call). Make that first call before starting any stream capture.
 *
 * All calls on a device share the array, and it keeps whatever the previous call left there. The
 * function clears the counters it needs on `stream` before the kernel; partial results are always
 * written before they are read. Two calls whose kernels can overlap on the GPU (different streams
 * without an ordering between them, or different host threads) race on the array and give wrong
 * results: order them.
 *
 * Returns 0 or a negative SUBGEN_E* code; asynchronous on `stream`. */
#define SUBGEN_NOALLOC_SCRATCH_BYTES (4u << 20)
int subgen_exact_attention_noalloc(const void* q, const void* K, const void* V, void* out, int B, int H, int Hkv,
                                   int d, int n, int dtype, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SUBGEN_H_ */
