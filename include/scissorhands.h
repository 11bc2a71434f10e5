/*
 * libscissorhands — budgeted KV-cache decode attention for NVIDIA B200 (sm_100a).
 *
 * C ABI of the data-parallel hot path of Scissorhands (arXiv 2305.17118):
 * per-step decode attention over a per-(sequence, head) KV cache held under a
 * fixed token budget B, fused with the importance-record update over the
 * history window w, and the compression step that evicts m tokens per
 * (sequence, head) once the cache fills while keeping the r most recent.
 *
 * Conventions
 *   - A "unit" is one independent (sequence, head) pair; a handle serves
 *     `heads` units (batch x heads of one layer).  Units never interact
 *     (Section 4.1 drops the layer and batch indices).
 *   - Every unit receives the same stream of calls, so the number of live
 *     tokens n and the step counter t are the same for all units and are kept
 *     on the host: no call below synchronises the device except sh_state,
 *     sh_export_unit and the *_host variants.
 *   - All device memory is owned by the caller.  The library allocates only a
 *     small host struct per handle.  Pointers named *_dev are device pointers,
 *     *_host are host pointers.  `stream` is a cudaStream_t passed as void*
 *     (NULL = the legacy default stream).  Calls enqueue work and return.
 *   - Every function returns an sh_status (0 = SH_OK, negative = error) and
 *     never aborts, throws or prints.  On error nothing has been enqueued
 *     unless stated otherwise.
 *   - A handle is not thread-safe: calls on one handle must not overlap (calls on
 *     different handles may, from any threads).  All calls that touch one
 *     handle's workspace should be given the same stream, or streams the
 *     caller has ordered; the library inserts no cross-stream dependencies.
 *   - Kernels that wait (on mbarriers) do so for a bounded time; one that gives
 *     up records a code in the workspace's error word, finishes without touching
 *     further state, and the next sh_state returns SH_EDEVICE.
 *   - Slots [0, n) of a unit's cache are live, in no particular order (a
 *     compression fills the holes it makes from the tail); sh_state's positions
 *     tell which token sits where.  With SH_OPT_COMPACTION = 0 compaction is
 *     stable and the slots stay sorted by stream position.
 */
#ifndef SCISSORHANDS_H_
#define SCISSORHANDS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sh_context *sh_handle;

typedef enum {
    SH_OK = 0,
    SH_EINVAL = -1, /* bad argument (NULL pointer, size out of range, bad dtype) */
    SH_EFULL = -2,  /* decode step on a full cache: call sh_compress first */
    SH_ESTATE = -3, /* call out of order (e.g. no workspace bound) */
    SH_ECUDA = -4,  /* a CUDA runtime call or launch failed; see sh_last_cuda_error */
    SH_ENOMEM = -5, /* host allocation failed or workspace too small */
    SH_ETOOBIG = -6, /* problem larger than a fixed-capacity entry point can take */
    SH_EDEVICE = -7  /* reported by sh_state: a kernel gave up one of its bounded waits on an
                        asynchronous copy and left its work undone */
} sh_status;

typedef enum {
    SH_F32 = 0,         /* K/V rows stored as fp32 */
    SH_F16 = 1,         /* fp16 */
    SH_BF16 = 2,        /* bf16 */
    SH_INT4_G64_F16 = 3 /* symmetric int4, groups of 64 along head_dim, fp16 scale per group;
                           q/k/v arrive as fp16 and rows are quantised when appended */
} sh_dtype;

typedef enum {
    SH_OPT_SOFTMAX_SCALE = 0, /* multiplier of the logits; default 1/sqrt(head_dim) */
    SH_OPT_SPLIT = 1,         /* CTAs cooperating on one unit (1, 2, 4 or 8); default chosen from `heads` */
    SH_OPT_AUTO_COMPRESS = 2, /* 1 (default): sh_decode_step compresses by itself when the cache fills;
                                 0: the caller calls sh_compress */
    SH_OPT_RECORD_MODE = 5,   /* 0 (default): the importance record is kept online, one comparison per cached
                                 token per step; 1: it is recomputed at every compression from the queries of
                                 the last w steps (the library keeps them: heads*w*head_dim extra elements)
                                 scored against the cache as it is then (Algorithm 2 as stated; Section 4.1,
                                 "Overhead Tradeoff").  Every storage type and head size (with
                                 SH_OPT_PREFILL_CHUNK = 2: fp16/bf16, head_dim 128 and budgets up to about 700
                                 only, else SH_EINVAL).  Set before sh_bind: it changes sh_workspace_bytes. */
    SH_OPT_COMPACTION = 6,    /* 1 (default): every hole left by a dropped token below n-m is filled with a kept
                                 row from the tail, so at most m rows move per compression; slots are then in no
                                 particular order: sh_state's pos tells which token sits where.
                                 0: stable left-compaction, slots stay sorted by stream position (nearly every
                                 surviving row moves: about three times the time per compression at B = 410,
                                 m = 64).  The kept set is the same either way: nothing in Algorithm 2 depends
                                 on where a token is stored. */
    SH_OPT_PREFILL_CHUNK = 4, /* 1 (default): sh_prefill hands the tokens between two compressions to a chunk
                                 kernel: the tcgen05 kernels for fp16/bf16/int4 with head_dim 128 (any budget;
                                 fp16/bf16: persistent CTAs fed by tiled TMA copies, up to 128 tokens a launch), the CUDA-core kernel for
                                 fp32 rows and for head_dim 64; 0: one decode step per token; 2: the warp-level
                                 MMA chunk kernel where it applies (fp16/bf16, head_dim 128, budgets up to about
                                 700); 3: as 1, but fp16/bf16 use the tcgen05 kernel with one CTA per unit and
                                 per-thread asynchronous copies; 4: the CUDA-core kernel for every shape */
    SH_OPT_DECODE_KERNEL = 3, /* 0 (default): chosen from the shape; 1: one CTA (or cluster) per unit with
                                 direct loads; 2: persistent CTAs fed by bulk asynchronous copies
                                 (stored rows of 256 bytes or more: fp32, and fp16/bf16 with head_dim 128; SH_OPT_SPLIT
                                 ignored; other shapes use 1) */
    SH_OPT_SELFTEST_SKIP_TILE = 7 /* -1 (default): off.  k >= 0: self-test of the give-up path of the bounded waits.
                                 In the kernel of SH_OPT_DECODE_KERNEL = 2 the first CTA never requests the k-th
                                 tile of rows it was due to stream, so the wait for that tile runs out after
                                 about a second, the CTA finishes without touching further cache state, and the
                                 next sh_state returns SH_EDEVICE.  Outputs of such a step are meaningless.
                                 The persistent tcgen05 chunk kernel (SH_OPT_PREFILL_CHUNK = 1, fp16/bf16,
                                 head_dim 128) honours it the same way: its first CTA never requests the k-th key
                                 tile of a launch (tiles counted over both sweeps), every role of that CTA gives up
                                 within a few seconds and releases its tensor memory. */
} sh_option;

/*
 * Create a handle.  Definition 4.1 and the inputs of Algorithms 1 and 2:
 * B = token budget per unit, r = recent window (never evicted), w = history
 * window of the importance record in steps, m = tokens dropped per
 * compression, heads = number of units, head_dim = d.
 * Requires 1 <= B <= 32768, r >= 0, 1 <= w <= 16384, 1 <= m <= B - r,
 * head_dim in {64, 128} (int4: 128 or 64), dtype an sh_dtype.
 * Errors: SH_EINVAL, SH_ENOMEM.
 */
int sh_create(int B, int r, int w, int m, int heads, int head_dim, int dtype, sh_handle *out);

/* Free the host struct.  Device memory stays with the caller. */
void sh_destroy(sh_handle h);

/* Bytes of device workspace the handle needs (K, V, scales, record bit-planes,
 * positions, selection scratch, staging for the *_host calls). */
size_t sh_workspace_bytes(sh_handle h);

/*
 * Give the handle its workspace: `bytes` >= sh_workspace_bytes(h) of device
 * memory aligned to 256 bytes, owned by the caller and kept alive until
 * sh_destroy.  The library zero-fills it on `stream` and resets n = t = 0.
 * Errors: SH_EINVAL (NULL, misaligned), SH_ENOMEM (too small), SH_ECUDA.
 */
int sh_bind(sh_handle h, void *slab_dev, size_t bytes, void *stream);

/* Set an option before the first step.  Errors: SH_EINVAL, SH_ESTATE. */
int sh_set_option(sh_handle h, int key, double value);

/*
 * One generation step of Algorithm 1 for every unit: append (k_new, v_new) as
 * the token at stream position t+1 (n <- n+1), attend with q over the n
 * cached tokens including the new one (estimator of Section 4.1:
 * alpha_j = softmax_j(scale*<q,K[j]>), out = sum_j alpha_j V[j]), and record
 * for every cached token whether alpha_j < 1/(t+1) as this step's entry of
 * the importance record (Algorithm 2's loop body, maintained online as the
 * "Overhead Tradeoff" paragraph describes).  With SH_OPT_AUTO_COMPRESS the
 * compression of Algorithm 2 follows when n == B.
 * q_dev, k_new_dev, v_new_dev: [heads][head_dim] in the handle's dtype (fp16
 * for the int4 store), 16-byte aligned.  attn_out_dev: [heads][head_dim] fp32,
 * 4-byte aligned.
 * Errors: SH_EFULL when n == B on entry, SH_EINVAL (NULL or misaligned pointer, more than
 * 2^24 - 1 tokens streamed), SH_ESTATE, SH_ECUDA.
 */
int sh_decode_step(sh_handle h, const void *q_dev, const void *k_new_dev, const void *v_new_dev,
                   float *attn_out_dev, void *stream);

/*
 * Same step with HOST buffers; returns after `stream` has been synchronised,
 * with attn_out_host filled.  Page-locked (pinned), 16-byte aligned buffers are
 * read and written by the kernel directly over PCIe, overlapped with the
 * streaming of K and V; pageable buffers are staged through the workspace with
 * cudaMemcpyAsync before and after the kernel.
 */
int sh_decode_step_host(sh_handle h, const void *q_host, const void *k_new_host, const void *v_new_host,
                        float *attn_out_host, void *stream);

/*
 * Prompt phase, stream semantics of Definition 4.1: equivalent to p calls of
 * sh_decode_step (each followed by a compression when the cache fills),
 * whatever SH_OPT_AUTO_COMPRESS says.  q_dev, k_dev, v_dev: time-major
 * [p][heads][head_dim].  out_dev: [p][heads][head_dim] fp32 or NULL to discard.
 * Between two compressions the steps only append, so they are evaluated up to
 * 64 at a time by a chunk kernel (causal attention of the chunk over the cache
 * and itself, one record bit-plane row per step: on the tensor cores for fp16,
 * bf16 and int4 stores with head_dim 128, on CUDA cores otherwise); the results
 * equal the per-token path up to fp32 summation order.  SH_OPT_PREFILL_CHUNK = 0
 * forces the per-token path.
 * At most 2^24 - 1 tokens may be streamed through a handle.
 */
int sh_prefill(sh_handle h, const void *q_dev, const void *k_dev, const void *v_dev, int p,
               float *out_dev, void *stream);

/*
 * The prompting stage read as a bulk operation (Section 2: the prompt's keys and values are computed
 * and cached in full before generation starts), as an alternative to the token stream of
 * Definition 4.1 that sh_prefill implements.  `src` holds a cache that was never compressed (a handle
 * whose budget exceeds the prompt, fed through sh_prefill: its outputs are full causal attention and
 * its record holds the prompt's last w steps).  Algorithm 2 is applied to it as often as needed with
 * dst's r and m - same record, m tokens per round, the r newest protected - until fewer than dst's
 * B tokens remain; the survivors with their record, positions (and stored queries) become the cache
 * of `dst`, which continues at t = src's t.  src is left compressed.
 * dst must be bound and fresh (nothing streamed); both must agree in heads, head_dim, dtype, w and
 * SH_OPT_RECORD_MODE, and neither may hold ragged sequences.  Asynchronous on `stream`.
 * Errors: SH_EINVAL (mismatch, or fewer than m candidates outside the recent window), SH_ESTATE, SH_ECUDA.
 */
int sh_import_compressed(sh_handle dst, sh_handle src, void *stream);

/*
 * The same in one call for a fresh handle h: the p prompt tokens (layout as sh_prefill, 1 <= p <= 32767)
 * are attended in full in a scratch workspace of sh_prefill_bulk_scratch_bytes(h, p) bytes (device
 * memory, 256-byte aligned, the caller's; it holds the whole prompt's keys and values and may be freed
 * or reused once `stream` has passed this call), then compressed into h as sh_import_compressed does.
 * out_dev: [p][heads][head_dim] fp32 or NULL.
 */
int sh_prefill_bulk(sh_handle h, const void *q_dev, const void *k_dev, const void *v_dev, int p, float *out_dev,
                    void *scratch_dev, size_t scratch_bytes, void *stream);
size_t sh_prefill_bulk_scratch_bytes(sh_handle h, int p);

/*
 * Prompts of different lengths (Section 4.1 treats one head of one sequence; a batch is many such
 * streams, and real batches are ragged).  The handle's units are n_sequences groups of
 * heads / n_sequences consecutive units; sequence i consumes the first lengths_host[i] <= p_max
 * tokens of its units' columns of the time-major blocks q/k/v [p_max][heads][head_dim] (the rest
 * is ignored), with compressions whenever its own cache fills.  Afterwards n and t differ per
 * sequence: they live in per-unit device arrays that the kernels read and advance, every
 * sh_decode_step appends one token to every sequence, a compression runs whenever some sequence's
 * cache is full and touches only those, and sh_sequence_state reports the per-sequence counters.
 * Needs a freshly bound handle (nothing streamed yet) and heads % n_sequences == 0.
 * Not available with SH_OPT_RECORD_MODE = 1; sh_prefill, sh_prefill_chunk and sh_restore are not
 * available afterwards (SH_ESTATE).  out_dev as for sh_prefill (rows past a sequence's length are
 * not written).
 */
int sh_prefill_ragged(sh_handle h, const void *q_dev, const void *k_dev, const void *v_dev, int p_max,
                      const int *lengths_host, int n_sequences, float *out_dev, void *stream);

/* Per-sequence live tokens and tokens streamed (one entry, the common values, unless
 * sh_prefill_ragged was used).  Fills at most `capacity` entries; returns the number of sequences. */
int sh_sequence_state(sh_handle h, int *n_host, long long *t_host, int capacity);

/*
 * One chunk of the prompt without the compression: steps t+1 .. t+count for
 * every unit in one launch (see sh_prefill).  Needs 1 <= count <=
 * sh_prefill_chunk_max(h) and count <= B - n; returns SH_EINVAL otherwise
 * (sh_prefill_chunk_max is min(128, w) on the default kernel of fp16/bf16 stores with head_dim 128,
 * min(64, w) on every other chunk kernel, or 0 where SH_OPT_PREFILL_CHUNK = 2 does not apply).
 * Layout as sh_prefill.  The caller compresses when n reaches B.
 */
int sh_prefill_chunk(sh_handle h, const void *q_dev, const void *k_dev, const void *v_dev, int count,
                     float *out_dev, void *stream);
int sh_prefill_chunk_max(sh_handle h);

/*
 * Algorithm 2 for every unit, if the cache is full (n == B): importance
 * record I_j = number of the last w steps at which token j was below the
 * threshold; the r newest tokens are not candidates; the m candidates with
 * the largest I are dropped, the oldest first among equal I; K, V, record and
 * positions of the survivors are compacted in place into slots [0, n-m) (see
 * SH_OPT_COMPACTION for their order); n <- n-m.
 * A no-op when n < B.  *evicted_per_unit (may be NULL) receives m or 0.
 */
int sh_compress(sh_handle h, void *stream, int *evicted_per_unit);

/*
 * sh_compress for callers that cannot allocate device memory.  (The paper has
 * no counterpart: this is a deployment variant of sh_compress, same result.)
 *
 * Some users of this library never get to call cudaMalloc after start-up: a
 * serving engine that gives all of HBM to its own KV-block pool has nothing
 * left to ask for, and code inside a latency-critical decode loop must avoid
 * the device-wide synchronisation an allocation implies.  For them this entry
 * point keeps the selection's result list (one int32 per unit and slot: the
 * source slot of every surviving row, or the list of moves, written by the
 * select-m kernel and read by the compaction kernel) in a static device array
 * inside the library instead of the workspace's region for it, and calls no
 * allocator of any kind.  Only that list is static: the record, the positions
 * and a per-unit move count stay in the handle's workspace, as for sh_compress.
 * Where one kernel does selection and compaction together (SH_OPT_COMPACTION = 1
 * with bit-planes that fit in shared memory) no list leaves the kernel and the
 * array is not touched.
 *
 * Limit: heads * B <= SH_STATIC_SCRATCH_MAX_ENTRIES (4 MiB of device memory,
 * held by every GPU that loads the library until the process exits); beyond it
 * the call returns SH_ETOOBIG and does nothing.  Inputs and outputs are the
 * handle's bound workspace, exactly as for sh_compress.
 * The first call on each device looks up the array's device address (with that
 * device current).  Make that first call at start-up: before any stream
 * capture, and before the rest of device memory is handed to a pool, since the
 * CUDA runtime may load the library's device code, and with it reserve the
 * array, only then.
 * All calls on a device share the one array and it keeps the previous call's
 * contents.  Nothing in it needs to start at zero: the selection writes every
 * entry the compaction reads.  Two calls whose kernels overlap on the GPU
 * (different streams, different handles) race on it: serialise them.
 */
#define SH_STATIC_SCRATCH_MAX_ENTRIES (1u << 20)
int sh_compress_static(sh_handle h, void *stream, int *evicted_per_unit);

/*
 * Selection of Algorithm 2 on caller-supplied records, for testing the
 * selection kernel on its own: counters_dev [units][n] uint16 (tokens in
 * position order); evicted_dev [units][m] int32 receives the indices of the
 * dropped tokens in ascending order.  Needs 0 <= r, 1 <= m <= n - r,
 * n <= SH_SELECT_MAX_N (counters and histogram share the CTA's shared memory),
 * every counter <= 16384; SH_EINVAL otherwise.  Uses no handle and no workspace.
 */
#define SH_SELECT_MAX_N 40000
int sh_select(const uint16_t *counters_dev, int units, int n, int r, int m, int32_t *evicted_dev,
              void *stream);

/*
 * Snapshot for checking and checkpointing; synchronises `stream`.  Any output
 * pointer may be NULL.  n_out: live tokens per unit (-1 after sh_prefill_ragged: they differ).
 * t_out: tokens streamed (the largest, after sh_prefill_ragged).
 * pos_host [heads][B] int32: stream positions (1-based) of slots [0,n), 0 beyond.
 * counters_host [heads][B] uint16: importance record I of Algorithm 2 at the
 * current step, 0 beyond n.  low_host [heads][ceil(B/32)] uint32: bit j%32 of
 * word j/32 = the last step's comparison alpha_j < 1/t for the token now in slot j
 * (a compression that followed the step has already moved the bits with their tokens).
 */
int sh_state(sh_handle h, void *stream, int *n_out, long long *t_out, int32_t *pos_host,
             uint16_t *counters_host, uint32_t *low_host);

/*
 * SH_OPT_RECORD_MODE = 1 only: recompute the record now (what sh_compress does first in that
 * mode): each query of the last w steps (t-w, t] is scored against the cached tokens that
 * already existed at its step, softmax over those, and alpha_j < 1/step becomes that step's
 * bit-plane row.  A following sh_compress at the same step uses the result as it stands.
 * Errors: SH_ESTATE when the handle keeps its record online.
 */
int sh_recompute_record(sh_handle h, void *stream);

/*
 * Analysis entry point (paper, "Ablation on Attention Score Error": the change ratio
 * (alpha_s - alpha_o) / alpha_o between the scores over a budgeted cache and over the full one).
 * Attention scores of query q ([heads][head_dim], device, the handle's input dtype) over each unit's
 * present cache: alpha_out[u][j] = softmax_j(scale * q_u . k_j) over the live slots j < n of unit u,
 * 0 for the other slots; alpha_out is device memory, fp32, [heads][B].  Nothing is appended, the
 * record and the counters do not change.  Asynchronous on `stream`.  int4 caches are scored on their
 * dequantised keys.  Errors: SH_EINVAL (NULL argument), SH_ESTATE (not bound), SH_ECUDA.
 */
int sh_scores(sh_handle h, const void *q, float *alpha_out, void *stream);

/* The record bit-planes of one unit, [w][ceil(B/32)] uint32 on the host: row (s mod w) holds, for
 * step s of the last w steps, bit j%32 of word j/32 = [alpha_j < 1/s] for the token now in slot j.
 * Synchronises. */
int sh_export_record(sh_handle h, int unit, uint32_t *planes_host, void *stream);

/* Stored K and V rows of one unit as fp32 (int4: dequantised), [B][head_dim]
 * each on the host; rows beyond n are whatever the slots hold.  Synchronises. */
int sh_export_unit(sh_handle h, int unit, float *K_host, float *V_host, void *stream);

/*
 * Resume from a workspace image: after the caller has copied back a saved
 * copy of the whole workspace, set the host counters that went with it
 * (0 <= n <= B, n <= t < 2^24; with n == B the next call must be sh_compress).
 * Not available once sh_prefill_ragged has run (SH_ESTATE): the per-sequence
 * counters then live in the workspace image itself and one (n, t) pair cannot
 * describe them.  Errors: SH_EINVAL, SH_ESTATE.
 */
int sh_restore(sh_handle h, int n, long long t);

/* Number of kernels this handle has launched since creation. */
long long sh_launch_count(sh_handle h);

/* Which fused decode kernel sh_decode_step launches for this handle's shape and options
 * (see SH_OPT_DECODE_KERNEL): 1 = one CTA or cluster per unit with direct loads, 2 = persistent
 * CTAs fed by bulk asynchronous copies, 3 = the int4 store's kernel for many units (codes unpacked
 * to fp16, dot products as tensor-core MMAs; chosen automatically from 592 units on with head_dim
 * 128, SH_OPT_DECODE_KERNEL = 1 keeps the CUDA-core kernel).  For reports and profiles. */
int sh_decode_kernel_choice(sh_handle h);

/* Text for a status code; never NULL. */
const char *sh_strerror(int status);

/* cudaGetErrorString of the last CUDA failure seen by this handle ("" if none). */
const char *sh_last_cuda_error(sh_handle h);

#ifdef __cplusplus
}
#endif
#endif /* SCISSORHANDS_H_ */
