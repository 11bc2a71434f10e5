// Internal declarations shared by the translation units of libscissorhands.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <vector>

#include "scissorhands.h"

// Byte offsets of the regions inside the caller's workspace slab.
struct ShLayout {
    size_t K, V;            // [U][B][row_bytes]
    size_t Ks, Vs;          // int4 only: [U][Bs][D/64] fp16 group scales (Bs = B rounded up to 8: every unit 16-byte aligned)
    size_t hist;            // [U][w][Bw] u32 bit-planes: row (step mod w), bit j = "slot j was low at that step"
    size_t pos;             // [U][B] int32 stream positions
    size_t src_idx;         // [U][B] int32 selection result: source slot of each surviving destination slot
    size_t counters;        // [U][B] u16 scratch for sh_state
    size_t xport;           // [2][B][D] fp32 scratch for sh_export_unit
    size_t stage_q, stage_k, stage_v, stage_out;  // staging for the *_host calls
    size_t err;             // one int: set by a kernel whose bounded wait gave up
    size_t qring;           // record_mode 1 only: [U][w][in_bytes] queries of the last w steps
    size_t n_arr, t_arr;    // [U] int32 each: per-unit live rows / tokens streamed (sequences of different lengths)
    size_t total;
};

struct sh_context {
    int B, r, w, m, U, D, dtype;
    int Bw;          // ceil(B / 32)
    int Bs;          // scale rows per unit of the int4 store: B rounded up to a multiple of 8
    int row_bytes;   // bytes of one stored K (or V) row, without int4 scales
    int in_bytes;    // bytes of one q / k_new / v_new row
    int n;           // live tokens per unit
    long long t;     // tokens streamed per unit
    float scale;
    int split;
    bool split_explicit;   // SH_OPT_SPLIT was set by the caller
    int auto_compress;
    int unordered;      // SH_OPT_COMPACTION: 0 stable left-compaction, 1 holes filled from the tail (slots unordered)
    int record_mode;    // SH_OPT_RECORD_MODE: 0 record kept online, 1 recomputed at compression from stored queries
    long long record_fresh_t;   // record_mode 1: step for which the bit-planes were last recomputed (-1: never)
    int prefill_chunk;  // SH_OPT_PREFILL_CHUNK: 1 = sh_prefill may batch tokens between compressions
    int kernel;      // SH_OPT_DECODE_KERNEL: 0 automatic, 1 direct loads, 2 pipelined bulk copies
    int selftest_skip_tile;   // SH_OPT_SELFTEST_SKIP_TILE: -1, or the tile CTA 0's producer leaves out
    bool started;    // a step has run: options are frozen
    char *slab;
    size_t slab_bytes;
    ShLayout L;
    long long launches;
    cudaError_t last_err;
    // Active range of units: normally all of them.  While a ragged prompt is streamed, one
    // sequence's units at a time, with n and t above holding for that sequence.
    int u0, ucount;
    // Sequences of different lengths (after sh_prefill_ragged): per-sequence mirrors of the
    // device arrays n_arr / t_arr; units_per_seq consecutive units form a sequence.
    bool ragged;
    int units_per_seq;
    std::vector<int> n_seq;
    std::vector<long long> t_seq;
};

// Programmatic dependent launch.  The decode kernels are launched with programmatic stream serialisation:
// the next kernel of the stream may be scheduled while this one still runs, which hides its launch latency
// and start-up behind this kernel's tail.  sh_pdl_launch_dependents() (first thing in the kernel) says the
// next kernel may be scheduled once every CTA of this one has got that far; sh_pdl_wait() returns when the
// preceding kernel of the stream has completed and its writes are visible: nothing that depends on earlier
// work (any global memory of the workspace or of the caller) is touched before it.
#ifdef __CUDACC__
__device__ __forceinline__ void sh_pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void sh_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

// Bounds-checked build (-DSH_DEBUG_BOUNDS, build.build(debug_bounds=True)): the stand-in for a memory checker.
// Every index a kernel derives from state it reads back from the workspace (per-unit row counts and step
// numbers, source slots, move lists) is range-checked before it is used; a violation records a code
// 0x7xx in the device error word and the unit, or the one access, is skipped, so nothing is read or written
// out of range and nothing traps.  sh_state then returns SH_EDEVICE.  In the normal build the checks vanish.
#ifdef SH_DEBUG_BOUNDS
#define SH_BOUNDS_OK(cond, err, code) ((cond) ? true : ((err) ? (atomicCAS((err), 0, (code)), false) : false))
#else
#define SH_BOUNDS_OK(cond, err, code) true
#endif

// Base pointers of the active unit range inside the workspace.
inline char *sh_pK(const sh_context *c) { return c->slab + c->L.K + (size_t)c->u0 * c->B * c->row_bytes; }
inline char *sh_pV(const sh_context *c) { return c->slab + c->L.V + (size_t)c->u0 * c->B * c->row_bytes; }
inline char *sh_pKs(const sh_context *c) { return c->slab + c->L.Ks + (size_t)c->u0 * c->Bs * (c->D / 64) * 2; }
inline char *sh_pVs(const sh_context *c) { return c->slab + c->L.Vs + (size_t)c->u0 * c->Bs * (c->D / 64) * 2; }
inline uint32_t *sh_phist(const sh_context *c) {
    return reinterpret_cast<uint32_t *>(c->slab + c->L.hist) + (size_t)c->u0 * c->w * c->Bw;
}
inline int32_t *sh_ppos(const sh_context *c) { return reinterpret_cast<int32_t *>(c->slab + c->L.pos) + (size_t)c->u0 * c->B; }
inline int32_t *sh_psrc(const sh_context *c) { return reinterpret_cast<int32_t *>(c->slab + c->L.src_idx) + (size_t)c->u0 * c->B; }
inline char *sh_pqring(const sh_context *c) {
    return c->record_mode ? c->slab + c->L.qring + (size_t)c->u0 * c->w * c->in_bytes : nullptr;
}
inline int *sh_pnarr(const sh_context *c) { return c->ragged ? reinterpret_cast<int *>(c->slab + c->L.n_arr) + c->u0 : nullptr; }
inline int *sh_ptarr(const sh_context *c) { return c->ragged ? reinterpret_cast<int *>(c->slab + c->L.t_arr) + c->u0 : nullptr; }

struct DecodeParams {
    const void *q, *k_new, *v_new;
    float *out;
    char *K, *V;
    char *Ks, *Vs;
    uint32_t *hist;
    int32_t *pos;
    char *qring;    // [U][w][row] ring of the last w queries (row = step mod w), or NULL
    int *n_arr, *t_arr;   // per-unit live rows / tokens streamed before this step (sequences of different
                          // lengths), updated by the kernel; NULL when n and t below hold for every unit
    int U, B, Bw, w;
    int Bs;         // scale rows per unit (int4 store)
    int n;          // live rows per unit including the token appended by this step
    int hist_row;   // t mod w
    int t;          // 1-based stream position of this step's token
    float scale_log2e;
    int *err;                 // device error word (bounds-checked build; a bounded wait that gave up)
    int selftest_skip_tile;   // pipelined kernel only: -1, or the tile (counted per CTA) that CTA 0's producer leaves out
};

struct CompactParams {
    char *K, *V, *Ks, *Vs;
    uint32_t *hist;
    int32_t *pos;
    const int32_t *src_idx;
    int U, B, Bw, w, n, m;
    int row_bytes, scale_bytes;
    int Bs;                     // scale rows per unit (int4 store)
    int chunk_bytes;            // set by the launcher: shared-memory gather buffer of the row kernel
    int rec_rows;               // set by the launcher: bit-plane rows staged per pass of the record kernel
    uint32_t bw_magic;          // set by the launcher: floor(2^32 / Bw) + 1
    int *err;                   // device error word (a bounded wait gave up)
    int unordered;              // moves (hole <- filler) listed in src_idx: holes from the front of the row, fillers
                                // from its back, their number in n_moves[u*B]
    const uint16_t *n_moves;
    int *n_arr;                 // per-unit live rows, or NULL: units whose cache is not full are skipped;
                                // the record kernel, which runs last, takes m off the ones it compacted
};

struct SelectParams {
    const uint32_t *hist;       // bit-planes, or
    const uint16_t *counters;   // [U][n] caller-supplied records
    int32_t *src_idx;           // [U][B] or NULL
    int32_t *evicted;           // [U][m] or NULL
    int U, B, Bw, w, n, r, m;
    int cmax;                   // largest possible counter value
    int *err;                   // device error word (bounds-checked build), or NULL
    const int *n_arr;           // per-unit live rows, or NULL: units whose cache is not full are skipped
    // unordered mode (holes are filled from the tail, so slots are not sorted by position): the recent
    // window and the tie-break go by the position array; the result is a list of (hole, filler) moves
    int unordered;
    const int32_t *pos;         // [U][B] stream positions
    const int *t_arr;           // per-unit tokens streamed, or NULL: t below holds for every unit
    int t;
    uint16_t *n_moves;          // [U][B] u16 scratch: entry u*B receives the number of moves of unit u
    int stage_planes;           // set by the launcher: copy the unit's bit-planes to shared memory first
    // fused unordered compression (set by the launcher when everything fits in shared memory): the selecting CTA
    // also moves the rows, the record bits and the positions of its unit; no move list leaves the CTA
    int fuse;
    int fuse_off;               // offset (in ints) of the fused path's shared arrays
    uint32_t bw_magic;          // floor(2^32 / Bw) + 1
    CompactParams mv;
};


// Chunked prompt step / recount (sh_prefill_chunk.cu, sh_chunk_umma.cu).
struct ChunkParams {
    const char *q, *k, *v;   // [c][U][D] time-major, 16-bit elements
    float *out;              // [c][U][D] fp32 or NULL
    char *K, *V;             // caches [U][B][D] (int4 store: [U][B][D/2] codes)
    char *Ks, *Vs;           // int4 store: fp16 group scales [U][Bs][D/64]
    int Bs;                  // int4 store: scale rows per unit
    uint32_t *hist;
    int32_t *pos;
    int U, B, Bw, w;
    int Utot;                // units of the whole handle: tokens of q/k/v/out are Utot rows apart
    int n0;                  // live rows before the chunk
    int c;                   // tokens in the chunk (<= CQ, <= w, n0 + c <= B)
    int t0;                  // tokens streamed before the chunk
    int SS;                  // row stride of S in floats
    float scale_log2e;
    char *qring;             // [U][w][D] queries of the last w steps (row = step mod w), or NULL
    // recount mode (the record recomputed at compression time): queries come from the ring,
    // steps first_step .. first_step + nsteps - 1, blockIdx.y selects CQ of them; keys are the
    // n0 cached rows, visible to a query when their position does not exceed its step
    int first_step, nsteps;
    int *err;                // device error word (a bounded wait gave up)
    int selftest_skip_tile;  // persistent tcgen05 kernel only: -1, or the key tile of its first unit that CTA 0 never requests
};

// tcgen05 version of the chunked prompt step (fp16/bf16, head_dim 128, any budget): tokens per launch, launcher.
int sh_chunk_umma_capacity();
cudaError_t sh_launch_chunk_umma(const ChunkParams &p, int dtype, cudaStream_t s);
cudaError_t sh_launch_recount_umma(const ChunkParams &p, int dtype, cudaStream_t s);
// the same chunk step with persistent CTAs and tiled TMA copies (sh_chunk_umma_tma.cu)
int sh_chunk_umma_tma_capacity();
cudaError_t sh_launch_chunk_umma_tma(const ChunkParams &p, int dtype, cudaStream_t s, int *launches);
cudaError_t sh_launch_recount_umma_tma(const ChunkParams &p, int dtype, cudaStream_t s);
// int4-g64 store: the chunked prompt step with codes unpacked into the tensor-core tiles (sh_chunk_umma_int4.cu).
cudaError_t sh_launch_chunk_umma_int4(const ChunkParams &p, cudaStream_t s);
cudaError_t sh_launch_recount_umma_int4(const ChunkParams &p, cudaStream_t s);

// CUDA-core chunk kernel: every storage type and head size (sh_chunk_simt.cu).
int sh_chunk_simt_capacity();
cudaError_t sh_launch_chunk_simt(const ChunkParams &p, int dtype, int D, cudaStream_t s);
cudaError_t sh_launch_recount_simt(const ChunkParams &p, int dtype, int D, cudaStream_t s);

// Launchers (each returns the cudaError_t of its launch and adds to *launches).
cudaError_t sh_launch_decode(const sh_context *c, const DecodeParams &p, cudaStream_t s, long long *launches);
// Scores of a query over the present caches (analysis; p.n = live rows, nothing appended).
cudaError_t sh_launch_scores(const sh_context *c, const DecodeParams &p, float *alpha_out, cudaStream_t s, long long *launches);
int sh_decode_kernel_for(const sh_context *c, int units);
// Pipelined (bulk-copy ring) variant of the decode kernel and its applicability test.
bool sh_decode_tma_supported(const sh_context *c);
cudaError_t sh_launch_decode_tma(const sh_context *c, const DecodeParams &p, cudaStream_t s, long long *launches);
// Chunked prompt kernel: tokens one launch can take for this handle (0 = unsupported), and its launcher.
int sh_prefill_chunk_capacity(const sh_context *c);
bool sh_recount_supported(const sh_context *c);
cudaError_t sh_launch_prefill_chunk(const sh_context *c, const void *q, const void *k, const void *v, float *out,
                                    int count, cudaStream_t s, long long *launches);
// Host bookkeeping shared by the compression entry points: is a compression due (some cache full),
// and the counter update once its kernels have been enqueued.
bool sh_compression_due(const sh_context *c);
void sh_after_compression(sh_context *c);
cudaError_t sh_launch_recount(const sh_context *c, cudaStream_t s, long long *launches);
// Recompute the record if the handle is in recompute mode and has not done so for the current step.
int sh_recount_if_needed(sh_context *c, cudaStream_t s);
cudaError_t sh_launch_select(const SelectParams &p, bool from_hist, cudaStream_t s, long long *launches);
// Unordered compression (SH_OPT_COMPACTION = 1): one fused launch where the unit's bit-planes fit in shared
// memory, else the selection followed by the hole-filling kernel.
cudaError_t sh_launch_compress_unordered(const SelectParams &sp, const CompactParams &cp, cudaStream_t s, long long *launches);
cudaError_t sh_launch_compact(const CompactParams &p, cudaStream_t s, long long *launches);
cudaError_t sh_launch_counters(const uint32_t *hist, uint16_t *counters, int U, int B, int Bw, int w, int n,
                               const int *n_arr, cudaStream_t s, long long *launches);
