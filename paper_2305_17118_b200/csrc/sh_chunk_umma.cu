// Chunked prompt step on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor memory).
//
// Same computation as the warp-level kernel of sh_prefill_chunk.cu: up to 64 consecutive steps of one
// unit in one CTA; step i attends with q_i over the n0 cached rows plus the chunk's tokens 0..i and
// writes its comparison bits into its own bit-plane row.  What differs is where the work runs:
//
//   * S = Q.K^T is issued by one thread as tcgen05.mma (M = 128, N = 64 keys per tile, K = 16 per
//     instruction), operands in shared memory in the canonical no-swizzle core-matrix order, the
//     fp32 result in tensor memory.  The 64 queries occupy rows 0..63 and again rows 64..127, so
//     that all 128 lanes of tensor memory carry data: thread i and thread i + 64 own the same
//     query and split the columns (keys) of every tile between them.
//   * The row statistics need every logit against the final row sum, and a whole row of logits
//     (B up to 32768) fits neither in tensor memory nor in shared memory.  So the logits are
//     computed twice - tensor-core time is cheap here: a first sweep over the key tiles keeps a
//     running maximum and sum per row (one thread per row: no shuffles), a second sweep recomputes
//     S tile by tile, forms e = 2^(s - M), packs the record bits of 32 keys into a word by plain
//     register arithmetic, and hands P (high and low 16-bit parts) to the second contraction.
//     No limit on B follows from this structure.
//   * O^T = V^T.P^T accumulates in tensor memory as [128 columns of d][64 queries]: V tiles are
//     the MN-major A operand exactly as they lie in the cache (rows of d), P the K-major B operand.
//
// Every mbarrier wait is bounded; tensor memory is released on every path.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "sh_async.cuh"
#include "sh_internal.h"
#include "sh_umma.cuh"

namespace {

using namespace shasync;
using namespace shumma;

constexpr int D = 128;            // head_dim served by this kernel
constexpr int TN = 64;            // keys per tile
constexpr int CQ = 64;            // queries per CTA
constexpr int NT = 256;           // threads per CTA: two per lane of tensor memory (warps w and w + 4 share a lane quadrant)
constexpr int GROUP = 2048;       // bytes of 8 rows of 256 B in core-matrix order: [16 chunks][8 rows][16 B]
constexpr int TILE = (TN / 8) * GROUP;          // 16 KB
constexpr int Q_BYTES = (2 * CQ / 8) * GROUP;   // 128 rows
constexpr int PG = (TN / 8) * 128;              // bytes of 8 rows of P (TN keys each) in core-matrix order
constexpr int P_BYTES = (CQ / 8) * PG;          // 64 rows x TN keys x 2 B
constexpr int HC = TN / 4;                      // columns of a tile per thread (four threads share a query row)
static_assert(HC == 16, "a thread reads its 16 columns with one tcgen05.ld and owns half a record word");
constexpr int TMEM_COLS = 256;    // power of two covering two S tiles and O^T; two CTAs fit in the 512 columns of an SM
constexpr int S_COL = 0;          // two S tiles: columns [0, TN) and [TN, 2 TN)
constexpr int O_COL = 2 * TN;     // O^T: CQ columns

constexpr int OFF_Q = 0;
constexpr int OFF_K = OFF_Q + Q_BYTES;
constexpr int OFF_V = OFF_K + 2 * TILE;
constexpr int OFF_PH = OFF_V + 2 * TILE;
constexpr int OFF_PL = OFF_PH + P_BYTES;
constexpr int OFF_STAT = OFF_PL + P_BYTES;      // M[64], L[64] floats (the per-thread m[128], l[128] of the first sweep
                                                // meet in the P buffer, which is idle between the sweeps)
constexpr int OFF_BAR = OFF_STAT + 4 * (64 + 64);
constexpr int SMEM_BYTES = OFF_BAR + 64;
static_assert(P_BYTES >= 4 * 2 * NT, "the first sweep's statistics alias the P buffer");
static_assert(2 * (SMEM_BYTES + 1024) <= 228 * 1024, "two CTAs per SM");

// Start filling a tile buffer with rows [j0, j0 + TN) of the unit's K or V as seen by the chunk
// (cached rows, then the chunk's own tokens, zeros beyond), 16-byte piece (row, ch) going to
// [row / 8][ch][row % 8]: the canonical no-swizzle order, K-major for K, MN-major for V.
__device__ __forceinline__ void load_tile(char *tile, const char *cache_u, const char *chunk, int j0, int n0, int n_tot,
                                          size_t chunk_stride) {
    // consecutive threads take the 8 rows of a core matrix, then the next 16-byte column: a warp writes 512
    // contiguous bytes of shared memory and reads 8 x 64 contiguous bytes of global memory.  With 256
    // threads a thread keeps its column and walks rows row0, row0 + 16, ...: two row groups further each time.
    static_assert(NT == 256, "piece idx = tid + 256 k lies 16 rows below piece tid");
    const int row0 = ((threadIdx.x >> 7) << 3) | (threadIdx.x & 7), ch = (threadIdx.x >> 3) & 15;
    char *dst = tile + (row0 >> 3) * GROUP + ch * 128 + (row0 & 7) * 16;
    const char *src_cache = cache_u + (size_t)(j0 + row0) * (D * 2) + ch * 16;
    const char *src_chunk = chunk + (ptrdiff_t)(j0 + row0 - n0) * (ptrdiff_t)chunk_stride + ch * 16;
#pragma unroll
    for (int k = 0; k < TN / 16; ++k) {
        const int j = j0 + row0 + 16 * k;
        if (j < n0) cp_async16(dst, src_cache);
        else if (j < n_tot) cp_async16(dst, src_chunk);
        else *reinterpret_cast<uint4 *>(dst) = make_uint4(0, 0, 0, 0);
        dst += 2 * GROUP;
        src_cache += 16 * (D * 2);
        src_chunk += 16 * (ptrdiff_t)chunk_stride;
    }
}


// RECOUNT: the record recomputed at compression time.  Queries come from the ring of the last w queries
// (steps first_step .. first_step + nsteps - 1, blockIdx.y selects 64 of them), keys are the n0 cached rows, a
// key is visible to a query when its position does not exceed the query's step (slots need not be sorted);
// nothing is appended and no output is formed: only the bit-plane rows of those steps are rewritten.
template <int DT, bool RECOUNT>
__global__ void __launch_bounds__(NT, 2) sh_chunk_umma_kernel(const ChunkParams p) {
    using SP = Split<DT>;
    extern __shared__ __align__(128) unsigned char sm[];
    char *Qs = reinterpret_cast<char *>(sm) + OFF_Q;
    char *Kt = reinterpret_cast<char *>(sm) + OFF_K;
    char *Vt = reinterpret_cast<char *>(sm) + OFF_V;
    char *Ph = reinterpret_cast<char *>(sm) + OFF_PH;
    char *Pl = reinterpret_cast<char *>(sm) + OFF_PL;
    float *m_sh = reinterpret_cast<float *>(sm + OFF_PH);
    float *l_sh = m_sh + NT;
    float *Mfin = reinterpret_cast<float *>(sm + OFF_STAT), *Lfin = Mfin + 64;
    uint64_t *bar_s = reinterpret_cast<uint64_t *>(sm + OFF_BAR);
    uint64_t *bar_pv = bar_s + 2;        // bar_s[0], bar_s[1]: one per S buffer
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bar_s + 3);

    const int u = blockIdx.x, tid = threadIdx.x, warp = tid >> 5;
    // this thread's query and its quarter of every tile's columns: warps w and w + 4 read the same 32 lanes
    const int i = tid & 63, quarter = ((tid >> 6) & 1) * 2 + (tid >> 7);
    const int qoff = RECOUNT ? (int)blockIdx.y * CQ : 0;
    const int n0 = p.n0, c = RECOUNT ? min(CQ, p.nsteps - qoff) : p.c, n_tot = RECOUNT ? n0 : n0 + c;
    const int ntiles = (n_tot + TN - 1) / TN;
    const int step0 = RECOUNT ? p.first_step + qoff : p.t0 + 1;     // step of this CTA's first query
    int *pos_sh = reinterpret_cast<int *>(sm + OFF_PL);             // [3][TN] positions of the key tiles (recount only: P is idle)
    const size_t tstride = (size_t)p.Utot * D * 2;       // bytes between consecutive tokens of one unit
    const char *Kc = p.K + (size_t)u * p.B * D * 2;
    const char *Vc = p.V + (size_t)u * p.B * D * 2;
    const char *kchunk = RECOUNT ? nullptr : p.k + (size_t)u * D * 2, *vchunk = RECOUNT ? nullptr : p.v + (size_t)u * D * 2;
    const int32_t *pos_u = p.pos + (size_t)u * p.B;
    // positions of key tile kt into pos_sh[buf] (slots beyond the cache: never visible)
    auto load_pos = [&](int buf, int kt) {
        if (RECOUNT && tid < TN) {
            const int j = kt * TN + tid;
            pos_sh[buf * TN + tid] = j < n0 ? pos_u[j] : 0x7fffffff;
        }
    };

    // ---- tensor memory, barriers
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        mbar_init(bar_s, 1);
        mbar_init(bar_s + 1, 1);
        mbar_init(bar_pv, 1);
        fence_barrier_init();
    }
    // The two sweeps form one sequence of G = 2 ntiles S tiles; tile g covers the keys of tile g mod ntiles.
    // S buffer, K buffer and mbarrier of tile g: g & 1.  V tile kt (second sweep only) sits in buffer kt & 1.
    const int G = 2 * ntiles;
    auto key_tile = [&](int g) { return g < ntiles ? g : g - ntiles; };
    load_tile(Kt, Kc, kchunk, 0, n0, n_tot, tstride);
    load_tile(Kt + TILE, Kc, kchunk, key_tile(1) * TN, n0, n_tot, tstride);
    load_pos(0, 0);          // positions of tile g sit in buffer g mod 3: written two iterations ahead of their use
    load_pos(1, key_tile(1));
    if (p.out) load_tile(Vt, Vc, vchunk, 0, n0, n_tot, tstride);     // idle until the second sweep: fetched early
    // ---- queries (rows beyond c are zero), twice: rows 0..63 and 64..127; asynchronous like the first tiles
    for (int idx = tid; idx < CQ * 16; idx += NT) {
        const int row = idx >> 4, ch = idx & 15;
        char *dst = Qs + (row >> 3) * GROUP + ch * 128 + (row & 7) * 16;
        if (row < c) {
            const char *src = RECOUNT ? p.qring + ((size_t)u * p.w + (step0 + row) % p.w) * (D * 2) + ch * 16
                                      : p.q + (size_t)row * tstride + (size_t)u * D * 2 + ch * 16;
            cp_async16(dst, src);
            cp_async16(dst + (CQ / 8) * GROUP, src);
        } else {
            *reinterpret_cast<uint4 *>(dst) = make_uint4(0, 0, 0, 0);
            *reinterpret_cast<uint4 *>(dst + (CQ / 8) * GROUP) = make_uint4(0, 0, 0, 0);
        }
    }
    // ---- while those copies fly: append the chunk's keys, values and positions to the cache (nothing in this
    // launch reads them back from there) and remember the queries for a later recount
    if (!RECOUNT && tid < c) p.pos[(size_t)u * p.B + n0 + tid] = step0 + tid;
    if constexpr (!RECOUNT) {
        // up to 64 rows x 16 pieces = 4 pieces per thread: all loads are issued before the first store, so the
        // thread waits for memory once, not once per piece
        constexpr int PER = CQ * 16 / NT;
        uint4 kk[PER], vv[PER], qq[PER];
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const int idx = tid + i * NT, row = idx >> 4, ch = idx & 15;
            if (row < c) {
                const size_t src = (size_t)row * tstride + (size_t)u * D * 2 + ch * 16;
                kk[i] = *reinterpret_cast<const uint4 *>(p.k + src);
                vv[i] = *reinterpret_cast<const uint4 *>(p.v + src);
                if (p.qring) qq[i] = *reinterpret_cast<const uint4 *>(p.q + src);
            }
        }
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const int idx = tid + i * NT, row = idx >> 4, ch = idx & 15;
            if (row < c) {
                const size_t dst = ((size_t)u * p.B + n0 + row) * (D * 2) + ch * 16;
                *reinterpret_cast<uint4 *>(p.K + dst) = kk[i];
                *reinterpret_cast<uint4 *>(p.V + dst) = vv[i];
                if (p.qring) *reinterpret_cast<uint4 *>(p.qring + ((size_t)u * p.w + (step0 + row) % p.w) * (D * 2) + ch * 16) = qq[i];
            }
        }
    }
    cp_async_commit();
    cp_async_wait_all();
    fence_async_shared();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = *tmem_slot;
    const uint32_t lane_addr = tbase + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t q_addr = smem_u32(Qs), k_addr = smem_u32(Kt), v_addr = smem_u32(Vt), ph_addr = smem_u32(Ph), pl_addr = smem_u32(Pl);
    const uint32_t idesc_s = instr_desc(SP::FMT, 0, 128, TN);
    const uint32_t idesc_pv = instr_desc(SP::FMT, 1, 128, CQ);
    auto issue_s = [&](int g) {        // S tile g = Q . K_tile^T into S buffer g & 1 (one thread)
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
            umma_f16(tbase + S_COL + (g & 1) * TN, smem_desc(q_addr + ks * 256, 128, GROUP),
                     smem_desc(k_addr + (g & 1) * TILE + ks * 256, 128, GROUP), idesc_s, ks > 0);
        umma_commit(bar_s + (g & 1));
    };

    // The tensor core runs one tile ahead: S(g + 1) is issued before the threads turn to S(g), and the K
    // tile of g + 2 is fetched as soon as S(g) has been computed from the buffer it reuses.
    uint32_t par_s = 0, par_pv = 0;      // bit b of par_s: parity the next wait on bar_s[b] expects
    bool ok = true;
    const int nv = n0 + i + 1;           // keys visible to this thread's query
    const bool live_row = i < c;
    float m_run = -INFINITY, l_run = 0.f;
    float Mi = 0.f, Li = 1.f;
    const float tf = (float)(step0 + i);
    uint32_t *hrow = p.hist + ((size_t)u * p.w + (step0 + i) % p.w) * p.Bw;
    if (tid == 0) issue_s(0);
    for (int g = 0; g < G; ++g) {
        const int kt = key_tile(g);
        const bool second = g >= ntiles;
        cp_async_wait_all();           // K(g + 1) and, in the second sweep, V(kt) have landed
        fence_async_shared();
        tc_fence_before();
        if (!__syncthreads_and(ok)) { ok = false; break; }
        if (tid == 0 && g + 1 < G) issue_s(g + 1);
        ok = mbar_wait(bar_s + (g & 1), (par_s >> (g & 1)) & 1, p.err, 0x501) && ok;
        par_s ^= 1u << (g & 1);
        if (second && kt > 0 && p.out) {     // the previous tile's P.V has finished: P and the V buffer it read are free
            ok = mbar_wait(bar_pv, par_pv, p.err, 0x502) && ok;
            par_pv ^= 1;
        }
        tc_fence_after();
        if (g + 2 < G) {
            load_tile(Kt + (g & 1) * TILE, Kc, kchunk, key_tile(g + 2) * TN, n0, n_tot, tstride);
            load_pos((g + 2) % 3, key_tile(g + 2));
        }
        if (p.out && second && kt + 1 < ntiles) load_tile(Vt + ((kt + 1) & 1) * TILE, Vc, vchunk, (kt + 1) * TN, n0, n_tot, tstride);
        cp_async_commit();
        float sv[HC];
        tmem_ld16(lane_addr + S_COL + (g & 1) * TN + quarter * HC, sv);
        const int j0 = kt * TN + quarter * HC;
        // bit jj of vm: column jj of this batch is visible to the query (causal prefix, or by position in a recount)
        uint32_t vm;
        if (RECOUNT) {
            vm = 0;
            const int *pt = pos_sh + (g % 3) * TN + quarter * HC;
#pragma unroll
            for (int jj = 0; jj < HC; ++jj) vm |= (uint32_t)(pt[jj] <= step0 + i) << jj;
            if (!live_row) vm = 0;
        } else {
            const int lim = live_row ? nv - j0 : 0;
            vm = lim <= 0 ? 0u : (lim >= HC ? 0xffffu : (1u << lim) - 1u);
        }
        if (!second) {
            // ---- first sweep: running maximum and sum of the row
            if (vm) {
                float bmax = -INFINITY;
#pragma unroll
                for (int jj = 0; jj < HC; ++jj) {
                    sv[jj] = ((vm >> jj) & 1u) ? sv[jj] * p.scale_log2e : -INFINITY;
                    bmax = fmaxf(bmax, sv[jj]);
                }
                const float m_new = fmaxf(m_run, bmax);
                float acc = 0.f;
#pragma unroll
                for (int jj = 0; jj < HC; ++jj) acc += ex2_approx(sv[jj] - m_new);
                l_run = l_run * ex2_approx(m_run - m_new) + acc;
                m_run = m_new;
            }
            if (g == ntiles - 1) {
                // the four parts of a row meet (in the P buffer, idle until the second sweep)
                m_sh[tid] = m_run;
                l_sh[tid] = l_run;
                __syncthreads();
                if (tid < CQ) {
                    float M = -INFINITY, L = 0.f;
#pragma unroll
                    for (int part = 0; part < NT / CQ; ++part) M = fmaxf(M, m_sh[tid + part * CQ]);
#pragma unroll
                    for (int part = 0; part < NT / CQ; ++part) {
                        const float mp = m_sh[tid + part * CQ];
                        if (mp > -INFINITY) L += l_sh[tid + part * CQ] * ex2_approx(mp - M);
                    }
                    Mfin[tid] = M;
                    Lfin[tid] = L;
                }
                __syncthreads();
                Mi = Mfin[i];
                Li = Lfin[i];
            }
            continue;
        }
        // ---- second sweep: probabilities, record bits, O^T += V^T . P^T
        uint32_t word = 0, hi[HC / 2], lo[HC / 2];
#pragma unroll
        for (int jj = 0; jj < HC; jj += 2) {
            const bool v0 = (vm >> jj) & 1u, v1 = (vm >> (jj + 1)) & 1u;
            const float e0 = v0 ? ex2_approx(sv[jj] * p.scale_log2e - Mi) : 0.f;
            const float e1 = v1 ? ex2_approx(sv[jj + 1] * p.scale_log2e - Mi) : 0.f;
            // step t: low_j = [alpha_j < 1/t] = [e_j * t < L]
            word |= (uint32_t)(e0 * tf < Li) << jj;
            word |= (uint32_t)(e1 * tf < Li) << (jj + 1);
            SP::run(e0, e1, hi[jj >> 1], lo[jj >> 1]);
        }
        word &= vm;     // a slot the query does not see has no bit
        // 16 slots: half a record word
        if (live_row && (j0 >> 5) < p.Bw) reinterpret_cast<uint16_t *>(hrow)[j0 >> 4] = (uint16_t)word;
        if (p.out) {
#pragma unroll
            for (int cc = 0; cc < HC / 8; ++cc) {
                const int off = (i >> 3) * PG + (quarter * (HC / 8) + cc) * 128 + (i & 7) * 16;
                *reinterpret_cast<uint4 *>(Ph + off) = make_uint4(hi[4 * cc], hi[4 * cc + 1], hi[4 * cc + 2], hi[4 * cc + 3]);
                *reinterpret_cast<uint4 *>(Pl + off) = make_uint4(lo[4 * cc], lo[4 * cc + 1], lo[4 * cc + 2], lo[4 * cc + 3]);
            }
            fence_async_shared();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < TN / 16; ++ks) {
                    const uint64_t a = smem_desc(v_addr + (kt & 1) * TILE + ks * 2 * GROUP, GROUP, 128);
                    umma_f16(tbase + O_COL, a, smem_desc(ph_addr + ks * 256, 128, PG), idesc_pv, (kt > 0 || ks > 0));
                    umma_f16(tbase + O_COL, a, smem_desc(pl_addr + ks * 256, 128, PG), idesc_pv, 1);
                }
                umma_commit(bar_pv);
            }
        }
    }
    if (ok) {
        // bit-plane words beyond the last tile hold no live slot
        if (live_row && quarter == 0)
            for (int wd = ntiles * (TN / 32); wd < p.Bw; ++wd) hrow[wd] = 0;
        if (p.out) {
            ok = mbar_wait(bar_pv, par_pv, p.err, 0x504) && ok;
            tc_fence_after();
        }
    }
    // ---- O^T: lane = output column, tensor-memory column = query
    if (p.out) {
        const int dcol = tid & 127, b = tid >> 7;      // output column (lane of tensor memory), half of the queries
        float ov[32];
        tmem_ld32(lane_addr + O_COL + b * 32, ov);
        if (ok) {
#pragma unroll
            for (int qq = 0; qq < 32; ++qq) {
                const int qi = b * 32 + qq;
                if (qi < c) p.out[((size_t)qi * p.Utot + u) * D + dcol] = ov[qq] / Lfin[qi];
            }
        }
    }
    cp_async_wait_all();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(TMEM_COLS) : "memory");
    }
}

template <int DT, bool RECOUNT>
cudaError_t launch(const ChunkParams &p, cudaStream_t s) {
    auto kern = sh_chunk_umma_kernel<DT, RECOUNT>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const unsigned gy = RECOUNT ? (unsigned)((p.nsteps + CQ - 1) / CQ) : 1u;
    kern<<<dim3(p.U, gy, 1), NT, SMEM_BYTES, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

int sh_chunk_umma_capacity() { return CQ; }

cudaError_t sh_launch_chunk_umma(const ChunkParams &p, int dtype, cudaStream_t s) {
    if (p.c < 1 || p.c > CQ) return cudaErrorInvalidValue;
    return dtype == SH_F16 ? launch<SH_F16, false>(p, s) : launch<SH_BF16, false>(p, s);
}

cudaError_t sh_launch_recount_umma(const ChunkParams &p, int dtype, cudaStream_t s) {
    if (p.nsteps < 1 || p.out) return cudaErrorInvalidValue;
    return dtype == SH_F16 ? launch<SH_F16, true>(p, s) : launch<SH_BF16, true>(p, s);
}
