// Chunked prompt step on the 5th-generation tensor cores, persistent CTAs fed by tiled TMA copies.
//
// The computation is the one of sh_chunk_umma.cu (up to 128 consecutive steps of one unit: step i attends with
// q_i over the n0 cached rows plus the chunk's tokens 0..i, writes its comparison bits into its own bit-plane
// row, and the chunk's keys, values and queries are appended), and so are the two sweeps over the key tiles and
// the split of P into a high and a low 16-bit part.  What differs is who moves the data and who waits for whom:
//
//   * a CTA is persistent: it walks over units blockIdx.x, blockIdx.x + gridDim.x, ...; tensor memory, the
//     barriers and the tensor maps are set up once, and the tiles of the next unit are requested while the
//     softmax threads still work on the present one;
//   * every key, value and query tile is brought in by cp.async.bulk.tensor (one elected thread, CTA-local
//     destination, no delivery to several CTAs) from 3-D tensor maps over the caches [U][B][128] and over the
//     chunk's queries [c][U][128]: boxes of 64 rows x 128 bytes in the 128-byte swizzle, which is the K-major
//     operand layout for Q and K and the MN-major one for V.  Rows past B (and queries past c) are filled with
//     zeros by the copy engine; rows between n0 + c and the end of the last tile are stale cache rows: their
//     logits are masked, and the softmax threads zero them in the last value tile before P.V reads it;
//   * the softmax warps (8 for chunks of up to 64 tokens, 16 for up to 128) do the arithmetic; after them comes one
//     warp each that issues the MMAs, requests query and key tiles, requests value tiles, and one or four warps
//     that append the chunk to the cache (plain loads and stores, then a proxy fence: the tiles that contain the
//     new rows are requested only after the append of their unit is visible).
//
// Every wait is bounded; a wait that gives up records its code in the device error word and raises a CTA-wide
// flag, on which every role leaves; tensor memory is released on every path.
#include <cuda.h>
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
constexpr int NT = 256;           // softmax threads of the narrow chunk kernel and of the recount: two per lane of tensor memory
constexpr int W_MMA = NT / 32, W_KQ = W_MMA + 1, W_V = W_MMA + 2;      // (recount: warp 10 gathers the queries)
constexpr int HALF_K = TN * 128;        // bytes of one box: 64 rows x 64 elements (half of head_dim)
constexpr int TILE = 2 * HALF_K;        // a key or value tile: [2 halves of d][64 rows][128 B]
constexpr int HALF_Q = 128 * 128;       // 128 query rows (M = 128) x 64 elements
constexpr int Q_BYTES = 2 * HALF_Q;
constexpr int PG = (TN / 8) * 128;      // bytes of 8 rows of P (TN keys each) in no-swizzle core-matrix order
constexpr int HC = TN / 4;              // columns of a tile per thread (four threads share a query row)
static_assert(HC == 16, "a thread reads its 16 columns with one tcgen05.ld and owns half a record word");
constexpr int S_COL = 0;
constexpr int O_COL = 2 * TN;           // columns [O_COL, O_COL + QR): V^T.P_hi^T, the next QR columns: V^T.P_lo^T

// Two shapes of the chunk kernel.  Narrow: up to 64 queries, which occupy rows 0..63 and again rows 64..127 of the
// MMA, 8 softmax warps, two CTAs per SM.  Wide: up to 128 queries, one per row of the MMA (half the S instructions
// per query), 16 softmax warps, four key tiles in flight, one CTA per SM.
template <bool WIDE> struct CK {
    static constexpr int QR = WIDE ? 128 : 64;            // queries per unit and launch
    static constexpr int NT = 4 * QR;                     // softmax threads: four per query (16 columns of a tile each)
    static constexpr int NAPP = WIDE ? 4 : 1;             // warps that append (a warp moves the 48 KB of 64 tokens in about 10 us)
    static constexpr int NTH = NT + 96 + 32 * NAPP;       // + the warps that issue MMAs, request K/Q tiles, request V tiles, append
    static constexpr int W_MMA = NT / 32, W_KQ = W_MMA + 1, W_V = W_MMA + 2, W_APPEND = W_MMA + 3;
    static constexpr int CTAS = WIDE ? 1 : 2;             // per SM
    static constexpr int KST = WIDE ? 4 : 2;              // key tiles in flight
    static constexpr int P_BYTES = (QR / 8) * PG;         // QR rows x TN keys x 2 B
    static constexpr int TMEM_COLS = WIDE ? 512 : 256;    // two S tiles, O^T from P_hi and from P_lo (QR columns each), power of two
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = OFF_Q + Q_BYTES;
    static constexpr int OFF_V = OFF_K + KST * TILE;
    static constexpr int OFF_PH = OFF_V + 2 * TILE;
    static constexpr int OFF_PL = OFF_PH + P_BYTES;       // P_hi and P_lo form one B operand of 2 QR rows
    static constexpr int OFF_STAT = OFF_PL + P_BYTES;     // M[QR], L[QR], 1/L[QR]
    static constexpr int OFF_BAR = OFF_STAT + 4 * 3 * QR;
    static constexpr int SMEM_BYTES = OFF_BAR + 192;
    static_assert(OFF_K % 1024 == 0 && OFF_V % 1024 == 0 && HALF_K % 1024 == 0, "swizzled tiles start on 1024-byte boundaries");
    static_assert(P_BYTES >= 4 * 2 * NT, "the first sweep's statistics alias the P buffer");
    static_assert(CTAS * (SMEM_BYTES + 1024) <= 228 * 1024, "CTAs per SM");
    static_assert(O_COL + 2 * QR <= TMEM_COLS && CTAS * TMEM_COLS <= 512, "tensor memory columns");
};

// Shared-memory matrix descriptor for the 128-byte swizzle (layout type 2 in bits 61..63).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
    return smem_desc(saddr, lbo, sbo) | (2ull << 61);
}

// One box of a 3-D tensor map into this CTA's shared memory; completion counted in bytes on `bar`.
__device__ __forceinline__ void tma_load_3d(void *smem_dst, const CUtensorMap *map, int c0, int c1, int c2, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
            smem_u32(smem_dst)),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(smem_u32(bar))
        : "memory");
}
// Order this thread's earlier plain stores (any state space) before later reads by the copy engine.
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

__device__ __forceinline__ void st_release_shared(int *p, int v) {
    asm volatile("st.release.cta.shared.u32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_acquire_shared(const int *p) {
    int v;
    asm volatile("ld.acquire.cta.shared.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
    return v;
}
// Wait until *ctr >= target; bounded like mbar_wait.
__device__ __forceinline__ bool counter_wait(const int *ctr, int target, int *err, int code) {
    if (ld_acquire_shared(ctr) >= target) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t i = 1; i < WAIT_POLLS; ++i) {
        if (ld_acquire_shared(ctr) >= target) return true;
        if ((i & 255u) == 0 && global_ns() - t0 > WAIT_NS) break;
    }
    if (err) atomicCAS(err, 0, code);
    return false;
}

template <int THREADS>
__device__ __forceinline__ void softmax_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(THREADS) : "memory"); }

struct Bars {
    uint64_t q_full, q_empty;          // the unit's queries landed / its last S has been computed
    uint64_t k_full[4], k_empty[4];
    uint64_t v_full[2], v_empty[2];
    uint64_t s_done[2], s_free[2];     // S(g) computed / read out of tensor memory by all softmax threads
    uint64_t p_ready, pv_done;         // P(kt) written / P.V(kt) computed
    uint64_t o_free;                   // O^T of the unit read out
    uint32_t tmem_slot;
    int abort_flag;                    // a bounded wait gave up somewhere: everybody leaves
    int appended[4];                   // per append warp: units whose share of the chunk's rows is in the cache
};
static_assert(sizeof(Bars) <= 192, "barrier block");

template <int DT, bool WIDE>
__global__ void __launch_bounds__(CK<WIDE>::NTH, CK<WIDE>::CTAS)
sh_chunk_umma_tma_kernel(const ChunkParams p, const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                         const __grid_constant__ CUtensorMap mapV) {
    using SP = Split<DT>;
    using C = CK<WIDE>;
    extern __shared__ __align__(1024) unsigned char sm[];
    char *Qs = reinterpret_cast<char *>(sm) + C::OFF_Q;
    char *Kt = reinterpret_cast<char *>(sm) + C::OFF_K;
    char *Vt = reinterpret_cast<char *>(sm) + C::OFF_V;
    char *Ph = reinterpret_cast<char *>(sm) + C::OFF_PH;
    char *Pl = reinterpret_cast<char *>(sm) + C::OFF_PL;
    float *m_sh = reinterpret_cast<float *>(sm + C::OFF_PH);
    float *l_sh = m_sh + C::NT;
    float *Mfin = reinterpret_cast<float *>(sm + C::OFF_STAT), *Lfin = Mfin + C::QR, *Linv = Lfin + C::QR;
    Bars *bars = reinterpret_cast<Bars *>(sm + C::OFF_BAR);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n0 = p.n0, c = p.c, n_tot = n0 + c;
    const int ntiles = (n_tot + TN - 1) / TN, G = 2 * ntiles;
    const int step0 = p.t0 + 1;
    const bool with_out = p.out != nullptr;
    const int nunits = ((int)p.U - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;     // units of this CTA
    auto key_tile = [&](int g) { return g < ntiles ? g : g - ntiles; };
    auto aborted = [&]() { return *(volatile int *)&bars->abort_flag != 0; };

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_slot)), "r"(C::TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        mbar_init(&bars->q_full, 1);
        mbar_init(&bars->q_empty, 1);
        for (int s = 0; s < C::KST; ++s) { mbar_init(&bars->k_full[s], 1); mbar_init(&bars->k_empty[s], 1); }
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars->v_full[s], 1); mbar_init(&bars->v_empty[s], 1);
            mbar_init(&bars->s_done[s], 1); mbar_init(&bars->s_free[s], C::NT);
        }
        mbar_init(&bars->p_ready, C::NT);
        mbar_init(&bars->pv_done, 1);
        mbar_init(&bars->o_free, C::NT);
        for (int a = 0; a < 4; ++a) bars->appended[a] = 0;
        bars->abort_flag = 0;
        if ((smem_u32(sm) & 1023u) != 0) {      // the swizzled tiles need the 1024-byte alignment the declaration asks for
            if (p.err) atomicCAS(p.err, 0, 0x520);
            bars->abort_flag = 1;
        }
        fence_barrier_init();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = bars->tmem_slot;
    const bool start_ok = !aborted();

    if (warp == C::W_MMA) {
        // --------------------------------------------------------------------------------------- the issuing thread
        if (lane == 0 && start_ok) {
            const uint32_t idesc_s = instr_desc(SP::FMT, 0, 128, TN);
            const uint32_t idesc_pv = instr_desc(SP::FMT, 1, 128, 2 * C::QR);     // N = the queries' high parts, then their low parts
            // the descriptors of query buffer, key stage 0, value buffer 0 and P, built once; the other stages and buffers
            // lie a fixed number of 16-byte units further
            uint64_t dq[D / 16], dk[D / 16], dv[TN / 16], dp[TN / 16];
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                dq[ks] = smem_desc_sw128(smem_u32(Qs) + (ks >> 2) * HALF_Q + (ks & 3) * 32, 16, 1024);
                dk[ks] = smem_desc_sw128(smem_u32(Kt) + (ks >> 2) * HALF_K + (ks & 3) * 32, 16, 1024);
            }
#pragma unroll
            for (int ks = 0; ks < TN / 16; ++ks) {
                dv[ks] = smem_desc_sw128(smem_u32(Vt) + ks * 2048, HALF_K, 1024);
                dp[ks] = smem_desc(smem_u32(Ph) + ks * 256, 128, PG);       // row groups of P_hi, then of P_lo
            }
            // Two streams of work, each in its own order: S tiles (up to two ahead of the softmax threads, across unit
            // boundaries too) and P.V tiles.  Whichever has its operands ready is issued next, so neither waits
            // behind the other's barrier; nothing is ready: poll, with the same bounds as mbar_wait.
            bool ok = true;
            int sk = 0, sg = 0;          // next S: unit index and tile (both sweeps) of this CTA
            int pk = 0, pt = 0;          // next P.V: unit index and key tile
            const int pv_units = with_out ? nunits : 0;
            uint32_t idle = 0;
            unsigned long long idle_t0 = 0;
            while (ok && (sk < nunits || pk < pv_units)) {
                bool did = false;
                if (sk < nunits) {
                    const int gk = sk * G + sg, bb = gk & 1, st = gk % C::KST;
                    if ((sg != 0 || mbar_test(&bars->q_full, sk & 1)) && mbar_test(&bars->k_full[st], (gk / C::KST) & 1) &&
                        (gk < 2 || mbar_test(&bars->s_free[bb], ((gk >> 1) - 1) & 1))) {      // S(gk - 2) has been read out
                        tc_fence_after();
                        const uint64_t koff = (uint64_t)(st * (TILE >> 4));
#pragma unroll
                        for (int ks = 0; ks < D / 16; ++ks) umma_f16(tbase + S_COL + bb * TN, dq[ks], dk[ks] + koff, idesc_s, ks > 0);
                        umma_commit(&bars->k_empty[st]);
                        umma_commit(&bars->s_done[bb]);
                        if (sg == G - 1) umma_commit(&bars->q_empty);
                        if (++sg == G) { sg = 0; ++sk; }
                        did = true;
                    }
                }
                if (pk < pv_units) {
                    const int gv = pk * ntiles + pt, bb = gv & 1;
                    if (mbar_test(&bars->p_ready, gv & 1) && mbar_test(&bars->v_full[bb], (gv >> 1) & 1) &&
                        (pt != 0 || pk == 0 || mbar_test(&bars->o_free, (pk - 1) & 1))) {      // the previous unit's O^T is in registers
                        tc_fence_after();
                        const uint64_t voff = (uint64_t)(bb * (TILE >> 4));
#pragma unroll
                        for (int ks = 0; ks < TN / 16; ++ks) umma_f16(tbase + O_COL, dv[ks] + voff, dp[ks], idesc_pv, (pt > 0 || ks > 0));
                        umma_commit(&bars->v_empty[bb]);
                        umma_commit(&bars->pv_done);
                        if (++pt == ntiles) { pt = 0; ++pk; }
                        did = true;
                    }
                }
                if (did) {
                    idle = 0;
                } else {
                    if (idle == 0) idle_t0 = global_ns();
                    ++idle;
                    if (idle >= WAIT_POLLS || ((idle & 255u) == 0 && global_ns() - idle_t0 > WAIT_NS)) {
                        if (p.err) atomicCAS(p.err, 0, 0x527);
                        ok = false;
                    }
                }
                if (aborted()) ok = false;
            }
            if (!ok) *(volatile int *)&bars->abort_flag = 1;
        }
    } else if (warp == C::W_KQ) {
        // --------------------------------------------------------------------------------------- query and key tiles
        if (lane == 0 && start_ok) {
            bool ok = true;
            int last = -1, q_last = -1;           // the last key tile (global index) and the last unit's queries requested
            for (int k = 0; k < nunits && ok; ++k) {
                const int u = blockIdx.x + k * gridDim.x;
                if (k > 0) ok = mbar_wait(&bars->q_empty, (k - 1) & 1, p.err, 0x531);
                if (!ok || aborted()) { ok = false; break; }
                mbar_arrive_expect_tx(&bars->q_full, Q_BYTES);
                q_last = k;
#pragma unroll
                for (int part = 0; part < 4; ++part)
                    tma_load_3d(Qs + (part >> 1) * HALF_Q + (part & 1) * 64 * 128, &mapQ, (part >> 1) * 64, u, WIDE ? (part & 1) * 64 : 0, &bars->q_full);
                bool appended = false;
                for (int g = 0; g < G; ++g) {
                    const int gk = k * G + g, s = gk % C::KST, kt = key_tile(g);
                    if (gk >= C::KST) ok = mbar_wait(&bars->k_empty[s], ((gk / C::KST) - 1) & 1, p.err, 0x532);
                    if (ok && !appended && (kt + 1) * TN > n0) {     // this tile holds rows of the chunk
                        for (int a = 0; a < C::NAPP; ++a) ok = ok && counter_wait(&bars->appended[a], k + 1, p.err, 0x533);
                        fence_proxy_async_all();
                        appended = true;
                    }
                    if (!ok || aborted()) { ok = false; break; }
                    // self-test of the give-up path: this tile is never requested (nothing is in flight for it), so the
                    // waits that depend on it run out and every role of this CTA leaves through the abort flag
                    if (p.selftest_skip_tile >= 0 && blockIdx.x == 0 && gk == p.selftest_skip_tile) continue;
                    mbar_arrive_expect_tx(&bars->k_full[s], TILE);
                    tma_load_3d(Kt + s * TILE, &mapK, 0, kt * TN, u, &bars->k_full[s]);
                    tma_load_3d(Kt + s * TILE + HALF_K, &mapK, 64, kt * TN, u, &bars->k_full[s]);
                    last = gk;
                }
            }
            if (!ok) *(volatile int *)&bars->abort_flag = 1;
            // if the others gave up, nobody waits for the copies requested last: let them land before the CTA goes away
            // (a phase that is past reads as complete, so this costs nothing otherwise)
            if (q_last >= 0) mbar_wait(&bars->q_full, q_last & 1, nullptr, 0);
            for (int gk = last; gk > last - C::KST && gk >= 0; --gk) mbar_wait(&bars->k_full[gk % C::KST], (gk / C::KST) & 1, nullptr, 0);
        }
    } else if (warp == C::W_V) {
        // --------------------------------------------------------------------------------------- value tiles
        if (lane == 0 && start_ok && with_out) {
            bool ok = true;
            int last = -1;
            for (int k = 0; k < nunits && ok; ++k) {
                const int u = blockIdx.x + k * gridDim.x;
                bool appended = false;
                for (int kt = 0; kt < ntiles; ++kt) {
                    const int gv = k * ntiles + kt, b = gv & 1;
                    if (gv >= 2) ok = mbar_wait(&bars->v_empty[b], ((gv >> 1) - 1) & 1, p.err, 0x541);
                    if (ok && !appended && (kt + 1) * TN > n0) {
                        for (int a = 0; a < C::NAPP; ++a) ok = ok && counter_wait(&bars->appended[a], k + 1, p.err, 0x542);
                        fence_proxy_async_all();
                        appended = true;
                    }
                    if (!ok || aborted()) { ok = false; break; }
                    mbar_arrive_expect_tx(&bars->v_full[b], TILE);
                    tma_load_3d(Vt + b * TILE, &mapV, 0, kt * TN, u, &bars->v_full[b]);
                    tma_load_3d(Vt + b * TILE + HALF_K, &mapV, 64, kt * TN, u, &bars->v_full[b]);
                    last = gv;
                }
            }
            if (!ok) *(volatile int *)&bars->abort_flag = 1;
            for (int gv = last; gv > last - 2 && gv >= 0; --gv) mbar_wait(&bars->v_full[gv & 1], (gv >> 1) & 1, nullptr, 0);
        }
    } else if (warp >= C::W_APPEND) {
        // --------------------------------------------------------------------------------------- the append
        // keys, values and positions of the chunk into the cache rows n0 .. n0 + c - 1, queries into the ring of the
        // last w queries; a row of 256 bytes is 16 pieces, the warp moves two rows per instruction
        if (start_ok) {
            for (int k = 0; k < nunits; ++k) {
                if (aborted()) break;
                const int u = blockIdx.x + k * gridDim.x;
                const size_t tstride = (size_t)p.Utot * D * 2;
                const int aw = warp - C::W_APPEND;        // this warp takes every NAPP-th batch of eight rows
                for (int base = aw * 4 * 32; base < c * 16; base += C::NAPP * 4 * 32) {
                    uint4 kk[4], vv[4], qq[4];
#pragma unroll
                    for (int a = 0; a < 4; ++a) {
                        const int idx = base + a * 32 + lane, row = idx >> 4, ch = idx & 15;
                        if (row < c) {
                            const size_t src = (size_t)row * tstride + (size_t)u * D * 2 + ch * 16;
                            kk[a] = *reinterpret_cast<const uint4 *>(p.k + src);
                            vv[a] = *reinterpret_cast<const uint4 *>(p.v + src);
                            if (p.qring) qq[a] = *reinterpret_cast<const uint4 *>(p.q + src);
                        }
                    }
#pragma unroll
                    for (int a = 0; a < 4; ++a) {
                        const int idx = base + a * 32 + lane, row = idx >> 4, ch = idx & 15;
                        if (row < c) {
                            const size_t dst = ((size_t)u * p.B + n0 + row) * (D * 2) + ch * 16;
                            *reinterpret_cast<uint4 *>(p.K + dst) = kk[a];
                            *reinterpret_cast<uint4 *>(p.V + dst) = vv[a];
                            if (p.qring) *reinterpret_cast<uint4 *>(p.qring + ((size_t)u * p.w + (step0 + row) % p.w) * (D * 2) + ch * 16) = qq[a];
                        }
                    }
                }
                if (aw == 0)
                    for (int row = lane; row < c; row += 32) p.pos[(size_t)u * p.B + n0 + row] = step0 + row;
                fence_proxy_async_all();
                __syncwarp();
                if (lane == 0) st_release_shared(&bars->appended[aw], k + 1);
            }
        }
    } else if (start_ok) {
        // --------------------------------------------------------------------------------------- softmax threads
        // this thread's query and its quarter of every tile's columns (64 queries: rows 64..127 repeat rows 0..63)
        const int i = tid & (C::QR - 1), quarter = WIDE ? (tid >> 7) : ((tid >> 6) & 1) * 2 + (tid >> 7);
        const uint32_t lane_addr = tbase + ((uint32_t)((warp & 3) * 32) << 16);
        uint32_t par_pv = 0;
        bool ok = true;
        const int nv = n0 + i + 1;           // keys visible to this thread's query
        const bool live_row = i < c;
        const float tf = (float)(step0 + i);
        for (int k = 0; k < nunits && ok; ++k) {
            const int u = blockIdx.x + k * gridDim.x;
            uint32_t *hrow = p.hist + ((size_t)u * p.w + (step0 + i) % p.w) * p.Bw;
            float m_run = -INFINITY, l_run = 0.f, Mi = 0.f, Li = 1.f;
            int g_exit = G;                  // the iteration a warp left the loop at, after a wait that gave up
            for (int g = 0; g < G; ++g) {
                const int gk = k * G + g, b = gk & 1, kt = key_tile(g);
                const bool second = g >= ntiles;
                ok = mbar_wait(&bars->s_done[b], (gk >> 1) & 1, p.err, 0x501) && ok;
                // (one decision per warp: the tensor-memory loads below are warp-wide)
                if (__any_sync(0xffffffffu, !ok || aborted())) {
                    ok = false;
                    *(volatile int *)&bars->abort_flag = 1;
                    g_exit = g;
                    break;
                }
                tc_fence_after();
                float sv[HC];
                tmem_ld16(lane_addr + S_COL + b * TN + quarter * HC, sv);
                tc_fence_before();
                mbar_arrive(&bars->s_free[b]);       // this thread's share of S is in registers
                const int j0 = kt * TN + quarter * HC;
                const int lim = live_row ? nv - j0 : 0;
                const uint32_t vm = lim <= 0 ? 0u : (lim >= HC ? 0xffffu : (1u << lim) - 1u);
                if (!second) {
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
                        m_sh[tid] = m_run;
                        l_sh[tid] = l_run;
                        softmax_barrier<C::NT>();
                        if (tid < C::QR) {
                            float M = -INFINITY, L = 0.f;
#pragma unroll
                            for (int part = 0; part < C::NT / C::QR; ++part) M = fmaxf(M, m_sh[tid + part * C::QR]);
#pragma unroll
                            for (int part = 0; part < C::NT / C::QR; ++part) {
                                const float mp = m_sh[tid + part * C::QR];
                                if (mp > -INFINITY) L += l_sh[tid + part * C::QR] * ex2_approx(mp - M);
                            }
                            Mfin[tid] = M;
                            Lfin[tid] = L;
                            Linv[tid] = 1.f / L;
                        }
                        softmax_barrier<C::NT>();
                        Mi = Mfin[i];
                        Li = Lfin[i];
                        softmax_barrier<C::NT>();       // everyone has its row's M and L: the P buffer (m_sh, l_sh) may be written
                    }
                    continue;
                }
                uint32_t word = 0, hi[HC / 2], lo[HC / 2];
#pragma unroll
                for (int jj = 0; jj < HC; jj += 2) {
                    const bool v0 = (vm >> jj) & 1u, v1 = (vm >> (jj + 1)) & 1u;
                    const float e0 = v0 ? ex2_approx(sv[jj] * p.scale_log2e - Mi) : 0.f;
                    const float e1 = v1 ? ex2_approx(sv[jj + 1] * p.scale_log2e - Mi) : 0.f;
                    word |= (uint32_t)(e0 * tf < Li) << jj;
                    word |= (uint32_t)(e1 * tf < Li) << (jj + 1);
                    SP::run(e0, e1, hi[jj >> 1], lo[jj >> 1]);
                }
                word &= vm;
                if (live_row && (j0 >> 5) < p.Bw) reinterpret_cast<uint16_t *>(hrow)[j0 >> 4] = (uint16_t)word;
                if (with_out) {
                    const int gv = k * ntiles + kt;
                    if (kt > 0) {                    // the previous tile's P.V has finished: P is free
                        ok = mbar_wait(&bars->pv_done, par_pv, p.err, 0x502) && ok;
                        par_pv ^= 1;
                    }
                    const int rz = n_tot - kt * TN;  // rows of this tile that exist
                    if (rz < TN) ok = mbar_wait(&bars->v_full[gv & 1], (gv >> 1) & 1, p.err, 0x503) && ok;
                    if (__any_sync(0xffffffffu, !ok)) {
                        ok = false;
                        *(volatile int *)&bars->abort_flag = 1;
                        g_exit = g;
                        break;
                    }
                    if (rz < TN) {                   // (the last tile only) stale cache rows beyond the chunk: zero them for P.V
                        char *vt = Vt + (gv & 1) * TILE;
                        for (int idx = tid; idx < (TN - rz) * 16; idx += C::NT) {
                            const int row = rz + (idx >> 4), piece = idx & 15;
                            *reinterpret_cast<uint4 *>(vt + (piece >> 3) * HALF_K + row * 128 + (piece & 7) * 16) = make_uint4(0, 0, 0, 0);
                        }
                    }
#pragma unroll
                    for (int cc = 0; cc < HC / 8; ++cc) {
                        const int off = (i >> 3) * PG + (quarter * (HC / 8) + cc) * 128 + (i & 7) * 16;
                        *reinterpret_cast<uint4 *>(Ph + off) = make_uint4(hi[4 * cc], hi[4 * cc + 1], hi[4 * cc + 2], hi[4 * cc + 3]);
                        *reinterpret_cast<uint4 *>(Pl + off) = make_uint4(lo[4 * cc], lo[4 * cc + 1], lo[4 * cc + 2], lo[4 * cc + 3]);
                    }
                    fence_async_shared();
                    mbar_arrive(&bars->p_ready);     // this thread's part of P(kt) is in place
                }
            }
            if (g_exit < ntiles) {               // the others may be waiting at the three barriers of the first sweep's end
                softmax_barrier<C::NT>();
                softmax_barrier<C::NT>();
                softmax_barrier<C::NT>();
            }
            if (!ok) break;
            if (live_row && quarter == 0)
                for (int wd = ntiles * (TN / 32); wd < p.Bw; ++wd) hrow[wd] = 0;
            if (with_out) {
                ok = mbar_wait(&bars->pv_done, par_pv, p.err, 0x504) && ok;
                par_pv ^= 1;
                if (__any_sync(0xffffffffu, !ok)) {
                    ok = false;
                    *(volatile int *)&bars->abort_flag = 1;
                    break;
                }
                tc_fence_after();
                const int dcol = tid & 127, bq = tid >> 7;      // this thread's column of d and its 32 queries
                float oh[2][16], ol[2][16];
#pragma unroll
                for (int part = 0; part < 2; ++part) {
                    tmem_ld16(lane_addr + O_COL + bq * 32 + part * 16, oh[part]);
                    tmem_ld16(lane_addr + O_COL + C::QR + bq * 32 + part * 16, ol[part]);
                }
                tc_fence_before();
                mbar_arrive(&bars->o_free);          // O^T may be overwritten by the next unit
#pragma unroll
                for (int qq = 0; qq < 32; ++qq) {
                    const int qi = bq * 32 + qq;
                    if (qi < c) p.out[((size_t)qi * p.Utot + u) * D + dcol] = (oh[qq >> 4][qq & 15] + ol[qq >> 4][qq & 15]) * Linv[qi];
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(C::TMEM_COLS) : "memory");
    }
}


// ---------------------------------------------------------------------------------------------------------------
// The record recomputed at compression time (Algorithm 2 as stated) on the same structure.  A work item is one
// unit and up to 128 of its last w steps: the queries come from the ring of stored queries and fill all 128 rows
// of the MMA (nothing is duplicated), the keys are the n0 cached rows, a key is visible to a query when its
// position does not exceed the query's step (slots need not be sorted).  Nothing is appended and no output is
// formed: two sweeps over the key tiles (row maxima and sums, then the comparison bits), and each step's bit-plane
// row is rewritten.  Warps 0..7: softmax arithmetic, two threads per query row, 32 columns each; warp 8: MMA issue;
// warp 9: key tiles by TMA and the tiles' positions; warp 10: the queries, gathered from the ring into the
// swizzled operand layout with plain loads and stores.
constexpr int RQ = 128;                 // queries per work item
constexpr int RKST = 2;                 // key tiles in flight
constexpr int RPD = 4;                  // position tiles in flight (>= RKST + 2: see the producer)
constexpr int RHC = TN / 2;             // columns of a tile per thread
constexpr int RTHREADS = NT + 96;
constexpr int R_TMEM_COLS = 2 * TN;     // two S tiles
constexpr int ROFF_K = 2 * Q_BYTES;     // two query buffers: the next item's queries are gathered during the present item
constexpr int ROFF_POS = ROFF_K + RKST * TILE;
constexpr int ROFF_PMAX = ROFF_POS + RPD * TN * 4;        // per position tile: the largest position in it
constexpr int ROFF_STAT = ROFF_PMAX + RPD * 4;            // m[256], l[256], M[128], L[128]
constexpr int ROFF_BAR = ROFF_STAT + 4 * (2 * NT + 2 * RQ);
constexpr int R_SMEM_BYTES = ROFF_BAR + 256;
static_assert(ROFF_K % 1024 == 0, "swizzled tiles start on 1024-byte boundaries");
static_assert(RPD >= RKST + 2 && (RPD & (RPD - 1)) == 0, "position ring");
static_assert(2 * (R_SMEM_BYTES + 1024) <= 228 * 1024, "two CTAs per SM");

struct RBars {
    uint64_t q_full[2], q_empty[2];
    uint64_t k_full[RKST], k_empty[RKST];
    uint64_t pos_full[RPD];
    uint64_t s_done[2], s_free[2];
    uint32_t tmem_slot;
    int abort_flag;
};
static_assert(sizeof(RBars) <= 256, "barrier block");

template <int DT>
__global__ void __launch_bounds__(RTHREADS, 2) sh_recount_umma_tma_kernel(const ChunkParams p, const __grid_constant__ CUtensorMap mapK) {
    using SP = Split<DT>;
    extern __shared__ __align__(1024) unsigned char sm[];
    char *Qs = reinterpret_cast<char *>(sm);
    char *Kt = reinterpret_cast<char *>(sm) + ROFF_K;
    int *pos_sh = reinterpret_cast<int *>(sm + ROFF_POS);
    int *pmax_sh = reinterpret_cast<int *>(sm + ROFF_PMAX);
    float *m_sh = reinterpret_cast<float *>(sm + ROFF_STAT), *l_sh = m_sh + NT, *Mfin = l_sh + NT, *Lfin = Mfin + RQ;
    RBars *bars = reinterpret_cast<RBars *>(sm + ROFF_BAR);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n0 = p.n0;
    const int ntiles = (n0 + TN - 1) / TN, G = 2 * ntiles;
    const int nblk = (p.nsteps + RQ - 1) / RQ;
    const int items = p.U * nblk;
    const int nitems = (items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;     // work items of this CTA
    auto key_tile = [&](int g) { return g < ntiles ? g : g - ntiles; };
    auto aborted = [&]() { return *(volatile int *)&bars->abort_flag != 0; };

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_slot)), "r"(R_TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        for (int s = 0; s < 2; ++s) { mbar_init(&bars->q_full[s], 1); mbar_init(&bars->q_empty[s], 1); }
        for (int s = 0; s < RKST; ++s) { mbar_init(&bars->k_full[s], 1); mbar_init(&bars->k_empty[s], 1); }
        for (int s = 0; s < RPD; ++s) mbar_init(&bars->pos_full[s], 1);
        for (int s = 0; s < 2; ++s) { mbar_init(&bars->s_done[s], 1); mbar_init(&bars->s_free[s], NT); }
        bars->abort_flag = 0;
        if ((smem_u32(sm) & 1023u) != 0) {
            if (p.err) atomicCAS(p.err, 0, 0x560);
            bars->abort_flag = 1;
        }
        fence_barrier_init();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = bars->tmem_slot;
    const bool start_ok = !aborted() && n0 > 0;

    if (warp == W_MMA) {
        // --------------------------------------------------------------------------------------- the issuing thread
        if (lane == 0 && start_ok) {
            const uint32_t idesc_s = instr_desc(SP::FMT, 0, 128, TN);
            // descriptors of query buffer 0 and key stage 0; the other buffers lie a fixed number of 16-byte units further
            uint64_t dq[D / 16], dk[D / 16];
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                dq[ks] = smem_desc_sw128(smem_u32(Qs) + (ks >> 2) * HALF_Q + (ks & 3) * 32, 16, 1024);
                dk[ks] = smem_desc_sw128(smem_u32(Kt) + (ks >> 2) * HALF_K + (ks & 3) * 32, 16, 1024);
            }
            bool ok = true;
            for (int k = 0; k < nitems && ok; ++k) {
                ok = mbar_wait(&bars->q_full[k & 1], (k >> 1) & 1, p.err, 0x561);
                for (int g = 0; g < G && ok; ++g) {
                    const int gk = k * G + g, s = gk % RKST, b = gk & 1;
                    ok = mbar_wait(&bars->k_full[s], (gk / RKST) & 1, p.err, 0x562);
                    if (gk >= 2) ok = ok && mbar_wait(&bars->s_free[b], ((gk >> 1) - 1) & 1, p.err, 0x563);   // S(gk - 2) has been read out
                    if (!ok || aborted()) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t qoff = (uint64_t)((k & 1) * (Q_BYTES >> 4)), koff = (uint64_t)(s * (TILE >> 4));
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) umma_f16(tbase + b * TN, dq[ks] + qoff, dk[ks] + koff, idesc_s, ks > 0);
                    umma_commit(&bars->k_empty[s]);
                    umma_commit(&bars->s_done[b]);
                    if (g == G - 1) umma_commit(&bars->q_empty[k & 1]);
                }
            }
            if (!ok) *(volatile int *)&bars->abort_flag = 1;
        }
    } else if (warp == W_KQ) {
        // --------------------------------------------------------------------------------------- key tiles and their positions
        // the whole warp walks the tiles: lane 0 waits and requests the copy, every lane stores two positions
        if (start_ok) {
            bool ok = true;
            int last = -1;
            // the positions of a tile are fetched one tile early, so that their latency falls into the wait for the stage
            auto fetch_pos = [&](int k, int g, int (&pv)[2]) {
                if (k >= nitems) return;
                const int u = (blockIdx.x + k * gridDim.x) / nblk, kt = key_tile(g);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int j = kt * TN + h * 32 + lane;
                    pv[h] = j < n0 ? p.pos[(size_t)u * p.B + j] : 0x7fffffff;      // slots beyond the cache: never visible
                }
            };
            int pv[2];
            fetch_pos(0, 0, pv);
            for (int k = 0; k < nitems && ok; ++k) {
                const int u = (blockIdx.x + k * gridDim.x) / nblk;
                for (int g = 0; g < G; ++g) {
                    const int gk = k * G + g, s = gk % RKST, kt = key_tile(g);
                    if (lane == 0) {
                        // S(gk - RKST) has been computed; it was issued after S(gk - RKST - 2) had been read out, and the
                        // softmax threads read a tile's positions before they release its S buffer: so the positions
                        // of tile gk - RPD are no longer needed, RPD >= RKST + 2
                        if (gk >= RKST) ok = mbar_wait(&bars->k_empty[s], ((gk / RKST) - 1) & 1, p.err, 0x571);
                        if (aborted()) ok = false;
                    }
                    ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                    if (!ok) break;
                    if (lane == 0) {
                        mbar_arrive_expect_tx(&bars->k_full[s], TILE);
                        tma_load_3d(Kt + s * TILE, &mapK, 0, kt * TN, u, &bars->k_full[s]);
                        tma_load_3d(Kt + s * TILE + HALF_K, &mapK, 64, kt * TN, u, &bars->k_full[s]);
                    }
                    int *pt = pos_sh + (gk % RPD) * TN;
                    pt[lane] = pv[0];
                    pt[32 + lane] = pv[1];
                    const int tile_max = __reduce_max_sync(0xffffffffu, max(pv[0], pv[1]));
                    if (lane == 0) pmax_sh[gk % RPD] = tile_max;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->pos_full[gk % RPD]);
                    last = gk;
                    if (g + 1 < G) fetch_pos(k, g + 1, pv);
                    else fetch_pos(k + 1, 0, pv);
                }
            }
            if (lane == 0) {
                if (!ok) *(volatile int *)&bars->abort_flag = 1;
                for (int gk = last; gk > last - RKST && gk >= 0; --gk) mbar_wait(&bars->k_full[gk % RKST], (gk / RKST) & 1, nullptr, 0);
            }
        }
    } else if (warp == W_V) {
        // --------------------------------------------------------------------------------------- the queries
        // rows (step mod w) of the unit's ring, 16 pieces of 16 bytes each, into the K-major 128-byte swizzle:
        // piece ch of row r goes to half ch / 8, row r, 16-byte column (ch % 8) ^ (r % 8)
        if (start_ok) {
            bool ok = true;
            for (int k = 0; k < nitems && ok; ++k) {
                const int item = blockIdx.x + k * gridDim.x, u = item / nblk, qb = item % nblk;
                const int s0 = p.first_step + qb * RQ, c = min(RQ, p.nsteps - qb * RQ);
                if (lane == 0) {
                    if (k >= 2) ok = mbar_wait(&bars->q_empty[k & 1], ((k >> 1) - 1) & 1, p.err, 0x581);     // item k - 2 has left this buffer
                    if (aborted()) ok = false;
                }
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
                char *Qb = Qs + (k & 1) * Q_BYTES;
                for (int base = 0; base < RQ * 16; base += 8 * 32) {
                    uint4 qq[8];
#pragma unroll
                    for (int a = 0; a < 8; ++a) {
                        const int idx = base + a * 32 + lane, row = idx >> 4, ch = idx & 15;
                        qq[a] = row < c ? *reinterpret_cast<const uint4 *>(p.qring + ((size_t)u * p.w + (s0 + row) % p.w) * (D * 2) + ch * 16)
                                        : make_uint4(0, 0, 0, 0);
                    }
#pragma unroll
                    for (int a = 0; a < 8; ++a) {
                        const int idx = base + a * 32 + lane, row = idx >> 4, ch = idx & 15;
                        *reinterpret_cast<uint4 *>(Qb + (ch >> 3) * HALF_Q + row * 128 + (((ch & 7) ^ (row & 7)) << 4)) = qq[a];
                    }
                }
                fence_async_shared();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars->q_full[k & 1]);
            }
            if (lane == 0 && !ok) *(volatile int *)&bars->abort_flag = 1;
        }
    } else if (start_ok) {
        // --------------------------------------------------------------------------------------- softmax threads
        const int i = tid & 127, half = tid >> 7;        // this thread's query row and its half of every tile's columns
        const uint32_t lane_addr = tbase + ((uint32_t)((warp & 3) * 32) << 16);
        bool ok = true;
        for (int k = 0; k < nitems && ok; ++k) {
            const int item = blockIdx.x + k * gridDim.x, u = item / nblk, qb = item % nblk;
            const int s0 = p.first_step + qb * RQ, c = min(RQ, p.nsteps - qb * RQ);
            const int step = s0 + i;
            const bool live_row = i < c;
            const float tf = (float)step;
            uint32_t *hrow = p.hist + ((size_t)u * p.w + step % p.w) * p.Bw;
            float m_run = -INFINITY, l_run = 0.f, Mi = 0.f, Li = 1.f;
            int g_exit = G;
            for (int g = 0; g < G; ++g) {
                const int gk = k * G + g, b = gk & 1, kt = key_tile(g);
                ok = mbar_wait(&bars->s_done[b], (gk >> 1) & 1, p.err, 0x551) && ok;
                ok = mbar_wait(&bars->pos_full[gk % RPD], (gk / RPD) & 1, p.err, 0x552) && ok;
                if (__any_sync(0xffffffffu, !ok || aborted())) {
                    ok = false;
                    *(volatile int *)&bars->abort_flag = 1;
                    g_exit = g;
                    break;
                }
                tc_fence_after();
                float sv[RHC];
                tmem_ld32(lane_addr + b * TN + half * RHC, sv);
                tc_fence_before();
                // bit jj of vm: column jj of this thread's half is visible to its query.  Most tiles hold only tokens older
                // than every query of the item (their largest position says so): nothing to compare
                uint32_t vm = 0xffffffffu;
                if (pmax_sh[gk % RPD] > step) {
                    vm = 0;
                    const int4 *pt = reinterpret_cast<const int4 *>(pos_sh + (gk % RPD) * TN + half * RHC);
#pragma unroll
                    for (int q4 = 0; q4 < RHC / 4; ++q4) {
                        const int4 pp = pt[q4];
                        vm |= (uint32_t)(pp.x <= step) << (4 * q4) | (uint32_t)(pp.y <= step) << (4 * q4 + 1) |
                              (uint32_t)(pp.z <= step) << (4 * q4 + 2) | (uint32_t)(pp.w <= step) << (4 * q4 + 3);
                    }
                }
                if (!live_row) vm = 0;
                mbar_arrive(&bars->s_free[b]);       // S is in registers and the tile's positions have been read
                if (g < ntiles) {
                    if (vm) {
                        float bmax = -INFINITY;
#pragma unroll
                        for (int jj = 0; jj < RHC; ++jj) {
                            sv[jj] = ((vm >> jj) & 1u) ? sv[jj] * p.scale_log2e : -INFINITY;
                            bmax = fmaxf(bmax, sv[jj]);
                        }
                        const float m_new = fmaxf(m_run, bmax);
                        float acc = 0.f;
#pragma unroll
                        for (int jj = 0; jj < RHC; ++jj) acc += ex2_approx(sv[jj] - m_new);
                        l_run = l_run * ex2_approx(m_run - m_new) + acc;
                        m_run = m_new;
                    }
                    if (g == ntiles - 1) {
                        m_sh[tid] = m_run;
                        l_sh[tid] = l_run;
                        softmax_barrier<NT>();
                        if (tid < RQ) {
                            const float ma = m_sh[tid], mb = m_sh[tid + RQ];
                            const float M = fmaxf(ma, mb);
                            float L = 0.f;
                            if (ma > -INFINITY) L += l_sh[tid] * ex2_approx(ma - M);
                            if (mb > -INFINITY) L += l_sh[tid + RQ] * ex2_approx(mb - M);
                            Mfin[tid] = M;
                            Lfin[tid] = L;
                        }
                        softmax_barrier<NT>();
                        Mi = Mfin[i];
                        Li = Lfin[i];
                        softmax_barrier<NT>();       // everyone has its row's M and L: the next item may overwrite them
                    }
                    continue;
                }
                uint32_t word = 0;
#pragma unroll
                for (int jj = 0; jj < RHC; ++jj) {
                    const float e = ((vm >> jj) & 1u) ? ex2_approx(sv[jj] * p.scale_log2e - Mi) : 0.f;
                    word |= (uint32_t)(e * tf < Li) << jj;
                }
                word &= vm;
                if (live_row && kt * 2 + half < p.Bw) hrow[kt * 2 + half] = word;
            }
            if (g_exit < ntiles) {               // the others may be waiting at the three barriers of the first sweep's end
                softmax_barrier<NT>();
                softmax_barrier<NT>();
                softmax_barrier<NT>();
            }
            if (!ok) break;
            if (live_row && half == 0)
                for (int wd = ntiles * (TN / 32); wd < p.Bw; ++wd) hrow[wd] = 0;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(R_TMEM_COLS) : "memory");
    }
}

typedef CUresult (*EncodeTiled)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime (the library does not link against the driver).
EncodeTiled encoder() {
    static EncodeTiled fn = [] {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            sym = nullptr;
        return reinterpret_cast<EncodeTiled>(sym);
    }();
    return fn;
}

// Map over rows of 128 16-bit elements: [dim2][dim1][128], boxes of 64 elements x (box1 x box2) rows, 128-byte swizzle,
// zeros outside the tensor.
bool make_map(CUtensorMap *m, const void *base, uint64_t dim1, uint64_t dim2, uint64_t stride1, uint64_t stride2, uint32_t box1,
              uint32_t box2) {
    EncodeTiled enc = encoder();
    if (!enc) return false;
    const cuuint64_t gdim[3] = {(cuuint64_t)D, dim1, dim2};
    const cuuint64_t gstride[2] = {stride1, stride2};
    const cuuint32_t box[3] = {64u, box1, box2};
    const cuuint32_t estr[3] = {1u, 1u, 1u};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT16, 3, const_cast<void *>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// SMs of the current device (asked on every launch: a process may drive several devices).
int sm_count() {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) v = 0;
    return v;
}

template <int DT, bool WIDE>
cudaError_t launch_tma(const ChunkParams &p, cudaStream_t s) {
    using C = CK<WIDE>;
    CUtensorMap mq, mk, mv;
    const uint64_t row = (uint64_t)D * 2;
    if (!make_map(&mq, p.q, (uint64_t)p.Utot, (uint64_t)p.c, row, (uint64_t)p.Utot * row, 1, 64) ||
        !make_map(&mk, p.K, (uint64_t)p.B, (uint64_t)p.U, row, (uint64_t)p.B * row, TN, 1) ||
        !make_map(&mv, p.V, (uint64_t)p.B, (uint64_t)p.U, row, (uint64_t)p.B * row, TN, 1))
        return cudaErrorNotSupported;
    auto kern = sh_chunk_umma_tma_kernel<DT, WIDE>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const int sms = sm_count();
    if (sms <= 0) return cudaErrorInvalidDevice;
    const int grid = p.U < C::CTAS * sms ? p.U : C::CTAS * sms;
    kern<<<dim3(grid, 1, 1), C::NTH, C::SMEM_BYTES, s>>>(p, mq, mk, mv);
    return cudaGetLastError();
}

template <int DT>
cudaError_t launch_recount_tma(const ChunkParams &p, cudaStream_t s) {
    CUtensorMap mk;
    const uint64_t row = (uint64_t)D * 2;
    if (!make_map(&mk, p.K, (uint64_t)p.B, (uint64_t)p.U, row, (uint64_t)p.B * row, TN, 1)) return cudaErrorNotSupported;
    auto kern = sh_recount_umma_tma_kernel<DT>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, R_SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const int sms = sm_count();
    if (sms <= 0) return cudaErrorInvalidDevice;
    const long long items = (long long)p.U * ((p.nsteps + RQ - 1) / RQ);
    const int grid = items < 2 * sms ? (int)items : 2 * sms;
    kern<<<dim3(grid, 1, 1), RTHREADS, R_SMEM_BYTES, s>>>(p, mk);
    return cudaGetLastError();
}

}  // namespace

cudaError_t sh_launch_recount_umma_tma(const ChunkParams &p, int dtype, cudaStream_t s) {
    if (p.nsteps < 1 || p.out || p.U < 1) return cudaErrorInvalidValue;
    if (p.n0 < 1) return cudaSuccess;
    return dtype == SH_F16 ? launch_recount_tma<SH_F16>(p, s) : launch_recount_tma<SH_BF16>(p, s);
}

int sh_chunk_umma_tma_capacity() { return CK<true>::QR; }

cudaError_t sh_launch_chunk_umma_tma(const ChunkParams &p, int dtype, cudaStream_t s, int *launches) {
    *launches = 0;
    if (p.c < 1 || p.c > CK<true>::QR || p.U < 1) return cudaErrorInvalidValue;
    cudaError_t e;
    if (p.c <= CK<false>::QR) {
        e = dtype == SH_F16 ? launch_tma<SH_F16, false>(p, s) : launch_tma<SH_BF16, false>(p, s);
        if (e == cudaSuccess) *launches = 1;
        return e;
    }
    // More than 64 tokens.  The wide shape runs one CTA per SM: it pays from about four units per SM on (1280 units:
    // 128 tokens in 0.79 of the time of two narrow launches; 256 units: 1.5 times slower, half the SMs would hold
    // one unit and wait for the others' second).  With fewer units the chunk goes as two narrow launches.
    if (p.U >= 4 * sm_count()) {
        e = dtype == SH_F16 ? launch_tma<SH_F16, true>(p, s) : launch_tma<SH_BF16, true>(p, s);
        if (e == cudaSuccess) *launches = 1;
        return e;
    }
    for (int done = 0; done < p.c; done += CK<false>::QR) {
        ChunkParams part = p;
        const size_t skip = (size_t)done * p.Utot * D;        // elements of q, k, v and out before token `done`
        part.q = p.q + skip * 2; part.k = p.k + skip * 2; part.v = p.v + skip * 2;
        part.out = p.out ? p.out + skip : nullptr;
        part.n0 = p.n0 + done; part.t0 = p.t0 + done;
        part.c = p.c - done < CK<false>::QR ? p.c - done : CK<false>::QR;
        e = dtype == SH_F16 ? launch_tma<SH_F16, false>(part, s) : launch_tma<SH_BF16, false>(part, s);
        if (e != cudaSuccess) return e;
        *launches += 1;
    }
    return cudaSuccess;
}
