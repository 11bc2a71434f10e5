// Chunked prompt step on an int4-g64 cache (tcgen05.mma, accumulators in tensor memory).
//
// Same structure as sh_chunk_umma.cu - 64 queries as rows 0..63 and again 64..127, key tiles of 64
// visited twice, four threads per query row - with the arithmetic arranged so that it equals the decode
// step's on the int4 store:
//
//   * The tensor-core operands are the integer codes themselves (exact in fp16), unpacked from the
//     cache into the tiles by the threads; the group scales never enter a 16-bit operand.
//   * A row has two groups of 64 dimensions with a scale each, so a logit is
//       s_j = scale * ( ks[j][0] * sum_{d<64} q_d c_jd  +  ks[j][1] * sum_{d>=64} q_d c_jd ):
//     the two sums are two accumulators in tensor memory (k-steps 0..3 and 4..7 of the tile) and the
//     threads combine them in fp32.
//   * out_d = sum_j p_j * vs[j][g(d)] * c_jd: the value scale is folded into the probabilities, one
//     set per group (P'_g = p * vs[.][g], as high and low fp16 parts), and O^T is accumulated once per
//     group; output column d takes its value from the accumulator of its own group.
//   * The chunk's own keys and values are quantised first (same rule as the decode step: a = max|x| over
//     the group, sc = fp16(a/7), code = clamp(rint(x/sc), -7, 7), IEEE fp32) and written to the cache;
//     every tile then comes from the cache.
//
// One CTA of 8 warps per unit and SM (384 columns of tensor memory, 130 KB of shared memory).  Every
// mbarrier wait is bounded; tensor memory is released on every path.
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
constexpr int NT = 256;           // threads per CTA: two per lane of tensor memory
constexpr int HC = TN / 4;        // columns of a tile per thread
constexpr int GROUP = 2048;       // bytes of 8 rows of 256 B in core-matrix order: [16 chunks][8 rows][16 B]
constexpr int TILE = (TN / 8) * GROUP;          // 16 KB: 64 rows of 128 fp16 codes
constexpr int Q_BYTES = (2 * CQ / 8) * GROUP;   // 128 rows
constexpr int PG = (TN / 8) * 128;              // bytes of 8 rows of P (TN keys each)
constexpr int P_BYTES = (CQ / 8) * PG;          // 64 rows x TN keys x 2 B
constexpr int ROWB = D / 2;                     // stored row: 64 bytes of codes
constexpr int TMEM_COLS = 512;
constexpr int S_COL = 0;          // S(buffer b, group g): columns (2 b + g) * TN
constexpr int O_COL = 4 * TN;     // O^T of group g: columns O_COL + g * CQ

constexpr int OFF_Q = 0;
constexpr int OFF_K = OFF_Q + Q_BYTES;
constexpr int OFF_V = OFF_K + 2 * TILE;
constexpr int OFF_P = OFF_V + 2 * TILE;         // [group][hi, lo]
constexpr int OFF_KS = OFF_P + 4 * P_BYTES;     // float [3][TN][2]: key scales of tile g in buffer g mod 3
constexpr int OFF_VS = OFF_KS + 3 * TN * 2 * 4; // float [2][TN][2]: value scales of tile kt in buffer kt & 1
constexpr int OFF_STAT = OFF_VS + 2 * TN * 2 * 4;
constexpr int OFF_BAR = OFF_STAT + 4 * (64 + 64);
constexpr int SMEM_BYTES = OFF_BAR + 64;
static_assert(4 * P_BYTES >= 4 * 2 * NT, "the first sweep's statistics alias the P buffers");
static_assert(HC == 16, "a thread reads its 16 columns with one tcgen05.ld and owns half a record word");

// 8 codes of one 32-bit word -> 8 exact fp16 integers (16 bytes), element order 0..7.
// Element e of a word sits in nibble (e >> 1) + 4 (e & 1), biased by +8.
__device__ __forceinline__ uint4 unpack8(uint32_t w) {
    const __half2 bias = __floats2half2_rn(1032.f, 1032.f);
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint32_t bits = ((w >> (4 * i)) & 0x000F000Fu) | 0x64006400u;
        const __half2 h = __hsub2(*reinterpret_cast<__half2 *>(&bits), bias);
        o[i] = *reinterpret_cast<const uint32_t *>(&h);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// One thread's share of a tile: the 16 bytes (32 codes) of piece (row, quarter) of the stored rows.
struct Piece {
    uint4 codes;
    float sc0, sc1;     // the row's two group scales (only the thread with quarter 0 keeps them)
};

// Rows [j0, j0 + TN) of the unit's K or V codes: thread tid takes row tid / 4, bytes 16 (tid % 4) .. +16.
__device__ __forceinline__ Piece load_piece(const char *codes_u, const __half *scales_u, int j0, int n_tot) {
    Piece pc;
    const int row = threadIdx.x >> 2, qt = threadIdx.x & 3, j = j0 + row;
    pc.codes = make_uint4(0x88888888u, 0x88888888u, 0x88888888u, 0x88888888u);     // code 0 in every nibble
    pc.sc0 = 0.f;
    pc.sc1 = 0.f;
    if (j < n_tot) {
        pc.codes = *reinterpret_cast<const uint4 *>(codes_u + (size_t)j * ROWB + qt * 16);
        if (qt == 0) {
            const __half2 s2 = *reinterpret_cast<const __half2 *>(scales_u + (size_t)j * 2);
            pc.sc0 = __low2float(s2);
            pc.sc1 = __high2float(s2);
        }
    }
    return pc;
}
// ... unpacked into the tile (canonical no-swizzle order [row / 8][16-byte column][row % 8]) and the scale table.
__device__ __forceinline__ void store_piece(const Piece &pc, char *tile, float *scales_sh) {
    const int row = threadIdx.x >> 2, qt = threadIdx.x & 3;
    char *dst = tile + (row >> 3) * GROUP + (qt * 4) * 128 + (row & 7) * 16;
    *reinterpret_cast<uint4 *>(dst) = unpack8(pc.codes.x);
    *reinterpret_cast<uint4 *>(dst + 128) = unpack8(pc.codes.y);
    *reinterpret_cast<uint4 *>(dst + 256) = unpack8(pc.codes.z);
    *reinterpret_cast<uint4 *>(dst + 384) = unpack8(pc.codes.w);
    if (qt == 0) {
        scales_sh[row * 2] = pc.sc0;
        scales_sh[row * 2 + 1] = pc.sc1;
    }
}

// Quantise one group of 64 values of an input row (fp16, 128 bytes at src) into 32 bytes of codes at
// dst and its scale: the decode step's rule, in IEEE fp32.
__device__ __forceinline__ void quantise_group(const char *src, char *dst, __half *scale_out) {
    float f[64];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const uint4 raw = *reinterpret_cast<const uint4 *>(src + 16 * k);
        const __half2 *h = reinterpret_cast<const __half2 *>(&raw);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 t = __half22float2(h[i]);
            f[8 * k + 2 * i] = t.x;
            f[8 * k + 2 * i + 1] = t.y;
        }
    }
    float a = 0.f;
#pragma unroll
    for (int i = 0; i < 64; ++i) a = fmaxf(a, fabsf(f[i]));
    const float sc = __half2float(__float2half_rn(__fdiv_rn(a, 7.0f)));
#pragma unroll
    for (int k = 0; k < 8; k += 4) {
        uint32_t w[4];
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            w[kk] = 0;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                float code = 0.f;
                if (sc != 0.f) code = fminf(fmaxf(rintf(__fdiv_rn(f[8 * (k + kk) + e], sc)), -7.f), 7.f);
                w[kk] |= (uint32_t)((int)code + 8) << (4 * ((e >> 1) + 4 * (e & 1)));
            }
        }
        *reinterpret_cast<uint4 *>(dst + 4 * k) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    *scale_out = __float2half_rn(sc);
}


// RECOUNT: the record recomputed at compression time - queries from the ring of the last w queries (blockIdx.y
// selects 64 of them), keys the n0 cached rows, a key visible to a query when its position does not exceed the
// query's step; nothing is appended, no output: only the bit-plane rows of those steps are rewritten.
template <bool RECOUNT>
__global__ void __launch_bounds__(NT, 1) sh_chunk_umma_int4_kernel(const ChunkParams p) {
    using SP = Split<SH_F16>;
    extern __shared__ __align__(128) unsigned char sm[];
    char *Qs = reinterpret_cast<char *>(sm) + OFF_Q;
    char *Kt = reinterpret_cast<char *>(sm) + OFF_K;
    char *Vt = reinterpret_cast<char *>(sm) + OFF_V;
    char *Pb = reinterpret_cast<char *>(sm) + OFF_P;        // P'[group][hi, lo]
    float *ks_sh = reinterpret_cast<float *>(sm + OFF_KS);
    float *vs_sh = reinterpret_cast<float *>(sm + OFF_VS);
    float *m_sh = reinterpret_cast<float *>(sm + OFF_P);     // the first sweep's per-thread statistics (P is idle then)
    float *l_sh = m_sh + NT;
    float *Mfin = reinterpret_cast<float *>(sm + OFF_STAT), *Lfin = Mfin + 64;
    uint64_t *bar_s = reinterpret_cast<uint64_t *>(sm + OFF_BAR);
    uint64_t *bar_pv = bar_s + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bar_s + 3);

    const int u = blockIdx.x, tid = threadIdx.x, warp = tid >> 5;
    const int i = tid & 63, quarter = ((tid >> 6) & 1) * 2 + (tid >> 7);
    const int qoff = RECOUNT ? (int)blockIdx.y * CQ : 0;
    const int n0 = p.n0, c = RECOUNT ? min(CQ, p.nsteps - qoff) : p.c, n_tot = RECOUNT ? n0 : n0 + c;
    const int ntiles = (n_tot + TN - 1) / TN;
    const int step0 = RECOUNT ? p.first_step + qoff : p.t0 + 1;     // step of this CTA's first query
    int *pos_sh = reinterpret_cast<int *>(sm + OFF_P + 4096);       // [3][TN] positions of the key tiles (recount: P is idle)
    const int32_t *pos_u = p.pos + (size_t)u * p.B;
    auto load_pos = [&](int buf, int kt) {
        if (RECOUNT && tid < TN) {
            const int j = kt * TN + tid;
            pos_sh[buf * TN + tid] = j < n0 ? pos_u[j] : 0x7fffffff;
        }
    };
    const size_t tstride = (size_t)p.Utot * D * 2;       // bytes between consecutive tokens of one unit (fp16 inputs)
    char *Kc = p.K + (size_t)u * p.B * ROWB;
    char *Vc = p.V + (size_t)u * p.B * ROWB;
    __half *Ksc = reinterpret_cast<__half *>(p.Ks) + (size_t)u * p.Bs * 2;
    __half *Vsc = reinterpret_cast<__half *>(p.Vs) + (size_t)u * p.Bs * 2;

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
    // ---- the chunk's tokens: quantise keys and values into the cache (thread = (row, group, K or V)), positions
    if (!RECOUNT) {
        const int row = tid >> 2, g = (tid >> 1) & 1, isv = tid & 1;
        if (row < c) {
            const char *src = (isv ? p.v : p.k) + (size_t)row * tstride + (size_t)u * D * 2 + g * 128;
            char *dst = (isv ? Vc : Kc) + (size_t)(n0 + row) * ROWB + g * 32;
            quantise_group(src, dst, (isv ? Vsc : Ksc) + (size_t)(n0 + row) * 2 + g);
        }
        if (tid < c) p.pos[(size_t)u * p.B + n0 + tid] = step0 + tid;
    }
    // ---- queries (rows beyond c are zero), twice: rows 0..63 and 64..127; remembered for a later recount
    for (int idx = tid; idx < CQ * 16; idx += NT) {
        const int row = idx >> 4, ch = idx & 15;
        uint4 val = make_uint4(0, 0, 0, 0);
        if (row < c) {
            char *ring_row = p.qring ? p.qring + ((size_t)u * p.w + (step0 + row) % p.w) * (D * 2) + ch * 16 : nullptr;
            if (RECOUNT) {
                val = *reinterpret_cast<const uint4 *>(ring_row);
            } else {
                val = *reinterpret_cast<const uint4 *>(p.q + (size_t)row * tstride + (size_t)u * D * 2 + ch * 16);
                if (ring_row) *reinterpret_cast<uint4 *>(ring_row) = val;
            }
        }
        char *dst = Qs + (row >> 3) * GROUP + ch * 128 + (row & 7) * 16;
        *reinterpret_cast<uint4 *>(dst) = val;
        *reinterpret_cast<uint4 *>(dst + (CQ / 8) * GROUP) = val;
    }
    __threadfence_block();
    __syncthreads();                 // the appended rows are in the cache for every thread of this CTA
    // The two sweeps form one sequence of G = 2 ntiles S tiles; tile g covers the keys of tile g mod ntiles.
    // S buffers, K buffer and mbarrier of tile g: g & 1; key scales: g mod 3.  V tile kt: buffer kt & 1.
    const int G = 2 * ntiles;
    auto key_tile = [&](int g) { return g < ntiles ? g : g - ntiles; };
    store_piece(load_piece(Kc, Ksc, 0, n_tot), Kt, ks_sh);
    store_piece(load_piece(Kc, Ksc, key_tile(1) * TN, n_tot), Kt + TILE, ks_sh + TN * 2);
    load_pos(0, 0);          // positions of tile g sit in buffer g mod 3
    load_pos(1, key_tile(1));
    if (p.out) store_piece(load_piece(Vc, Vsc, 0, n_tot), Vt, vs_sh);
    fence_async_shared();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = *tmem_slot;
    const uint32_t lane_addr = tbase + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t q_addr = smem_u32(Qs), k_addr = smem_u32(Kt), v_addr = smem_u32(Vt), p_addr = smem_u32(Pb);
    const uint32_t idesc_s = instr_desc(SP::FMT, 0, 128, TN);
    const uint32_t idesc_pv = instr_desc(SP::FMT, 1, 128, CQ);
    auto issue_s = [&](int g) {        // the two group sums of S tile g into S(g & 1, 0) and S(g & 1, 1) (one thread)
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
            umma_f16(tbase + S_COL + ((g & 1) * 2 + (ks >> 2)) * TN, smem_desc(q_addr + ks * 256, 128, GROUP),
                     smem_desc(k_addr + (g & 1) * TILE + ks * 256, 128, GROUP), idesc_s, (ks & 3) > 0);
        umma_commit(bar_s + (g & 1));
    };

    uint32_t par_s = 0, par_pv = 0;
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
        fence_async_shared();          // the tiles stored at the end of the previous iteration
        tc_fence_before();
        if (!__syncthreads_and(ok)) { ok = false; break; }
        if (tid == 0 && g + 1 < G) issue_s(g + 1);
        ok = mbar_wait(bar_s + (g & 1), (par_s >> (g & 1)) & 1, p.err, 0x511) && ok;
        par_s ^= 1u << (g & 1);
        if (second && kt > 0 && p.out) {     // the previous tile's P.V has finished: P and the V buffer it read are free
            ok = mbar_wait(bar_pv, par_pv, p.err, 0x512) && ok;
            par_pv ^= 1;
        }
        tc_fence_after();
        // the next tiles' codes start their way from the cache now and are unpacked at the end of the iteration
        const bool want_k = g + 2 < G, want_v = p.out && second && kt + 1 < ntiles;
        Piece pk = {}, pv = {};
        if (want_k) pk = load_piece(Kc, Ksc, key_tile(g + 2) * TN, n_tot);
        if (want_v) pv = load_piece(Vc, Vsc, (kt + 1) * TN, n_tot);
        float s0[HC], s1[HC];
        tmem_ld16(lane_addr + S_COL + ((g & 1) * 2) * TN + quarter * HC, s0);
        tmem_ld16(lane_addr + S_COL + ((g & 1) * 2 + 1) * TN + quarter * HC, s1);
        const float *ksc = ks_sh + (g % 3) * TN * 2 + quarter * HC * 2;
        const int j0 = kt * TN + quarter * HC;
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
        float sv[HC];
#pragma unroll
        for (int jj = 0; jj < HC; ++jj) sv[jj] = (s0[jj] * ksc[2 * jj] + s1[jj] * ksc[2 * jj + 1]) * p.scale_log2e;
        if (!second) {
            if (vm) {
                float bmax = -INFINITY;
#pragma unroll
                for (int jj = 0; jj < HC; ++jj) {
                    sv[jj] = ((vm >> jj) & 1u) ? sv[jj] : -INFINITY;
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
        } else {
            // ---- second sweep: probabilities, record bits, P' = p * value scale per group, O^T_g += V^T . P'_g^T
            const float *vsc = vs_sh + (kt & 1) * TN * 2 + quarter * HC * 2;
            uint32_t word = 0, h0[HC / 2], l0[HC / 2], h1[HC / 2], l1[HC / 2];
#pragma unroll
            for (int jj = 0; jj < HC; jj += 2) {
                const bool v0 = (vm >> jj) & 1u, v1 = (vm >> (jj + 1)) & 1u;
                const float e0 = v0 ? ex2_approx(sv[jj] - Mi) : 0.f;
                const float e1 = v1 ? ex2_approx(sv[jj + 1] - Mi) : 0.f;
                word |= (uint32_t)(e0 * tf < Li) << jj;
                word |= (uint32_t)(e1 * tf < Li) << (jj + 1);
                SP::run(e0 * vsc[2 * jj], e1 * vsc[2 * jj + 2], h0[jj >> 1], l0[jj >> 1]);
                SP::run(e0 * vsc[2 * jj + 1], e1 * vsc[2 * jj + 3], h1[jj >> 1], l1[jj >> 1]);
            }
            word &= vm;
            if (live_row && (j0 >> 5) < p.Bw) reinterpret_cast<uint16_t *>(hrow)[j0 >> 4] = (uint16_t)word;
            if (p.out) {
#pragma unroll
                for (int cc = 0; cc < HC / 8; ++cc) {
                    const int off = (i >> 3) * PG + (quarter * (HC / 8) + cc) * 128 + (i & 7) * 16;
                    *reinterpret_cast<uint4 *>(Pb + off) = make_uint4(h0[4 * cc], h0[4 * cc + 1], h0[4 * cc + 2], h0[4 * cc + 3]);
                    *reinterpret_cast<uint4 *>(Pb + P_BYTES + off) = make_uint4(l0[4 * cc], l0[4 * cc + 1], l0[4 * cc + 2], l0[4 * cc + 3]);
                    *reinterpret_cast<uint4 *>(Pb + 2 * P_BYTES + off) = make_uint4(h1[4 * cc], h1[4 * cc + 1], h1[4 * cc + 2], h1[4 * cc + 3]);
                    *reinterpret_cast<uint4 *>(Pb + 3 * P_BYTES + off) = make_uint4(l1[4 * cc], l1[4 * cc + 1], l1[4 * cc + 2], l1[4 * cc + 3]);
                }
                fence_async_shared();
                tc_fence_before();
                __syncthreads();
                if (tid == 0) {
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < TN / 16; ++ks) {
                        const uint64_t a = smem_desc(v_addr + (kt & 1) * TILE + ks * 2 * GROUP, GROUP, 128);
#pragma unroll
                        for (int gg = 0; gg < 2; ++gg) {
                            umma_f16(tbase + O_COL + gg * CQ, a, smem_desc(p_addr + (2 * gg) * P_BYTES + ks * 256, 128, PG), idesc_pv,
                                     (kt > 0 || ks > 0));
                            umma_f16(tbase + O_COL + gg * CQ, a, smem_desc(p_addr + (2 * gg + 1) * P_BYTES + ks * 256, 128, PG), idesc_pv, 1);
                        }
                    }
                    umma_commit(bar_pv);
                }
            }
        }
        // ---- the next tiles go into the buffers that S(g) and the previous P.V have released
        if (want_k) {
            store_piece(pk, Kt + (g & 1) * TILE, ks_sh + ((g + 2) % 3) * TN * 2);
            load_pos((g + 2) % 3, key_tile(g + 2));
        }
        if (want_v) store_piece(pv, Vt + ((kt + 1) & 1) * TILE, vs_sh + ((kt + 1) & 1) * TN * 2);
    }
    if (ok) {
        if (live_row && quarter == 0)
            for (int wd = ntiles * (TN / 32); wd < p.Bw; ++wd) hrow[wd] = 0;
        if (p.out) {
            ok = mbar_wait(bar_pv, par_pv, p.err, 0x514) && ok;
            tc_fence_after();
        }
    }
    // ---- O^T: lane = output column (its group's accumulator), tensor-memory column = query
    if (p.out) {
        const int dcol = tid & 127, b = tid >> 7;
        float ov[32];
        tmem_ld32(lane_addr + O_COL + (dcol >> 6) * CQ + b * 32, ov);
        if (ok) {
#pragma unroll
            for (int qq = 0; qq < 32; ++qq) {
                const int qi = b * 32 + qq;
                if (qi < c) p.out[((size_t)qi * p.Utot + u) * D + dcol] = ov[qq] / Lfin[qi];
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(TMEM_COLS) : "memory");
    }
}

}  // namespace

cudaError_t sh_launch_chunk_umma_int4(const ChunkParams &p, cudaStream_t s) {
    if (p.c < 1 || p.c > CQ) return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(sh_chunk_umma_int4_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    sh_chunk_umma_int4_kernel<false><<<p.U, NT, SMEM_BYTES, s>>>(p);
    return cudaGetLastError();
}

cudaError_t sh_launch_recount_umma_int4(const ChunkParams &p, cudaStream_t s) {
    if (p.nsteps < 1 || p.out) return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(sh_chunk_umma_int4_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    sh_chunk_umma_int4_kernel<true><<<dim3(p.U, (unsigned)((p.nsteps + CQ - 1) / CQ), 1), NT, SMEM_BYTES, s>>>(p);
    return cudaGetLastError();
}
