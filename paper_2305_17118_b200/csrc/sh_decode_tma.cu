// Fused decode step, persistent pipelined variant: one CTA per SM walks over
// its share of the units while a producer thread streams their K and V rows
// into a shared-memory ring with bulk asynchronous copies (1-D TMA) and the
// consumer warps attend out of shared memory.
//
// Why: a unit's K and V rows are contiguous in HBM, so a whole tile of rows is
// one copy descriptor; the ring keeps ~190 KB per SM in flight across the
// softmax of one unit and the start of the next, which plain per-thread loads
// (bounded by registers, drained at every CTA boundary) cannot.  A read-only
// stream measured 7.1 TB/s on B200 this way.
//
// Per unit each group of LR lanes (a stored row is split over LR lanes, two
// 16-byte chunks each for 256-byte rows) keeps its own running softmax state (max, sum, weighted V sum) over the rows it is
// dealt, flash-decoding style, so K and V tiles are consumed together and no
// barrier sits between the logits and P.V.  Scaled logits are parked in shared
// memory; once the groups' states are merged, the record bits
// (alpha_j < 1/t  <=>  2^(s_j - M) * t < L) are formed from them with the
// final M and L.  The token of the step arrives with the unit's first tile,
// is appended to the cache and scored by group 0.
//
// All waits on copy barriers are bounded; a wait that gives up sets the device
// error word and switches the CTA to a drain mode in which nobody waits again.
#include <cuda_fp16.h>

#include "sh_async.cuh"
#include "sh_internal.h"

namespace {

using namespace shasync;

// d0 += a0*b, d1 += a1*b in one packed fp32 instruction (sm_100 FFMA2).
__device__ __forceinline__ void ffma2(float &d0, float &d1, float a0, float a1, float b) {
    asm("{.reg .b64 ra, rb, rc;\n\t"
        "mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %4}; mov.b64 rc, {%0, %1};\n\t"
        "fma.rn.f32x2 rc, ra, rb, rc;\n\t"
        "mov.b64 {%0, %1}, rc;}"
        : "+f"(d0), "+f"(d1)
        : "f"(a0), "f"(a1), "f"(b));
}

// Element traits.  A 16-byte chunk holds EPL elements.
//   dot:  a0 += sum of even-pair products, a1 += odd-pair products of q*k for one chunk, using
//         the mixed-precision FMA (16-bit inputs, fp32 product and sum: exact products, no
//         separate conversions).
//   axpy: acc[0..EPL) += p * v for one chunk: convert pairs, then packed fp32 FMAs.
template <int DT> struct ElemT;
template <> struct ElemT<SH_F32> {
    static constexpr int EPL = 4, BYTES = 4;
    static __device__ __forceinline__ void dot(const uint4 &q, const uint4 &k, float &a0, float &a1) {
        a0 = fmaf(__uint_as_float(q.x), __uint_as_float(k.x), a0);
        a1 = fmaf(__uint_as_float(q.y), __uint_as_float(k.y), a1);
        a0 = fmaf(__uint_as_float(q.z), __uint_as_float(k.z), a0);
        a1 = fmaf(__uint_as_float(q.w), __uint_as_float(k.w), a1);
    }
    static __device__ __forceinline__ void axpy(float *acc, float pe, const uint4 &v) {
        ffma2(acc[0], acc[1], __uint_as_float(v.x), __uint_as_float(v.y), pe);
        ffma2(acc[2], acc[3], __uint_as_float(v.z), __uint_as_float(v.w), pe);
    }
};
template <> struct ElemT<SH_F16> {
    static constexpr int EPL = 8, BYTES = 2;
    static __device__ __forceinline__ void dot(const uint4 &q, const uint4 &k, float &a0, float &a1) {
        asm("{.reg .b16 kl, kh, ql, qh;\n\t"
            "mov.b32 {kl, kh}, %2; mov.b32 {ql, qh}, %6; fma.rn.f32.f16 %0, ql, kl, %0; fma.rn.f32.f16 %1, qh, kh, %1;\n\t"
            "mov.b32 {kl, kh}, %3; mov.b32 {ql, qh}, %7; fma.rn.f32.f16 %0, ql, kl, %0; fma.rn.f32.f16 %1, qh, kh, %1;\n\t"
            "mov.b32 {kl, kh}, %4; mov.b32 {ql, qh}, %8; fma.rn.f32.f16 %0, ql, kl, %0; fma.rn.f32.f16 %1, qh, kh, %1;\n\t"
            "mov.b32 {kl, kh}, %5; mov.b32 {ql, qh}, %9; fma.rn.f32.f16 %0, ql, kl, %0; fma.rn.f32.f16 %1, qh, kh, %1;}"
            : "+f"(a0), "+f"(a1)
            : "r"(k.x), "r"(k.y), "r"(k.z), "r"(k.w), "r"(q.x), "r"(q.y), "r"(q.z), "r"(q.w));
    }
    static __device__ __forceinline__ void axpy(float *acc, float pe, const uint4 &v) {
        const __half2 *h = reinterpret_cast<const __half2 *>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 t = __half22float2(h[i]);
            ffma2(acc[2 * i], acc[2 * i + 1], t.x, t.y, pe);
        }
    }
};
template <> struct ElemT<SH_BF16> {
    static constexpr int EPL = 8, BYTES = 2;
    static __device__ __forceinline__ void dot(const uint4 &q, const uint4 &k, float &a0, float &a1) {
        asm("{.reg .b16 kl, kh, ql, qh;\n\t"
            "mov.b32 {kl, kh}, %2; mov.b32 {ql, qh}, %6; fma.rn.f32.bf16 %0, ql, kl, %0; fma.rn.f32.bf16 %1, qh, kh, %1;\n\t"
            "mov.b32 {kl, kh}, %3; mov.b32 {ql, qh}, %7; fma.rn.f32.bf16 %0, ql, kl, %0; fma.rn.f32.bf16 %1, qh, kh, %1;\n\t"
            "mov.b32 {kl, kh}, %4; mov.b32 {ql, qh}, %8; fma.rn.f32.bf16 %0, ql, kl, %0; fma.rn.f32.bf16 %1, qh, kh, %1;\n\t"
            "mov.b32 {kl, kh}, %5; mov.b32 {ql, qh}, %9; fma.rn.f32.bf16 %0, ql, kl, %0; fma.rn.f32.bf16 %1, qh, kh, %1;}"
            : "+f"(a0), "+f"(a1)
            : "r"(k.x), "r"(k.y), "r"(k.z), "r"(k.w), "r"(q.x), "r"(q.y), "r"(q.z), "r"(q.w));
    }
    static __device__ __forceinline__ void axpy(float *acc, float pe, const uint4 &v) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
            ffma2(acc[2 * i], acc[2 * i + 1], __uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u), pe);
    }
};

__device__ __forceinline__ void consumer_barrier(int threads) {
    asm volatile("bar.sync 1, %0;" ::"r"(threads) : "memory");
}
// 2^x, with 2^(-inf) = 0
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// DT dtype, D head_dim, NWC consumer warps, SR rows per tile, NST ring stages,
// LR lanes per row (each lane owns CH = row_bytes/16/LR chunks of 16 bytes, LR apart),
// CPS CTAs per SM the shared-memory footprint is sized for.
template <int DT, int D, int NWC, int SR, int NST, int LR, int CPS>
__global__ void __launch_bounds__(NWC * 32 + 32, CPS) sh_decode_tma_kernel(const DecodeParams p, int *err) {
    using E = ElemT<DT>;
    constexpr int EPL = E::EPL;
    constexpr int ROWB = D * E::BYTES;      // stored row == input row for these dtypes
    constexpr int CH = ROWB / 16 / LR;      // chunks per lane
    constexpr int EL = CH * EPL;            // elements per lane
    constexpr int RPW = 32 / LR;            // row groups per warp
    constexpr int NG = NWC * RPW;           // row groups per CTA
    constexpr int RG = SR / NG;             // rows per group per tile
    constexpr int TILE = SR * ROWB;
    constexpr int STAGE = 2 * TILE + 3 * ROWB;   // K tile | V tile | q | k_new | v_new
    static_assert(CH >= 1 && CH * LR * 16 == ROWB, "row must split into whole chunks per lane");
    static_assert(SR % NG == 0 && RG >= 1, "tile rows must split evenly over the groups");
    static_assert(D <= NWC * 32 && NWC <= 32, "merge needs one consumer thread per output column");
    constexpr int NCT = NWC * 32;

    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t full[NST], empty[NST];
    __shared__ int drain;                   // set once any bounded wait has given up
    __shared__ int issued;                  // tiles the producer has armed
    const int B = p.B;
    const int capw = (B + 31) & ~31;
    unsigned char *ring = smem;
    float *s_all = reinterpret_cast<float *>(smem + (size_t)NST * STAGE);   // [2][capw] scaled logits
    float *part = s_all + 2 * capw;                                         // [2][NWC][D] weighted V sums
    float *ml = part + 2 * NWC * D;                                         // [2][NWC][2] (max, sum)

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // rows already cached for unit u (the same for all units unless sequences differ in length)
    auto cached_rows = [&](int u) { return p.n_arr ? p.n_arr[u] : p.n - 1; };
    auto tiles_of = [](int n_old) { return n_old > 0 ? (n_old + SR - 1) / SR : 1; };   // the first tile also carries q and the new token

    sh_pdl_launch_dependents();
    if (tid == 0) {
        for (int s = 0; s < NST; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], NWC); }
        drain = 0;
        issued = 0;
        fence_barrier_init();
    }
    __syncthreads();
    sh_pdl_wait();            // the preceding kernel of the stream is complete: global memory may be touched

    if (warp == NWC) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            int it = 0, s = 0;
            uint32_t ph = 0;                // parity of the "stage is free" phase to wait for (first used on the second lap)
            bool stop = false;
            for (int u = blockIdx.x; u < p.U && !stop; u += gridDim.x) {
                const char *Kb = p.K + (size_t)u * B * ROWB;
                const char *Vb = p.V + (size_t)u * B * ROWB;
                const int n_old = cached_rows(u), ntiles = tiles_of(n_old);
                if (!SH_BOUNDS_OK(n_old >= 0 && n_old < B && (!p.t_arr || p.t_arr[u] >= n_old), err, 0x704)) continue;   // the consumers skip the unit too
                for (int tl = 0; tl < ntiles; ++tl) {
                    if (it >= NST && !mbar_wait(&empty[s], ph, err, 2)) *(volatile int *)&drain = 1;
                    if (*(volatile int *)&drain) { stop = true; break; }
                    const int rows = max(0, min(SR, n_old - tl * SR));
                    unsigned char *st = ring + (size_t)s * STAGE;
                    // self-test of the give-up path: one tile is never armed and never copied, so the
                    // consumers' bounded wait for it runs out (no copy is in flight for it)
                    const bool skip = p.selftest_skip_tile >= 0 && blockIdx.x == 0 && it == p.selftest_skip_tile;
                    if (!skip) mbar_arrive_expect_tx(&full[s], (uint32_t)(2 * rows * ROWB + (tl == 0 ? 3 * ROWB : 0)));
                    if (rows && !skip) {
                        bulk_g2s(st, Kb + (size_t)tl * TILE, (uint32_t)rows * ROWB, &full[s]);
                        bulk_g2s(st + TILE, Vb + (size_t)tl * TILE, (uint32_t)rows * ROWB, &full[s]);
                    }
                    if (tl == 0 && !skip) {
                        bulk_g2s(st + 2 * TILE, reinterpret_cast<const char *>(p.q) + (size_t)u * ROWB, ROWB, &full[s]);
                        bulk_g2s(st + 2 * TILE + ROWB, reinterpret_cast<const char *>(p.k_new) + (size_t)u * ROWB, ROWB, &full[s]);
                        bulk_g2s(st + 2 * TILE + 2 * ROWB, reinterpret_cast<const char *>(p.v_new) + (size_t)u * ROWB, ROWB, &full[s]);
                    }
                    ++it;
                    issued = it;
                    if (++s == NST) { s = 0; if (it > NST) ph ^= 1; }
                }
            }
        }
    } else {
        // ------------------------------------------------------------ consumers
        const int sub = lane / LR, c = lane % LR;
        const int g = warp * RPW + sub;                 // row group of this lane
        const float sc = p.scale_log2e;
        int s = 0, par = 0;
        uint32_t ph = 0;
        bool dead = false;                              // this thread has given up a wait: touch no more data
        for (int u = blockIdx.x; u < p.U; u += gridDim.x, par ^= 1) {
            float *s_sh = s_all + par * capw;
            const int n_old = cached_rows(u), ntiles = tiles_of(n_old), n = n_old + 1;
            if (!SH_BOUNDS_OK(n_old >= 0 && n_old < B && (!p.t_arr || p.t_arr[u] >= n_old), err, 0x704)) continue;
            const int t_step = p.t_arr ? p.t_arr[u] + 1 : p.t;
            const int hist_row = p.t_arr ? t_step % p.w : p.hist_row;
            const float tf = (float)t_step;
            uint4 qraw[CH];
            float m_run = -INFINITY, l_run = 0.f;
            float acc[EL];
#pragma unroll
            for (int e = 0; e < EL; ++e) acc[e] = 0.f;

            for (int tl = 0; tl < ntiles; ++tl) {
                int rows = max(0, min(SR, n_old - tl * SR));
                if (!dead && !mbar_wait(&full[s], ph, err, 3)) { dead = true; *(volatile int *)&drain = 1; }
                if (dead) rows = 0;                     // drain mode: keep the barriers moving, nothing else
                const unsigned char *st = ring + (size_t)s * STAGE;
                if (tl == 0) {
#pragma unroll
                    for (int k = 0; k < CH; ++k) qraw[k] = *reinterpret_cast<const uint4 *>(st + 2 * TILE + (c + k * LR) * 16);
                    if (p.qring && warp == 0 && sub == 0 && !dead) {     // remembered for a recount at compression time
#pragma unroll
                        for (int k = 0; k < CH; ++k)
                            *reinterpret_cast<uint4 *>(p.qring + ((size_t)u * p.w + hist_row) * ROWB + (c + k * LR) * 16) = qraw[k];
                    }
                }
                // ---- this group's rows of the tile: K chunks -> partial dot, V chunks parked in registers
                float sv[RG];
                uint4 vraw[RG][CH];
#pragma unroll
                for (int i = 0; i < RG; ++i) {
                    const int r = g + i * NG;
                    float a = 0.f, a1 = 0.f;
                    if (r < rows) {
                        const unsigned char *kr = st + (size_t)r * ROWB + c * 16;
#pragma unroll
                        for (int k = 0; k < CH; ++k) {
                            const uint4 kraw = *reinterpret_cast<const uint4 *>(kr + k * LR * 16);
                            vraw[i][k] = *reinterpret_cast<const uint4 *>(kr + TILE + k * LR * 16);
                            E::dot(qraw[k], kraw, a, a1);
                        }
                        a += a1;
                    } else {
#pragma unroll
                        for (int k = 0; k < CH; ++k) vraw[i][k] = make_uint4(0, 0, 0, 0);
                    }
                    sv[i] = a;
                }
                // ---- the token of this step rides on the unit's first tile: warp 0 scores it, group 0 owns it
                float s_new = -INFINITY;
                uint4 vnew[CH];
                if (tl == 0 && warp == 0 && !dead) {
                    float a = 0.f, a1 = 0.f;
                    uint4 kraw[CH];
#pragma unroll
                    for (int k = 0; k < CH; ++k) {
                        kraw[k] = *reinterpret_cast<const uint4 *>(st + 2 * TILE + ROWB + (c + k * LR) * 16);
                        vnew[k] = *reinterpret_cast<const uint4 *>(st + 2 * TILE + 2 * ROWB + (c + k * LR) * 16);
                        E::dot(qraw[k], kraw[k], a, a1);
                    }
                    a += a1;
#pragma unroll
                    for (int o = LR / 2; o; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
                    if (sub == 0) {
                        s_new = a * sc;
#pragma unroll
                        for (int k = 0; k < CH; ++k) {
                            *reinterpret_cast<uint4 *>(p.K + ((size_t)u * B + n_old) * ROWB + (c + k * LR) * 16) = kraw[k];
                            *reinterpret_cast<uint4 *>(p.V + ((size_t)u * B + n_old) * ROWB + (c + k * LR) * 16) = vnew[k];
                        }
                        if (c == 0) {
                            s_sh[n_old] = s_new;
                            p.pos[(size_t)u * B + n_old] = t_step;
                        }
                    }
                }
                // ---- the tile's data is in registers: hand the stage back to the producer
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[s]);
                if (++s == NST) { s = 0; ph ^= 1; }

                // ---- finish the dot products across the LR lanes of the group (every lane gets the sum)
#pragma unroll
                for (int o = LR / 2; o; o >>= 1) {
#pragma unroll
                    for (int i = 0; i < RG; ++i) sv[i] += __shfl_xor_sync(0xffffffffu, sv[i], o);
                }
                float mx = s_new;
#pragma unroll
                for (int i = 0; i < RG; ++i) {
                    const int r = g + i * NG;
                    sv[i] = (r < rows) ? sv[i] * sc : -INFINITY;
                    if (r < rows && c == 0) s_sh[tl * SR + r] = sv[i];
                    mx = fmaxf(mx, sv[i]);
                }
                // ---- running softmax of the group
                if (mx > m_run) {
                    const float corr = ex2(m_run - mx);     // 0 on the first rows (m_run = -inf)
                    l_run *= corr;
#pragma unroll
                    for (int e = 0; e < EL; ++e) acc[e] *= corr;
                    m_run = mx;
                }
                if (m_run != -INFINITY) {
#pragma unroll
                    for (int i = 0; i < RG; ++i) {
                        const float pe = ex2(sv[i] - m_run);    // 0 for rows that do not exist
                        l_run += pe;
#pragma unroll
                        for (int k = 0; k < CH; ++k) E::axpy(acc + k * EPL, pe, vraw[i][k]);
                    }
                    if (s_new != -INFINITY) {
                        const float pe = ex2(s_new - m_run);
                        l_run += pe;
#pragma unroll
                        for (int k = 0; k < CH; ++k) E::axpy(acc + k * EPL, pe, vnew[k]);
                    }
                }
            }
            // ---- merge the groups of the warp
#pragma unroll
            for (int o = LR; o < 32; o <<= 1) {
                const float m_o = __shfl_xor_sync(0xffffffffu, m_run, o);
                const float l_o = __shfl_xor_sync(0xffffffffu, l_run, o);
                const float m_n = fmaxf(m_run, m_o);
                const float wa = (m_run == -INFINITY) ? 0.f : ex2(m_run - m_n);
                const float wb = (m_o == -INFINITY) ? 0.f : ex2(m_o - m_n);
                l_run = wa * l_run + wb * l_o;
#pragma unroll
                for (int e = 0; e < EL; ++e) {
                    const float a_o = __shfl_xor_sync(0xffffffffu, acc[e], o);
                    acc[e] = wa * acc[e] + wb * a_o;
                }
                m_run = m_n;
            }
            float *pp = part + (size_t)par * NWC * D;
            float *pml = ml + par * NWC * 2;
            if (sub == 0) {
#pragma unroll
                for (int k = 0; k < CH; ++k)
#pragma unroll
                    for (int e = 0; e < EPL; ++e) pp[warp * D + (c + k * LR) * EPL + e] = acc[k * EPL + e];
                if (c == 0) { pml[warp * 2] = m_run; pml[warp * 2 + 1] = l_run; }
            }
            consumer_barrier(NCT);
            // ---- merge the warps: lane i of every warp weighs warp i's state, shuffles spread the result
            float mw = (lane < NWC) ? pml[lane * 2] : -INFINITY;
            float M = mw;
#pragma unroll
            for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
            const float wgt = (mw == -INFINITY) ? 0.f : ex2(mw - M);
            float L = (lane < NWC) ? wgt * pml[lane * 2 + 1] : 0.f;
#pragma unroll
            for (int o = 16; o; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
            if (warp * 32 < D) {       // warps that own output columns
                float o = 0.f;
#pragma unroll
                for (int i = 0; i < NWC; ++i) o = fmaf(__shfl_sync(0xffffffffu, wgt, i), pp[i * D + tid], o);
                if (tid < D) p.out[(size_t)u * D + tid] = o / L;
            }
            // ---- record bits of every slot, one ballot word per 32 slots
            uint32_t *hrow = p.hist + ((size_t)u * p.w + hist_row) * p.Bw;
            for (int wd = warp; wd < p.Bw; wd += NWC) {
                const int j = (wd << 5) + lane;
                bool low = false;
                if (j < n && !dead) low = ex2(s_sh[j] - M) * tf < L;
                const uint32_t word = __ballot_sync(0xffffffffu, low);
                if (lane == 0) hrow[wd] = word;
            }
            if (p.n_arr && tid == 0) {      // all warps are past the barrier: everyone has used the old values
                p.n_arr[u] = n;
                p.t_arr[u] = t_step;
            }
        }
    }

    // ------------------------------------------------------------ drain mode only
    __syncthreads();
    if (tid == 0 && drain) {
        // copies that were armed but never consumed must land before shared memory is released
        const int done = issued;
        for (int it = max(0, done - NST); it < done; ++it) mbar_wait(&full[it % NST], (it / NST) & 1, nullptr, 0);
    }
}

template <int DT, int D, int NWC, int SR, int NST, int LR, int CPS>
cudaError_t launch_tma(const sh_context *c, const DecodeParams &p, cudaStream_t s) {
    using E = ElemT<DT>;
    constexpr int ROWB = D * E::BYTES;
    constexpr int STAGE = 2 * SR * ROWB + 3 * ROWB;
    const int capw = (c->B + 31) & ~31;
    const size_t smem = (size_t)NST * STAGE + sizeof(float) * ((size_t)2 * capw + (size_t)2 * NWC * D + (size_t)2 * NWC * 2);
    if (smem > 227 * 1024) return cudaErrorInvalidValue;
    auto kern = sh_decode_tma_kernel<DT, D, NWC, SR, NST, LR, CPS>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int sms = 148;
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int grid = p.U < sms * CPS ? p.U : sms * CPS;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(NWC * 32 + 32, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, p, reinterpret_cast<int *>(c->slab + c->L.err));
}

}  // namespace

// Chosen by a sweep on B200 at 9216 units of 256-byte rows (consumer warps / rows per tile / ring stages /
// lanes per row: 8/128/3/8 273 us; 12/96/4/8 275; 16/128/3/8 278; 8/128/3/4 283; 8/64/6/8 290; 4/128/3/8 363).
constexpr int TMA_NWC = 8, TMA_SR = 128, TMA_NST = 3, TMA_LR = 8, TMA_CPS = 1;

namespace {

// Tile shapes per stored row size; 256-byte rows take the tuned shape above.
//   row bytes   SR    NST   LR   stage     row groups x rows per group per tile
//   256        128     3     8   64 KB     32 x 4
//   512         64     3    16   64 KB     16 x 4
// 128-byte rows (16-bit stores with head_dim 64) are left to the direct-load kernel: with half
// the bytes per row the per-row work of this one dominates (best of four shapes tried on B200:
// 190 us against 184 us for the OPT-66B-shaped workload with head_dim 64).
template <int DT, int D> struct Shape {
    static constexpr int RB = D * ElemT<DT>::BYTES;
    static constexpr int SR = RB == 512 ? 64 : TMA_SR, NST = TMA_NST, LR = RB == 512 ? 16 : TMA_LR;
};

template <int DT, int D> size_t shape_smem(int B) {
    using S = Shape<DT, D>;
    const int capw = (B + 31) & ~31;
    return (size_t)S::NST * (2 * S::SR * S::RB + 3 * S::RB) +
           sizeof(float) * ((size_t)2 * capw + (size_t)2 * TMA_NWC * D + (size_t)2 * TMA_NWC * 2);
}

template <int DT> size_t smem_for(int D, int B) {
    if constexpr (DT == SH_F32) {
        if (D == 64) return shape_smem<DT, 64>(B);
    }
    return shape_smem<DT, 128>(B);
}

template <int DT>
cudaError_t launch_dt(const sh_context *c, const DecodeParams &p, cudaStream_t s) {
    if constexpr (DT == SH_F32) {
        if (c->D == 64)
            return launch_tma<DT, 64, TMA_NWC, Shape<DT, 64>::SR, Shape<DT, 64>::NST, Shape<DT, 64>::LR, TMA_CPS>(c, p, s);
    }
    if constexpr (DT != SH_F32) {
        // Between one and two units per SM a single CTA per SM would run two units one after the other on most SMs
        // and one on the rest; two CTAs per SM with tiles of half the rows take every unit at once.
        int sms = 148, dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const int capw = (c->B + 31) & ~31;
        const size_t small = (size_t)TMA_NST * (2 * 64 * 256 + 3 * 256) + sizeof(float) * ((size_t)2 * capw + (size_t)2 * TMA_NWC * 128 + (size_t)2 * TMA_NWC * 2);
        if (p.U > sms && p.U <= 2 * sms && 2 * (small + 1024) <= 228 * 1024)
            return launch_tma<DT, 128, TMA_NWC, 64, TMA_NST, TMA_LR, 2>(c, p, s);
    }
    return launch_tma<DT, 128, TMA_NWC, Shape<DT, 128>::SR, Shape<DT, 128>::NST, Shape<DT, 128>::LR, TMA_CPS>(c, p, s);
}

}  // namespace

// Whether the pipelined kernel can serve this handle (dtype, shape, shared memory).
bool sh_decode_tma_supported(const sh_context *c) {
    if (c->D != 64 && c->D != 128) return false;
    if (c->row_bytes < 256) return false;
    size_t need;
    if (c->dtype == SH_F32) need = smem_for<SH_F32>(c->D, c->B);
    else if (c->dtype == SH_F16) need = smem_for<SH_F16>(c->D, c->B);
    else if (c->dtype == SH_BF16) need = smem_for<SH_BF16>(c->D, c->B);
    else return false;
    return need <= 227 * 1024;
}

cudaError_t sh_launch_decode_tma(const sh_context *c, const DecodeParams &p, cudaStream_t s, long long *launches) {
    cudaError_t e = cudaErrorInvalidValue;
    if (c->dtype == SH_F32) e = launch_dt<SH_F32>(c, p, s);
    else if (c->dtype == SH_F16) e = launch_dt<SH_F16>(c, p, s);
    else if (c->dtype == SH_BF16) e = launch_dt<SH_BF16>(c, p, s);
    if (e == cudaSuccess) *launches += 1;
    return e;
}
