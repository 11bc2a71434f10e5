// Chunked prompt step and recount on CUDA cores, for the storage types and head sizes the tensor-core
// chunk kernels do not take: fp32 rows (whose products do not fit 16-bit tensor-core operands without
// splitting), and every store with head_dim 64.
//
// Same contract as the other chunk kernels (sh_prefill_chunk.cu): step i of the chunk attends with q_i
// over the n0 cached rows plus the chunk's tokens 0..i and writes its own bit-plane row; in recount mode
// the queries come from the ring of the last w queries and a cached slot is visible when its position
// does not exceed the query's step.  K and V are read once per 64 queries instead of once per query.
//
// One CTA of 256 threads per (unit, block of 64 queries).  Keys go through shared memory 64 at a time,
// converted to fp32 (int4: dequantised, code x scale is exact), K transposed so that the logits are a
// register-tiled fp32 product: thread (ty, tx) of a 16 x 16 grid owns queries 4ty..4ty+3 and keys
// 4tx..4tx+3 of the tile, one 128-bit shared load of each operand per 16 FMAs.  A row of logits fits
// neither registers nor shared memory for large budgets, so the key tiles are visited twice: the first
// sweep keeps a running maximum and sum per query, the second recomputes the logits (same instructions,
// same values), forms e = 2^(s - M), the record bits e t < L, and accumulates P.V with the V tile, thread
// (ty, tx) owning queries 4ty..4ty+3 and D/16 output columns.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "sh_internal.h"

namespace {

constexpr int CQ = 64;            // queries per CTA
constexpr int KT = 64;            // keys per tile
constexpr int TS = 68;            // row stride (floats) of the transposed tiles: 16-byte aligned, 4 banks off per row
constexpr int NT = 256;

__device__ __forceinline__ float ex2a(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 16 bytes of a stored row -> EPL fp32 values.
template <int DT> struct Cvt;
template <> struct Cvt<SH_F32> {
    static constexpr int EPL = 4;
    static __device__ __forceinline__ void run(const uint4 &r, float, float *f) {
        f[0] = __uint_as_float(r.x); f[1] = __uint_as_float(r.y); f[2] = __uint_as_float(r.z); f[3] = __uint_as_float(r.w);
    }
};
template <> struct Cvt<SH_F16> {
    static constexpr int EPL = 8;
    static __device__ __forceinline__ void run(const uint4 &r, float, float *f) {
        const __half2 *h = reinterpret_cast<const __half2 *>(&r);
#pragma unroll
        for (int i = 0; i < 4; ++i) { const float2 t = __half22float2(h[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
    }
};
template <> struct Cvt<SH_BF16> {
    static constexpr int EPL = 8;
    static __device__ __forceinline__ void run(const uint4 &r, float, float *f) {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(w[i] << 16); f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
    }
};
// int4 store: word k of a chunk holds elements 8k..8k+7, element e in nibble (e>>1) + 4(e&1), biased by 8
template <> struct Cvt<SH_INT4_G64_F16> {
    static constexpr int EPL = 32;
    static __device__ __forceinline__ void run(const uint4 &r, float sc, float *f) {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int k = 0; k < 4; ++k)
#pragma unroll
            for (int e = 0; e < 8; ++e)
                f[8 * k + e] = (float)((int)((w[k] >> (4 * ((e >> 1) + 4 * (e & 1)))) & 0xFu) - 8) * sc;
    }
};

template <int DT> __host__ __device__ constexpr int stored_row_bytes(int D) {
    return DT == SH_F32 ? D * 4 : (DT == SH_INT4_G64_F16 ? D / 2 : D * 2);
}
template <int DT> __host__ __device__ constexpr int input_row_bytes(int D) { return DT == SH_F32 ? D * 4 : D * 2; }

// One input element (q, k_new, v_new rows: fp32, or 16-bit; the int4 store takes fp16) as fp32.
template <int DT> __device__ __forceinline__ float input_elem(const char *row, int i) {
    if constexpr (DT == SH_F32) return reinterpret_cast<const float *>(row)[i];
    else if constexpr (DT == SH_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(row)[i]);
    else return __half2float(reinterpret_cast<const __half *>(row)[i]);
}

// Rows [j0, j0 + 64) of a unit's K (transposed: Kt[element][key]) or V (Vs[key][element]) as fp32, zeros
// beyond n_tot.  Consecutive lanes take consecutive keys, so the transposed stores hit distinct banks.
template <int DT, int D, bool TRANSPOSE>
__device__ __forceinline__ void load_tile(float *dst, const char *rows, const __half *scales, int j0, int n_tot) {
    using C = Cvt<DT>;
    constexpr int EPL = C::EPL, ROWB = stored_row_bytes<DT>(D), CH = ROWB / 16, VST = D + 4;
    for (int idx = threadIdx.x; idx < KT * CH; idx += NT) {
        const int key = idx % KT, ch = idx / KT, j = j0 + key;
        float f[EPL];
        if (j < n_tot) {
            const uint4 raw = *reinterpret_cast<const uint4 *>(rows + (size_t)j * ROWB + ch * 16);
            float sc = 1.f;
            if constexpr (DT == SH_INT4_G64_F16) sc = __half2float(scales[(size_t)j * (D / 64) + (ch * 32) / 64]);
            C::run(raw, sc, f);
        } else {
#pragma unroll
            for (int e = 0; e < EPL; ++e) f[e] = 0.f;
        }
        if constexpr (TRANSPOSE) {
#pragma unroll
            for (int e = 0; e < EPL; ++e) dst[(ch * EPL + e) * TS + key] = f[e];
        } else {
#pragma unroll
            for (int e = 0; e < EPL; e += 4)
                *reinterpret_cast<float4 *>(dst + key * VST + ch * EPL + e) = make_float4(f[e], f[e + 1], f[e + 2], f[e + 3]);
        }
    }
}

// Append the chunk's keys and values to the cache (int4: quantised by the decode step's rule, IEEE fp32:
// a = max|x| over a group of 64, sc = fp16(a / 7), code = clamp(rint(x / sc), -7, 7)), their positions, and
// remember the queries in the ring if the handle keeps one.
template <int DT, int D>
__device__ __forceinline__ void append_chunk(const ChunkParams &p, int u, int c) {
    constexpr int ROWB = stored_row_bytes<DT>(D), INB = input_row_bytes<DT>(D);
    const int tid = threadIdx.x;
    const size_t tstride = (size_t)p.Utot * INB;
    if (tid < c) p.pos[(size_t)u * p.B + p.n0 + tid] = p.t0 + 1 + tid;
    if (p.qring) {
        for (int idx = tid; idx < c * (INB / 16); idx += NT) {
            const int row = idx / (INB / 16), ch = idx % (INB / 16);
            *reinterpret_cast<uint4 *>(p.qring + ((size_t)u * p.w + (p.t0 + 1 + row) % p.w) * INB + ch * 16) =
                *reinterpret_cast<const uint4 *>(p.q + (size_t)row * tstride + (size_t)u * INB + ch * 16);
        }
    }
    if constexpr (DT == SH_INT4_G64_F16) {
        // one warp per (token, K or V, group of 64): lane l holds elements 2l, 2l+1 of the group
        const int warp = tid >> 5, lane = tid & 31;
        constexpr int G = D / 64;
        for (int item = warp; item < c * 2 * G; item += NT / 32) {
            const int row = item / (2 * G), which = (item / G) & 1, g = item % G;
            const char *src = (which ? p.v : p.k) + (size_t)row * tstride + (size_t)u * INB;
            const __half2 h2 = reinterpret_cast<const __half2 *>(src)[g * 32 + lane];
            const float x0 = __low2float(h2), x1 = __high2float(h2);
            float a = fmaxf(fabsf(x0), fabsf(x1));
#pragma unroll
            for (int o = 16; o; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
            const float sc = __half2float(__float2half_rn(__fdiv_rn(a, 7.0f)));
            float c0 = 0.f, c1 = 0.f;
            if (sc != 0.f) {
                c0 = fminf(fmaxf(rintf(__fdiv_rn(x0, sc)), -7.f), 7.f);
                c1 = fminf(fmaxf(rintf(__fdiv_rn(x1, sc)), -7.f), 7.f);
            }
            // elements 2l, 2l+1 sit in word (2l % 32) / 8 of chunk 2l / 32, nibbles (e>>1) and (e>>1) + 4 with e = 2l % 8
            const int e = (2 * lane) & 7;
            uint32_t word = ((uint32_t)((int)c0 + 8) << (4 * (e >> 1))) | ((uint32_t)((int)c1 + 8) << (4 * ((e >> 1) + 4)));
            word |= __shfl_xor_sync(0xffffffffu, word, 1);
            word |= __shfl_xor_sync(0xffffffffu, word, 2);
            const size_t slot = (size_t)u * p.B + p.n0 + row;
            if ((lane & 3) == 0)
                reinterpret_cast<uint32_t *>((which ? p.V : p.K) + slot * ROWB)[g * 8 + (lane >> 2)] = word;
            if (lane == 0)
                reinterpret_cast<__half *>(which ? p.Vs : p.Ks)[((size_t)u * p.Bs + p.n0 + row) * G + g] = __float2half_rn(sc);
        }
    } else {
        for (int idx = tid; idx < c * (ROWB / 16); idx += NT) {
            const int row = idx / (ROWB / 16), ch = idx % (ROWB / 16);
            const size_t src = (size_t)row * tstride + (size_t)u * INB + ch * 16;
            const size_t dst = ((size_t)u * p.B + p.n0 + row) * ROWB + ch * 16;
            *reinterpret_cast<uint4 *>(p.K + dst) = *reinterpret_cast<const uint4 *>(p.k + src);
            *reinterpret_cast<uint4 *>(p.V + dst) = *reinterpret_cast<const uint4 *>(p.v + src);
        }
    }
}

template <int DT, int D, bool RECOUNT>
__global__ void __launch_bounds__(NT, 2) sh_chunk_simt_kernel(const ChunkParams p) {
    constexpr int ROWB = stored_row_bytes<DT>(D), INB = input_row_bytes<DT>(D);
    constexpr int VST = D + 4;          // row stride of the V tile
    constexpr int DPT = D / 16;         // output columns per thread
    extern __shared__ __align__(16) float sm[];
    float *Qt = sm;                     // [D][TS]   queries, transposed
    float *Kt = Qt + D * TS;            // [D][TS]   key tile, transposed; reused as Ps[KT][TS] (probabilities, [key][query])
    float *Vs = Kt + D * TS;            // [KT][VST] value tile
    uint32_t *bits = reinterpret_cast<uint32_t *>(Vs + KT * VST);   // [CQ][2] record bits of the tile
    int *pos_t = reinterpret_cast<int *>(bits + 2 * CQ);            // [KT] positions of the tile's slots (recount mode)

    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    const int ty = tid >> 4, tx = tid & 15;
    const int qoff = RECOUNT ? (int)blockIdx.y * CQ : 0;
    const int step0 = (RECOUNT ? p.first_step : p.t0 + 1) + qoff;
    const int c = min(CQ, (RECOUNT ? p.nsteps : p.c) - qoff);
    const int n0 = p.n0;
    const int n_tot = RECOUNT ? n0 : n0 + c;
    const int ntiles = (n_tot + KT - 1) / KT;
    const char *Kc = p.K + (size_t)u * p.B * ROWB;
    const char *Vc = p.V + (size_t)u * p.B * ROWB;
    const __half *Ksc = DT == SH_INT4_G64_F16 ? reinterpret_cast<const __half *>(p.Ks) + (size_t)u * p.Bs * (D / 64) : nullptr;
    const __half *Vsc = DT == SH_INT4_G64_F16 ? reinterpret_cast<const __half *>(p.Vs) + (size_t)u * p.Bs * (D / 64) : nullptr;
    const int32_t *pos_u = p.pos + (size_t)u * p.B;

    // ---- bit-plane rows of this CTA's steps start at zero (words beyond the visited tiles stay so)
    for (int idx = tid; idx < c * p.Bw; idx += NT) {
        const int i = idx / p.Bw, wd = idx % p.Bw;
        p.hist[((size_t)u * p.w + (step0 + i) % p.w) * p.Bw + wd] = 0u;
    }
    if constexpr (!RECOUNT) append_chunk<DT, D>(p, u, c);
    // ---- queries, transposed (columns beyond c are zero)
    for (int idx = tid; idx < CQ * D; idx += NT) {
        const int qi = idx % CQ, i = idx / CQ;
        float val = 0.f;
        if (qi < c) {
            const char *row = RECOUNT ? p.qring + ((size_t)u * p.w + (step0 + qi) % p.w) * INB
                                      : p.q + (size_t)qi * p.Utot * INB + (size_t)u * INB;
            val = input_elem<DT>(row, i);
        }
        Qt[i * TS + qi] = val;
    }
    __syncthreads();          // the appended rows are visible to this CTA's loads from here on

    // logits of this thread's 4 queries x 4 keys of tile kt; -inf where the query may not see the key
    auto logits = [&](int kt, float (&s)[4][4]) {
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) s[a][b] = 0.f;
        // blocks of 16 elements are summed on their own and then added up: the rounding error of a long
        // sequential fp32 sum would otherwise eat the 1e-5 tolerance of fp32 stores at large logits
        for (int i0 = 0; i0 < D; i0 += 16) {
            float part[4][4];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) part[a][b] = 0.f;
#pragma unroll
            for (int i = i0; i < i0 + 16; ++i) {
                const float4 q4 = *reinterpret_cast<const float4 *>(Qt + i * TS + 4 * ty);
                const float4 k4 = *reinterpret_cast<const float4 *>(Kt + i * TS + 4 * tx);
                const float qa[4] = {q4.x, q4.y, q4.z, q4.w}, kb[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = 0; b < 4; ++b) part[a][b] = fmaf(qa[a], kb[b], part[a][b]);
            }
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) s[a][b] += part[a][b];
        }
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const int qi = 4 * ty + a;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int jl = 4 * tx + b, j = kt * KT + jl;
                const bool live = qi < c && (RECOUNT ? (j < n0 && pos_t[jl] <= step0 + qi) : j < n0 + qi + 1);
                s[a][b] = live ? s[a][b] * p.scale_log2e : -INFINITY;
            }
        }
    };

    // ---- sweep 1: running maximum and sum of every query row (replicated over the 16 threads of a row)
    float m_run[4], l_run[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) { m_run[a] = -INFINITY; l_run[a] = 0.f; }
    for (int kt = 0; kt < ntiles; ++kt) {
        load_tile<DT, D, true>(Kt, Kc, Ksc, kt * KT, n_tot);
        if (RECOUNT && tid < KT) pos_t[tid] = kt * KT + tid < n0 ? pos_u[kt * KT + tid] : 0x7fffffff;
        __syncthreads();
        float s[4][4];
        logits(kt, s);
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            float mx = fmaxf(fmaxf(s[a][0], s[a][1]), fmaxf(s[a][2], s[a][3]));
#pragma unroll
            for (int o = 8; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            // (no branch around the shuffles: the two query rows of a warp may differ in what they see)
            const float m_new = fmaxf(m_run[a], mx);
            const float ref = m_new == -INFINITY ? 0.f : m_new;      // nothing visible yet: every term below is 2^(-inf) = 0
            float sum = ex2a(s[a][0] - ref) + ex2a(s[a][1] - ref) + ex2a(s[a][2] - ref) + ex2a(s[a][3] - ref);
#pragma unroll
            for (int o = 8; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            l_run[a] = l_run[a] * ex2a(m_run[a] - ref) + sum;
            m_run[a] = m_new;
        }
        __syncthreads();      // tile consumed
    }

    // ---- sweep 2: probabilities, record bits, P.V
    float acc[4][DPT];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int e = 0; e < DPT; ++e) acc[a][e] = 0.f;
    float *Ps = Kt;
    for (int kt = 0; kt < ntiles; ++kt) {
        load_tile<DT, D, true>(Kt, Kc, Ksc, kt * KT, n_tot);
        if constexpr (!RECOUNT) load_tile<DT, D, false>(Vs, Vc, Vsc, kt * KT, n_tot);
        if (RECOUNT && tid < KT) pos_t[tid] = kt * KT + tid < n0 ? pos_u[kt * KT + tid] : 0x7fffffff;
        if (tid < 2 * CQ) bits[tid] = 0u;
        __syncthreads();
        float s[4][4];
        logits(kt, s);
        __syncthreads();      // every thread is done with the key tile: it becomes the probability tile
        uint32_t mine[4];
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const float tf = (float)(step0 + 4 * ty + a);
            mine[a] = 0u;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const float e = s[a][b] == -INFINITY ? 0.f : ex2a(s[a][b] - m_run[a]);
                if (s[a][b] != -INFINITY && e * tf < l_run[a]) mine[a] |= 1u << b;     // alpha_j < 1/t
                s[a][b] = e;
            }
        }
#pragma unroll
        for (int b = 0; b < 4; ++b)
            *reinterpret_cast<float4 *>(Ps + (4 * tx + b) * TS + 4 * ty) = make_float4(s[0][b], s[1][b], s[2][b], s[3][b]);
#pragma unroll
        for (int a = 0; a < 4; ++a)
            if (mine[a]) atomicOr(&bits[(4 * ty + a) * 2 + (tx >> 3)], mine[a] << (4 * (tx & 7)));
        __syncthreads();
        if (tid < 2 * CQ) {
            const int qi = tid >> 1, wd = kt * 2 + (tid & 1);
            if (qi < c && wd < p.Bw) p.hist[((size_t)u * p.w + (step0 + qi) % p.w) * p.Bw + wd] = bits[tid];
        }
        if constexpr (!RECOUNT) {
#pragma unroll 4
            for (int key = 0; key < KT; ++key) {
                const float4 p4 = *reinterpret_cast<const float4 *>(Ps + key * TS + 4 * ty);
                const float pa[4] = {p4.x, p4.y, p4.z, p4.w};
                float vv[DPT];
#pragma unroll
                for (int e = 0; e < DPT; e += 4) {
                    const float4 v4 = *reinterpret_cast<const float4 *>(Vs + key * VST + tx * DPT + e);
                    vv[e] = v4.x; vv[e + 1] = v4.y; vv[e + 2] = v4.z; vv[e + 3] = v4.w;
                }
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int e = 0; e < DPT; ++e) acc[a][e] = fmaf(pa[a], vv[e], acc[a][e]);
            }
        }
        __syncthreads();      // tiles and bit words consumed
    }
    if constexpr (!RECOUNT) {
        if (p.out) {
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const int qi = 4 * ty + a;
                if (qi < c) {
                    const float inv = 1.f / l_run[a];
                    float *o = p.out + ((size_t)qi * p.Utot + u) * D + tx * DPT;
#pragma unroll
                    for (int e = 0; e < DPT; e += 4)
                        *reinterpret_cast<float4 *>(o + e) = make_float4(acc[a][e] * inv, acc[a][e + 1] * inv, acc[a][e + 2] * inv, acc[a][e + 3] * inv);
                }
            }
        }
    }
    (void)lane;
}

template <int DT, int D, bool RECOUNT>
cudaError_t launch_simt(const ChunkParams &p, cudaStream_t s) {
    const size_t smem = sizeof(float) * ((size_t)2 * D * TS + (size_t)KT * (D + 4)) + sizeof(int) * (2 * CQ + KT);
    auto kern = sh_chunk_simt_kernel<DT, D, RECOUNT>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const unsigned gy = RECOUNT ? (unsigned)((p.nsteps + CQ - 1) / CQ) : 1u;
    kern<<<dim3(p.U, gy, 1), NT, smem, s>>>(p);
    return cudaGetLastError();
}

template <bool RECOUNT>
cudaError_t launch_any(const ChunkParams &p, int dtype, int D, cudaStream_t s) {
    if (D != 64 && D != 128) return cudaErrorInvalidValue;
    switch (dtype) {
        case SH_F32: return D == 64 ? launch_simt<SH_F32, 64, RECOUNT>(p, s) : launch_simt<SH_F32, 128, RECOUNT>(p, s);
        case SH_F16: return D == 64 ? launch_simt<SH_F16, 64, RECOUNT>(p, s) : launch_simt<SH_F16, 128, RECOUNT>(p, s);
        case SH_BF16: return D == 64 ? launch_simt<SH_BF16, 64, RECOUNT>(p, s) : launch_simt<SH_BF16, 128, RECOUNT>(p, s);
        case SH_INT4_G64_F16:
            return D == 64 ? launch_simt<SH_INT4_G64_F16, 64, RECOUNT>(p, s) : launch_simt<SH_INT4_G64_F16, 128, RECOUNT>(p, s);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

int sh_chunk_simt_capacity() { return CQ; }
cudaError_t sh_launch_chunk_simt(const ChunkParams &p, int dtype, int D, cudaStream_t s) { return launch_any<false>(p, dtype, D, s); }
cudaError_t sh_launch_recount_simt(const ChunkParams &p, int dtype, int D, cudaStream_t s) { return launch_any<true>(p, dtype, D, s); }
