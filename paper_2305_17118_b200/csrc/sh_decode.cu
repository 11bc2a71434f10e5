// Fused decode step: append + logits + stable softmax + P.V + importance-record
// bits, one CTA (or one cluster of S CTAs) per (sequence, head) unit.  This is
// the kernel for the int4 store, for 16-bit stores with head_dim 64 and for
// launches with few units; stores with rows of 256 bytes or more go through the
// pipelined kernel of sh_decode_tma.cu at scale (sh_launch_decode picks).
//
// The work is a GEMV per unit (one query against n cached rows), so it is bound
// by HBM bandwidth and runs on CUDA cores.  Layout of the work inside a CTA:
// a K (or V) row of D elements is D*es bytes = LPR lanes x 16 bytes, so a warp
// reads RPW = 32/LPR whole rows per 128-bit load instruction, fully coalesced,
// and every lane keeps R such loads in flight before it touches the data.
// Logits stay in shared memory until the softmax denominator is known, so K and
// V are each read from HBM exactly once per step and the record bits
// (alpha_j < 1/t  <=>  e_j * t < L) cost one ballot word per 32 slots.
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "sh_internal.h"

namespace cg = cooperative_groups;

namespace {

// ---------------------------------------------------------------- loads / stores
__device__ __forceinline__ uint4 ld_stream(const void *p) {
    // read-only, read-once data: keep it out of L1
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ uint4 ld_plain(const void *p) { return *reinterpret_cast<const uint4 *>(p); }
__device__ __forceinline__ void st_plain(void *p, const uint4 &v) { *reinterpret_cast<uint4 *>(p) = v; }

// d0 += a0*b, d1 += a1*b in one packed fp32 instruction (sm_100 FFMA2).
__device__ __forceinline__ void ffma2(float &d0, float &d1, float a0, float a1, float b) {
    asm("{.reg .b64 ra, rb, rc;\n\t"
        "mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %4}; mov.b64 rc, {%0, %1};\n\t"
        "fma.rn.f32x2 rc, ra, rb, rc;\n\t"
        "mov.b64 {%0, %1}, rc;}"
        : "+f"(d0), "+f"(d1)
        : "f"(a0), "f"(a1), "f"(b));
}
// a0 += q.lo*k.lo, a1 += q.hi*k.hi for one packed pair: mixed-precision FMA (16-bit inputs,
// exact fp32 product and sum), so no separate conversion instructions are needed.
__device__ __forceinline__ void fma_pair_f16(float &a0, float &a1, uint32_t q2, uint32_t k2) {
    asm("{.reg .b16 kl, kh, ql, qh;\n\t"
        "mov.b32 {kl, kh}, %2; mov.b32 {ql, qh}, %3;\n\t"
        "fma.rn.f32.f16 %0, ql, kl, %0; fma.rn.f32.f16 %1, qh, kh, %1;}"
        : "+f"(a0), "+f"(a1)
        : "r"(k2), "r"(q2));
}

// ---------------------------------------------------------------- element traits
// A "chunk" is the 16 bytes one lane loads from a stored row; EPL elements.
//   Q:    this lane's EPL elements of the query, in the form `dot` wants them
//   dot:  sum over the chunk of q*k (fp32 accumulation; int4: of q*code, scale applied by the caller)
//   axpy: acc[0..EPL) += p * v (int4: p * code)
template <int DT> struct Elem;

template <> struct Elem<SH_F32> {
    static constexpr int EPL = 4;        // elements per 16-byte chunk of a stored row
    static __device__ __forceinline__ void cvt(const uint4 &r, float *f) {
        f[0] = __uint_as_float(r.x); f[1] = __uint_as_float(r.y);
        f[2] = __uint_as_float(r.z); f[3] = __uint_as_float(r.w);
    }
    struct Q { float f[4]; };
    static __device__ __forceinline__ void load_q(const void *row, int c, Q &q) { cvt(ld_plain(reinterpret_cast<const char *>(row) + c * 16), q.f); }
    static __device__ __forceinline__ void q_floats(const Q &q, float *f) {
#pragma unroll
        for (int e = 0; e < 4; ++e) f[e] = q.f[e];
    }
    static __device__ __forceinline__ float dot(const Q &q, const uint4 &r) {
        float a = __uint_as_float(r.x) * q.f[0];
        a = fmaf(__uint_as_float(r.y), q.f[1], a);
        a = fmaf(__uint_as_float(r.z), q.f[2], a);
        return fmaf(__uint_as_float(r.w), q.f[3], a);
    }
    static __device__ __forceinline__ void axpy(float *acc, float p, const uint4 &r) {
        acc[0] = fmaf(p, __uint_as_float(r.x), acc[0]); acc[1] = fmaf(p, __uint_as_float(r.y), acc[1]);
        acc[2] = fmaf(p, __uint_as_float(r.z), acc[2]); acc[3] = fmaf(p, __uint_as_float(r.w), acc[3]);
    }
};
template <> struct Elem<SH_F16> {
    static constexpr int EPL = 8;
    static __device__ __forceinline__ void cvt(const uint4 &r, float *f) {
        const __half2 *h = reinterpret_cast<const __half2 *>(&r);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 t = __half22float2(h[i]);
            f[2 * i] = t.x; f[2 * i + 1] = t.y;
        }
    }
    // With one CTA per unit and ~5 CTAs per SM this kernel is sensitive to register count:
    // convert-then-FMA (48 registers) measured faster here than the mixed-precision and packed
    // forms the pipelined kernel uses (62 registers, one CTA per SM fewer).
    struct Q { float f[8]; };
    static __device__ __forceinline__ void load_q(const void *row, int c, Q &q) { cvt(ld_plain(reinterpret_cast<const char *>(row) + c * 16), q.f); }
    static __device__ __forceinline__ void q_floats(const Q &q, float *f) {
#pragma unroll
        for (int e = 0; e < 8; ++e) f[e] = q.f[e];
    }
    static __device__ __forceinline__ float dot(const Q &q, const uint4 &r) {
        float f[8];
        cvt(r, f);
        float a = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) a = fmaf(q.f[e], f[e], a);
        return a;
    }
    static __device__ __forceinline__ void axpy(float *acc, float p, const uint4 &r) {
        float f[8];
        cvt(r, f);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = fmaf(p, f[e], acc[e]);
    }
};
template <> struct Elem<SH_BF16> {
    static constexpr int EPL = 8;
    static __device__ __forceinline__ void cvt(const uint4 &r, float *f) {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    struct Q { float f[8]; };
    static __device__ __forceinline__ void load_q(const void *row, int c, Q &q) { cvt(ld_plain(reinterpret_cast<const char *>(row) + c * 16), q.f); }
    static __device__ __forceinline__ void q_floats(const Q &q, float *f) {
#pragma unroll
        for (int e = 0; e < 8; ++e) f[e] = q.f[e];
    }
    static __device__ __forceinline__ float dot(const Q &q, const uint4 &r) {
        float f[8];
        cvt(r, f);
        float a = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) a = fmaf(q.f[e], f[e], a);
        return a;
    }
    static __device__ __forceinline__ void axpy(float *acc, float p, const uint4 &r) {
        float f[8];
        cvt(r, f);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = fmaf(p, f[e], acc[e]);
    }
};
// int4 store: a chunk is 32 codes.  Word k of the chunk holds elements 8k..8k+7;
// element e of a word sits in nibble (e>>1) + 4*(e&1), biased by +8, so that
// ((word >> 4i) & 0x000F000F) | 0x64006400 is the half2 (1024+e_{2i}, 1024+e_{2i+1}).
template <> struct Elem<SH_INT4_G64_F16> {
    static constexpr int EPL = 32;
    static __device__ __forceinline__ void cvt(const uint4 &r, float *f) {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
        const __half2 bias = __floats2half2_rn(1032.f, 1032.f);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t bits = ((w[k] >> (4 * i)) & 0x000F000Fu) | 0x64006400u;
                __half2 h = __hsub2(*reinterpret_cast<__half2 *>(&bits), bias);
                float2 t = __half22float2(h);
                f[8 * k + 2 * i] = t.x; f[8 * k + 2 * i + 1] = t.y;
            }
        }
    }
    // the query's 32 fp16 elements of this chunk: word 4k+i holds elements 8k+2i, 8k+2i+1,
    // the same pairing the code extraction below produces
    struct Q { uint4 raw[4]; };
    static __device__ __forceinline__ void load_q(const void *row, int c, Q &q) {
#pragma unroll
        for (int k = 0; k < 4; ++k) q.raw[k] = ld_plain(reinterpret_cast<const char *>(row) + c * 64 + 16 * k);
    }
    static __device__ __forceinline__ void q_floats(const Q &q, float *f) {
#pragma unroll
        for (int k = 0; k < 4; ++k) Elem<SH_F16>::cvt(q.raw[k], f + 8 * k);
    }
    static __device__ __forceinline__ float dot(const Q &q, const uint4 &r) {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
        const __half2 bias = __floats2half2_rn(1032.f, 1032.f);
        float a0 = 0.f, a1 = 0.f;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t qw[4] = {q.raw[k].x, q.raw[k].y, q.raw[k].z, q.raw[k].w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t bits = ((w[k] >> (4 * i)) & 0x000F000Fu) | 0x64006400u;
                const __half2 h = __hsub2(*reinterpret_cast<__half2 *>(&bits), bias);   // exact small integers
                fma_pair_f16(a0, a1, qw[i], *reinterpret_cast<const uint32_t *>(&h));
            }
        }
        return a0 + a1;
    }
    static __device__ __forceinline__ void axpy(float *acc, float p, const uint4 &r) {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
        const __half2 bias = __floats2half2_rn(1032.f, 1032.f);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t bits = ((w[k] >> (4 * i)) & 0x000F000Fu) | 0x64006400u;
                const float2 t = __half22float2(__hsub2(*reinterpret_cast<__half2 *>(&bits), bias));
                ffma2(acc[8 * k + 2 * i], acc[8 * k + 2 * i + 1], t.x, t.y, p);
            }
        }
    }
};

template <int DT> __device__ __forceinline__ int stored_row_bytes(int D) {
    return DT == SH_F32 ? D * 4 : (DT == SH_INT4_G64_F16 ? D / 2 : D * 2);
}

// Load this lane's EPL elements of a q / k_new / v_new row as fp32.
template <int DT> __device__ __forceinline__ void load_input(const void *row, int c, float *f) {
    using E = Elem<DT>;
    if constexpr (DT == SH_INT4_G64_F16) {
        const char *p = reinterpret_cast<const char *>(row) + c * 64;
#pragma unroll
        for (int k = 0; k < 4; ++k) Elem<SH_F16>::cvt(ld_plain(p + 16 * k), f + 8 * k);
    } else {
        E::cvt(ld_plain(reinterpret_cast<const char *>(row) + c * 16), f);
    }
}

// Quantisation of a row of the int4 store, all in IEEE fp32: a = max|x| over a group of 64, sc = fp16(a / 7),
// code = clamp(rint(x / sc), -7, 7), stored value code * sc.  The row is spread over a whole warp: lane l holds elements EPT*l .. EPT*l + EPT - 1 of a
// row of D fp16 values (EPT = D / 32; a scale group of 64 is 64 / EPT lanes, an 8-code word 8 / EPT lanes).
// Writes the row's codes and scales and leaves the dequantised values in x.
template <int D>
__device__ __forceinline__ void int4_append_row(const char *src_row, char *dst_row, __half *dst_scales, float (&x)[D / 32], int lane) {
    constexpr int EPT = D / 32, GL = 64 / EPT, LPW = 8 / EPT;
    static_assert(EPT == 2 || EPT == 4, "head_dim 64 or 128");
    if constexpr (EPT == 4) {
        const uint2 in = *reinterpret_cast<const uint2 *>(src_row + 8 * lane);
        const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&in.x)), b = __half22float2(*reinterpret_cast<const __half2 *>(&in.y));
        x[0] = a.x; x[1] = a.y; x[2] = b.x; x[3] = b.y;
    } else {
        const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(src_row + 4 * lane));
        x[0] = a.x; x[1] = a.y;
    }
    float amax = 0.f;
#pragma unroll
    for (int e = 0; e < EPT; ++e) amax = fmaxf(amax, fabsf(x[e]));
#pragma unroll
    for (int o = GL / 2; o; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const float sc = __half2float(__float2half_rn(__fdiv_rn(amax, 7.0f)));
    uint32_t word = 0;
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
        float code = 0.f;
        if (sc != 0.f) code = fminf(fmaxf(rintf(__fdiv_rn(x[e], sc)), -7.f), 7.f);
        x[e] = code * sc;
        const int ew = EPT * (lane % LPW) + e;              // element within its 8-code word
        word |= (uint32_t)((int)code + 8) << (4 * ((ew >> 1) + 4 * (ew & 1)));
    }
#pragma unroll
    for (int o = LPW / 2; o; o >>= 1) word |= __shfl_xor_sync(0xffffffffu, word, o);
    if (lane % LPW == 0) reinterpret_cast<uint32_t *>(dst_row)[lane / LPW] = word;
    if (lane % GL == 0) dst_scales[lane / GL] = __float2half_rn(sc);
}

// ---------------------------------------------------------------- reductions
// Reduce CNT per-lane values across the LPR lanes of a row group so that the
// lanes end up owning different rows: at each halving a lane keeps the upper or
// lower half of its values according to one bit of its chunk index and adds
// what its partner sends.  Costs CNT-1 shuffles instead of CNT*log2(LPR).
template <int CNT, int HALF> struct TransposeReduce {
    static __device__ __forceinline__ void run(float *v, int c, int &rowi) {
        if constexpr (HALF >= 1) {
            if constexpr (CNT > 1) {
                const bool up = (c & HALF) != 0;
#pragma unroll
                for (int k = 0; k < CNT / 2; ++k) {
                    const float send = up ? v[k] : v[k + CNT / 2];
                    const float keep = up ? v[k + CNT / 2] : v[k];
                    v[k] = keep + __shfl_xor_sync(0xffffffffu, send, HALF);
                }
                rowi += up ? CNT / 2 : 0;
                TransposeReduce<CNT / 2, HALF / 2>::run(v, c, rowi);
            } else {
                v[0] += __shfl_xor_sync(0xffffffffu, v[0], HALF);
                TransposeReduce<1, HALF / 2>::run(v, c, rowi);
            }
        }
    }
};

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ---------------------------------------------------------------- the kernel
// DT dtype, D head_dim, NW warps per CTA, R rows in flight per lane,
// S CTAs per unit (a thread-block cluster when S > 1).
template <int DT, int D, int NW, int R, int S>
// (CTAs of 4 warps are the many-units shape: capped at 64 registers so that 8 of them share an SM - measured
// at 9216 units, int4 289 -> 237 us, int4 with head_dim 64 249 -> 173 us, 16-bit rows of 128 bytes unchanged;
// fp32 rows of 512 bytes would spill and keep the compiler's choice)
__global__ void __launch_bounds__(NW * 32, NW == 4 ? ((DT == SH_F32 && D == 128) ? 4 : 8) : 0) sh_decode_kernel(const DecodeParams p) {
    static_assert((R & (R - 1)) == 0, "the row-sum transposition halves R at every step");
    using E = Elem<DT>;
    constexpr int EPL = E::EPL;
    constexpr int LPR = D / EPL;     // lanes per row
    constexpr int RPW = 32 / LPR;    // rows per warp-wide load
    constexpr int PASS = NW * RPW;   // rows per CTA-wide load
    constexpr bool Q4 = (DT == SH_INT4_G64_F16);
    static_assert(LPR >= 1 && LPR <= 32 && (LPR & (LPR - 1)) == 0, "row must be 1..32 chunks");
    static_assert(D <= NW * 32, "output reduction needs one thread per column");
    const int ROWB = stored_row_bytes<DT>(D);
    const int INB = (DT == SH_F32) ? D * 4 : D * 2;

    extern __shared__ __align__(16) float smem[];
    // s_sh[cap] | red[NW*D] | wred[NW] | xM[8] | xL[8] | xo[D] | vn[D]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sub = lane / LPR, c = lane % LPR;
    const int u = blockIdx.x / S;
    const int cr = (S > 1) ? (int)(blockIdx.x % S) : 0;
    const int B = p.B;
    sh_pdl_launch_dependents();
    sh_pdl_wait();            // the preceding kernel of the stream is complete: global memory may be touched
    // live rows including this step's token, the step number and its bit-plane row: the same for
    // every unit (kernel arguments) unless the handle serves sequences of different lengths
    int n = p.n, t_step = p.t, hist_row = p.hist_row;
    if (p.n_arr) {
        n = p.n_arr[u] + 1;
        t_step = p.t_arr[u] + 1;
        hist_row = t_step % p.w;
    }
    // (the same for every CTA of a cluster: all of them leave before the first cluster barrier)
    if (!SH_BOUNDS_OK(n >= 1 && n <= B && t_step >= n && hist_row >= 0 && hist_row < p.w, p.err, 0x701)) return;
    const int n_old = n - 1;

    int chunk, lo;
    if constexpr (S > 1) {
        chunk = (((n + S - 1) / S) + 31) & ~31;
        lo = cr * chunk;
    } else {
        chunk = (B + 31) & ~31;
        lo = 0;
    }
    const int cap = (S > 1) ? ((((B + S - 1) / S) + 31) & ~31) : ((B + 31) & ~31);
    float *s_sh = smem;
    float *red = s_sh + cap;
    float *wred = red + NW * D;
    float *xM = wred + NW;
    float *xL = xM + 8;
    float *xo = xL + 8;
    float *vn = xo + D;                 // int4 store: dequantised value row of this step's token

    if constexpr (S > 1) cg::this_cluster().sync();   // every CTA of the cluster is running: its shared memory may be written

    const int hi_all = min(n, lo + chunk);   // this CTA owns slots [lo, hi_all)
    const int hi = min(n_old, hi_all);       // ... of which [lo, hi) are already cached
    const bool has_new = (n_old >= lo) && (n_old < lo + chunk);
    const int cnt = max(hi_all - lo, 0);

    // ---- q chunk of this lane, fp32
    typename E::Q qv;
    E::load_q(reinterpret_cast<const char *>(p.q) + (size_t)u * INB, c, qv);
    if (p.qring && warp == 0 && sub == 0 && cr == 0) {           // remembered for a recount at compression time
        constexpr int QCH = Q4 ? 4 : 1;                          // 16-byte pieces of q per lane (int4: a lane covers 32 elements)
#pragma unroll
        for (int k = 0; k < QCH; ++k)
            st_plain(p.qring + ((size_t)u * p.w + hist_row) * INB + (c * QCH + k) * 16,
                     ld_plain(reinterpret_cast<const char *>(p.q) + (size_t)u * INB + (c * QCH + k) * 16));
    }

    const char *Kb = p.K + (size_t)u * B * ROWB;
    const char *Vb = p.V + (size_t)u * B * ROWB;
    const __half *Ksb = Q4 ? reinterpret_cast<const __half *>(p.Ks) + (size_t)u * p.Bs * (D / 64) : nullptr;
    const __half *Vsb = Q4 ? reinterpret_cast<const __half *>(p.Vs) + (size_t)u * p.Bs * (D / 64) : nullptr;

    // ---- logits of the cached rows
    float lmax = -INFINITY;
    for (int b0 = lo; b0 < hi; b0 += PASS * R) {
        uint4 raw[R];
        float rs[R];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int j = b0 + i * PASS + warp * RPW + sub;
            raw[i] = make_uint4(0, 0, 0, 0);
            rs[i] = 1.f;
            if (j < hi) {
                raw[i] = ld_stream(Kb + (size_t)j * ROWB + c * 16);
                if constexpr (Q4) rs[i] = __half2float(Ksb[(size_t)j * (D / 64) + (c >> 1)]);
            }
        }
        float part[R];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const float a = E::dot(qv, raw[i]);
            part[i] = Q4 ? a * rs[i] : a;
        }
        int rowi = 0;
        TransposeReduce<R, LPR / 2>::run(part, c, rowi);
        constexpr int NV = (LPR >= R) ? 1 : R / LPR;   // complete sums per lane
        constexpr int WF = (LPR > R) ? LPR / R : 1;    // lanes holding the same sum
        if ((c & (WF - 1)) == 0) {
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int j = b0 + (rowi + k) * PASS + warp * RPW + sub;
                if (j < hi) {
                    const float s = part[k] * p.scale_log2e;
                    s_sh[j - lo] = s;
                    lmax = fmaxf(lmax, s);
                }
            }
        }
    }

    // ---- the token of this step: append it and score it (warp 0 of the owning CTA)
    float fv_new[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) fv_new[e] = 0.f;
    if constexpr (Q4) {
        // warp 0 quantises, appends and scores the key row, warp 1 quantises and appends the value row
        if (has_new && warp < 2) {
            constexpr int EPT = D / 32;
            float x[EPT];
            const char *src = reinterpret_cast<const char *>(warp == 0 ? p.k_new : p.v_new) + (size_t)u * INB;
            int4_append_row<D>(src, (warp == 0 ? p.K : p.V) + ((size_t)u * B + n_old) * ROWB,
                               reinterpret_cast<__half *>(warp == 0 ? p.Ks : p.Vs) + ((size_t)u * p.Bs + n_old) * (D / 64), x, lane);
            if (warp == 0) {
                const __half *qh = reinterpret_cast<const __half *>(reinterpret_cast<const char *>(p.q) + (size_t)u * INB) + EPT * lane;
                float a = 0.f;
#pragma unroll
                for (int e = 0; e < EPT; ++e) a = fmaf(__half2float(qh[e]), x[e], a);
                a = warp_sum(a);
                const float s = a * p.scale_log2e;
                if (lane == 0) {
                    s_sh[n_old - lo] = s;
                    p.pos[(size_t)u * B + n_old] = t_step;
                }
                lmax = fmaxf(lmax, s);
            } else {
#pragma unroll
                for (int e = 0; e < EPT; ++e) vn[EPT * lane + e] = x[e];
            }
        }
    } else if (has_new && warp == 0) {
        float fk[EPL];
        load_input<DT>(reinterpret_cast<const char *>(p.k_new) + (size_t)u * INB, c, fk);
        load_input<DT>(reinterpret_cast<const char *>(p.v_new) + (size_t)u * INB, c, fv_new);
        char *kdst = p.K + ((size_t)u * B + n_old) * ROWB + c * 16;
        char *vdst = p.V + ((size_t)u * B + n_old) * ROWB + c * 16;
        if (sub == 0) {
            st_plain(kdst, ld_plain(reinterpret_cast<const char *>(p.k_new) + (size_t)u * INB + c * 16));
            st_plain(vdst, ld_plain(reinterpret_cast<const char *>(p.v_new) + (size_t)u * INB + c * 16));
        }
        float a = 0.f;
        {
            float qf[EPL];
            E::q_floats(qv, qf);
#pragma unroll
            for (int e = 0; e < EPL; ++e) a = fmaf(qf[e], fk[e], a);
        }
#pragma unroll
        for (int o = LPR / 2; o; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        const float s = a * p.scale_log2e;
        if (lane == 0) s_sh[n_old - lo] = s;
        lmax = fmaxf(lmax, s);
        if (lane == 0) p.pos[(size_t)u * B + n_old] = t_step;
    }

    // ---- max over the unit
    lmax = warp_max(lmax);
    if (lane == 0) wred[warp] = lmax;
    __syncthreads();
    float M = wred[0];
#pragma unroll
    for (int i = 1; i < NW; ++i) M = fmaxf(M, wred[i]);
    if constexpr (S > 1) {
        cg::cluster_group cluster = cg::this_cluster();
        if (tid < S) cluster.map_shared_rank(xM, tid)[cr] = M;
        cluster.sync();
        M = xM[0];
#pragma unroll
        for (int i = 1; i < S; ++i) M = fmaxf(M, xM[i]);
    }

    // ---- exponentials and the denominator
    float lsum = 0.f;
    for (int j = tid; j < cnt; j += NW * 32) {
        const float e = exp2f(s_sh[j] - M);
        s_sh[j] = e;
        lsum += e;
    }
    lsum = warp_sum(lsum);
    __syncthreads();   // every thread has read wred (max) before it is reused
    if (lane == 0) wred[warp] = lsum;
    __syncthreads();
    float L = 0.f;
#pragma unroll
    for (int i = 0; i < NW; ++i) L += wred[i];

    // ---- P.V
    float acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
    for (int b0 = lo; b0 < hi; b0 += PASS * R) {
        uint4 raw[R];
        float pe[R];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int j = b0 + i * PASS + warp * RPW + sub;
            raw[i] = make_uint4(0, 0, 0, 0);
            pe[i] = 0.f;
            if (j < hi) {
                raw[i] = ld_stream(Vb + (size_t)j * ROWB + c * 16);
                pe[i] = s_sh[j - lo];
                if constexpr (Q4) pe[i] *= __half2float(Vsb[(size_t)j * (D / 64) + (c >> 1)]);
            }
        }
#pragma unroll
        for (int i = 0; i < R; ++i) E::axpy(acc, pe[i], raw[i]);
    }
    if (!Q4 && has_new && warp == 0 && sub == 0) {
        const float e_new = s_sh[n_old - lo];
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] = fmaf(e_new, fv_new[e], acc[e]);
    }
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
    }
    if (sub == 0) {
#pragma unroll
        for (int e = 0; e < EPL; ++e) red[warp * D + c * EPL + e] = acc[e];
    }
    __syncthreads();
    float o = 0.f;
    if (tid < D) {
#pragma unroll
        for (int i = 0; i < NW; ++i) o += red[i * D + tid];
        if (Q4 && has_new) o = fmaf(s_sh[n_old - lo], vn[tid], o);      // the step's own token (int4 store: see above)
    }

    if constexpr (S > 1) {
        cg::cluster_group cluster = cg::this_cluster();
        if (tid < D) xo[tid] = o;
        if (tid < S) cluster.map_shared_rank(xL, tid)[cr] = L;
        cluster.sync();
        float Lt = 0.f;
#pragma unroll
        for (int i = 0; i < S; ++i) Lt += xL[i];
        L = Lt;
        if (cr == 0 && tid < D) {
            float ot = 0.f;
#pragma unroll
            for (int i = 0; i < S; ++i) ot += cluster.map_shared_rank(xo, i)[tid];
            p.out[(size_t)u * D + tid] = ot / L;
        }
    } else {
        if (tid < D) p.out[(size_t)u * D + tid] = o / L;
    }

    // ---- record: low_j = [alpha_j < 1/t] = [e_j * t < L], one bit-plane row per step
    {
        const float tf = (float)t_step;
        uint32_t *hrow = p.hist + ((size_t)u * p.w + hist_row) * p.Bw;
        const int w_lo = lo >> 5;
        const int w_hi = (S > 1 && cr != S - 1) ? min(p.Bw, (lo + chunk) >> 5) : p.Bw;
        for (int wd = w_lo + warp; wd < w_hi; wd += NW) {
            const int j = (wd << 5) + lane;   // slot
            bool low = false;
            if (j < hi_all) low = s_sh[j - lo] * tf < L;
            const uint32_t word = __ballot_sync(0xffffffffu, low);
            if (lane == 0) hrow[wd] = word;
        }
    }
    if constexpr (S > 1) {
        // peers may still be reading this CTA's shared memory
        cg::this_cluster().sync();
    }
    if (p.n_arr && tid == 0 && cr == 0) {    // every CTA of the unit has read the old values
        p.n_arr[u] = n;
        p.t_arr[u] = t_step;
    }
}

#include "sh_decode_int4_mma.inl"

template <int DT, int D, int NW, int R, int S>
cudaError_t launch_one(const sh_context *c, const DecodeParams &p, cudaStream_t s) {
    const int B = c->B;
    const int cap = (S > 1) ? ((((B + S - 1) / S) + 31) & ~31) : ((B + 31) & ~31);
    const size_t smem = sizeof(float) * ((size_t)cap + (size_t)NW * D + NW + 8 + 8 + 2 * D);
    auto kern = sh_decode_kernel<DT, D, NW, R, S>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.U * S), 1, 1);
    cfg.blockDim = dim3(NW * 32, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (S > 1) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = S;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    return cudaLaunchKernelEx(&cfg, kern, p);
}

// Attention scores of one query over each unit's present cache, written out in full: alpha_j =
// softmax_j(scale * q.k_j) over the live slots, 0 beyond them.  Nothing is appended and no state
// changes.  Analysis only (the score change ratio of the paper's "Ablation on Attention Score Error"
// compares these between a budgeted cache and a full one); one CTA per unit, plain loads.
template <int DT, int D>
__global__ void __launch_bounds__(256) sh_scores_kernel(const DecodeParams p, float *alpha_out) {
    using E = Elem<DT>;
    constexpr int EPL = E::EPL, LPR = D / EPL, RPW = 32 / LPR, NW = 8;
    constexpr bool Q4 = (DT == SH_INT4_G64_F16);
    const int ROWB = stored_row_bytes<DT>(D);
    const int INB = (DT == SH_F32) ? D * 4 : D * 2;
    extern __shared__ __align__(16) float smem[];
    float *s_sh = smem;                       // [B rounded up]
    float *wred = s_sh + ((p.B + 31) & ~31);  // [NW]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sub = lane / LPR, c = lane % LPR;
    const int u = blockIdx.x, B = p.B;
    const int n = p.n_arr ? p.n_arr[u] : p.n;
    if (!SH_BOUNDS_OK(n >= 0 && n <= B, p.err, 0x702)) return;
    typename E::Q qv;
    E::load_q(reinterpret_cast<const char *>(p.q) + (size_t)u * INB, c, qv);
    const char *Kb = p.K + (size_t)u * B * ROWB;
    const __half *Ksb = Q4 ? reinterpret_cast<const __half *>(p.Ks) + (size_t)u * p.Bs * (D / 64) : nullptr;
    float lmax = -INFINITY;
    for (int j0 = warp * RPW; j0 < n; j0 += NW * RPW) {
        const int j = j0 + sub;
        float a = 0.f;
        if (j < n) {
            a = E::dot(qv, ld_plain(Kb + (size_t)j * ROWB + c * 16));
            if constexpr (Q4) a *= __half2float(Ksb[(size_t)j * (D / 64) + (c >> 1)]);
        }
#pragma unroll
        for (int o = LPR / 2; o; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        if (j < n && c == 0) {
            const float sc = a * p.scale_log2e;
            s_sh[j] = sc;
            lmax = fmaxf(lmax, sc);
        }
    }
    lmax = warp_max(lmax);
    if (lane == 0) wred[warp] = lmax;
    __syncthreads();
    float M = wred[0];
#pragma unroll
    for (int i = 1; i < NW; ++i) M = fmaxf(M, wred[i]);
    __syncthreads();
    float lsum = 0.f;
    for (int j = tid; j < n; j += NW * 32) {
        const float e = exp2f(s_sh[j] - M);
        s_sh[j] = e;
        lsum += e;
    }
    lsum = warp_sum(lsum);
    if (lane == 0) wred[warp] = lsum;
    __syncthreads();
    float L = 0.f;
#pragma unroll
    for (int i = 0; i < NW; ++i) L += wred[i];
    for (int j = tid; j < B; j += NW * 32) alpha_out[(size_t)u * B + j] = j < n ? s_sh[j] / L : 0.f;
}

template <int DT, int D>
cudaError_t launch_scores(const DecodeParams &p, float *alpha_out, cudaStream_t s) {
    const size_t smem = sizeof(float) * ((size_t)((p.B + 31) & ~31) + 8);
    auto kern = sh_scores_kernel<DT, D>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    kern<<<p.U, 256, smem, s>>>(p, alpha_out);
    return cudaGetLastError();
}

template <int DT, int D, int NW, int R>
cudaError_t launch_split(const sh_context *c, const DecodeParams &p, cudaStream_t s) {
    switch (c->split) {
        case 1: return launch_one<DT, D, NW, R, 1>(c, p, s);
        case 2: return launch_one<DT, D, NW, R, 2>(c, p, s);
        case 4: return launch_one<DT, D, NW, R, 4>(c, p, s);
        case 8: return launch_one<DT, D, NW, R, 8>(c, p, s);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

cudaError_t sh_launch_scores(const sh_context *c, const DecodeParams &p, float *alpha_out, cudaStream_t s, long long *launches) {
    cudaError_t e = cudaErrorInvalidValue;
    switch (c->dtype) {
        case SH_F32: e = c->D == 64 ? launch_scores<SH_F32, 64>(p, alpha_out, s) : launch_scores<SH_F32, 128>(p, alpha_out, s); break;
        case SH_F16: e = c->D == 64 ? launch_scores<SH_F16, 64>(p, alpha_out, s) : launch_scores<SH_F16, 128>(p, alpha_out, s); break;
        case SH_BF16: e = c->D == 64 ? launch_scores<SH_BF16, 64>(p, alpha_out, s) : launch_scores<SH_BF16, 128>(p, alpha_out, s); break;
        case SH_INT4_G64_F16:
            e = c->D == 64 ? launch_scores<SH_INT4_G64_F16, 64>(p, alpha_out, s) : launch_scores<SH_INT4_G64_F16, 128>(p, alpha_out, s);
            break;
        default: break;
    }
    if (e == cudaSuccess) *launches += 1;
    return e;
}

// Which decode kernel serves `units` units of this handle: 2 = pipelined (sh_decode_tma.cu), 3 = int4 rows on the
// tensor cores (sh_decode_int4_mma.inl), 1 = direct loads.
int sh_decode_kernel_for(const sh_context *c, int units) {
    // Shapes of launch (crossovers measured on B200, rows of 256 bytes: equal at 12 units per SM, the direct
    // kernel 6 % ahead from 16 per SM on, the pipelined one 15 % ahead at 8.6).  With very many units per SM
    // the direct-load kernel in its many-units shape is the fastest for every storage type: CTAs of 4 warps
    // capped at 64 registers, eight per SM, hide the load latency by occupancy (9216 units, fp16 rows of 256
    // bytes: 261 us against 273 us for the pipelined kernel).  Below 16 units per SM, rows of 256 bytes or
    // more stream through the persistent pipelined kernel from 128 units on; the direct kernel takes the
    // rest, with 4-warp CTAs from 4 units per SM on and 8-warp CTAs (and a cluster split for very few units)
    // below.  SH_OPT_DECODE_KERNEL = 1 / 2 forces the direct / pipelined kernel.
    const bool many = units >= 4 * 148 && c->split == 1;
    const bool pipelined_ok = sh_decode_tma_supported(c);
    const bool prefer_direct = many && (!pipelined_ok || units >= 16 * 148);
    if (c->kernel != 1 && pipelined_ok &&
        (c->kernel == 2 || (!prefer_direct && units >= 128 && !(c->split_explicit && c->split > 1))))
        return 2;
    // int4 store, many units: codes unpacked to fp16 and multiplied on the tensor cores (9216 units: 158 us against
    // 223 us on CUDA cores), unless the caller asked for the CUDA-core kernel or the budget outgrows its shared memory
    if (many && c->kernel != 1 && c->dtype == SH_INT4_G64_F16 && c->D == 128 && int4_mma_smem(c->B) <= 200 * 1024) return 3;
    return 1;
}

cudaError_t sh_launch_decode(const sh_context *c, const DecodeParams &p, cudaStream_t s, long long *launches) {
    const bool many = p.U >= 4 * 148 && c->split == 1;
    const int which = sh_decode_kernel_for(c, p.U);
    if (which == 2) return sh_launch_decode_tma(c, p, s, launches);
    cudaError_t e = cudaErrorInvalidValue;
    // Two shapes of CTA.  With few units per SM the step is latency-bound and a CTA of 8 warps with 8 row
    // loads in flight per thread finishes a unit soonest.  With many units per SM (no cluster split then)
    // CTAs of 4 warps (16 row loads in flight per thread; int4, whose loads carry 32 elements each: 2), spend less on barriers and on the cross-warp merge:
    // measured at 9216 units on B200, int4 428 -> 289 us, fp16 with head_dim 64 183 -> 149 us, fp32 with
    // head_dim 64 369 -> 263 us, 16-bit rows of 256 bytes 283 -> 261 us.
    switch (c->dtype) {
        case SH_F32:
            if (c->D == 64) e = many ? launch_one<SH_F32, 64, 4, 16, 1>(c, p, s) : launch_split<SH_F32, 64, 8, 8>(c, p, s);
            else if (c->D == 128) e = many ? launch_one<SH_F32, 128, 4, 16, 1>(c, p, s) : launch_split<SH_F32, 128, 8, 8>(c, p, s);
            break;
        case SH_F16:
            if (c->D == 64) e = many ? launch_one<SH_F16, 64, 4, 16, 1>(c, p, s) : launch_split<SH_F16, 64, 8, 8>(c, p, s);
            else if (c->D == 128) e = many ? launch_one<SH_F16, 128, 4, 8, 1>(c, p, s) : launch_split<SH_F16, 128, 8, 8>(c, p, s);
            break;
        case SH_BF16:
            if (c->D == 64) e = many ? launch_one<SH_BF16, 64, 4, 16, 1>(c, p, s) : launch_split<SH_BF16, 64, 8, 8>(c, p, s);
            else if (c->D == 128) e = many ? launch_one<SH_BF16, 128, 4, 8, 1>(c, p, s) : launch_split<SH_BF16, 128, 8, 8>(c, p, s);
            break;
        case SH_INT4_G64_F16:
            if (c->D == 64) e = many ? launch_one<SH_INT4_G64_F16, 64, 4, 2, 1>(c, p, s) : launch_split<SH_INT4_G64_F16, 64, 8, 4>(c, p, s);
            else if (c->D == 128) {
                // many units: unpacked codes go to the tensor cores (sh_decode_int4_mma.inl) unless the caller
                // asked for the CUDA-core kernel by name
                if (many) e = which == 3 ? launch_int4_mma<4, 1, 1, 8>(c, p, s) : launch_one<SH_INT4_G64_F16, 128, 4, 2, 1>(c, p, s);
                else e = launch_split<SH_INT4_G64_F16, 128, 8, 4>(c, p, s);
            }
            break;
        default: break;
    }
    if (e == cudaSuccess) *launches += 1;
    return e;
}
