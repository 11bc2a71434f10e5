// Fused decode step for the int4-g64 store with many units per launch, dot products on the tensor cores.
// Included by sh_decode.cu inside its unnamed namespace (it uses that file's helpers).
//
// On an int4 cache the CUDA-core kernel is bound by instruction issue, not by memory: unpacking a 4-bit
// code, converting it and multiplying costs about five instructions per code.  Here a code is only
// unpacked to fp16 (a shift, one logic operation and half of a packed subtract: exact small integers) and
// the multiply-adds run as warp-level MMAs (m16n8k16, fp16 inputs, fp32 accumulation; products of fp16
// values are exact in fp32).  One query per unit is a matrix-vector product, so most of an MMA's columns
// stay empty; the tensor pipe has that much room to spare, the issue slots do not.
//
// q.K^T: an MMA's 16 rows are 8 keys x the 2 scale groups of a row (rows g and g+8: key g, dims 0..63 and
// 64..127), its k-dimension runs over the 64 dims of a group in 4 steps, column 0 of B holds q[0..63] and
// column 1 q[64..127].  C[g][0] and C[g+8][1] are the two group sums of key g; the thread that holds both
// (lane 4g) combines them with the key's two fp16 scales in fp32.  The assignment of dims to k-indices is
// free as long as A and B agree: thread (g, tg) takes the 8-byte piece tg of each group (16 codes).
//
// P.V: O^T = V^T . c with c_j = e_j * (value scale of key j and of the column's group): an MMA's rows are 16
// output dims, its k-dimension 16 keys.  Thread (g, tg) loads 8 bytes (dims 16g..16g+15) of keys
// 4tg..4tg+3 of a 16-key block; codes of two keys are paired into one register by a byte permute.  The
// coefficient enters as fp16 high and low parts in separate columns of B (columns 0/1: group 0 hi/lo,
// 2/3: group 1 hi/lo), so the product keeps ~fp32 accuracy; rows of dims below 64 read columns 0+1, the
// others 2+3.
//
// The step's own token is quantised and appended by warps 0 (key, which it also scores) and 1 (value) in fp32
// with the arithmetic of the CUDA-core kernel; softmax, record bits and the cross-warp merge are the same as there.

__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// codes of elements (2i, 2i+1) of an 8-code word as a half2 of exact integers in [-8, 7]
__device__ __forceinline__ uint32_t codes_pair(uint32_t word, int i) {
    uint32_t bits = ((word >> (4 * i)) & 0x000F000Fu) | 0x64006400u;       // (1024 + c0, 1024 + c1)
    const __half2 bias = __floats2half2_rn(1032.f, 1032.f);
    const __half2 h = __hsub2(*reinterpret_cast<__half2 *>(&bits), bias);
    return *reinterpret_cast<const uint32_t *>(&h);
}
__device__ __forceinline__ uint2 ld_stream8(const void *p) {
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
    const __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<const uint32_t *>(&h);
}

// NW warps per CTA, RK (RV) key blocks in flight per warp in the K (V) pass.
template <int NW, int RK, int RV, int MB>
__global__ void __launch_bounds__(NW * 32, MB) sh_decode_int4_mma_kernel(const DecodeParams p) {
    static_assert(NW % 4 == 0, "one thread per output column, and 16-byte aligned shared arrays behind wred[NW]");
    constexpr int D = 128, ROWB = 64, INB = 256, G = 2;
    constexpr int KB = 8;        // keys per warp step in the K pass
    constexpr int VB = 16;       // keys per warp step in the V pass
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, tg = lane & 3;
    const int u = blockIdx.x, B = p.B;
    sh_pdl_launch_dependents();
    sh_pdl_wait();
    int n = p.n, t_step = p.t, hist_row = p.hist_row;
    if (p.n_arr) {
        n = p.n_arr[u] + 1;
        t_step = p.t_arr[u] + 1;
        hist_row = t_step % p.w;
    }
    if (!SH_BOUNDS_OK(n >= 1 && n <= B && t_step >= n && hist_row >= 0 && hist_row < p.w, p.err, 0x703)) return;
    const int n_old = n - 1;
    const int cap = (B + 31) & ~31;
    float *s_sh = smem;                 // [cap] scaled logits, then e_j
    float *red = s_sh + cap;            // [NW][D] partial outputs
    float *wred = red + NW * D;         // [NW]
    float *vnew_sh = wred + NW;         // [D] dequantised value row of the step's token
    const int capk = (B + 15) & ~15;
    __half *cT = reinterpret_cast<__half *>(vnew_sh + D);   // [4][capk] P.V coefficients e_j * scale: group 0 high, low, group 1 high, low

    const char *qrow = reinterpret_cast<const char *>(p.q) + (size_t)u * INB;
    // B fragments of q: column g of B is q restricted to scale group g (columns 2..7 are zero)
    uint32_t qb[4][2];
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        qb[s][0] = qb[s][1] = 0u;
        if (g < G) {
            qb[s][0] = *reinterpret_cast<const uint32_t *>(qrow + (64 * g + 16 * tg + 2 * s) * 2);
            qb[s][1] = *reinterpret_cast<const uint32_t *>(qrow + (64 * g + 16 * tg + 8 + 2 * s) * 2);
        }
    }
    if (p.qring && tid < INB / 16)
        st_plain(p.qring + ((size_t)u * p.w + hist_row) * INB + tid * 16, ld_plain(qrow + tid * 16));

    const char *Kb = p.K + (size_t)u * B * ROWB;
    const char *Vb = p.V + (size_t)u * B * ROWB;
    const __half *Ksb = reinterpret_cast<const __half *>(p.Ks) + (size_t)u * p.Bs * G;
    const __half *Vsb = reinterpret_cast<const __half *>(p.Vs) + (size_t)u * p.Bs * G;

    // ---- logits of the cached rows: 8 keys per warp step, RK steps in flight
    float lmax = -INFINITY;
    for (int b0 = 0; b0 < n_old; b0 += NW * KB * RK) {
        uint2 raw[RK][2];
        __half2 sc2[RK];
#pragma unroll
        for (int i = 0; i < RK; ++i) {
            const int j = b0 + (i * NW + warp) * KB + g;
            raw[i][0] = raw[i][1] = make_uint2(0u, 0u);
            sc2[i] = __floats2half2_rn(0.f, 0.f);
            if (j < n_old) {
                raw[i][0] = ld_stream8(Kb + (size_t)j * ROWB + 8 * tg);          // group 0, piece tg
                raw[i][1] = ld_stream8(Kb + (size_t)j * ROWB + 32 + 8 * tg);     // group 1, piece tg
                sc2[i] = *reinterpret_cast<const __half2 *>(Ksb + (size_t)j * G);
            }
        }
#pragma unroll
        for (int i = 0; i < RK; ++i) {
            float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int s = 0; s < 4; ++s)
                mma_f16(c, codes_pair(raw[i][0].x, s), codes_pair(raw[i][1].x, s), codes_pair(raw[i][0].y, s),
                        codes_pair(raw[i][1].y, s), qb[s][0], qb[s][1]);
            const int j = b0 + (i * NW + warp) * KB + g;
            if (tg == 0 && j < n_old) {
                const float2 sc = __half22float2(sc2[i]);
                const float sl = (c[0] * sc.x + c[3] * sc.y) * p.scale_log2e;
                s_sh[j] = sl;
                lmax = fmaxf(lmax, sl);
            }
        }
    }

    // ---- the token of this step: warp 0 quantises and appends its key and scores it, warp 1 does the value row
    if (warp < 2) {
        float x[4];
        int4_append_row<D>(reinterpret_cast<const char *>(warp == 0 ? p.k_new : p.v_new) + (size_t)u * INB,
                           (warp == 0 ? p.K : p.V) + ((size_t)u * B + n_old) * ROWB,
                           reinterpret_cast<__half *>(warp == 0 ? p.Ks : p.Vs) + ((size_t)u * p.Bs + n_old) * G, x, lane);
        if (warp == 0) {
            const uint2 qin = *reinterpret_cast<const uint2 *>(qrow + 8 * lane);
            const float2 q01 = __half22float2(*reinterpret_cast<const __half2 *>(&qin.x));
            const float2 q23 = __half22float2(*reinterpret_cast<const __half2 *>(&qin.y));
            float dot = fmaf(q23.y, x[3], fmaf(q23.x, x[2], fmaf(q01.y, x[1], q01.x * x[0])));
            dot = warp_sum(dot);
            const float sl = dot * p.scale_log2e;
            if (lane == 0) {
                s_sh[n_old] = sl;
                p.pos[(size_t)u * B + n_old] = t_step;
            }
            lmax = fmaxf(lmax, sl);
        } else {
            *reinterpret_cast<float4 *>(vnew_sh + 4 * lane) = make_float4(x[0], x[1], x[2], x[3]);
        }
    }

    // ---- max, exponentials, denominator
    lmax = warp_max(lmax);
    if (lane == 0) wred[warp] = lmax;
    __syncthreads();
    float M = wred[0];
#pragma unroll
    for (int i = 1; i < NW; ++i) M = fmaxf(M, wred[i]);
    float lsum = 0.f;
    for (int j = tid; j < n; j += NW * 32) {
        const float e = exp2f(s_sh[j] - M);
        s_sh[j] = e;
        lsum += e;
    }
    // coefficient of every cached key in the second contraction, once per key: e_j times the value scale of each
    // group, as an fp16 high part and what it missed (zero beyond the cached rows: the blocks of 16 keys run over)
    for (int j = tid; j < ((n_old + 15) & ~15); j += NW * 32) {
        float c0 = 0.f, c1 = 0.f;
        if (j < n_old) {
            const float2 vs = __half22float2(*reinterpret_cast<const __half2 *>(Vsb + (size_t)j * G));
            c0 = s_sh[j] * vs.x;
            c1 = s_sh[j] * vs.y;
        }
        const __half h0 = __float2half_rn(c0), h1 = __float2half_rn(c1);
        cT[j] = h0;
        cT[capk + j] = __float2half_rn(c0 - __half2float(h0));
        cT[2 * capk + j] = h1;
        cT[3 * capk + j] = __float2half_rn(c1 - __half2float(h1));
    }
    lsum = warp_sum(lsum);
    __syncthreads();
    if (lane == 0) wred[warp] = lsum;
    __syncthreads();
    float L = 0.f;
#pragma unroll
    for (int i = 0; i < NW; ++i) L += wred[i];

    // ---- P.V: 16 keys per warp step, RV steps in flight; thread (g, tg): dims 16g..16g+15 of keys 4tg..4tg+3
    float oacc[8][4];
#pragma unroll
    for (int b = 0; b < 8; ++b)
#pragma unroll
        for (int e = 0; e < 4; ++e) oacc[b][e] = 0.f;
    for (int b0 = 0; b0 < n_old; b0 += NW * VB * RV) {
        uint2 raw[RV][4];
        uint32_t cb[RV][2];
#pragma unroll
        for (int i = 0; i < RV; ++i) {
            const int jb = b0 + (i * NW + warp) * VB + 4 * tg;
#pragma unroll
            for (int kx = 0; kx < 4; ++kx) {
                raw[i][kx] = make_uint2(0u, 0u);
                if (jb + kx < n_old) raw[i][kx] = ld_stream8(Vb + (size_t)(jb + kx) * ROWB + 8 * g);
            }
            // column g of B (g < 4) for this thread's four keys; the other columns stay empty
            uint2 cc = make_uint2(0u, 0u);
            if (g < 4 && jb < n_old) cc = *reinterpret_cast<const uint2 *>(cT + g * capk + jb);
            cb[i][0] = cc.x;
            cb[i][1] = cc.y;
        }
#pragma unroll
        for (int i = 0; i < RV; ++i) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                // The codes of two keys are interleaved once per word, 16-bit half by half: nibble i of the low halves
                // holds element 2i of both keys, nibble i of the high halves element 2i + 1 (element e of a word sits
                // in nibble (e>>1) + 4(e&1)); one mask then pulls out a (key, key + 1) pair of the same dim.
                const uint32_t w0 = h ? raw[i][0].y : raw[i][0].x, w1 = h ? raw[i][1].y : raw[i][1].x;
                const uint32_t w2 = h ? raw[i][2].y : raw[i][2].x, w3 = h ? raw[i][3].y : raw[i][3].x;
                const uint32_t ev01 = __byte_perm(w0, w1, 0x5410), od01 = __byte_perm(w0, w1, 0x7632);
                const uint32_t ev23 = __byte_perm(w2, w3, 0x5410), od23 = __byte_perm(w2, w3, 0x7632);
#pragma unroll
                for (int ix = 0; ix < 4; ++ix) {
                    // block b = 4h + ix: rows g / g+8 are dims 16g + 2b and 16g + 2b + 1; k-indices 2tg, 2tg+1 / 2tg+8, 2tg+9
                    // are this thread's keys 0, 1 / 2, 3
                    mma_f16(oacc[4 * h + ix], codes_pair(ev01, ix), codes_pair(od01, ix), codes_pair(ev23, ix), codes_pair(od23, ix),
                            cb[i][0], cb[i][1]);
                }
            }
        }
    }
    // dims below 64 (g < 4) take columns 0 + 1, held by the lane with tg = 0; the others columns 2 + 3, tg = 1
    if (tg == (g >> 2)) {
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            red[warp * D + 16 * g + 2 * b] = oacc[b][0] + oacc[b][1];
            red[warp * D + 16 * g + 2 * b + 1] = oacc[b][2] + oacc[b][3];
        }
    }
    __syncthreads();
    if (tid < D) {
        float o = s_sh[n_old] * vnew_sh[tid];
#pragma unroll
        for (int i = 0; i < NW; ++i) o += red[i * D + tid];
        p.out[(size_t)u * D + tid] = o / L;
    }

    // ---- record: low_j = [alpha_j < 1/t] = [e_j * t < L], one bit-plane row per step
    {
        const float tf = (float)t_step;
        uint32_t *hrow = p.hist + ((size_t)u * p.w + hist_row) * p.Bw;
        for (int wd = warp; wd < p.Bw; wd += NW) {
            const int j = (wd << 5) + lane;
            bool low = false;
            if (j < n) low = s_sh[j] * tf < L;
            const uint32_t word = __ballot_sync(0xffffffffu, low);
            if (lane == 0) hrow[wd] = word;
        }
    }
    if (p.n_arr && tid == 0) {
        p.n_arr[u] = n;
        p.t_arr[u] = t_step;
    }
}

// Shared memory of the kernel with 4 warps: logits, partial outputs, the token's value row, P.V coefficients.
inline size_t int4_mma_smem(int B) {
    return sizeof(float) * ((size_t)((B + 31) & ~31) + 4 * 128 + 4 + 128) + 8 * (size_t)((B + 15) & ~15);
}

template <int NW, int RK, int RV, int MB>
cudaError_t launch_int4_mma(const sh_context *c, const DecodeParams &p, cudaStream_t s) {
    static_assert(NW == 4, "int4_mma_smem assumes 4 warps");
    const size_t smem = int4_mma_smem(c->B);
    auto kern = sh_decode_int4_mma_kernel<NW, RK, RV, MB>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.U, 1, 1);
    cfg.blockDim = dim3(NW * 32, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, p);
}
