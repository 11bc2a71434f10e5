// Chunked prompt step: c consecutive tokens of the stream handled in one launch.  This file holds the
// warp-level (mma.sync) kernel, chosen with SH_OPT_PREFILL_CHUNK = 2, and the dispatch between it and the
// tcgen05 kernel of sh_chunk_umma.cu, which is the default.
//
// Between two compressions the method's steps only append, so c steps can be
// evaluated together: step i (0 <= i < c) attends with q_i over the n0 cached
// rows plus the chunk's own tokens 0..i (causal), and records its comparison
// bits in its own bit-plane row.  The results are those of c calls of the
// decode step; K and V are read from HBM once per chunk instead of once per
// token, and the two contractions S = Q.K^T  [c x n x d] and O = P.V [c x d x n]
// are dense enough (about 50 FLOP per byte) to belong on the tensor cores.
//
// One CTA of 8 warps per unit.  S is kept whole in shared memory in fp32
// ([CQ][n] - the record bits need every probability against the final row sum),
// K and V pass through a 64-row tile buffer.  MMAs are warp-level
// m16n8k16 with fp32 accumulation: q.k products of 16-bit inputs are exact;
// P is fed as a high and a low 16-bit part so that P.V keeps ~fp32 accuracy.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "sh_internal.h"

namespace {

constexpr int D = 128;          // head_dim served by this kernel
constexpr int KT = 64;          // keys per tile
constexpr int ROWH = D + 8;     // padded row length in 16-bit elements (272 bytes: conflict-free ldmatrix)
constexpr int NTHREADS = 256;

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void *row_ptr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(smem_addr(row_ptr)));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void *row_ptr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(smem_addr(row_ptr)));
}

// 2^x (one MUFU instruction; 2^-inf = 0)
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int DT> struct Mma;
template <> struct Mma<SH_F16> {
    static __device__ __forceinline__ void run(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    }
    // p0, p1 in [0, 1] -> packed high parts and packed low parts (p = hi + lo up to ~2^-22)
    static __device__ __forceinline__ void split(float p0, float p1, uint32_t &hi, uint32_t &lo) {
        const __half2 h = __floats2half2_rn(p0, p1);
        const float2 hf = __half22float2(h);
        const __half2 l = __floats2half2_rn(p0 - hf.x, p1 - hf.y);
        hi = *reinterpret_cast<const uint32_t *>(&h);
        lo = *reinterpret_cast<const uint32_t *>(&l);
    }
};
template <> struct Mma<SH_BF16> {
    static __device__ __forceinline__ void run(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    }
    static __device__ __forceinline__ void split(float p0, float p1, uint32_t &hi, uint32_t &lo) {
        const __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
        const float2 hf = __bfloat1622float2(h);
        const __nv_bfloat162 l = __floats2bfloat162_rn(p0 - hf.x, p1 - hf.y);
        hi = *reinterpret_cast<const uint32_t *>(&h);
        lo = *reinterpret_cast<const uint32_t *>(&l);
    }
};


__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Start filling a 64-row tile buffer with rows [j0, j0+64) of the unit's K or V as seen by
// the chunk: cached rows, then the chunk's own tokens, zeros beyond.  Asynchronous: the
// caller commits the group and waits for it before reading the tile.
__device__ __forceinline__ void load_tile_async(uint16_t *tile, const char *cache_u, const char *chunk, int j0, int n0,
                                                int n_tot, size_t chunk_stride) {
    for (int idx = threadIdx.x; idx < KT * (D / 8); idx += NTHREADS) {
        const int row = idx / (D / 8), ch = idx % (D / 8);
        const int j = j0 + row;
        uint16_t *dst = tile + row * ROWH + ch * 8;
        if (j < n0) cp_async16(dst, cache_u + (size_t)j * (D * 2) + ch * 16);
        else if (j < n_tot) cp_async16(dst, chunk + (size_t)(j - n0) * chunk_stride + ch * 16);
        else *reinterpret_cast<uint4 *>(dst) = make_uint4(0, 0, 0, 0);
    }
}

// CQ queries per CTA (64 or 32).  Warps form a WM x WN grid: WM row blocks of 16 queries,
// WN groups that split the 64 keys of a tile (logits) or the 128 output columns (P.V).
template <int DT, int CQ, bool RECOUNT>
__global__ void __launch_bounds__(NTHREADS, CQ == 32 ? 2 : 1) sh_prefill_chunk_kernel(const ChunkParams p) {
    constexpr int WM = CQ / 16, WN = 8 / WM;
    constexpr int NBK = KT / WN / 8;     // 8-key blocks per warp in the logits phase
    constexpr int NBD = D / WN / 8;      // 8-column blocks per warp in the P.V phase
    static_assert(NBK % 2 == 0 && NBD % 2 == 0, "ldmatrix.x4 covers two 8-wide blocks");
    using M = Mma<DT>;

    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint16_t *Qs = reinterpret_cast<uint16_t *>(smem_raw);              // [CQ][ROWH]
    uint16_t *tile0 = Qs + CQ * ROWH;                                   // [2][KT][ROWH] double-buffered K/V tiles
    float *S = reinterpret_cast<float *>(tile0 + 2 * KT * ROWH);        // [CQ][SS]
    float *rowL = S + (size_t)CQ * p.SS;                                // [CQ] row sums
    int *nvs = reinterpret_cast<int *>(rowL + CQ);                      // [CQ] keys visible to each query
    int *pos_sh = nvs + CQ;                                             // [SS] stream positions of the cached slots (recount mode)

    const int u = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int wm = warp % WM, wn = warp / WM;
    const int n0 = p.n0, SS = p.SS;
    // first step handled by this CTA and how many
    // blockIdx.y selects CQ consecutive queries (of the window in recount mode, of the chunk otherwise)
    const int qoff = (int)blockIdx.y * CQ;
    const int step0 = (RECOUNT ? p.first_step : p.t0 + 1) + qoff;
    const int c = min(CQ, (RECOUNT ? p.nsteps : p.c) - qoff);
    // keys this CTA needs: the cache, and the chunk's tokens up to its own last query
    const int n_tot = RECOUNT ? p.n0 : p.n0 + qoff + c;
    const size_t tstride = (size_t)p.Utot * D * 2;       // bytes between consecutive tokens of one unit
    const char *Kc = p.K + (size_t)u * p.B * D * 2;
    const char *Vc = p.V + (size_t)u * p.B * D * 2;
    const int ntiles = (n_tot + KT - 1) / KT;

    // ---- queries of the chunk (rows beyond c are zero)
    for (int idx = tid; idx < CQ * (D / 8); idx += NTHREADS) {
        const int row = idx / (D / 8), ch = idx % (D / 8);
        uint4 val = make_uint4(0, 0, 0, 0);
        if (row < c) {
            char *ring_row = p.qring ? p.qring + ((size_t)u * p.w + (step0 + row) % p.w) * (D * 2) + ch * 16 : nullptr;
            if (RECOUNT) {
                val = *reinterpret_cast<const uint4 *>(ring_row);
            } else {
                val = *reinterpret_cast<const uint4 *>(p.q + (size_t)(qoff + row) * tstride + (size_t)u * D * 2 + ch * 16);
                if (ring_row) *reinterpret_cast<uint4 *>(ring_row) = val;     // remembered for a later recount
            }
        }
        *reinterpret_cast<uint4 *>(Qs + row * ROWH + ch * 8) = val;
    }
    const int32_t *pos_u = p.pos + (size_t)u * p.B;
    if (RECOUNT) {
        // a query sees the cached slots whose position does not exceed its step (slots need not be sorted);
        // every cached slot is scanned, the invisible ones carry a logit of -inf
        for (int i = tid; i < CQ; i += NTHREADS) nvs[i] = (i < c) ? n0 : 0;
        for (int j = tid; j < n0; j += NTHREADS) pos_sh[j] = pos_u[j];
    } else {
        for (int i = tid; i < CQ; i += NTHREADS) nvs[i] = (i < c) ? n0 + qoff + i + 1 : 0;
        if (tid < c) p.pos[(size_t)u * p.B + n0 + qoff + tid] = step0 + tid;
        // append the chunk's keys and values to the cache (nothing in this launch reads them back from there)
        for (int idx = tid; idx < c * (D / 8); idx += NTHREADS) {
            const int row = idx / (D / 8), ch = idx % (D / 8);
            const size_t src = (size_t)(qoff + row) * tstride + (size_t)u * D * 2 + ch * 16;
            const size_t dst = ((size_t)u * p.B + n0 + qoff + row) * (D * 2) + ch * 16;
            *reinterpret_cast<uint4 *>(p.K + dst) = *reinterpret_cast<const uint4 *>(p.k + src);
            *reinterpret_cast<uint4 *>(p.V + dst) = *reinterpret_cast<const uint4 *>(p.v + src);
        }
    }
    const char *kchunk = RECOUNT ? nullptr : p.k + (size_t)u * D * 2, *vchunk = RECOUNT ? nullptr : p.v + (size_t)u * D * 2;
    load_tile_async(tile0, Kc, kchunk, 0, n0, n_tot, tstride);      // first K tile is on its way
    cp_async_commit();
    __syncthreads();

    // A fragments of this warp's 16 queries, all 8 k-steps, kept in registers
    uint32_t qa[D / 16][4];
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
        const int mi = lane >> 3, r = lane & 7;   // matrix index, row within it
        ldmatrix_x4(qa[ks], Qs + (wm * 16 + (mi & 1) * 8 + r) * ROWH + ks * 16 + (mi >> 1) * 8);
    }

    // ---- phase 1: S = scale * Q.K^T, causal inside the chunk
    for (int kt = 0; kt < ntiles; ++kt) {
        uint16_t *tile = tile0 + (kt & 1) * KT * ROWH;
        // prefetch the next K tile (or the first V tile) into the other buffer, then wait for this one
        if (kt + 1 < ntiles) load_tile_async(tile0 + ((kt + 1) & 1) * KT * ROWH, Kc, kchunk, (kt + 1) * KT, n0, n_tot, tstride);
        else if (!RECOUNT) load_tile_async(tile0 + ((kt + 1) & 1) * KT * ROWH, Vc, vchunk, 0, n0, n_tot, tstride);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        float acc[NBK][4];
#pragma unroll
        for (int nb = 0; nb < NBK; ++nb)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[nb][e] = 0.f;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
            for (int nbp = 0; nbp < NBK / 2; ++nbp) {
                uint32_t b[4];
                const int mi = lane >> 3, r = lane & 7;
                ldmatrix_x4(b, tile + (wn * (KT / WN) + nbp * 16 + (mi >> 1) * 8 + r) * ROWH + ks * 16 + (mi & 1) * 8);
                M::run(acc[2 * nbp], qa[ks], b[0], b[1]);
                M::run(acc[2 * nbp + 1], qa[ks], b[2], b[3]);
            }
        }
#pragma unroll
        for (int nb = 0; nb < NBK; ++nb) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int i = wm * 16 + (lane >> 2) + (e >> 1) * 8;                 // query row
                const int j = kt * KT + wn * (KT / WN) + nb * 8 + (lane & 3) * 2 + (e & 1);   // key slot
                // cached rows (and chunk tokens 0..i) the query may see
                const bool live = RECOUNT ? (j < nvs[i] && pos_sh[j] <= step0 + i) : j < nvs[i];
                S[(size_t)i * SS + j] = live ? acc[nb][e] * p.scale_log2e : -INFINITY;
            }
        }
        __syncthreads();      // tile consumed: its buffer may be refilled by the next iteration's prefetch
    }

    // ---- softmax rows and record bits: one warp per query row
    for (int i = warp; i < CQ; i += NTHREADS / 32) {
        float *Si = S + (size_t)i * SS;
        const int nv = nvs[i];
        float mx = -INFINITY;
        for (int j = lane; j < nv; j += 32) mx = fmaxf(mx, Si[j]);
#pragma unroll
        for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float sum = 0.f;
        for (int j = lane; j < ntiles * KT; j += 32) {
            const float e = (j < nv && Si[j] != -INFINITY) ? ex2_approx(Si[j] - mx) : 0.f;
            Si[j] = e;
            sum += e;
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == 0) rowL[i] = sum;
        if (i < c) {
            // step t: low_j = [alpha_j < 1/t] = [e_j * t < L]
            const int t = step0 + i;
            const float tf = (float)t;
            uint32_t *hrow = p.hist + ((size_t)u * p.w + (t % p.w)) * p.Bw;
            __syncwarp();
            for (int wd = 0; wd < p.Bw; ++wd) {
                const int j = (wd << 5) + lane;
                const bool low = j < nv && (!RECOUNT || pos_sh[j] <= t) && Si[j] * tf < sum;
                const uint32_t word = __ballot_sync(0xffffffffu, low);
                if (lane == 0) hrow[wd] = word;
            }
        }
    }

    if constexpr (RECOUNT) {
        cp_async_wait<0>();
    } else {
    // ---- phase 2: O = P.V
    float oacc[NBD][4];
#pragma unroll
    for (int nb = 0; nb < NBD; ++nb)
#pragma unroll
        for (int e = 0; e < 4; ++e) oacc[nb][e] = 0.f;
    for (int kt = 0; kt < ntiles; ++kt) {
        // V tile kt sits in buffer (ntiles + kt) & 1: the first one was prefetched behind the last K tile
        uint16_t *tile = tile0 + ((ntiles + kt) & 1) * KT * ROWH;
        if (kt + 1 < ntiles) load_tile_async(tile0 + ((ntiles + kt + 1) & 1) * KT * ROWH, Vc, vchunk, (kt + 1) * KT, n0, n_tot, tstride);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();      // tile landed for everyone; on the first pass also: P complete
#pragma unroll
        for (int ks = 0; ks < KT / 16; ++ks) {
            // A fragments of P: rows r0 = wm*16 + lane/4 and r0 + 8, key columns j0 + {0,1} and j0 + 8 + {0,1}
            const int r0 = wm * 16 + (lane >> 2);
            const int j0 = kt * KT + ks * 16 + (lane & 3) * 2;
            const float2 p00 = *reinterpret_cast<const float2 *>(S + (size_t)r0 * SS + j0);
            const float2 p10 = *reinterpret_cast<const float2 *>(S + (size_t)(r0 + 8) * SS + j0);
            const float2 p01 = *reinterpret_cast<const float2 *>(S + (size_t)r0 * SS + j0 + 8);
            const float2 p11 = *reinterpret_cast<const float2 *>(S + (size_t)(r0 + 8) * SS + j0 + 8);
            uint32_t ahi[4], alo[4];
            M::split(p00.x, p00.y, ahi[0], alo[0]);
            M::split(p10.x, p10.y, ahi[1], alo[1]);
            M::split(p01.x, p01.y, ahi[2], alo[2]);
            M::split(p11.x, p11.y, ahi[3], alo[3]);
#pragma unroll
            for (int nbp = 0; nbp < NBD / 2; ++nbp) {
                uint32_t b[4];
                const int mi = lane >> 3, r = lane & 7;
                ldmatrix_x4_trans(b, tile + (ks * 16 + (mi & 1) * 8 + r) * ROWH + wn * (D / WN) + nbp * 16 + (mi >> 1) * 8);
                M::run(oacc[2 * nbp], ahi, b[0], b[1]);
                M::run(oacc[2 * nbp], alo, b[0], b[1]);
                M::run(oacc[2 * nbp + 1], ahi, b[2], b[3]);
                M::run(oacc[2 * nbp + 1], alo, b[2], b[3]);
            }
        }
        __syncthreads();      // tile consumed before the next prefetch overwrites the other buffer's partner
    }
    cp_async_wait<0>();
    if (p.out) {
#pragma unroll
        for (int nb = 0; nb < NBD; ++nb) {
#pragma unroll
            for (int hrow = 0; hrow < 2; ++hrow) {
                const int i = wm * 16 + (lane >> 2) + hrow * 8;
                if (i < c) {
                    const float inv = 1.f / rowL[i];
                    const int col = wn * (D / WN) + nb * 8 + (lane & 3) * 2;
                    float2 o2 = make_float2(oacc[nb][2 * hrow] * inv, oacc[nb][2 * hrow + 1] * inv);
                    *reinterpret_cast<float2 *>(p.out + ((size_t)(qoff + i) * p.Utot + u) * D + col) = o2;
                }
            }
        }
    }
    }   // !RECOUNT
}

template <int DT, int CQ, bool RECOUNT>
cudaError_t launch_chunk(const ChunkParams &p, cudaStream_t s) {
    const size_t smem = sizeof(uint16_t) * (size_t)(CQ + 2 * KT) * ROWH + sizeof(float) * ((size_t)CQ * p.SS + 2 * CQ) + sizeof(int) * (size_t)p.SS;
    auto kern = sh_prefill_chunk_kernel<DT, CQ, RECOUNT>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const unsigned gy = (unsigned)(((RECOUNT ? p.nsteps : p.c) + CQ - 1) / CQ);
    kern<<<dim3(p.U, gy, 1), NTHREADS, smem, s>>>(p);
    return cudaGetLastError();
}

int s_stride(int B) { return ((B + KT - 1) / KT) * KT + 8; }
size_t smem_need(int CQ, int B) {
    return sizeof(uint16_t) * (size_t)(CQ + 2 * KT) * ROWH + sizeof(float) * ((size_t)CQ * s_stride(B) + 2 * CQ) + sizeof(int) * (size_t)s_stride(B);
}

}  // namespace

// Largest number of tokens one chunk launch can take for this handle (0: not supported).
// Does the CUDA-core chunk kernel serve this handle?  It takes what the tensor-core kernels do not (fp32 rows,
// head_dim 64), and everything when SH_OPT_PREFILL_CHUNK = 4 asks for it.
static bool use_simt(const sh_context *c) { return c->prefill_chunk == 4 || c->D != 128 || c->dtype == SH_F32; }

int sh_prefill_chunk_capacity(const sh_context *c) {
    if (use_simt(c)) return sh_chunk_simt_capacity() < c->w ? sh_chunk_simt_capacity() : c->w;
    if (c->dtype == SH_INT4_G64_F16) {       // int4 store: the tcgen05 kernel only
        if (c->prefill_chunk == 2) return 0;
        return sh_chunk_umma_capacity() < c->w ? sh_chunk_umma_capacity() : c->w;
    }
    if (c->dtype != SH_F16 && c->dtype != SH_BF16) return 0;
    int cq = 0;
    if (c->prefill_chunk == 1) cq = sh_chunk_umma_tma_capacity();      // persistent tcgen05 kernel: any budget, up to 128 tokens
    else if (c->prefill_chunk != 2) cq = sh_chunk_umma_capacity();     // tcgen05 kernel with one CTA per unit: any budget
    else if (smem_need(32, c->B) <= 200 * 1024) cq = 64;          // warp-level kernel: one or two CTAs of 32 queries, or one of 64
    if (cq > c->w) cq = c->w;     // every step of a chunk needs its own bit-plane row
    return cq;
}

// The recount (record recomputed at compression time): any budget on the tcgen05 kernel; the warp-level
// kernel keeps a whole row of logits in shared memory (budgets up to about 700).
bool sh_recount_supported(const sh_context *c) {
    if (use_simt(c)) return true;
    if (c->dtype == SH_INT4_G64_F16) return c->prefill_chunk != 2;      // int4 store: the tcgen05 kernel only
    if (c->dtype != SH_F16 && c->dtype != SH_BF16) return false;
    return c->prefill_chunk != 2 || smem_need(32, c->B) <= 200 * 1024;
}

// Steps t0+1 .. t0+count (count <= capacity, n0 + count <= B) in one launch.
cudaError_t sh_launch_prefill_chunk(const sh_context *c, const void *q, const void *k, const void *v, float *out,
                                    int count, cudaStream_t s, long long *launches) {
    ChunkParams p = {};
    p.q = static_cast<const char *>(q); p.k = static_cast<const char *>(k); p.v = static_cast<const char *>(v);
    p.out = out;
    p.K = sh_pK(c); p.V = sh_pV(c);
    p.Ks = sh_pKs(c); p.Vs = sh_pVs(c); p.Bs = c->Bs;
    p.hist = sh_phist(c);
    p.pos = sh_ppos(c);
    p.U = c->ucount; p.Utot = c->U; p.B = c->B; p.Bw = c->Bw; p.w = c->w;
    p.n0 = c->n; p.c = count; p.t0 = (int)c->t;
    p.SS = s_stride(c->B);
    p.scale_log2e = (float)((double)c->scale * 1.4426950408889634);
    p.qring = sh_pqring(c);
    p.err = reinterpret_cast<int *>(c->slab + c->L.err);
    p.selftest_skip_tile = c->selftest_skip_tile;
    cudaError_t e = cudaErrorInvalidValue;
    if (count < 1 || count > sh_prefill_chunk_capacity(c)) return e;
    if (use_simt(c)) {
        e = sh_launch_chunk_simt(p, c->dtype, c->D, s);
        if (e == cudaSuccess) *launches += 1;
        return e;
    }
    if (c->dtype == SH_INT4_G64_F16) {
        e = sh_launch_chunk_umma_int4(p, s);
        if (e == cudaSuccess) *launches += 1;
        return e;
    }
    if (c->prefill_chunk != 2) {
        int nl = 0;
        e = c->prefill_chunk == 1 ? sh_launch_chunk_umma_tma(p, c->dtype, s, &nl) : cudaErrorNotSupported;
        if (e == cudaSuccess) {
            *launches += nl;
            return e;
        }
        if (e == cudaErrorNotSupported) {       // option 3, or a driver without the tensor-map encoder: the per-unit tcgen05 kernel,
            (void)cudaGetLastError();           // which takes 64 tokens at a time (the steps of a chunk are consecutive: it splits)
            const int cap = sh_chunk_umma_capacity();
            e = cudaSuccess;
            for (int done = 0; done < count && e == cudaSuccess; done += cap) {
                ChunkParams part = p;
                const size_t skip = (size_t)done * c->U * c->D;       // elements of q, k, v and out before token `done`
                part.q = p.q + skip * 2; part.k = p.k + skip * 2; part.v = p.v + skip * 2;
                part.out = p.out ? p.out + skip : nullptr;
                part.n0 = p.n0 + done; part.t0 = p.t0 + done;
                part.c = count - done < cap ? count - done : cap;
                e = sh_launch_chunk_umma(part, c->dtype, s);
                if (e == cudaSuccess && done > 0) *launches += 1;
            }
        }
        if (e == cudaSuccess) *launches += 1;
        return e;
    }
    // 32 queries per CTA when two such CTAs fit on an SM (the second half of a longer chunk goes to a
    // sibling CTA that re-reads the keys): more warps in flight hide the latencies of this kernel better
    // than sharing the K/V tiles between 64 queries does
    const bool two_per_sm = smem_need(32, c->B) <= 112 * 1024;
    if (count <= 32 || two_per_sm || smem_need(64, c->B) > 200 * 1024)
        e = c->dtype == SH_F16 ? launch_chunk<SH_F16, 32, false>(p, s) : launch_chunk<SH_BF16, 32, false>(p, s);
    else e = c->dtype == SH_F16 ? launch_chunk<SH_F16, 64, false>(p, s) : launch_chunk<SH_BF16, 64, false>(p, s);
    if (e == cudaSuccess) *launches += 1;
    return e;
}

// The record of Algorithm 2 recomputed from the queries of the last w steps against the
// present cache: rewrites the unit's bit-plane rows of those steps.
cudaError_t sh_launch_recount(const sh_context *c, cudaStream_t s, long long *launches) {
    ChunkParams p = {};
    p.selftest_skip_tile = -1;
    p.K = sh_pK(c); p.V = sh_pV(c);
    p.hist = sh_phist(c);
    p.pos = sh_ppos(c);
    p.U = c->ucount; p.Utot = c->U; p.B = c->B; p.Bw = c->Bw; p.w = c->w;
    p.n0 = c->n; p.c = 0; p.t0 = (int)c->t;
    p.SS = s_stride(c->B);
    p.scale_log2e = (float)((double)c->scale * 1.4426950408889634);
    p.qring = sh_pqring(c);
    p.nsteps = c->t < c->w ? (int)c->t : c->w;
    p.first_step = (int)c->t - p.nsteps + 1;
    if (p.nsteps < 1) return cudaSuccess;
    p.err = reinterpret_cast<int *>(c->slab + c->L.err);
    p.Ks = sh_pKs(c); p.Vs = sh_pVs(c); p.Bs = c->Bs;
    cudaError_t e;
    if (use_simt(c)) {
        e = sh_launch_recount_simt(p, c->dtype, c->D, s);
        if (e == cudaSuccess) *launches += 1;
        return e;
    }
    if (c->dtype == SH_INT4_G64_F16) {
        e = sh_launch_recount_umma_int4(p, s);
        if (e == cudaSuccess) *launches += 1;
        return e;
    }
    if (c->prefill_chunk != 2) {
        e = c->prefill_chunk == 1 ? sh_launch_recount_umma_tma(p, c->dtype, s) : cudaErrorNotSupported;
        if (e == cudaErrorNotSupported) {
            (void)cudaGetLastError();
            e = sh_launch_recount_umma(p, c->dtype, s);
        }
        if (e == cudaSuccess) *launches += 1;
        return e;
    }
    if (smem_need(64, c->B) <= 200 * 1024) e = c->dtype == SH_F16 ? launch_chunk<SH_F16, 64, true>(p, s) : launch_chunk<SH_BF16, 64, true>(p, s);
    else e = c->dtype == SH_F16 ? launch_chunk<SH_F16, 32, true>(p, s) : launch_chunk<SH_BF16, 32, true>(p, s);
    if (e == cudaSuccess) *launches += 1;
    return e;
}
