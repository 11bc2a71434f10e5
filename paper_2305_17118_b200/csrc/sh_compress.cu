// Compression step (Algorithm 2): importance record from the bit-planes,
// select-m with a deterministic tie-break, and stable in-place compaction of
// K, V, scales, bit-planes and positions.  One CTA per unit for the selection,
// three CTAs per unit (K, V, record+positions) for the compaction.
#include "sh_internal.h"

namespace {

constexpr int SEL_THREADS = 256;
constexpr int CMP_THREADS = 256;

// Exclusive prefix count of a per-thread flag over the CTA.  `wsum` is shared
// scratch of >= 32 ints.  Returns this thread's rank; total in *total.
__device__ __forceinline__ int block_flag_scan(bool flag, int *wsum, int *total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const uint32_t b = __ballot_sync(0xffffffffu, flag);
    const int in_warp = __popc(b & ((1u << lane) - 1u));
    __syncthreads();                 // wsum free for reuse
    if (lane == 0) wsum[warp] = __popc(b);
    __syncthreads();
    int before = 0, tot = 0;
    for (int i = 0; i < nw; ++i) {
        const int v = wsum[i];
        if (i < warp) before += v;
        tot += v;
    }
    *total = tot;
    return before + in_warp;
}

// I_j = number of set bits of slot j over the w bit-plane rows of its unit.
__device__ __forceinline__ int slot_counter(const uint32_t *hist_u, int w, int Bw, int j) {
    const uint32_t *col = hist_u + (j >> 5);
    const int sh = j & 31;
    int cnt = 0;
    for (int s = 0; s < w; ++s) cnt += (col[(size_t)s * Bw] >> sh) & 1u;
    return cnt;
}

// Selection: among slots [0, n-r) drop the m with the largest key
// (counter descending, slot ascending).  Radix-select on the counter value by
// a shared-memory histogram, then an exact prefix count in slot order inside
// the tie class at the cut.
template <bool FROM_HIST>
__global__ void __launch_bounds__(SEL_THREADS) sh_select_kernel(const SelectParams p) {
    extern __shared__ int sm[];
    int *cnt_sh = sm;                      // [n]
    int *bins = cnt_sh + p.n;              // [cmax + 1]
    int *wsum = bins + (p.cmax + 1);       // [32]
    int *cut = wsum + 32;                  // [2] = {cstar, need}
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    const int n = p.n, ncand = p.n - p.r, m = p.m;

    for (int i = tid; i <= p.cmax; i += SEL_THREADS) bins[i] = 0;
    for (int j = tid; j < n; j += SEL_THREADS) {
        int I;
        if (FROM_HIST) I = slot_counter(p.hist + (size_t)u * p.w * p.Bw, p.w, p.Bw, j);
        else I = min((int)p.counters[(size_t)u * n + j], p.cmax);
        cnt_sh[j] = I;
    }
    __syncthreads();
    for (int j = tid; j < ncand; j += SEL_THREADS) atomicAdd(&bins[cnt_sh[j]], 1);
    __syncthreads();

    // Cut: largest c with #{I >= c} >= m.  Warp 0 scans the bins from the top, 32 at a time.
    if (tid < 32) {
        int above = 0;   // candidates with a counter beyond the 32 bins under inspection
        for (int base = p.cmax; base >= 0; base -= 32) {
            const int cidx = base - lane;
            const int v = cidx >= 0 ? bins[cidx] : 0;
            int incl = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int x = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += x;
            }
            const uint32_t hit = __ballot_sync(0xffffffffu, above + incl >= m);
            if (hit) {
                const int f = __ffs(hit) - 1;
                if (lane == f) {
                    cut[0] = cidx;
                    cut[1] = m - (above + incl - v);   // how many of the tie class go
                }
                break;
            }
            above += __shfl_sync(0xffffffffu, incl, 31);
        }
    }
    __syncthreads();
    const int cstar = cut[0], need = cut[1];

    int tie_carry = 0, keep_carry = 0, ev_carry = 0;
    for (int j0 = 0; j0 < n; j0 += SEL_THREADS) {
        const int j = j0 + tid;
        const int I = j < n ? cnt_sh[j] : -1;
        const bool cand = j < ncand;
        const bool tie = cand && I == cstar;
        int tot;
        const int tie_rank = tie_carry + block_flag_scan(tie, wsum, &tot);
        tie_carry += tot;
        const bool ev = cand && (I > cstar || (tie && tie_rank < need));
        const bool keep = j < n && !ev;
        const int dst = keep_carry + block_flag_scan(keep, wsum, &tot);
        keep_carry += tot;
        const int eidx = ev_carry + block_flag_scan(ev, wsum, &tot);
        ev_carry += tot;
        if (keep && p.src_idx) p.src_idx[(size_t)u * p.B + dst] = j;
        if (ev && p.evicted) p.evicted[(size_t)u * m + eidx] = j;
    }
}

// Rows of `row_bytes` (a multiple of 16) moved dst <- src_idx[dst] for dst in
// [0, n_keep).  Destinations never exceed their sources and sources increase
// with the destination, so batches in ascending order with all reads of a batch
// before its writes never overwrite a row that is still needed.
__device__ void compact_rows(char *base, const int32_t *src, int n_keep, int row_bytes) {
    constexpr int RR = 4;
    const int lpr = row_bytes >> 4;                 // 16-byte chunks per row
    const int rpp = CMP_THREADS / lpr;              // rows per pass
    const int row_in_pass = threadIdx.x / lpr, ch = threadIdx.x % lpr;
    const bool active = row_in_pass < rpp;
    for (int b = 0; b < n_keep; b += rpp * RR) {
        uint4 v[RR];
        int sj[RR];
#pragma unroll
        for (int i = 0; i < RR; ++i) {
            const int dst = b + i * rpp + row_in_pass;
            sj[i] = -1;
            if (active && dst < n_keep) {
                const int s = src[dst];
                if (s != dst) {
                    sj[i] = s;
                    v[i] = *reinterpret_cast<const uint4 *>(base + (size_t)s * row_bytes + ch * 16);
                }
            }
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < RR; ++i) {
            const int dst = b + i * rpp + row_in_pass;
            if (sj[i] >= 0) *reinterpret_cast<uint4 *>(base + (size_t)dst * row_bytes + ch * 16) = v[i];
        }
    }
}

// Same for small per-slot items (positions, int4 scales); slots [n_keep, n) get `fill`.
template <typename T>
__device__ void compact_items(T *base, const int32_t *src, int n_keep, int n, T fill) {
    for (int b = 0; b < n; b += CMP_THREADS) {
        const int dst = b + threadIdx.x;
        T val = fill;
        if (dst < n_keep) val = base[src[dst]];
        __syncthreads();
        if (dst < n) base[dst] = val;
    }
}

// Bit-planes: every row (one past step) is gathered through src_idx.  A warp
// owns a row: it stages the row's words in shared memory, then writes the
// gathered words; bits of the freed slots become 0.
__device__ void compact_hist(uint32_t *hist_u, const int32_t *src, int n_keep, int w, int Bw, uint32_t *stage) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = CMP_THREADS / 32;
    uint32_t *st = stage + warp * Bw;
    for (int s = warp; s < w; s += nw) {
        uint32_t *row = hist_u + (size_t)s * Bw;
        for (int k = lane; k < Bw; k += 32) st[k] = row[k];
        __syncwarp();
        for (int k = 0; k < Bw; ++k) {
            const int dst = (k << 5) + lane;
            bool bit = false;
            if (dst < n_keep) {
                const int sj = src[dst];
                bit = (st[sj >> 5] >> (sj & 31)) & 1u;
            }
            const uint32_t word = __ballot_sync(0xffffffffu, bit);
            if (lane == 0) row[k] = word;
        }
        __syncwarp();
    }
}

__global__ void __launch_bounds__(CMP_THREADS) sh_compact_kernel(const CompactParams p) {
    extern __shared__ uint32_t stage[];
    const int u = blockIdx.x, what = blockIdx.y;
    const int n_keep = p.n - p.m;
    const int32_t *src = p.src_idx + (size_t)u * p.B;
    if (what == 0 || what == 1) {
        char *rows = (what == 0 ? p.K : p.V) + (size_t)u * p.B * p.row_bytes;
        compact_rows(rows, src, n_keep, p.row_bytes);
        if (p.scale_bytes == 4) {
            uint32_t *sc = reinterpret_cast<uint32_t *>(what == 0 ? p.Ks : p.Vs) + (size_t)u * p.B;
            compact_items<uint32_t>(sc, src, n_keep, p.n, 0u);
        } else if (p.scale_bytes == 2) {
            uint16_t *sc = reinterpret_cast<uint16_t *>(what == 0 ? p.Ks : p.Vs) + (size_t)u * p.B;
            compact_items<uint16_t>(sc, src, n_keep, p.n, (uint16_t)0);
        }
    } else {
        compact_hist(p.hist + (size_t)u * p.w * p.Bw, src, n_keep, p.w, p.Bw, stage);
        compact_items<int32_t>(p.pos + (size_t)u * p.B, src, n_keep, p.n, 0);
    }
}

__global__ void __launch_bounds__(256) sh_counters_kernel(const uint32_t *hist, uint16_t *counters, int B, int Bw,
                                                          int w, int n) {
    const int u = blockIdx.x;
    for (int j = threadIdx.x; j < B; j += blockDim.x) {
        int I = 0;
        if (j < n) I = slot_counter(hist + (size_t)u * w * Bw, w, Bw, j);
        counters[(size_t)u * B + j] = (uint16_t)I;
    }
}

}  // namespace

cudaError_t sh_launch_select(const SelectParams &p, bool from_hist, cudaStream_t s, long long *launches) {
    const size_t smem = sizeof(int) * ((size_t)p.n + p.cmax + 1 + 32 + 2);
    cudaError_t e;
    if (from_hist) {
        if (smem > 48 * 1024) {
            e = cudaFuncSetAttribute(sh_select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
        }
        sh_select_kernel<true><<<p.U, SEL_THREADS, smem, s>>>(p);
    } else {
        if (smem > 48 * 1024) {
            e = cudaFuncSetAttribute(sh_select_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
        }
        sh_select_kernel<false><<<p.U, SEL_THREADS, smem, s>>>(p);
    }
    e = cudaGetLastError();
    if (e == cudaSuccess && launches) *launches += 1;
    return e;
}

cudaError_t sh_launch_compact(const CompactParams &p, cudaStream_t s, long long *launches) {
    const size_t smem = sizeof(uint32_t) * (size_t)(CMP_THREADS / 32) * p.Bw;
    sh_compact_kernel<<<dim3(p.U, 3, 1), CMP_THREADS, smem, s>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess && launches) *launches += 1;
    return e;
}

cudaError_t sh_launch_counters(const uint32_t *hist, uint16_t *counters, int U, int B, int Bw, int w, int n,
                               cudaStream_t s, long long *launches) {
    sh_counters_kernel<<<U, 256, 0, s>>>(hist, counters, B, Bw, w, n);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess && launches) *launches += 1;
    return e;
}
