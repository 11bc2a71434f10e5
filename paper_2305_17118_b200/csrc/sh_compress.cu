// Compression step (Algorithm 2): importance record from the bit-planes,
// select-m with a deterministic tie-break, and stable in-place compaction of
// K, V, scales, bit-planes and positions.  One CTA per unit for the selection;
// the compaction is two kernels: K/V rows through bulk asynchronous copies
// (two CTAs per unit), and record bit-planes + positions (one CTA per unit).
#include "sh_async.cuh"
#include "sh_internal.h"

namespace {

constexpr int SEL_THREADS = 128;
constexpr int CMP_THREADS = 256;
constexpr int SEL_TIE_CAP = 1024;     // tie classes up to this size are searched from a shared-memory list

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

// Three flags at once: ranks and totals packed 10 bits each (a CTA of at most 1023 threads), one barrier pair.
__device__ __forceinline__ int block_flag_scan3(bool a, bool b, bool c, int *wsum, int *total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const uint32_t lt = (1u << lane) - 1u;
    const uint32_t ba = __ballot_sync(0xffffffffu, a), bb = __ballot_sync(0xffffffffu, b), bc = __ballot_sync(0xffffffffu, c);
    const int in_warp = __popc(ba & lt) | (__popc(bb & lt) << 10) | (__popc(bc & lt) << 20);
    __syncthreads();                 // wsum free for reuse
    if (lane == 0) wsum[warp] = __popc(ba) | (__popc(bb) << 10) | (__popc(bc) << 20);
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
#pragma unroll 8
    for (int s = 0; s < w; ++s) cnt += (col[s * Bw] >> sh) & 1u;
    return cnt;
}

// Bit compress of one word (keep the bits under mask m, squeezed to the right) with the five
// butterfly masks of the classic network, which depend on m alone.
__device__ __forceinline__ uint32_t compress_bits(uint32_t x, uint32_t m, const uint32_t *mv) {
    x &= m;
#pragma unroll
    for (int i = 0; i < 5; ++i) {
        const uint32_t t = x & mv[i];
        x = (x ^ t) | (t >> (1 << i));
    }
    return x;
}

// Inverse of compress_bits: the low popc(m) bits of x spread to the set bits of m (same masks, reverse order).
__device__ __forceinline__ uint32_t expand_bits(uint32_t x, uint32_t m, const uint32_t *mv) {
#pragma unroll
    for (int i = 4; i >= 0; --i) {
        const uint32_t t = x << (1 << i);
        x = (x & ~mv[i]) | (t & mv[i]);
    }
    return x & m;
}

__device__ __forceinline__ void compress_masks(uint32_t m, uint32_t *mv_out) {
    uint32_t mk = ~m << 1;
#pragma unroll
    for (int i = 0; i < 5; ++i) {
        uint32_t mp = mk ^ (mk << 1);
        mp ^= mp << 2; mp ^= mp << 4; mp ^= mp << 8; mp ^= mp << 16;
        const uint32_t mv = mp & m;
        mv_out[i] = mv;
        m = (m ^ mv) | (mv >> (1 << i));
        mk &= ~mp;
    }
}

// Unordered compaction, record part.  Per-word masks of the holes (slots below n - m that were dropped)
// and of the fillers (kept slots at or beyond n - m), their butterfly masks, and the number of holes
// before each word.  hmask..fmv: shared arrays of Bw, Bw, Bw, 5 Bw, 5 Bw words.  Ends with a barrier.
template <class HoleOf, class FillerOf>
__device__ __forceinline__ void build_fill_masks(HoleOf hole_of, FillerOf filler_of, int h, int Bw, uint32_t *hmask,
                                                 uint32_t *fmask, uint32_t *hoff, uint32_t *hmv, uint32_t *fmv,
                                                 int n_keep, int n, int *err) {
    const int tid = threadIdx.x, nt = blockDim.x;
    for (int k = tid; k < Bw; k += nt) { hmask[k] = 0; fmask[k] = 0; }
    __syncthreads();
    for (int k = tid; k < h; k += nt) {
        const int d = hole_of(k), sj = filler_of(k);
        if (!SH_BOUNDS_OK(d >= 0 && d < n_keep && sj >= n_keep && sj < n, err, 0x711)) continue;
        atomicOr(&hmask[d >> 5], 1u << (d & 31));
        atomicOr(&fmask[sj >> 5], 1u << (sj & 31));
    }
    __syncthreads();
    for (int k = tid; k < Bw; k += nt) {
        compress_masks(hmask[k], hmv + k * 5);
        compress_masks(fmask[k], fmv + k * 5);
    }
    if (tid == 0) {
        uint32_t run = 0;
        for (int k = 0; k < Bw; ++k) { hoff[k] = run; run += __popc(hmask[k]); }
    }
    __syncthreads();
}

// In every one of the nr staged bit-plane rows (row stride `stride` words, one thread per row) the
// fillers' bits, taken in slot order, go to the holes in slot order: the tail words are compressed by the
// filler mask into a bit stream (written over the tail, which is dead afterwards), each head word takes
// its share of the stream expanded to its holes, and the bits from n_keep on are cleared.
__device__ __forceinline__ void fill_record_rows(uint32_t *rows_sh, int stride, int nr, int n, int n_keep, int Bw,
                                                 const uint32_t *hmask, const uint32_t *fmask, const uint32_t *hoff,
                                                 const uint32_t *hmv, const uint32_t *fmv) {
    const int k0 = n_keep >> 5, k_end = (n + 31) >> 5;         // tail words: [k0, k_end)
    const uint32_t low0 = (n_keep & 31) ? ((1u << (n_keep & 31)) - 1u) : 0u;   // head bits of word k0
    for (int r = threadIdx.x; r < nr; r += blockDim.x) {
        uint32_t *rw = rows_sh + r * stride;
        const uint32_t saved0 = rw[k0] & low0;
        unsigned long long acc = 0;
        int fill = 0, o = k0;
        for (int k = k0; k < k_end; ++k) {
            const uint32_t mk = fmask[k];
            const uint32_t c = compress_bits(rw[k], mk, fmv + k * 5);
            acc |= (unsigned long long)c << fill;
            fill += __popc(mk);
            if (fill >= 32) {
                rw[o++] = (uint32_t)acc;      // o <= k: the word was already consumed
                acc >>= 32;
                fill -= 32;
            }
        }
        if (o < Bw) rw[o] = (uint32_t)acc;
        const int head_words = low0 ? k0 + 1 : k0;
        for (int wd = 0; wd < head_words; ++wd) {
            const uint32_t hm = hmask[wd];
            uint32_t val = (wd == k0) ? saved0 : rw[wd];
            if (hm) {
                const int off = hoff[wd], sw = k0 + (off >> 5), sb = off & 31;
                const uint32_t lo = rw[sw], hi = (sw + 1 < Bw) ? rw[sw + 1] : 0u;
                const uint32_t bits = __funnelshift_r(lo, hi, sb);          // stream bits off .. off+31
                val = (val & ~hm) | expand_bits(bits, hm, hmv + wd * 5);
            }
            if (wd == k0) val &= low0;
            rw[wd] = val;               // word k0 comes last: the stream's first word is no longer needed
        }
        for (int wd = head_words; wd < Bw; ++wd) rw[wd] = 0;
    }
}

// K and V rows (and int4 scales) of the h moves of one unit: hole <- filler.  Sources and destinations
// are disjoint.  Four independent 16-byte pieces per thread are in flight: the loads of a batch are
// issued before its stores.  what: 0 = K, 1 = V, 2 = both.
template <class HoleOf, class FillerOf>
__device__ __forceinline__ void fill_rows(const CompactParams &p, int u, int what, int h, HoleOf hole_of, FillerOf filler_of) {
    const int tid = threadIdx.x, nt = blockDim.x;
    const int lpr = p.row_bytes >> 4, lsh = __ffs(lpr) - 1;     // 16-byte chunks per row: a power of two
    const int per = h * lpr, first = what == 1 ? per : 0, last = what == 0 ? per : 2 * per;
    char *Kr = p.K + (size_t)u * p.B * p.row_bytes, *Vr = p.V + (size_t)u * p.B * p.row_bytes;
    for (int base = first + tid; base < last; base += 4 * nt) {
        uint4 val[4];
        char *dst[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int idx = base + i * nt;
            dst[i] = nullptr;
            if (idx < last) {
                char *rows = idx >= per ? Vr : Kr;
                const int rem = idx >= per ? idx - per : idx;
                const int k = rem >> lsh, ch = rem & (lpr - 1);
                if (!SH_BOUNDS_OK(hole_of(k) >= 0 && hole_of(k) < p.n - p.m && filler_of(k) >= p.n - p.m && filler_of(k) < p.n, p.err, 0x712)) continue;
                dst[i] = rows + (size_t)hole_of(k) * p.row_bytes + ch * 16;
                val[i] = *reinterpret_cast<const uint4 *>(rows + (size_t)filler_of(k) * p.row_bytes + ch * 16);
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (dst[i]) *reinterpret_cast<uint4 *>(dst[i]) = val[i];
    }
    for (int side = (what == 1 ? 1 : 0); side <= (what == 0 ? 0 : 1); ++side) {
        if (p.scale_bytes == 4) {
            uint32_t *sc = reinterpret_cast<uint32_t *>(side == 0 ? p.Ks : p.Vs) + (size_t)u * p.Bs;
            for (int k = tid; k < h; k += nt) sc[hole_of(k)] = sc[filler_of(k)];
        } else if (p.scale_bytes == 2) {
            uint16_t *sc = reinterpret_cast<uint16_t *>(side == 0 ? p.Ks : p.Vs) + (size_t)u * p.Bs;
            for (int k = tid; k < h; k += nt) sc[hole_of(k)] = sc[filler_of(k)];
        }
    }
}

// Positions of the h moves of one unit, then the freed tail is zeroed and the unit's row count updated.
template <class HoleOf, class FillerOf>
__device__ __forceinline__ void fill_positions(const CompactParams &p, int u, int h, HoleOf hole_of, FillerOf filler_of) {
    const int tid = threadIdx.x, nt = blockDim.x, n_keep = p.n - p.m;
    int32_t *pos = p.pos + (size_t)u * p.B;
    for (int k = tid; k < h; k += nt)
        if (SH_BOUNDS_OK(hole_of(k) >= 0 && hole_of(k) < n_keep && filler_of(k) >= n_keep && filler_of(k) < p.n, p.err, 0x713))
            pos[hole_of(k)] = pos[filler_of(k)];
    __syncthreads();                                 // every filler is read before the tail is zeroed
    for (int j = n_keep + tid; j < p.n; j += nt) pos[j] = 0;
    if (p.n_arr && tid == 0) p.n_arr[u] = n_keep;    // the unit is compacted
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
    int *cut = wsum + 32;                  // [8] = {cstar, need, size of the tie class, pstar, tie list fill}
    int *tie_list = cut + 8;               // [SEL_TIE_CAP] positions of the tie class (unordered mode only)
    uint32_t *planes = reinterpret_cast<uint32_t *>(tie_list + (p.unordered ? SEL_TIE_CAP : 0));   // [w * Bw] when staged, then [G][5][Bw] partial sums
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    const int n = p.n, ncand = p.n - p.r, m = p.m;
    if (p.n_arr && p.n_arr[u] != n) {            // this unit's cache is not full (whole CTA leaves)
        if (tid == 0 && p.unordered && p.n_moves) p.n_moves[(size_t)u * p.B] = 0;   // tells the move kernel to skip it too
        return;
    }

    if (!SH_BOUNDS_OK(n >= 1 && n <= p.B && m >= 1 && m <= n - p.r, p.err, 0x717)) return;
    for (int i = tid; i <= p.cmax; i += SEL_THREADS) bins[i] = 0;
    if (FROM_HIST) {
        const uint32_t *hist_u = p.hist + (size_t)u * p.w * p.Bw;
        if (p.stage_planes) {
            // One coalesced pass brings the unit's bit-planes to shared memory.  Then the
            // rows are summed 32 slots at a time: thread (g, k) adds rows g, g+G, ... of
            // word column k into a 5-plane bit-sliced counter (at most 31 rows each), and
            // every slot finally picks its bits out of the G partial counters.
            // (the fused path works on the staged rows later, one thread per row: odd row stride there)
            const int Bw = p.Bw, w = p.w, G = (w + 30) / 31, pst = p.fuse ? (Bw | 1) : Bw;
            if (pst != Bw) {
                for (int i = tid; i < w * Bw; i += SEL_THREADS) {
                    const int rr = Bw > 1 ? (int)__umulhi((uint32_t)i, p.bw_magic) : i;      // i / Bw
                    planes[rr * pst + (i - rr * Bw)] = hist_u[i];
                }
            } else {
                for (int i = tid; i < w * Bw; i += SEL_THREADS) planes[i] = hist_u[i];
            }
            __syncthreads();
            uint32_t *part = planes + w * pst;
            for (int item = tid; item < G * Bw; item += SEL_THREADS) {
                const int g = item / Bw, k = item % Bw;
                uint32_t c0 = 0, c1 = 0, c2 = 0, c3 = 0, c4 = 0;
                for (int s = g; s < w; s += G) {
                    uint32_t x = planes[s * pst + k], t;
                    t = c0 & x; c0 ^= x; x = t;
                    t = c1 & x; c1 ^= x; x = t;
                    t = c2 & x; c2 ^= x; x = t;
                    t = c3 & x; c3 ^= x; x = t;
                    c4 ^= x;
                }
                uint32_t *o = part + (size_t)g * 5 * Bw + k;
                o[0] = c0; o[Bw] = c1; o[2 * Bw] = c2; o[3 * Bw] = c3; o[4 * Bw] = c4;
            }
            __syncthreads();
            for (int j = tid; j < n; j += SEL_THREADS) {
                const uint32_t *col = part + (j >> 5);
                const int sh = j & 31;
                int cnt = 0;
                for (int g = 0; g < G; ++g) {
#pragma unroll
                    for (int pl = 0; pl < 5; ++pl) cnt += ((col[(g * 5 + pl) * Bw] >> sh) & 1u) << pl;
                }
                cnt_sh[j] = cnt;
            }
        } else {
            for (int j = tid; j < n; j += SEL_THREADS) cnt_sh[j] = slot_counter(hist_u, p.w, p.Bw, j);
        }
    } else {
        for (int j = tid; j < n; j += SEL_THREADS) cnt_sh[j] = min((int)p.counters[(size_t)u * n + j], p.cmax);
    }
    __syncthreads();
    // Candidates: everything but the r most recent tokens.  With position-sorted slots those are the
    // last r slots; otherwise the positions say (one token per step: the r newest have pos > t - r).
    const int32_t *pos_u = p.unordered ? p.pos + (size_t)u * p.B : nullptr;
    const int t_cut = p.unordered ? (p.t_arr ? p.t_arr[u] : p.t) - p.r : 0;
    auto is_cand = [&](int j) { return p.unordered ? (j < n && pos_u[j] <= t_cut) : j < ncand; };
    if (p.unordered && p.fuse && m == 1) {
        // Steady state with one token dropped per step: the candidate with the largest counter goes,
        // the oldest among equals; the newest row takes its slot.  No histogram, no lists, no bit
        // networks: a block-wide maximum of (counter, -position), one row pair to move, and in every
        // bit-plane row one bit to carry from the last slot to the freed one.
        unsigned long long key = 0;                       // 0: no candidate seen
        for (int j = tid; j < n; j += SEL_THREADS)
            if (is_cand(j)) {
                const unsigned long long kj = ((unsigned long long)(cnt_sh[j] + 1) << 32) | (uint32_t)(0x7fffffff - pos_u[j]);
                key = kj > key ? kj : key;
            }
        unsigned long long best = key;
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
            best = other > best ? other : best;
        }
        if (lane == 0) {                                  // per-warp maxima as two words each in the scan scratch
            wsum[tid >> 5] = (int)(uint32_t)(best >> 32);
            wsum[16 + (tid >> 5)] = (int)(uint32_t)best;
        }
        __syncthreads();
        best = 0;
        for (int i = 0; i < SEL_THREADS / 32; ++i) {
            const unsigned long long bi = ((unsigned long long)(uint32_t)wsum[i] << 32) | (uint32_t)wsum[16 + i];
            best = bi > best ? bi : best;
        }
        for (int j = tid; j < n; j += SEL_THREADS)
            if (is_cand(j) && (((unsigned long long)(cnt_sh[j] + 1) << 32) | (uint32_t)(0x7fffffff - pos_u[j])) == best) cut[0] = j;
        __syncthreads();
        const int hole = cut[0], last = n - 1;            // positions are unique: exactly one thread wrote
        const CompactParams &c = p.mv;
        if (tid == 0 && p.evicted) p.evicted[u] = hole;
        if (hole != last) {
            const int lpr = c.row_bytes >> 4;
            if (tid < 2 * lpr) {
                char *rows = (tid < lpr ? c.K : c.V) + (size_t)u * c.B * c.row_bytes;
                const int ch = tid < lpr ? tid : tid - lpr;
                *reinterpret_cast<uint4 *>(rows + (size_t)hole * c.row_bytes + ch * 16) =
                    *reinterpret_cast<const uint4 *>(rows + (size_t)last * c.row_bytes + ch * 16);
            }
            if (tid < 2 && c.scale_bytes) {
                char *sc = (tid == 0 ? c.Ks : c.Vs) + (size_t)u * c.Bs * c.scale_bytes;
                for (int b = 0; b < c.scale_bytes; ++b) sc[(size_t)hole * c.scale_bytes + b] = sc[(size_t)last * c.scale_bytes + b];
            }
        }
        {
            const int Bw = p.Bw, pst = Bw | 1;
            uint32_t *hist_w = c.hist + (size_t)u * p.w * Bw;
            for (int rr = tid; rr < p.w; rr += SEL_THREADS) {
                const uint32_t *rw = planes + rr * pst;
                const uint32_t bit = (rw[last >> 5] >> (last & 31)) & 1u;
                if ((hole >> 5) == (last >> 5)) {
                    uint32_t x = rw[last >> 5] & ~(1u << (last & 31));
                    if (hole != last) x = (x & ~(1u << (hole & 31))) | (bit << (hole & 31));
                    hist_w[(size_t)rr * Bw + (last >> 5)] = x;
                } else {
                    hist_w[(size_t)rr * Bw + (last >> 5)] = rw[last >> 5] & ~(1u << (last & 31));
                    hist_w[(size_t)rr * Bw + (hole >> 5)] = (rw[hole >> 5] & ~(1u << (hole & 31))) | (bit << (hole & 31));
                }
            }
        }
        if (tid == 0) {
            int32_t *pos_w = c.pos + (size_t)u * c.B;
            if (hole != last) pos_w[hole] = pos_w[last];
            pos_w[last] = 0;
            if (c.n_arr) c.n_arr[u] = n - 1;
        }
        return;
    }
    for (int j = tid; j < n; j += SEL_THREADS)
        if (is_cand(j)) atomicAdd(&bins[cnt_sh[j]], 1);
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
                    cut[2] = v;
                    cut[4] = 0;
                }
                break;
            }
            above += __shfl_sync(0xffffffffu, incl, 31);
        }
    }
    __syncthreads();
    const int cstar = cut[0], need = cut[1];

    if (p.unordered) {
        // Tie class at the cut: the `need` members with the smallest positions go.  Positions are unique
        // and at most t_cut, so a binary search on the position value finds the largest one that goes.
        const int tie_size = cut[2];
        int pstar = -1;
        if (need >= tie_size) {
            pstar = t_cut;                   // the whole class goes
        } else if (need > 0 && tie_size <= SEL_TIE_CAP) {
            // small class (the usual case): its positions are listed in shared memory and one warp searches
            for (int j = tid; j < n; j += SEL_THREADS)
                if (is_cand(j) && cnt_sh[j] == cstar) tie_list[atomicAdd(&cut[4], 1)] = pos_u[j];
            __syncthreads();
            if (tid < 32) {
                int lo = 0, hi = t_cut;      // smallest value with #{tie, pos <= value} >= need lies in (lo, hi]
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    int cntv = 0;
                    for (int i = lane; i < tie_size; i += 32) cntv += tie_list[i] <= mid;
                    cntv = __reduce_add_sync(0xffffffffu, cntv);
                    if (cntv >= need) hi = mid; else lo = mid;
                }
                if (lane == 0) cut[3] = hi;
            }
            __syncthreads();
            pstar = cut[3];
        } else if (need > 0) {
            int lo = 0, hi = t_cut;          // same search with block-wide counts over all slots
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                int cntv = 0;
                for (int j0 = 0; j0 < n; j0 += SEL_THREADS) {
                    const int j = j0 + tid;
                    const bool in = j < n && is_cand(j) && cnt_sh[j] == cstar && pos_u[j] <= mid;
                    cntv += __syncthreads_count(in);
                }
                if (cntv >= need) hi = mid; else lo = mid;
            }
            pstar = hi;
        }
        // Holes (dropped slots below n - m) are filled, in order, by the kept slots at or beyond n - m.
        const int n_keep = n - m;
        int hole_carry = 0, fill_carry = 0, ev_carry = 0;
        for (int j0 = 0; j0 < n; j0 += SEL_THREADS) {
            const int j = j0 + tid;
            const int I = j < n ? cnt_sh[j] : -1;
            const bool ev = j < n && is_cand(j) && (I > cstar || (I == cstar && pos_u[j] <= pstar));
            const bool hole = ev && j < n_keep, filler = j >= n_keep && j < n && !ev;
            int tot;
            const int rk = block_flag_scan3(hole, filler, ev, wsum, &tot);
            const int hk = hole_carry + (rk & 1023), fk = fill_carry + ((rk >> 10) & 1023), eidx = ev_carry + (rk >> 20);
            hole_carry += tot & 1023;
            fill_carry += (tot >> 10) & 1023;
            ev_carry += tot >> 20;
            // (ranks stay below m as long as the positions of a unit are distinct, which the library
            // maintains; the bounds keep a workspace restored from foreign data from writing out of range)
            if (p.fuse) {
                if (hole && hk < m) sm[p.fuse_off + hk] = j;
                if (filler && fk < m) sm[p.fuse_off + m + fk] = j;
            } else if (p.src_idx) {
                if (hole && hk < m) p.src_idx[(size_t)u * p.B + hk] = j;
                if (filler && fk < m) p.src_idx[(size_t)u * p.B + (p.B - 1 - fk)] = j;
            }
            if (ev && eidx < m && p.evicted) p.evicted[(size_t)u * m + eidx] = j;
        }
        hole_carry = min(min(hole_carry, fill_carry), m);
        if (!p.fuse) {
            if (tid == 0 && p.n_moves) p.n_moves[(size_t)u * p.B] = (uint16_t)(0x8000 | hole_carry);   // bit 15: unit selected
            return;
        }
        // Fused path: the move list stays in shared memory and this CTA carries the moves out.
        __syncthreads();
        const int h = hole_carry;
        const int *hole_sh = sm + p.fuse_off, *fill_sh = hole_sh + m;
        auto hole_of = [&](int k) { return hole_sh[k]; };
        auto filler_of = [&](int k) { return fill_sh[k]; };
        fill_rows(p.mv, u, 2, h, hole_of, filler_of);       // K and V rows: loads in flight during the record work
        {
            const int Bw = p.Bw, w = p.w, pst = Bw | 1;
            uint32_t *hmask = reinterpret_cast<uint32_t *>(sm + p.fuse_off + 2 * m);
            uint32_t *fmask = hmask + Bw, *hoff = fmask + Bw, *hmv = hoff + Bw, *fmv = hmv + 5 * Bw;
            build_fill_masks(hole_of, filler_of, h, Bw, hmask, fmask, hoff, hmv, fmv, n_keep, n, p.mv.err);
            fill_record_rows(planes, pst, w, n, n_keep, Bw, hmask, fmask, hoff, hmv, fmv);   // the rows staged for counting
            __syncthreads();
            uint32_t *hist_w = p.mv.hist + (size_t)u * w * Bw;
            if (pst != Bw) {
                for (int i = tid; i < w * Bw; i += SEL_THREADS) {
                    const int rr = (int)__umulhi((uint32_t)i, p.bw_magic);
                    hist_w[i] = planes[rr * pst + (i - rr * Bw)];
                }
            } else {
                for (int i = tid; i < w * Bw; i += SEL_THREADS) hist_w[i] = planes[i];
            }
        }
        fill_positions(p.mv, u, h, hole_of, filler_of);
        return;
    }
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
        const int rk = block_flag_scan3(keep, ev, false, wsum, &tot);
        const int dst = keep_carry + (rk & 1023), eidx = ev_carry + ((rk >> 10) & 1023);
        keep_carry += tot & 1023;
        ev_carry += (tot >> 10) & 1023;
        if (keep && p.src_idx) p.src_idx[(size_t)u * p.B + dst] = j;
        if (ev && p.evicted) p.evicted[(size_t)u * m + eidx] = j;
    }
}

// K or V rows of one unit, moved dst <- src_idx[dst] for dst in [0, n_keep).
// Destinations never exceed their sources and sources increase with the
// destination, so everything from the first moved row on can be handled in
// ascending chunks, each read completely before it is written.  A chunk is
// gathered into shared memory by bulk asynchronous copies (one per run of
// consecutive source rows, all counted on one mbarrier) and written back to its
// contiguous destination by a single bulk store.
constexpr int ROWS_THREADS = 128;

__global__ void __launch_bounds__(ROWS_THREADS) sh_compact_rows_kernel(const CompactParams p) {
    extern __shared__ __align__(128) unsigned char buf[];
    __shared__ __align__(8) uint64_t bar;
    __shared__ int first_moved;
    const int u = blockIdx.x, what = blockIdx.y, tid = threadIdx.x;
    const int n_keep = p.n - p.m, rb = p.row_bytes;
    if (p.n_arr && p.n_arr[u] != p.n) return;    // this unit's cache is not full (whole CTA leaves)
    const int32_t *src = p.src_idx + (size_t)u * p.B;
    char *rows = (what == 0 ? p.K : p.V) + (size_t)u * p.B * rb;

    if (tid == 0) {
        first_moved = n_keep;
        shasync::mbar_init(&bar, 1);
        shasync::fence_barrier_init();
    }
    __syncthreads();
    {
        int mine = n_keep;
        for (int d = tid; d < n_keep; d += ROWS_THREADS)
            if (src[d] != d) { mine = d; break; }
        if (mine < n_keep) atomicMin(&first_moved, mine);
    }
    __syncthreads();
    const int d0 = first_moved;
    const int chunk_rows = p.chunk_bytes / rb;
    uint32_t phase = 0;
    bool ok = true;
    for (int a = d0; a < n_keep && ok; a += chunk_rows) {
        const int b = min(n_keep, a + chunk_rows);
        if (tid == 0) shasync::mbar_arrive_expect_tx(&bar, (uint32_t)(b - a) * rb);
        __syncthreads();   // the expectation is posted before any copy can complete
        for (int d = a + tid; d < b; d += ROWS_THREADS) {
            const int s0 = src[d];
            if (d != a && src[d - 1] + 1 == s0) continue;        // inside someone else's run
            int len = 1;
            while (d + len < b && src[d + len] == s0 + len) ++len;
            // (bounds-checked build: a run out of range is replaced by the rows already at its destination, so the
            // barrier's byte count still holds and nothing out of range is read)
            const int s_ok = SH_BOUNDS_OK(s0 >= d && s0 + len <= p.n, p.err, 0x714) ? s0 : d;
            shasync::bulk_g2s(buf + (size_t)(d - a) * rb, rows + (size_t)s_ok * rb, (uint32_t)len * rb, &bar);
        }
        ok = __syncthreads_and(shasync::mbar_wait(&bar, phase, p.err, 1));   // uniform across the CTA
        phase ^= 1;
        if (tid == 0 && ok) {
            shasync::fence_async_shared();
            shasync::bulk_s2g(rows + (size_t)a * rb, buf, (uint32_t)(b - a) * rb);
            shasync::bulk_commit();
            shasync::bulk_wait_read_all();    // the buffer may be refilled
        }
        __syncthreads();
    }
    if (tid == 0) shasync::bulk_wait_all();

    // int4 group scales travel with their rows
    if (p.scale_bytes) {
        __syncthreads();
        if (p.scale_bytes == 4) {
            uint32_t *sc = reinterpret_cast<uint32_t *>(what == 0 ? p.Ks : p.Vs) + (size_t)u * p.Bs;
            for (int base = 0; base < p.n; base += ROWS_THREADS) {
                const int d = base + tid;
                uint32_t val = 0;
                if (d < n_keep && SH_BOUNDS_OK(src[d] >= d && src[d] < p.n, p.err, 0x716)) val = sc[src[d]];
                __syncthreads();
                if (d < p.n) sc[d] = val;
            }
        } else {
            uint16_t *sc = reinterpret_cast<uint16_t *>(what == 0 ? p.Ks : p.Vs) + (size_t)u * p.Bs;
            for (int base = 0; base < p.n; base += ROWS_THREADS) {
                const int d = base + tid;
                uint16_t val = 0;
                if (d < n_keep && SH_BOUNDS_OK(src[d] >= d && src[d] < p.n, p.err, 0x716)) val = sc[src[d]];
                __syncthreads();
                if (d < p.n) sc[d] = val;
            }
        }
    }
}

// Record bit-planes and positions of one unit.  Removing the dropped slots
// from a bit-plane row is a bit compress (keep the bits under a mask, squeezed
// to the right).  The mask is the same for all w rows, so the five butterfly
// masks of the classic compress network are computed once per 32-slot word and
// every row is then handled by one thread: 20 logic operations per source word
// plus a funnel shift into the output stream.  Bits of the freed slots become 0.
__global__ void __launch_bounds__(CMP_THREADS) sh_compact_record_kernel(const CompactParams p) {
    extern __shared__ uint32_t rec_sm[];
    const int u = blockIdx.x, tid = threadIdx.x;
    const int n_keep = p.n - p.m, Bw = p.Bw, w = p.w;
    if (p.n_arr && p.n_arr[u] != p.n) return;        // this unit's cache is not full (whole CTA leaves)
    const int stride = Bw | 1;                       // odd row stride: no bank conflicts
    const uint32_t bw_magic = p.bw_magic;
    auto row_of = [&](int i) { return Bw > 1 ? (int)__umulhi((uint32_t)i, bw_magic) : i; };   // i / Bw
    const int32_t *src = p.src_idx + (size_t)u * p.B;
    uint32_t *hist_u = p.hist + (size_t)u * w * Bw;
    uint32_t *keep = rec_sm;                         // [Bw] keep mask per source word
    uint32_t *mvs = keep + Bw;                       // [Bw][5] butterfly masks
    uint32_t *rows = mvs + 5 * Bw;                   // [p.rec_rows][stride] staged bit-plane rows

    for (int k = tid; k < Bw; k += CMP_THREADS) keep[k] = 0;
    __syncthreads();
    for (int d = tid; d < n_keep; d += CMP_THREADS) {
        const int sj = src[d];
        if (!SH_BOUNDS_OK(sj >= d && sj < p.n, p.err, 0x715)) continue;
        atomicOr(&keep[sj >> 5], 1u << (sj & 31));
    }
    __syncthreads();
    for (int k = tid; k < Bw; k += CMP_THREADS) {
        uint32_t m = keep[k], mk = ~m << 1;
#pragma unroll
        for (int i = 0; i < 5; ++i) {
            uint32_t mp = mk ^ (mk << 1);
            mp ^= mp << 2; mp ^= mp << 4; mp ^= mp << 8; mp ^= mp << 16;
            const uint32_t mv = mp & m;
            mvs[k * 5 + i] = mv;
            m = (m ^ mv) | (mv >> (1 << i));
            mk &= ~mp;
        }
    }
    __syncthreads();
    for (int s0 = 0; s0 < w; s0 += p.rec_rows) {
        const int nr = min(p.rec_rows, w - s0);
        for (int i = tid; i < nr * Bw; i += CMP_THREADS) { const int rr = row_of(i); rows[rr * stride + (i - rr * Bw)] = hist_u[(size_t)s0 * Bw + i]; }
        __syncthreads();
        for (int r = tid; r < nr; r += CMP_THREADS) {
            uint32_t *row = rows + r * stride;
            unsigned long long acc = 0;
            int fill = 0, o = 0;
            for (int k = 0; k < Bw; ++k) {
                const uint32_t m = keep[k];
                const uint32_t c = compress_bits(row[k], m, mvs + k * 5);
                acc |= (unsigned long long)c << fill;
                fill += __popc(m);
                if (fill >= 32) {
                    row[o++] = (uint32_t)acc;     // o <= k: the word was already consumed
                    acc >>= 32;
                    fill -= 32;
                }
            }
            if (o < Bw) row[o++] = (uint32_t)acc;
            for (; o < Bw; ++o) row[o] = 0;
        }
        __syncthreads();
        for (int i = tid; i < nr * Bw; i += CMP_THREADS) { const int rr = row_of(i); hist_u[(size_t)s0 * Bw + i] = rows[rr * stride + (i - rr * Bw)]; }
        __syncthreads();
    }
    // positions: read a batch, barrier, write it (destinations never pass sources)
    int32_t *pos = p.pos + (size_t)u * p.B;
    for (int base = 0; base < p.n; base += CMP_THREADS) {
        const int d = base + threadIdx.x;
        int32_t val = 0;
        if (d < n_keep && SH_BOUNDS_OK(src[d] >= d && src[d] < p.n, p.err, 0x715)) val = pos[src[d]];
        __syncthreads();
        if (d < p.n) pos[d] = val;
    }
    if (p.n_arr && tid == 0) p.n_arr[u] = n_keep;    // last kernel of the compression: the unit is compacted
}

// Unordered compaction: each hole takes the row of its filler.  Holes lie below n - m, fillers at or
// beyond it, so sources and destinations are disjoint and the moves are independent.  blockIdx.x % 3:
// 0 = K rows (+ int4 scales), 1 = V rows (+ scales), 2 = record bit-planes and positions.
__global__ void __launch_bounds__(CMP_THREADS) sh_fill_holes_kernel(const CompactParams p) {
    extern __shared__ uint32_t fh_sm[];
    // the three jobs of a unit sit next to each other in the grid: row traffic and the latency-bound
    // record work then overlap on every SM instead of running one after the other
    const int u = blockIdx.x / 3, what = blockIdx.x % 3, tid = threadIdx.x;
    // The selection kernel marked the units it handled (the three CTAs of a unit must agree, and the
    // third one updates the unit's row count, so that count cannot be the test here).
    const int marked = p.n_moves[(size_t)u * p.B];
    if (!(marked & 0x8000)) return;
    const int n_keep = p.n - p.m, h = marked & 0x7fff;
    const int32_t *row = p.src_idx + (size_t)u * p.B;
    auto hole_of = [&](int k) { return row[k]; };
    auto filler_of = [&](int k) { return row[p.B - 1 - k]; };
    if (what < 2) {
        fill_rows(p, u, what, h, hole_of, filler_of);
        return;
    }
    const int Bw = p.Bw, w = p.w, stride = Bw | 1;
    const uint32_t bw_magic = p.bw_magic;
    auto row_of = [&](int i) { return Bw > 1 ? (int)__umulhi((uint32_t)i, bw_magic) : i; };   // i / Bw
    uint32_t *hist_u = p.hist + (size_t)u * w * Bw;
    uint32_t *hmask = fh_sm;                 // [Bw] holes per word
    uint32_t *fmask = hmask + Bw;            // [Bw] fillers per word
    uint32_t *hoff = fmask + Bw;             // [Bw] holes before this word
    uint32_t *hmv = hoff + Bw;               // [Bw][5]
    uint32_t *fmv = hmv + 5 * Bw;            // [Bw][5]
    uint32_t *rows_sh = fmv + 5 * Bw;        // [p.rec_rows][stride]
    auto stage_rows = [&](int s0) {
        const int nr = min(p.rec_rows, w - s0);
        for (int i = tid; i < nr * Bw; i += CMP_THREADS) { const int rr = row_of(i); rows_sh[rr * stride + (i - rr * Bw)] = hist_u[(size_t)s0 * Bw + i]; }
    };
    stage_rows(0);                           // does not depend on the move list: in flight while the masks are built
    build_fill_masks(hole_of, filler_of, h, Bw, hmask, fmask, hoff, hmv, fmv, n_keep, p.n, p.err);
    for (int s0 = 0; s0 < w; s0 += p.rec_rows) {
        const int nr = min(p.rec_rows, w - s0);
        if (s0) {
            stage_rows(s0);
            __syncthreads();
        }
        fill_record_rows(rows_sh, stride, nr, p.n, n_keep, Bw, hmask, fmask, hoff, hmv, fmv);
        __syncthreads();
        for (int i = tid; i < nr * Bw; i += CMP_THREADS) { const int rr = row_of(i); hist_u[(size_t)s0 * Bw + i] = rows_sh[rr * stride + (i - rr * Bw)]; }
        __syncthreads();
    }
    fill_positions(p, u, h, hole_of, filler_of);     // last job of the compression for this unit
}

__global__ void __launch_bounds__(256) sh_counters_kernel(const uint32_t *hist, uint16_t *counters, int B, int Bw,
                                                          int w, int n_all, const int *n_arr) {
    const int u = blockIdx.x;
    const int n = n_arr ? n_arr[u] : n_all;
    for (int j = threadIdx.x; j < B; j += blockDim.x) {
        int I = 0;
        if (j < n) I = slot_counter(hist + (size_t)u * w * Bw, w, Bw, j);
        counters[(size_t)u * B + j] = (uint16_t)I;
    }
}

}  // namespace

namespace {
// fuse_with != NULL: take the fused unordered path if its shared arrays fit (reported in *fused)
cudaError_t launch_select(const SelectParams &p_in, bool from_hist, cudaStream_t s, long long *launches,
                          const CompactParams *fuse_with, bool *fused) {
    SelectParams p = p_in;
    p.fuse = 0;
    p.bw_magic = p.Bw > 1 ? (uint32_t)(0x100000000ULL / (unsigned)p.Bw) + 1u : 0u;
    size_t smem = sizeof(int) * ((size_t)p.n + p.cmax + 1 + 32 + 8 + (p.unordered ? SEL_TIE_CAP : 0));
    const size_t partial = sizeof(uint32_t) * (size_t)((p.w + 30) / 31) * 5 * p.Bw;
    const size_t planes = from_hist ? sizeof(uint32_t) * (size_t)p.w * p.Bw + partial : 0;
    if (fuse_with && from_hist && p.unordered) {
        const size_t planes_odd = sizeof(uint32_t) * (size_t)p.w * (p.Bw | 1) + partial;
        const size_t lists = sizeof(int) * (2 * (size_t)p.m + 13 * (size_t)p.Bw);
        if (smem + planes_odd + lists <= 96 * 1024) {
            p.fuse = 1;
            p.stage_planes = 1;
            p.fuse_off = (int)((smem + planes_odd) / sizeof(int));
            p.mv = *fuse_with;
            smem += planes_odd + lists;
        }
    }
    if (!p.fuse) {
        p.stage_planes = from_hist && smem + planes <= 96 * 1024;
        if (p.stage_planes) smem += planes;
    }
    if (fused) *fused = p.fuse != 0;
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
}  // namespace

cudaError_t sh_launch_select(const SelectParams &p, bool from_hist, cudaStream_t s, long long *launches) {
    return launch_select(p, from_hist, s, launches, nullptr, nullptr);
}

cudaError_t sh_launch_compress_unordered(const SelectParams &sp, const CompactParams &cp, cudaStream_t s, long long *launches) {
    bool fused = false;
    cudaError_t e = launch_select(sp, true, s, launches, &cp, &fused);
    if (e != cudaSuccess || fused) return e;
    return sh_launch_compact(cp, s, launches);
}

cudaError_t sh_launch_compact(const CompactParams &p_in, cudaStream_t s, long long *launches) {
    CompactParams p = p_in;
    // i / Bw as a multiply-high: exact while i * Bw < 2^32 (i stays below rows-per-pass * Bw <= 2^18)
    p.bw_magic = p.Bw > 1 ? (uint32_t)(0x100000000ULL / (unsigned)p.Bw) + 1u : 0u;
    if (p.unordered) {
        const int stride = p.Bw | 1;
        const size_t fixed = sizeof(uint32_t) * 13 * (size_t)p.Bw;     // masks, offsets, butterfly masks
        int rec_rows = (int)((96 * 1024 - fixed) / (stride * 4));
        if (rec_rows > CMP_THREADS) rec_rows = CMP_THREADS;
        if (rec_rows > p.w) rec_rows = p.w;
        if (rec_rows < 1) rec_rows = 1;
        p.rec_rows = rec_rows;
        const size_t smem = fixed + sizeof(uint32_t) * (size_t)rec_rows * stride;
        if (smem > 48 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(sh_fill_holes_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
        }
        sh_fill_holes_kernel<<<3 * p.U, CMP_THREADS, smem, s>>>(p);
        cudaError_t e = cudaGetLastError();
        if (e == cudaSuccess && launches) *launches += 1;
        return e;
    }
    // K/V rows: chunks of ~32 KB keep several CTAs per SM, so the reads of one
    // overlap the writes of another (measured best on B200 among 16..100 KB)
    const int max_chunk = p.row_bytes > 32 * 1024 ? p.row_bytes : 32 * 1024;
    int chunk_rows = max_chunk / p.row_bytes;
    if (chunk_rows > p.n - p.m) chunk_rows = p.n - p.m;
    if (chunk_rows < 1) chunk_rows = 1;
    p.chunk_bytes = chunk_rows * p.row_bytes;
    cudaError_t e;
    if (p.n - p.m > 0) {
        if (p.chunk_bytes > 40 * 1024) {
            e = cudaFuncSetAttribute(sh_compact_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, p.chunk_bytes);
            if (e != cudaSuccess) return e;
        }
        sh_compact_rows_kernel<<<dim3(p.U, 2, 1), ROWS_THREADS, p.chunk_bytes, s>>>(p);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        if (launches) *launches += 1;
    }
    // bit-plane rows staged per pass: up to one per thread, within ~64 KB
    const int stride = p.Bw | 1;
    int rec_rows = (64 * 1024) / (stride * 4);
    if (rec_rows > CMP_THREADS) rec_rows = CMP_THREADS;
    if (rec_rows > p.w) rec_rows = p.w;
    if (rec_rows < 1) rec_rows = 1;
    p.rec_rows = rec_rows;
    const size_t smem = sizeof(uint32_t) * ((size_t)6 * p.Bw + (size_t)rec_rows * stride);
    if (smem > 48 * 1024) {
        e = cudaFuncSetAttribute(sh_compact_record_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    sh_compact_record_kernel<<<p.U, CMP_THREADS, smem, s>>>(p);
    e = cudaGetLastError();
    if (e == cudaSuccess && launches) *launches += 1;
    return e;
}

cudaError_t sh_launch_counters(const uint32_t *hist, uint16_t *counters, int U, int B, int Bw, int w, int n,
                               const int *n_arr, cudaStream_t s, long long *launches) {
    sh_counters_kernel<<<U, 256, 0, s>>>(hist, counters, B, Bw, w, n, n_arr);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess && launches) *launches += 1;
    return e;
}
