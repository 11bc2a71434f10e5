// C ABI and host state machine of libscissorhands.  The number of live tokens
// n and the step counter t are the same for every unit (each unit appends one
// token per step and drops exactly m when full), so they live on the host and
// no call needs to read anything back from the device to schedule its work.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>

#include "sh_internal.h"

namespace {

constexpr double LOG2E = 1.4426950408889634;

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

void make_layout(sh_context *c) {
    ShLayout &L = c->L;
    const size_t U = c->U, B = c->B, D = c->D;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t at = off;
        off = align_up(off + bytes, 256);
        return at;
    };
    L.K = take(U * B * c->row_bytes);
    L.V = take(U * B * c->row_bytes);
    const size_t sc = c->dtype == SH_INT4_G64_F16 ? U * (size_t)c->Bs * (D / 64) * 2 : 0;
    L.Ks = take(sc);
    L.Vs = take(sc);
    L.hist = take(U * (size_t)c->w * c->Bw * 4);
    L.pos = take(U * B * 4);
    L.src_idx = take(U * B * 4);
    L.counters = take(U * B * 2);
    L.xport = take(2 * B * D * 4);
    L.stage_q = take(U * (size_t)c->in_bytes);
    L.stage_k = take(U * (size_t)c->in_bytes);
    L.stage_v = take(U * (size_t)c->in_bytes);
    L.stage_out = take(U * D * 4);
    L.err = take(256);
    L.qring = take(c->record_mode ? U * (size_t)c->w * c->in_bytes : 0);
    L.n_arr = take(U * 4);
    L.t_arr = take(U * 4);
    L.total = off;
}

int cuda_fail(sh_context *c, cudaError_t e) {
    if (c) c->last_err = e;
    return SH_ECUDA;
}

int default_split(int U, int B) {
    // A cluster split pays for itself only when there are fewer units than SMs (measured on B200:
    // with 256 units, 1 CTA per unit beats 2 for the int4 store, 22 us against 31 us, and is level
    // for fp16), and only while every CTA still owns a few dozen rows.
    int s = 1;
    while (s < 8 && (long long)U * s < 148 && B / (2 * s) >= 32) s *= 2;
    return s;
}

// Stored rows -> fp32, for sh_export_unit.
__global__ void sh_export_kernel(const char *K, const char *V, const __half *Ks, const __half *Vs, float *dst,
                                 int B, int D, int dtype, int row_bytes) {
    const int total = B * D;
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < 2 * total; idx += gridDim.x * blockDim.x) {
        const int which = idx / total, rem = idx % total, j = rem / D, i = rem % D;
        const char *row = (which ? V : K) + (size_t)j * row_bytes;
        float val;
        if (dtype == SH_F32) val = reinterpret_cast<const float *>(row)[i];
        else if (dtype == SH_F16) val = __half2float(reinterpret_cast<const __half *>(row)[i]);
        else if (dtype == SH_BF16) val = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(row)[i]);
        else {
            const uint32_t word = reinterpret_cast<const uint32_t *>(row)[i >> 3];
            const int e = i & 7, nib = (e >> 1) + 4 * (e & 1);
            const int code = (int)((word >> (4 * nib)) & 0xFu) - 8;
            const __half *sc = (which ? Vs : Ks) + (size_t)j * (D / 64);
            val = (float)code * __half2float(sc[i >> 6]);
        }
        dst[idx] = val;
    }
}

__global__ void sh_fill_counts_kernel(int *n_arr, int *t_arr, int count, int n, int t) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) { n_arr[i] = n; t_arr[i] = t; }
}

// Algorithm 2 on every unit of the active range holding n live rows each: the r newest are protected, m go.
// The handle's own compression is (B, r, m) of its creation; a prompt cached in full is brought under
// another handle's budget with that handle's r and m (sh_import_compressed).
int do_compress_at(sh_context *c, cudaStream_t s, int n, int r, int m, bool own) {
    int rrc = sh_recount_if_needed(c, s);
    if (rrc != SH_OK) return rrc;
    SelectParams sp = {};
    sp.hist = sh_phist(c);
    sp.counters = nullptr;
    sp.src_idx = sh_psrc(c);
    sp.evicted = nullptr;
    sp.U = c->ucount; sp.B = c->B; sp.Bw = c->Bw; sp.w = c->w; sp.n = n; sp.r = r; sp.m = m;
    sp.cmax = c->w;
    sp.err = reinterpret_cast<int *>(c->slab + c->L.err);
    sp.n_arr = sh_pnarr(c);
    sp.unordered = c->unordered;
    sp.pos = sh_ppos(c);
    sp.t_arr = sh_ptarr(c);
    sp.t = (int)c->t;
    sp.n_moves = reinterpret_cast<uint16_t *>(c->slab + c->L.counters) + (size_t)c->u0 * c->B;
    CompactParams cp = {};
    cp.K = sh_pK(c); cp.V = sh_pV(c);
    cp.Ks = sh_pKs(c); cp.Vs = sh_pVs(c);
    cp.hist = sh_phist(c);
    cp.pos = sh_ppos(c);
    cp.src_idx = sp.src_idx;
    cp.U = c->ucount; cp.B = c->B; cp.Bw = c->Bw; cp.w = c->w; cp.n = n; cp.m = m;
    cp.row_bytes = c->row_bytes;
    cp.scale_bytes = c->dtype == SH_INT4_G64_F16 ? (c->D / 64) * 2 : 0;
    cp.Bs = c->Bs;
    cp.err = reinterpret_cast<int *>(c->slab + c->L.err);
    cp.n_arr = sh_pnarr(c);
    cp.unordered = c->unordered;
    cp.n_moves = sp.n_moves;
    cudaError_t e;
    if (c->unordered) {
        e = sh_launch_compress_unordered(sp, cp, s, &c->launches);
    } else {
        e = sh_launch_select(sp, true, s, &c->launches);
        if (e == cudaSuccess) e = sh_launch_compact(cp, s, &c->launches);
    }
    if (e != cudaSuccess) return cuda_fail(c, e);
    if (own) sh_after_compression(c);
    else c->n -= m;
    return SH_OK;
}

int do_compress(sh_context *c, cudaStream_t s) { return do_compress_at(c, s, c->B, c->r, c->m, true); }

// Rows [0, n) of every unit's K, V, scales, positions, bit-planes and (if kept) query ring, from one
// workspace layout to another (the budgets, hence the strides, differ).  One CTA per unit.
struct RepackParams {
    const char *sK, *sV, *sKs, *sVs, *sq;
    const uint32_t *shist;
    const int32_t *spos;
    char *dK, *dV, *dKs, *dVs, *dq;
    uint32_t *dhist;
    int32_t *dpos;
    int n, w, row_bytes, scale_bytes, in_bytes;
    int sB, dB, sBw, dBw, sBs, dBs;
};

__global__ void __launch_bounds__(256) sh_repack_kernel(const RepackParams p) {
    const size_t u = blockIdx.x;
    const int tid = threadIdx.x, nt = blockDim.x;
    const int pieces = p.n * (p.row_bytes / 16);
    const uint4 *sk = reinterpret_cast<const uint4 *>(p.sK + u * p.sB * p.row_bytes);
    const uint4 *sv = reinterpret_cast<const uint4 *>(p.sV + u * p.sB * p.row_bytes);
    uint4 *dk = reinterpret_cast<uint4 *>(p.dK + u * p.dB * p.row_bytes);
    uint4 *dv = reinterpret_cast<uint4 *>(p.dV + u * p.dB * p.row_bytes);
    for (int i = tid; i < pieces; i += nt) { dk[i] = sk[i]; dv[i] = sv[i]; }
    if (p.scale_bytes) {
        const int cnt = p.n * (p.scale_bytes / 2);
        const uint16_t *a = reinterpret_cast<const uint16_t *>(p.sKs + u * p.sBs * p.scale_bytes);
        const uint16_t *b = reinterpret_cast<const uint16_t *>(p.sVs + u * p.sBs * p.scale_bytes);
        uint16_t *c = reinterpret_cast<uint16_t *>(p.dKs + u * p.dBs * p.scale_bytes);
        uint16_t *d = reinterpret_cast<uint16_t *>(p.dVs + u * p.dBs * p.scale_bytes);
        for (int i = tid; i < cnt; i += nt) { c[i] = a[i]; d[i] = b[i]; }
    }
    for (int i = tid; i < p.n; i += nt) p.dpos[u * p.dB + i] = p.spos[u * p.sB + i];
    const int words = p.sBw < p.dBw ? p.sBw : p.dBw;
    for (int i = tid; i < p.w * words; i += nt) {
        const int row = i / words, k = i - row * words;
        p.dhist[(u * p.w + row) * p.dBw + k] = p.shist[(u * p.w + row) * p.sBw + k];
    }
    if (p.sq && p.dq) {
        const int qp = p.w * (p.in_bytes / 16);
        const uint4 *a = reinterpret_cast<const uint4 *>(p.sq + u * p.w * p.in_bytes);
        uint4 *b = reinterpret_cast<uint4 *>(p.dq + u * p.w * p.in_bytes);
        for (int i = tid; i < qp; i += nt) b[i] = a[i];
    }
}

}  // namespace

bool sh_compression_due(const sh_context *c) {
    if (!c->ragged) return c->n == c->B;
    for (int n : c->n_seq)
        if (n == c->B) return true;
    return false;
}

void sh_after_compression(sh_context *c) {
    if (!c->ragged) { c->n -= c->m; return; }
    for (int &n : c->n_seq)
        if (n == c->B) n -= c->m;
}

int sh_recount_if_needed(sh_context *c, cudaStream_t s) {
    if (!c->record_mode || c->record_fresh_t == c->t) return SH_OK;
    cudaError_t e = sh_launch_recount(c, s, &c->launches);
    if (e != cudaSuccess) { c->last_err = e; return SH_ECUDA; }
    c->record_fresh_t = c->t;
    return SH_OK;
}

namespace {

int do_step(sh_context *c, const void *q, const void *k, const void *v, float *out, cudaStream_t s,
            bool compress_after) {
    DecodeParams p = {};
    p.q = q; p.k_new = k; p.v_new = v; p.out = out;
    p.K = sh_pK(c); p.V = sh_pV(c);
    p.Ks = sh_pKs(c); p.Vs = sh_pVs(c);
    p.hist = sh_phist(c);
    p.pos = sh_ppos(c);
    p.qring = sh_pqring(c);
    p.n_arr = sh_pnarr(c); p.t_arr = sh_ptarr(c);
    p.U = c->ucount; p.B = c->B; p.Bw = c->Bw; p.w = c->w; p.Bs = c->Bs;
    p.n = c->n + 1;
    p.t = (int)(c->t + 1);
    p.hist_row = (int)((c->t + 1) % c->w);
    p.scale_log2e = (float)((double)c->scale * LOG2E);
    p.selftest_skip_tile = c->selftest_skip_tile;
    p.err = reinterpret_cast<int *>(c->slab + c->L.err);
    cudaError_t e = sh_launch_decode(c, p, s, &c->launches);
    if (e != cudaSuccess) return cuda_fail(c, e);
    c->started = true;
    c->t += 1;
    if (c->ragged) {
        for (size_t i = 0; i < c->n_seq.size(); ++i) { c->n_seq[i] += 1; c->t_seq[i] += 1; }
    } else {
        c->n += 1;
    }
    if (compress_after && sh_compression_due(c)) return do_compress(c, s);
    return SH_OK;
}

// Is any cache full (the next step would overflow it)?
bool cache_full(const sh_context *c) { return sh_compression_due(c); }

bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

}  // namespace

extern "C" {

int sh_create(int B, int r, int w, int m, int heads, int head_dim, int dtype, sh_handle *out) {
    if (!out) return SH_EINVAL;
    *out = nullptr;
    // B is bounded by the shared memory that holds one unit's logits (4 bytes per slot)
    if (B < 1 || B > 32768 || r < 0 || w < 1 || w > 16384 || m < 1 || m > B - r || heads < 1) return SH_EINVAL;
    if (head_dim != 64 && head_dim != 128) return SH_EINVAL;
    if (dtype < SH_F32 || dtype > SH_INT4_G64_F16) return SH_EINVAL;
    sh_context *c = new (std::nothrow) sh_context();
    if (!c) return SH_ENOMEM;
    c->B = B; c->r = r; c->w = w; c->m = m; c->U = heads; c->D = head_dim; c->dtype = dtype;
    c->Bw = (B + 31) / 32;
    c->Bs = (B + 7) / 8 * 8;
    c->row_bytes = dtype == SH_F32 ? head_dim * 4 : (dtype == SH_INT4_G64_F16 ? head_dim / 2 : head_dim * 2);
    c->in_bytes = dtype == SH_F32 ? head_dim * 4 : head_dim * 2;
    c->n = 0; c->t = 0;
    c->scale = (float)(1.0 / std::sqrt((double)head_dim));
    c->split = default_split(heads, B);
    c->split_explicit = false;
    c->auto_compress = 1;
    c->kernel = 0;
    c->prefill_chunk = 1;
    c->record_mode = 0;
    c->unordered = 1;
    c->record_fresh_t = -1;
    c->selftest_skip_tile = -1;
    c->started = false;
    c->slab = nullptr; c->slab_bytes = 0;
    c->launches = 0;
    c->last_err = cudaSuccess;
    c->u0 = 0; c->ucount = heads;
    c->ragged = false;
    c->units_per_seq = heads;
    make_layout(c);
    *out = c;
    return SH_OK;
}

void sh_destroy(sh_handle h) { delete h; }

size_t sh_workspace_bytes(sh_handle h) { return h ? h->L.total : 0; }

int sh_bind(sh_handle h, void *slab_dev, size_t bytes, void *stream) {
    if (!h || !slab_dev) return SH_EINVAL;
    if (reinterpret_cast<uintptr_t>(slab_dev) & 255u) return SH_EINVAL;
    if (bytes < h->L.total) return SH_ENOMEM;
    cudaError_t e = cudaMemsetAsync(slab_dev, 0, h->L.total, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(h, e);
    h->slab = static_cast<char *>(slab_dev);
    h->slab_bytes = bytes;
    h->n = 0; h->t = 0;
    h->started = false;
    h->ragged = false;
    h->n_seq.clear(); h->t_seq.clear();
    h->u0 = 0; h->ucount = h->U;
    h->record_fresh_t = -1;
    return SH_OK;
}

int sh_set_option(sh_handle h, int key, double value) {
    if (!h) return SH_EINVAL;
    if (h->started) return SH_ESTATE;
    switch (key) {
        case SH_OPT_SOFTMAX_SCALE:
            if (!(value > 0.0) || !std::isfinite(value)) return SH_EINVAL;
            h->scale = (float)value;
            return SH_OK;
        case SH_OPT_SPLIT: {
            const int s = (int)value;
            if (s != 1 && s != 2 && s != 4 && s != 8) return SH_EINVAL;
            h->split = s;
            h->split_explicit = true;
            return SH_OK;
        }
        case SH_OPT_AUTO_COMPRESS:
            h->auto_compress = value != 0.0;
            return SH_OK;
        case SH_OPT_RECORD_MODE: {
            const int mode = (int)value;
            if (mode != 0 && mode != 1) return SH_EINVAL;
            if (h->slab) return SH_ESTATE;                       // changes the workspace layout
            if (mode == 1 && !sh_recount_supported(h)) return SH_EINVAL;   // needs the recount kernel's shapes
            h->record_mode = mode;
            make_layout(h);
            return SH_OK;
        }
        case SH_OPT_COMPACTION: {
            const int mode = (int)value;
            if (mode != 0 && mode != 1) return SH_EINVAL;
            h->unordered = mode;
            return SH_OK;
        }
        case SH_OPT_PREFILL_CHUNK: {
            const int mode = (int)value;
            if (mode < 0 || mode > 4) return SH_EINVAL;
            const int before = h->prefill_chunk;
            h->prefill_chunk = mode;
            if (h->record_mode && !sh_recount_supported(h)) {     // the recount would not fit the chosen kernel
                h->prefill_chunk = before;
                return SH_EINVAL;
            }
            return SH_OK;
        }
        case SH_OPT_DECODE_KERNEL: {
            const int k = (int)value;
            if (k < 0 || k > 2) return SH_EINVAL;
            h->kernel = k;
            return SH_OK;
        }
        case SH_OPT_SELFTEST_SKIP_TILE: {
            if (!(value >= -1.0 && value < 1e9)) return SH_EINVAL;
            h->selftest_skip_tile = (int)value;
            return SH_OK;
        }
        default: return SH_EINVAL;
    }
}

int sh_decode_step(sh_handle h, const void *q_dev, const void *k_new_dev, const void *v_new_dev,
                   float *attn_out_dev, void *stream) {
    if (!h || !q_dev || !k_new_dev || !v_new_dev || !attn_out_dev) return SH_EINVAL;
    if (misaligned(q_dev) || misaligned(k_new_dev) || misaligned(v_new_dev)) return SH_EINVAL;
    if (reinterpret_cast<uintptr_t>(attn_out_dev) & 3u) return SH_EINVAL;
    if (!h->slab) return SH_ESTATE;
    if (cache_full(h)) return SH_EFULL;
    if (h->t + 1 >= (1 << 24)) return SH_EINVAL;   // the threshold test multiplies by t in fp32
    return do_step(h, q_dev, k_new_dev, v_new_dev, attn_out_dev, (cudaStream_t)stream, h->auto_compress != 0);
}

// Device-visible alias of a pinned host buffer (unified addressing maps pinned
// host memory into the device's address space), or NULL if the buffer is
// pageable or misaligned and has to be staged through the workspace.
static void *pinned_alias(const void *host_ptr) {
    if (misaligned(host_ptr)) return nullptr;
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, host_ptr) != cudaSuccess) {
        (void)cudaGetLastError();
        return nullptr;
    }
    if (a.type != cudaMemoryTypeHost || !a.devicePointer) return nullptr;
    return a.devicePointer;
}

int sh_decode_step_host(sh_handle h, const void *q_host, const void *k_new_host, const void *v_new_host,
                        float *attn_out_host, void *stream) {
    if (!h || !q_host || !k_new_host || !v_new_host || !attn_out_host) return SH_EINVAL;
    if (reinterpret_cast<uintptr_t>(attn_out_host) & 3u) return SH_EINVAL;
    if (!h->slab) return SH_ESTATE;
    if (cache_full(h)) return SH_EFULL;
    if (h->t + 1 >= (1 << 24)) return SH_EINVAL;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t inb = (size_t)h->U * h->in_bytes, outb = (size_t)h->U * h->D * 4;
    cudaError_t e;
    // Pinned buffers are read and written by the kernel itself over PCIe, so
    // the transfers overlap the streaming of K and V instead of preceding and
    // following it; pageable ones go through staging copies.
    const void *src[3] = {q_host, k_new_host, v_new_host};
    const size_t stage_off[3] = {h->L.stage_q, h->L.stage_k, h->L.stage_v};
    const void *in[3];
    for (int i = 0; i < 3; ++i) {
        in[i] = pinned_alias(src[i]);
        if (!in[i]) {
            char *st = h->slab + stage_off[i];
            if ((e = cudaMemcpyAsync(st, src[i], inb, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(h, e);
            in[i] = st;
        }
    }
    float *out = static_cast<float *>(pinned_alias(attn_out_host));
    const bool stage_out = out == nullptr;
    if (stage_out) out = reinterpret_cast<float *>(h->slab + h->L.stage_out);
    int rc = do_step(h, in[0], in[1], in[2], out, s, false);
    if (rc != SH_OK) return rc;
    // The result leaves before any compression that follows.
    if (stage_out &&
        (e = cudaMemcpyAsync(attn_out_host, out, outb, cudaMemcpyDeviceToHost, s)) != cudaSuccess)
        return cuda_fail(h, e);
    if (h->auto_compress && sh_compression_due(h)) {
        rc = do_compress(h, s);
        if (rc != SH_OK) return rc;
    }
    if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return cuda_fail(h, e);
    return SH_OK;
}

// Tokens [0, count) of a time-major block through the chunk kernel; no compression.
static int do_chunk(sh_context *c, const char *q, const char *k, const char *v, float *out, int count, cudaStream_t s) {
    cudaError_t e = sh_launch_prefill_chunk(c, q, k, v, out, count, s, &c->launches);
    if (e != cudaSuccess) return cuda_fail(c, e);
    c->started = true;
    c->n += count;
    c->t += count;
    return SH_OK;
}

int sh_prefill_chunk(sh_handle h, const void *q_dev, const void *k_dev, const void *v_dev, int count, float *out_dev,
                     void *stream) {
    if (!h || !q_dev || !k_dev || !v_dev || count < 1) return SH_EINVAL;
    if (misaligned(q_dev) || misaligned(k_dev) || misaligned(v_dev)) return SH_EINVAL;
    if (!h->slab || h->ragged) return SH_ESTATE;
    if (h->n >= h->B) return SH_EFULL;
    const int cap = sh_prefill_chunk_capacity(h);
    if (cap == 0 || count > cap || count > h->B - h->n) return SH_EINVAL;
    if (h->t + count >= (1 << 24)) return SH_EINVAL;
    return do_chunk(h, static_cast<const char *>(q_dev), static_cast<const char *>(k_dev),
                    static_cast<const char *>(v_dev), out_dev, count, (cudaStream_t)stream);
}

int sh_prefill_chunk_max(sh_handle h) { return h ? sh_prefill_chunk_capacity(h) : 0; }

// p tokens of the active unit range (q, k, v, out already point at that range's first unit;
// consecutive tokens are h->U rows apart): chunks where the shape allows, decode steps otherwise,
// a compression whenever the cache fills.
static int prefill_range(sh_context *h, const char *q_dev, const char *k_dev, const char *v_dev, int p, float *out_dev,
                         cudaStream_t s) {
    const size_t in_stride = (size_t)h->U * h->in_bytes, out_stride = (size_t)h->U * h->D;
    float *sink = reinterpret_cast<float *>(h->slab + h->L.stage_out);
    const int cap = h->prefill_chunk ? sh_prefill_chunk_capacity(h) : 0;
    int i = 0;
    while (i < p) {
        const char *q = q_dev + i * in_stride, *k = k_dev + i * in_stride, *v = v_dev + i * in_stride;
        int cnt = p - i;
        if (cnt > h->B - h->n) cnt = h->B - h->n;
        if (cnt > cap) cnt = cap;
        int rc;
        if (cnt >= 2) {
            // the steps up to the next compression only append: take them in one launch
            rc = do_chunk(h, q, k, v, out_dev ? out_dev + i * out_stride : nullptr, cnt, s);
        } else {
            cnt = 1;
            rc = do_step(h, q, k, v, out_dev ? out_dev + i * out_stride : sink, s, false);
        }
        if (rc != SH_OK) return rc;
        if (h->n == h->B && (rc = do_compress(h, s)) != SH_OK) return rc;
        i += cnt;
    }
    return SH_OK;
}

int sh_prefill(sh_handle h, const void *q_dev, const void *k_dev, const void *v_dev, int p, float *out_dev,
               void *stream) {
    if (!h || !q_dev || !k_dev || !v_dev || p < 0) return SH_EINVAL;
    if (misaligned(q_dev) || misaligned(k_dev) || misaligned(v_dev)) return SH_EINVAL;
    if (!h->slab || h->ragged) return SH_ESTATE;
    if (h->n >= h->B) return SH_EFULL;
    if (h->t + p >= (1 << 24)) return SH_EINVAL;
    return prefill_range(h, static_cast<const char *>(q_dev), static_cast<const char *>(k_dev),
                         static_cast<const char *>(v_dev), p, out_dev, (cudaStream_t)stream);
}

int sh_import_compressed(sh_handle dst, sh_handle src, void *stream) {
    if (!dst || !src || dst == src) return SH_EINVAL;
    if (!dst->slab || !src->slab) return SH_ESTATE;
    if (dst->started || dst->t != 0 || dst->n != 0 || dst->ragged || src->ragged) return SH_ESTATE;
    if (dst->U != src->U || dst->D != src->D || dst->dtype != src->dtype || dst->w != src->w ||
        dst->record_mode != src->record_mode)
        return SH_EINVAL;
    cudaStream_t s = (cudaStream_t)stream;
    // Algorithm 2 on the record as it stands, as often as needed: fewer than dst->B tokens must remain
    while (src->n >= dst->B) {
        if (src->n - dst->r < dst->m) return SH_EINVAL;
        const int rc = do_compress_at(src, s, src->n, dst->r, dst->m, false);
        if (rc != SH_OK) return rc;
    }
    RepackParams rp = {};
    rp.sK = sh_pK(src); rp.sV = sh_pV(src); rp.sKs = sh_pKs(src); rp.sVs = sh_pVs(src); rp.sq = sh_pqring(src);
    rp.shist = sh_phist(src); rp.spos = sh_ppos(src);
    rp.dK = sh_pK(dst); rp.dV = sh_pV(dst); rp.dKs = sh_pKs(dst); rp.dVs = sh_pVs(dst); rp.dq = sh_pqring(dst);
    rp.dhist = sh_phist(dst); rp.dpos = sh_ppos(dst);
    rp.n = src->n; rp.w = src->w; rp.row_bytes = src->row_bytes;
    rp.scale_bytes = src->dtype == SH_INT4_G64_F16 ? (src->D / 64) * 2 : 0;
    rp.in_bytes = src->in_bytes;
    rp.sB = src->B; rp.dB = dst->B; rp.sBw = src->Bw; rp.dBw = dst->Bw; rp.sBs = src->Bs; rp.dBs = dst->Bs;
    if (rp.n > 0) {
        sh_repack_kernel<<<dst->U, 256, 0, s>>>(rp);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(dst, e);
        dst->launches += 1;
    }
    dst->n = src->n;
    dst->t = src->t;
    dst->started = true;
    dst->record_fresh_t = -1;
    return SH_OK;
}

// A context for the whole prompt: budget p + 1 (never fills), the options of h that shape the kernels.
static sh_context *bulk_context(const sh_context *h, int p) {
    sh_handle t = nullptr;
    if (sh_create(p + 1, 0, h->w, 1, h->U, h->D, h->dtype, &t) != SH_OK) return nullptr;
    t->scale = h->scale;
    t->kernel = h->kernel;
    t->prefill_chunk = h->prefill_chunk;
    t->unordered = h->unordered;
    if (h->split_explicit) { t->split = h->split; t->split_explicit = true; }
    if (h->record_mode && sh_set_option(t, SH_OPT_RECORD_MODE, 1.0) != SH_OK) { sh_destroy(t); return nullptr; }
    return t;
}

size_t sh_prefill_bulk_scratch_bytes(sh_handle h, int p) {
    if (!h || p < 1 || p > 32767) return 0;
    sh_context *t = bulk_context(h, p);
    if (!t) return 0;
    const size_t bytes = t->L.total;
    sh_destroy(t);
    return bytes;
}

int sh_prefill_bulk(sh_handle h, const void *q_dev, const void *k_dev, const void *v_dev, int p, float *out_dev,
                    void *scratch_dev, size_t scratch_bytes, void *stream) {
    if (!h || !q_dev || !k_dev || !v_dev || !scratch_dev || p < 1 || p > 32767) return SH_EINVAL;
    if (!h->slab) return SH_ESTATE;
    if (h->started || h->t != 0 || h->ragged) return SH_ESTATE;
    sh_context *t = bulk_context(h, p);
    if (!t) return SH_EINVAL;
    int rc = sh_bind(t, scratch_dev, scratch_bytes, stream);
    if (rc == SH_OK) rc = sh_prefill(t, q_dev, k_dev, v_dev, p, out_dev, stream);
    if (rc == SH_OK) rc = sh_import_compressed(h, t, stream);
    if (rc == SH_ECUDA) h->last_err = t->last_err != cudaSuccess ? t->last_err : h->last_err;
    h->launches += t->launches;
    sh_destroy(t);
    return rc;
}

int sh_prefill_ragged(sh_handle h, const void *q_dev, const void *k_dev, const void *v_dev, int p_max,
                      const int *lengths_host, int n_sequences, float *out_dev, void *stream) {
    if (!h || !q_dev || !k_dev || !v_dev || !lengths_host || p_max < 0 || n_sequences < 1) return SH_EINVAL;
    if (misaligned(q_dev) || misaligned(k_dev) || misaligned(v_dev)) return SH_EINVAL;
    if (!h->slab) return SH_ESTATE;
    if (h->ragged || h->t != 0 || h->n != 0) return SH_ESTATE;       // a fresh handle only
    if (h->record_mode) return SH_EINVAL;                            // the recompute variant assumes one schedule
    if (h->U % n_sequences) return SH_EINVAL;
    for (int sq = 0; sq < n_sequences; ++sq)
        if (lengths_host[sq] < 0 || lengths_host[sq] > p_max) return SH_EINVAL;
    if (p_max >= (1 << 24)) return SH_EINVAL;
    cudaStream_t s = (cudaStream_t)stream;
    const int ups = h->U / n_sequences;
    h->units_per_seq = ups;
    h->n_seq.assign(n_sequences, 0);
    h->t_seq.assign(n_sequences, 0);
    long long t_max = 0;
    int rc = SH_OK;
    for (int sq = 0; sq < n_sequences && rc == SH_OK; ++sq) {
        // this sequence's units alone, with its own n and t: the uniform machinery on a sub-range
        h->u0 = sq * ups; h->ucount = ups; h->n = 0; h->t = 0;
        const size_t in_off = (size_t)h->u0 * h->in_bytes;
        rc = prefill_range(h, static_cast<const char *>(q_dev) + in_off, static_cast<const char *>(k_dev) + in_off,
                           static_cast<const char *>(v_dev) + in_off, lengths_host[sq],
                           out_dev ? out_dev + (size_t)h->u0 * h->D : nullptr, s);
        if (rc != SH_OK) break;
        h->n_seq[sq] = h->n;
        h->t_seq[sq] = h->t;
        if (h->t > t_max) t_max = h->t;
        int *na = reinterpret_cast<int *>(h->slab + h->L.n_arr) + h->u0;
        int *ta = reinterpret_cast<int *>(h->slab + h->L.t_arr) + h->u0;
        sh_fill_counts_kernel<<<(ups + 255) / 256, 256, 0, s>>>(na, ta, ups, h->n, (int)h->t);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) rc = cuda_fail(h, e);
        else h->launches += 1;
    }
    h->u0 = 0; h->ucount = h->U;
    h->n = 0;
    h->t = t_max;
    if (rc != SH_OK) return rc;
    h->ragged = true;
    h->started = true;
    return SH_OK;
}

int sh_sequence_state(sh_handle h, int *n_host, long long *t_host, int capacity) {
    if (!h || capacity < 0) return SH_EINVAL;
    if (!h->ragged) {
        if (capacity >= 1) { if (n_host) n_host[0] = h->n; if (t_host) t_host[0] = h->t; }
        return 1;
    }
    const int ns = (int)h->n_seq.size();
    for (int i = 0; i < ns && i < capacity; ++i) {
        if (n_host) n_host[i] = h->n_seq[i];
        if (t_host) t_host[i] = h->t_seq[i];
    }
    return ns;
}

int sh_recompute_record(sh_handle h, void *stream) {
    if (!h) return SH_EINVAL;
    if (!h->slab || !h->record_mode) return SH_ESTATE;
    h->record_fresh_t = -1;
    return sh_recount_if_needed(h, (cudaStream_t)stream);
}

int sh_export_record(sh_handle h, int unit, uint32_t *planes_host, void *stream) {
    if (!h || unit < 0 || unit >= h->U || !planes_host) return SH_EINVAL;
    if (!h->slab) return SH_ESTATE;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t bytes = (size_t)h->w * h->Bw * 4;
    cudaError_t e = cudaMemcpyAsync(planes_host, h->slab + h->L.hist + (size_t)unit * bytes, bytes,
                                    cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail(h, e);
    if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return cuda_fail(h, e);
    return SH_OK;
}

int sh_scores(sh_handle h, const void *q, float *alpha_out, void *stream) {
    if (!h || !q || !alpha_out) return SH_EINVAL;
    if (!h->slab) return SH_ESTATE;
    DecodeParams p = {};
    p.q = q;
    p.K = sh_pK(h); p.Ks = sh_pKs(h);
    p.n_arr = sh_pnarr(h);
    p.U = h->ucount; p.B = h->B; p.Bs = h->Bs;
    p.n = h->n;
    p.scale_log2e = (float)((double)h->scale * LOG2E);
    p.err = reinterpret_cast<int *>(h->slab + h->L.err);
    cudaError_t e = sh_launch_scores(h, p, alpha_out, (cudaStream_t)stream, &h->launches);
    if (e != cudaSuccess) return cuda_fail(h, e);
    return SH_OK;
}

int sh_compress(sh_handle h, void *stream, int *evicted_per_unit) {
    if (!h) return SH_EINVAL;
    if (!h->slab) return SH_ESTATE;
    if (evicted_per_unit) *evicted_per_unit = 0;
    if (!sh_compression_due(h)) return SH_OK;
    int rc = do_compress(h, (cudaStream_t)stream);
    if (rc == SH_OK && evicted_per_unit) *evicted_per_unit = h->m;
    return rc;
}

int sh_select(const uint16_t *counters_dev, int units, int n, int r, int m, int32_t *evicted_dev, void *stream) {
    if (!counters_dev || !evicted_dev || units < 1 || n < 1 || n > SH_SELECT_MAX_N || r < 0 || m < 1 || m > n - r)
        return SH_EINVAL;
    SelectParams sp = {};
    sp.hist = nullptr;
    sp.counters = counters_dev;
    sp.src_idx = nullptr;
    sp.evicted = evicted_dev;
    sp.U = units; sp.B = n; sp.Bw = (n + 31) / 32; sp.w = 0; sp.n = n; sp.r = r; sp.m = m;
    sp.cmax = 16384;
    cudaError_t e = sh_launch_select(sp, false, (cudaStream_t)stream, nullptr);
    return e == cudaSuccess ? SH_OK : SH_ECUDA;
}

int sh_state(sh_handle h, void *stream, int *n_out, long long *t_out, int32_t *pos_host, uint16_t *counters_host,
             uint32_t *low_host) {
    if (!h) return SH_EINVAL;
    if (!h->slab) return SH_ESTATE;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e;
    if (n_out) *n_out = h->ragged ? -1 : h->n;      // sequences differ: see sh_sequence_state
    if (t_out) *t_out = h->t;
    const size_t U = h->U, B = h->B;
    if (pos_host) {
        e = cudaMemcpyAsync(pos_host, h->slab + h->L.pos, U * B * 4, cudaMemcpyDeviceToHost, s);
        if (e != cudaSuccess) return cuda_fail(h, e);
    }
    if (counters_host) {
        uint16_t *cd = reinterpret_cast<uint16_t *>(h->slab + h->L.counters);
        e = sh_launch_counters(reinterpret_cast<const uint32_t *>(h->slab + h->L.hist), cd, h->U, h->B, h->Bw, h->w,
                               h->n, sh_pnarr(h), s, &h->launches);
        if (e != cudaSuccess) return cuda_fail(h, e);
        e = cudaMemcpyAsync(counters_host, cd, U * B * 2, cudaMemcpyDeviceToHost, s);
        if (e != cudaSuccess) return cuda_fail(h, e);
    }
    if (low_host) {
        // the bit-plane row of each sequence's own last step
        const size_t row_b = (size_t)h->Bw * 4, unit_b = (size_t)h->w * row_b;
        const int nsq = h->ragged ? (int)h->t_seq.size() : 1, ups = h->ragged ? h->units_per_seq : h->U;
        for (int sq = 0; sq < nsq; ++sq) {
            const int row = (int)((h->ragged ? h->t_seq[sq] : h->t) % h->w);
            const char *src = h->slab + h->L.hist + (size_t)sq * ups * unit_b + (size_t)row * row_b;
            e = cudaMemcpy2DAsync(reinterpret_cast<char *>(low_host) + (size_t)sq * ups * row_b, row_b, src, unit_b, row_b,
                                  ups, cudaMemcpyDeviceToHost, s);
            if (e != cudaSuccess) return cuda_fail(h, e);
        }
    }
    int dev_err = 0;
    e = cudaMemcpyAsync(&dev_err, h->slab + h->L.err, sizeof(int), cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail(h, e);
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(h, e);
    return dev_err ? SH_EDEVICE : SH_OK;
}

int sh_export_unit(sh_handle h, int unit, float *K_host, float *V_host, void *stream) {
    if (!h || unit < 0 || unit >= h->U || !K_host || !V_host) return SH_EINVAL;
    if (!h->slab) return SH_ESTATE;
    cudaStream_t s = (cudaStream_t)stream;
    float *dst = reinterpret_cast<float *>(h->slab + h->L.xport);
    const size_t B = h->B, D = h->D;
    const char *K = h->slab + h->L.K + (size_t)unit * B * h->row_bytes;
    const char *V = h->slab + h->L.V + (size_t)unit * B * h->row_bytes;
    const __half *Ks = reinterpret_cast<const __half *>(h->slab + h->L.Ks) + (size_t)unit * h->Bs * (D / 64);
    const __half *Vs = reinterpret_cast<const __half *>(h->slab + h->L.Vs) + (size_t)unit * h->Bs * (D / 64);
    sh_export_kernel<<<64, 256, 0, s>>>(K, V, Ks, Vs, dst, h->B, h->D, h->dtype, h->row_bytes);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(h, e);
    h->launches += 1;
    if ((e = cudaMemcpyAsync(K_host, dst, B * D * 4, cudaMemcpyDeviceToHost, s)) != cudaSuccess) return cuda_fail(h, e);
    if ((e = cudaMemcpyAsync(V_host, dst + B * D, B * D * 4, cudaMemcpyDeviceToHost, s)) != cudaSuccess)
        return cuda_fail(h, e);
    if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return cuda_fail(h, e);
    return SH_OK;
}

int sh_restore(sh_handle h, int n, long long t) {
    if (!h || n < 0 || n > h->B || t < n || t >= (1 << 24)) return SH_EINVAL;
    if (!h->slab) return SH_ESTATE;
    if (h->ragged) return SH_ESTATE;      // per-sequence counters live on the device: one (n, t) cannot describe them
    h->n = n;
    h->t = t;
    h->started = true;
    h->record_fresh_t = -1;
    return SH_OK;
}

long long sh_launch_count(sh_handle h) { return h ? h->launches : 0; }

int sh_decode_kernel_choice(sh_handle h) { return h ? sh_decode_kernel_for(h, h->U) : SH_EINVAL; }

const char *sh_strerror(int status) {
    switch (status) {
        case SH_OK: return "ok";
        case SH_EINVAL: return "invalid argument";
        case SH_EFULL: return "cache is full: compress before the next step";
        case SH_ESTATE: return "call out of order (no workspace bound, or option set after the first step)";
        case SH_ECUDA: return "CUDA runtime error";
        case SH_ENOMEM: return "allocation failed or workspace too small";
        case SH_ETOOBIG: return "problem exceeds the fixed capacity of this entry point";
        case SH_EDEVICE: return "a kernel gave up a bounded wait (device error word set); state is unreliable";
        default: return "unknown status";
    }
}

const char *sh_last_cuda_error(sh_handle h) {
    if (!h || h->last_err == cudaSuccess) return "";
    return cudaGetErrorString(h->last_err);
}

}  // extern "C"
