// sh_compress_static: the compression step with the selection's result list held
// in a static device array instead of the caller's workspace.
//
// Who needs this: an inference server that hands all of HBM to its own KV-block
// pool at start-up has nothing left for cudaMalloc afterwards, and a caller
// inside a latency-critical decode loop cannot afford cudaMalloc's implicit
// device synchronisation.  This entry point runs the compression without
// touching any allocator.  Only the int32 list that the selection kernel hands
// to the compaction kernel (source slot per surviving row, or the hole/filler
// moves) lives in the static array; the per-unit move count, like the record and
// the positions, stays in the handle's workspace.
#include <mutex>

#include "sh_internal.h"

namespace {

// One int32 per (unit, slot): source slot of every surviving destination slot.
// Held by every device that loads the library, until the process exits.
constexpr size_t SH_STATIC_SCRATCH_ENTRIES = SH_STATIC_SCRATCH_MAX_ENTRIES;
static __device__ __align__(256) int32_t g_static_src_idx[SH_STATIC_SCRATCH_ENTRIES];

constexpr int MAX_DEVICES = 64;
std::mutex g_mu;
int32_t *g_scratch_ptr[MAX_DEVICES] = {};   // device address of g_static_src_idx, per device

// The array's name is only a host-side stand-in in host code; the device
// address comes from cudaGetSymbolAddress, asked once per device while that
// device is current.
cudaError_t scratch_address(int32_t **out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_src_idx);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[dev] = static_cast<int32_t *>(p);
    }
    *out = g_scratch_ptr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" int sh_compress_static(sh_handle h, void *stream, int *evicted_per_unit) {
    if (!h) return SH_EINVAL;
    if (!h->slab) return SH_ESTATE;
    if (evicted_per_unit) *evicted_per_unit = 0;
    if ((size_t)h->U * (size_t)h->B > SH_STATIC_SCRATCH_ENTRIES) return SH_ETOOBIG;
    if (!sh_compression_due(h)) return SH_OK;
    int32_t *src_idx = nullptr;
    cudaError_t e = scratch_address(&src_idx);
    if (e != cudaSuccess) { h->last_err = e; return SH_ECUDA; }
    cudaStream_t s = (cudaStream_t)stream;
    const int rrc = sh_recount_if_needed(h, s);
    if (rrc != SH_OK) return rrc;

    SelectParams sp = {};
    sp.hist = sh_phist(h);
    sp.counters = nullptr;
    sp.src_idx = src_idx;
    sp.evicted = nullptr;
    sp.U = h->U; sp.B = h->B; sp.Bw = h->Bw; sp.w = h->w; sp.n = h->B; sp.r = h->r; sp.m = h->m;
    sp.cmax = h->w;
    sp.err = reinterpret_cast<int *>(h->slab + h->L.err);
    sp.n_arr = sh_pnarr(h);
    sp.unordered = h->unordered;
    sp.pos = sh_ppos(h);
    sp.t_arr = sh_ptarr(h);
    sp.t = (int)h->t;
    sp.n_moves = reinterpret_cast<uint16_t *>(h->slab + h->L.counters);
    CompactParams cp = {};
    cp.K = sh_pK(h); cp.V = sh_pV(h);
    cp.Ks = sh_pKs(h); cp.Vs = sh_pVs(h);
    cp.hist = sh_phist(h);
    cp.pos = sh_ppos(h);
    cp.src_idx = src_idx;
    cp.U = h->U; cp.B = h->B; cp.Bw = h->Bw; cp.w = h->w; cp.n = h->B; cp.m = h->m;
    cp.n_arr = sh_pnarr(h);
    cp.unordered = h->unordered;
    cp.n_moves = sp.n_moves;
    cp.row_bytes = h->row_bytes;
    cp.scale_bytes = h->dtype == SH_INT4_G64_F16 ? (h->D / 64) * 2 : 0;
    cp.Bs = h->Bs;
    cp.err = reinterpret_cast<int *>(h->slab + h->L.err);
    if (h->unordered) {
        e = sh_launch_compress_unordered(sp, cp, s, &h->launches);
    } else {
        e = sh_launch_select(sp, true, s, &h->launches);
        if (e == cudaSuccess) e = sh_launch_compact(cp, s, &h->launches);
    }
    if (e != cudaSuccess) { h->last_err = e; return SH_ECUDA; }
    sh_after_compression(h);
    if (evicted_per_unit) *evicted_per_unit = h->m;
    return SH_OK;
}
