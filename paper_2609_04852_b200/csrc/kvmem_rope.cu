// Position-consistent keys (Sec. 4.4: RoPE is applied to raw K at the block's assigned compact
// position while the block is materialised, V is copied unchanged, sine/cosine come from a
// precomputed table; Sec. 4.3: the same transformation, inverted, brings keys and queries into the
// position-independent space of the index).
//
// Rotary variant: element i pairs with i + d/2; the table row of a position holds (cos, sin) per pair.
// A rotated element is defined as fp32 products and sums without fused multiply-add followed by one
// round-to-nearest-even to bf16, so the view's keys are a reproducible code.
//
// gather_rope_kernel does the work of the plain gather (one tile = one selected block x K|V x layer x
// KV head) but K tiles pass through registers: a thread loads 8 low and the 8 matching high dimensions
// of one token (two 128-bit loads), the 8 (cos, sin) pairs of the token's compact position (four
// 128-bit loads that hit L2 for 7 of the 8 KV heads), and stores two 128-bit results.  V tiles are
// copied with 128-bit loads and stores.  HBM-bound: 1 read + 1 write per view byte plus the table.
#include <algorithm>

#include "kvmem_internal.cuh"
#include "kvmem_rope.cuh"

namespace kvmem {

// y[r][v] = RoPE(x[r][v], positions[r]) (or the inverse); one thread per (row, vector, 8-pair chunk)
__global__ void __launch_bounds__(256)
rope_rotate_kernel(const __nv_bfloat16* __restrict__ x, __nv_bfloat16* __restrict__ y, long long n_rows, int n_vec, int d,
                   const int32_t* __restrict__ positions, const float2* __restrict__ rope, int rope_positions, float sgn,
                   int32_t* __restrict__ status) {
    const int half = d / 2, chunks = half / 8;
    const long long total = n_rows * n_vec * chunks;
    for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(e % chunks);
        const long long rv = e / chunks;
        const long long r = rv / n_vec;
        const int pos = positions[r];
        if (pos < 0 || pos >= rope_positions) { atomicExch(status, (int)KVMEM_E_DEVICE_RANGE); continue; }
        const __nv_bfloat16* src = x + rv * d + c * 8;
        __nv_bfloat16* dst = y + rv * d + c * 8;
        const uint4 lo = *reinterpret_cast<const uint4*>(src), hi = *reinterpret_cast<const uint4*>(src + half);
        uint4 lo_o, hi_o;
        rotate8(lo, hi, rope + (size_t)pos * half + c * 8, sgn, lo_o, hi_o);
        *reinterpret_cast<uint4*>(dst) = lo_o;
        *reinterpret_cast<uint4*>(dst + half) = hi_o;
    }
}

struct GatherRopeArgs {
    const __nv_bfloat16* pages;
    const int32_t* tables;
    const int32_t* nblocks_dev;
    const int32_t* sel_ids;
    const int32_t* n_sel;
    __nv_bfloat16* view_k;
    __nv_bfloat16* view_v;
    const float2* rope;
    int32_t* status;
    int session_first, sel_stride, max_bps, max_blocks, LG, B, d, cap_tokens, first_position, rope_positions, in_block;
    size_t page_elems;
};

__global__ void __launch_bounds__(256)
gather_rope_kernel(GatherRopeArgs a) {
    pdl_wait();        // everything earlier in the stream is complete and visible from here on
    const int s = blockIdx.y;
    const int NB = a.nblocks_dev[a.session_first + s];
    int n_blk = a.n_sel[s];
    const int cap_blocks = a.cap_tokens / a.B;
    if (n_blk > a.sel_stride || n_blk > cap_blocks) {
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE);
        n_blk = min(min(n_blk, a.sel_stride), cap_blocks);
    }
    n_blk = max(n_blk, 0);
    const int per_block = 2 * a.LG;
    const long long n_tiles = (long long)n_blk * per_block;
    const long long t_begin = n_tiles * blockIdx.x / gridDim.x, t_end = n_tiles * (blockIdx.x + 1) / gridDim.x;
    const int tile_elems = a.B * a.d, half = a.d / 2, chunks = half / 8;
    int cached_j = -1, page = -1;
    for (long long tile = t_begin; tile < t_end; ++tile) {
        const int j = (int)(tile / per_block), w = (int)(tile % per_block);
        const int kv = w / a.LG, lg = w % a.LG;
        if (j != cached_j) {
            cached_j = j;
            const int id = a.sel_ids[(size_t)s * a.sel_stride + j];
            page = -1;
            if (id >= 0 && id < NB) page = a.tables[(size_t)(a.session_first + s) * a.max_bps + id];
            if (page < 0 || page >= a.max_blocks) { atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE); page = -1; }
        }
        if (page < 0) continue;
        const __nv_bfloat16* src = a.pages + (size_t)page * a.page_elems + (size_t)w * tile_elems;
        __nv_bfloat16* dst = (kv ? a.view_v : a.view_k) + (((size_t)s * a.LG + lg) * a.cap_tokens + (size_t)j * a.B) * a.d;
        if (kv) {                                           // values: unchanged
            const uint4* s4 = reinterpret_cast<const uint4*>(src);
            uint4* d4 = reinterpret_cast<uint4*>(dst);
            for (int v = threadIdx.x; v < tile_elems / 8; v += 256) d4[v] = __ldg(s4 + v);
        } else {                                            // keys: rotate to the compact position
            for (int e = threadIdx.x; e < a.B * chunks; e += 256) {
                const int t = e / chunks, c = e % chunks;
                const int pos = a.first_position + j * a.B + (a.in_block ? 0 : t);      // in-block layout: t is already in the stored key
                if (pos >= a.rope_positions) { atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE); continue; }
                const __nv_bfloat16* row = src + (size_t)t * a.d + c * 8;
                const uint4 lo = __ldg(reinterpret_cast<const uint4*>(row)), hi = __ldg(reinterpret_cast<const uint4*>(row + half));
                uint4 lo_o, hi_o;
                rotate8(lo, hi, a.rope + (size_t)pos * half + c * 8, 1.0f, lo_o, hi_o);
                __nv_bfloat16* orow = dst + (size_t)t * a.d + c * 8;
                *reinterpret_cast<uint4*>(orow) = lo_o;
                *reinterpret_cast<uint4*>(orow + half) = hi_o;
            }
        }
    }
}

cudaError_t launch_rope_rotate(const kvmem_pool& p, const __nv_bfloat16* x, __nv_bfloat16* y, long long n_rows, int n_vec,
                               const int32_t* positions, int inverse, cudaStream_t st) {
    const int d = p.geo.d;
    const long long total = n_rows * n_vec * (d / 16);
    const int blocks = (int)std::min<long long>((total + 255) / 256, (long long)p.sm_count * 8);
    rope_rotate_kernel<<<std::max(blocks, 1), 256, 0, st>>>(x, y, n_rows, n_vec, d, positions, p.rope_dev,
                                                          p.cfg.rope_max_positions, inverse ? -1.0f : 1.0f, p.status_dev);
    return cudaGetLastError();
}

cudaError_t launch_gather_rope(const kvmem_pool& p, int session_first, int n_sessions, const int32_t* sel_ids,
                               int sel_stride, const int32_t* n_sel, __nv_bfloat16* view_k, __nv_bfloat16* view_v,
                               int view_cap_tokens, int first_position, cudaStream_t st) {
    const Geometry& g = p.geo;
    GatherRopeArgs a{};
    a.pages = p.pages; a.tables = p.tables; a.nblocks_dev = p.nblocks_dev; a.sel_ids = sel_ids; a.n_sel = n_sel;
    a.view_k = view_k; a.view_v = view_v; a.rope = p.rope_dev; a.status = p.status_dev;
    a.session_first = session_first; a.sel_stride = sel_stride; a.max_bps = g.max_bps; a.max_blocks = g.max_blocks;
    a.LG = g.L * g.G; a.B = g.B; a.d = g.d; a.cap_tokens = view_cap_tokens; a.first_position = first_position;
    a.rope_positions = p.cfg.rope_max_positions; a.page_elems = p.lay.page_elems; a.in_block = p.cfg.rope_in_block_keys;
    // many short-lived CTAs (about 64 per SM over the kernel's life, 8 resident): a CTA rotates a K tile with long
    // dependent chains (table row, then arithmetic) or copies a V tile; the hardware scheduler overlaps and balances them
    // better than 8 persistent CTAs per SM do (measured at 1M: 397 us with 8 per SM, 355 us with 64)
    const int ctas = g_gather_ctas > 0 ? g_gather_ctas : std::max(1, p.sm_count * 64 / n_sessions + 1);
    launch_pdl(gather_rope_kernel, dim3(dim3((unsigned)ctas, (unsigned)n_sessions)), dim3(256), 0, st, a);
    return cudaGetLastError();
}

}  // namespace kvmem
