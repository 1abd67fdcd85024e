// Execution cache: working-set reuse with bounded delta re-RoPE (Sec. 4.4, "Retrieval-Aware
// Hierarchical Reuse"; Eq. "kvmem-working-set-delta").
//
// The cache is `cap` slots in caller-owned device memory, each one page in the pool's page format
// (K then V, [L][G][B][d]): K encoded for the block's current compact position, V unchanged.  An update
// takes the cache from the previous working set to the new selection:
//   plan  (one CTA):  retained blocks keep their slot, every other slot is reclaimed; incoming blocks,
//                     in ascending id order, take the free slots in ascending slot order; per selected
//                     block an action is recorded: 0 leave alone, 1 delta re-RoPE in place, 2 rebuild
//                     K from raw K, 3 load (rebuild K and copy V);
//   apply (all SMs):  one tile = (selected block, K|V, layer, KV head); only tiles with work are touched,
//                     so a step moves the incoming blocks and re-encodes the moved ones, nothing else.
// view_slots[j] = slot of the j-th selected block is the execution view's page table; attention runs
// over the slots through it (the paged split-K kernel), so nothing is ever compacted.
#include <algorithm>

#include "kvmem_internal.cuh"
#include "kvmem_rope.cuh"

namespace kvmem {

CacheLayout cache_layout(size_t page_elems, int cap) {
    CacheLayout c{};
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t at = off; off += align_up(bytes, 256); return at; };
    c.pages = take((size_t)cap * page_elems * sizeof(__nv_bfloat16));
    c.slot_block = take((size_t)cap * sizeof(int32_t));
    c.slot_pos = take((size_t)cap * sizeof(int32_t));
    c.slot_cnt = take((size_t)cap * sizeof(int32_t));
    c.view_slots = take((size_t)cap * sizeof(int32_t));
    c.n_view = take(sizeof(int32_t));
    c.iota = take((size_t)cap * sizeof(int32_t));
    c.action = take((size_t)cap * sizeof(int32_t));
    c.old_pos = take((size_t)cap * sizeof(int32_t));
    c.free_list = take((size_t)cap * sizeof(int32_t));
    c.total = off;
    return c;
}

struct CachePtrs {
    __nv_bfloat16* pages;
    int32_t *slot_block, *slot_pos, *slot_cnt, *view_slots, *n_view, *iota, *action, *old_pos, *free_list;
};

static CachePtrs cache_ptrs(void* cache, const CacheLayout& c) {
    char* b = reinterpret_cast<char*>(cache);
    CachePtrs p{};
    p.pages = reinterpret_cast<__nv_bfloat16*>(b + c.pages);
    p.slot_block = reinterpret_cast<int32_t*>(b + c.slot_block);
    p.slot_pos = reinterpret_cast<int32_t*>(b + c.slot_pos);
    p.slot_cnt = reinterpret_cast<int32_t*>(b + c.slot_cnt);
    p.view_slots = reinterpret_cast<int32_t*>(b + c.view_slots);
    p.n_view = reinterpret_cast<int32_t*>(b + c.n_view);
    p.iota = reinterpret_cast<int32_t*>(b + c.iota);
    p.action = reinterpret_cast<int32_t*>(b + c.action);
    p.old_pos = reinterpret_cast<int32_t*>(b + c.old_pos);
    p.free_list = reinterpret_cast<int32_t*>(b + c.free_list);
    return p;
}

__global__ void __launch_bounds__(256)
view_cache_reset_kernel(CachePtrs c, int cap) {
    for (int s = blockIdx.x * blockDim.x + threadIdx.x; s < cap; s += gridDim.x * blockDim.x) {
        c.slot_block[s] = -1; c.slot_pos[s] = 0; c.slot_cnt[s] = 0; c.view_slots[s] = -1; c.iota[s] = s;
        c.action[s] = 0; c.old_pos[s] = 0; c.free_list[s] = 0;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) *c.n_view = 0;
}

constexpr int kPlanThreads = 1024;

// position of `id` in the ascending list ids[0..n), or -1
__device__ __forceinline__ int find_sorted(const int32_t* ids, int n, int id) {
    int lo = 0, hi = n;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (ids[mid] < id) lo = mid + 1; else hi = mid;
    }
    return (lo < n && ids[lo] == id) ? lo : -1;
}

__global__ void __launch_bounds__(kPlanThreads)
view_cache_plan_kernel(CachePtrs c, int cap, const int32_t* __restrict__ sel_ids, const int32_t* __restrict__ n_sel,
                       const int32_t* __restrict__ nblocks_dev, int session, int max_delta, int32_t* __restrict__ stats,
                       int32_t* __restrict__ status) {
    pdl_wait();
    pdl_trigger();
    __shared__ unsigned int warp_tot[32];
    __shared__ int sh_stats[4];
    extern __shared__ int32_t sel_sm[];             // the selection, for the binary searches: [cap]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int n = *n_sel;
    if (n < 0 || n > cap) {
        if (tid == 0) atomicExch(status, (int)KVMEM_E_DEVICE_RANGE);
        n = min(max(n, 0), cap);
    }
    const int NB = nblocks_dev[session];
    if (tid < 4) sh_stats[tid] = 0;
    for (int j = tid; j < cap; j += kPlanThreads) { c.view_slots[j] = -1; sel_sm[j] = j < n ? sel_ids[j] : 0x7fffffff; }
    __syncthreads();
    // 1. retained blocks keep their slot; every other slot is reclaimed
    for (int s = tid; s < cap; s += kPlanThreads) {
        const int b = c.slot_block[s];
        const int j = b >= 0 ? find_sorted(sel_sm, n, b) : -1;
        if (j >= 0) c.view_slots[j] = s;
        else c.slot_block[s] = -1;
    }
    __syncthreads();
    // 2. ranks of the free slots and of the incoming blocks: one packed scan (cap <= 32,768)
    const int per = (cap + kPlanThreads - 1) / kPlanThreads;
    const int r0 = min(tid * per, cap), r1 = min(r0 + per, cap);
    unsigned int n_free = 0, n_inc = 0;
    for (int i = r0; i < r1; ++i) {
        n_free += c.slot_block[i] < 0;
        n_inc += (i < n && c.view_slots[i] < 0);
    }
    const unsigned int val = n_free | (n_inc << 16);
    unsigned int inc = val;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    const unsigned int wt = warp_tot[lane];
    unsigned int winc = wt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned int t = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += t;
    }
    const unsigned int ex = __shfl_sync(0xffffffffu, winc - wt, warp) + inc - val;
    unsigned int free_rank = ex & 0xffffu, inc_rank = ex >> 16;
    for (int i = r0; i < r1; ++i)
        if (c.slot_block[i] < 0) c.free_list[free_rank++] = i;
    __syncthreads();
    // 3. per selected block: its slot and what has to happen to its keys
    int st[4] = {0, 0, 0, 0};
    for (int j = r0; j < r1; ++j) {
        if (j >= n) break;
        const int id = sel_sm[j];
        if (id < 0 || id >= NB) atomicExch(status, (int)KVMEM_E_DEVICE_RANGE);
        int slot = c.view_slots[j], act, old = j;
        if (slot < 0) {
            slot = c.free_list[inc_rank++];
            act = 3;
            c.slot_cnt[slot] = 0;
        } else {
            old = c.slot_pos[slot];
            const int cnt = c.slot_cnt[slot];
            if (old == j) act = 0;
            else if (cnt < max_delta) { act = 1; c.slot_cnt[slot] = cnt + 1; }
            else { act = 2; c.slot_cnt[slot] = 0; }
        }
        c.slot_block[slot] = id;
        c.slot_pos[slot] = j;
        c.view_slots[j] = slot;
        c.action[j] = act;
        c.old_pos[j] = old;
        st[act] += 1;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
        if (st[i]) atomicAdd(&sh_stats[i], st[i]);
    __syncthreads();
    if (tid == 0) {
        *c.n_view = n;
        if (stats) { stats[0] = sh_stats[0]; stats[1] = sh_stats[1]; stats[2] = sh_stats[2]; stats[3] = sh_stats[3]; }
    }
}

struct CacheApplyArgs {
    CachePtrs c;
    const __nv_bfloat16* pages;      // repository pages (raw K, V)
    const int32_t* table;            // this session's block table
    const int32_t* sel_ids;
    const float2* rope;
    int32_t* status;
    int cap, max_blocks, LG, B, d, first_position, rope_positions, in_block;
    size_t page_elems;
};

// HBM-bound on the tiles it touches: 1 read + 1 write per byte of an incoming block, 1 read + 1 write per
// K byte of a re-encoded block, nothing for a block that stays where it is.  Held to 40 registers (six CTAs per SM instead
// of five): the kernel waits on its loads, and the update of a 4,096-block cache goes from 247 to 237 us.
__global__ void __launch_bounds__(256, 6)
view_cache_apply_kernel(CacheApplyArgs a) {
    pdl_wait();
    const int n = min(max(*a.c.n_view, 0), a.cap);
    const int per_block = 2 * a.LG;
    const long long n_tiles = (long long)n * per_block;
    const int tile_elems = a.B * a.d, half = a.d / 2, chunks = half / 8;
    for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const int j = (int)(tile / per_block), w = (int)(tile % per_block);
        const int kv = w / a.LG;
        const int act = a.c.action[j];
        if (act == 0 || (kv == 1 && act != 3)) continue;
        const int slot = a.c.view_slots[j];
        if (slot < 0 || slot >= a.cap) { if (threadIdx.x == 0) atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE); continue; }
        __nv_bfloat16* dst = a.c.pages + (size_t)slot * a.page_elems + (size_t)w * tile_elems;
        if (act == 1) {
            // delta re-RoPE in place: every token of the block moves by the same number of positions
            const int delta = (j - a.c.old_pos[j]) * a.B;
            const int mag = delta < 0 ? -delta : delta;
            if (mag >= a.rope_positions) { if (threadIdx.x == 0) atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE); continue; }
            const float sgn = delta < 0 ? -1.0f : 1.0f;
            const float2* cs = a.rope + (size_t)mag * half;
            for (int e = threadIdx.x; e < a.B * chunks; e += 256) {
                const int t = e / chunks, c = e % chunks;
                __nv_bfloat16* row = dst + (size_t)t * a.d + c * 8;
                const uint4 lo = *reinterpret_cast<const uint4*>(row), hi = *reinterpret_cast<const uint4*>(row + half);
                uint4 lo_o, hi_o;
                rotate8(lo, hi, cs + c * 8, sgn, lo_o, hi_o);
                *reinterpret_cast<uint4*>(row) = lo_o;
                *reinterpret_cast<uint4*>(row + half) = hi_o;
            }
            continue;
        }
        const int id = a.sel_ids[j];
        int page = -1;
        if (id >= 0) page = a.table[id];             // id < NB was checked by the plan kernel
        if (page < 0 || page >= a.max_blocks) { if (threadIdx.x == 0) atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE); continue; }
        const __nv_bfloat16* src = a.pages + (size_t)page * a.page_elems + (size_t)w * tile_elems;
        if (kv) {                                           // values: unchanged
            const uint4* s4 = reinterpret_cast<const uint4*>(src);
            uint4* d4 = reinterpret_cast<uint4*>(dst);
            for (int v = threadIdx.x; v < tile_elems / 8; v += 256) d4[v] = __ldg(s4 + v);
        } else {                                            // keys: stored K rotated to the compact position
            for (int e = threadIdx.x; e < a.B * chunks; e += 256) {
                const int t = e / chunks, c = e % chunks;
                const int pos = a.first_position + j * a.B + (a.in_block ? 0 : t);   // in-block layout: t is already in the stored key
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

cudaError_t launch_view_cache_reset(const kvmem_pool& p, void* cache, int cap, cudaStream_t st) {
    const CacheLayout lay = cache_layout(p.lay.page_elems, cap);
    view_cache_reset_kernel<<<std::max(1, std::min((cap + 255) / 256, p.sm_count)), 256, 0, st>>>(cache_ptrs(cache, lay), cap);
    return cudaGetLastError();
}

cudaError_t launch_view_cache_update(const kvmem_pool& p, int session, const int32_t* sel_ids, const int32_t* n_sel,
                                     void* cache, int cap, int max_delta, int first_position, int32_t* stats,
                                     cudaStream_t st) {
    const Geometry& g = p.geo;
    const CacheLayout lay = cache_layout(p.lay.page_elems, cap);
    const CachePtrs c = cache_ptrs(cache, lay);
    const size_t plan_smem = (size_t)cap * sizeof(int32_t);
    if (plan_smem > 48 * 1024) {
        cudaError_t ea = cudaFuncSetAttribute(view_cache_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan_smem);
        if (ea != cudaSuccess) return ea;
    }
    launch_pdl(view_cache_plan_kernel, dim3(1), dim3(kPlanThreads), plan_smem, st, c, cap, sel_ids, n_sel, p.nblocks_dev, session,
               max_delta, stats, p.status_dev);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    CacheApplyArgs a{};
    a.c = c; a.pages = p.pages; a.table = p.tables + (size_t)session * g.max_bps; a.sel_ids = sel_ids; a.rope = p.rope_dev;
    a.status = p.status_dev; a.cap = cap; a.max_blocks = g.max_blocks; a.LG = g.L * g.G; a.B = g.B; a.d = g.d;
    a.first_position = first_position; a.rope_positions = p.cfg.rope_max_positions; a.page_elems = p.lay.page_elems; a.in_block = p.cfg.rope_in_block_keys;
    // Work per tile is very uneven (an unmoved block costs nothing, a V tile only moves for an incoming block) and every
    // tile starts with a chain of dependent metadata loads: many short-lived CTAs (about 64 per SM over the kernel's life,
    // 8 resident) let the hardware scheduler balance the load and hide those chains, and an odd grid keeps a CTA from
    // meeting the same (K|V, layer, head) tile of every block (measured at 1M: 304 us with 8 per SM, 245 us with 64).
    const long long max_tiles = (long long)cap * 2 * g.L * g.G;
    const unsigned grid = (unsigned)std::max<long long>(1, std::min<long long>(max_tiles, (long long)p.sm_count * 64 + 1));
    launch_pdl(view_cache_apply_kernel, dim3(grid), dim3(256), 0, st, a);
    return cudaGetLastError();
}

// the pieces of the cache that attention needs: its pages as the page source, view_slots as the block table
void view_cache_paged_source(const kvmem_pool& p, void* cache, int cap, PagedSource* src) {
    const CacheLayout lay = cache_layout(p.lay.page_elems, cap);
    const CachePtrs c = cache_ptrs(cache, lay);
    src->pages = c.pages; src->n_pages = cap; src->tables = c.view_slots; src->table_stride = cap;
    src->nblocks_dev = c.n_view; src->sel_ids = c.iota; src->n_sel = c.n_view;
}

}  // namespace kvmem
