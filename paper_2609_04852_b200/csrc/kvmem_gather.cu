// Execution-view assembly (Sec. 4.4 "execution view"; Sec. 5.2: selected blocks, chronological,
// contiguous compact positions).  View tokens [j*B, (j+1)*B) of a session are the K and V of
// block sel_ids[j], fetched through the block table.  It is a pure byte copy: 2 bytes moved
// (one read, one write) per view byte.
//
// The unit of work is one tile = (selected block j, K|V, layer, KV head): B*d*2 bytes, contiguous
// both in the page and in the view.  A session's tiles, ordered (j, K|V, l, g), are cut into equal
// contiguous ranges, one per CTA, so consecutive tiles of a CTA share one page lookup.
//
// Two kernels do the same copy:
//   * gather_bulk_kernel: one warp per CTA drives the TMA engine.  Tiles travel
//     global -> shared with cp.async.bulk (mbarrier completion) and shared -> global with
//     cp.async.bulk (bulk-group completion) through a ring of shared-memory stages; no register
//     ever holds payload.  Lookups for the next 32 blocks are done lane-parallel ahead of use.
//   * gather_ldst_kernel: 256 threads copy each tile with 128-bit ld.global.nc / st.global.
//     Kept as the comparison point for the profiles.
#include "kvmem_internal.cuh"
#include "kvmem_ptx.cuh"

namespace kvmem {

struct GatherArgs {
    const __nv_bfloat16* pages;
    const int32_t* tables;       // [max_sessions][max_bps]
    const int32_t* nblocks_dev;  // [max_sessions]
    const int32_t* sel_ids;      // [n_sessions][sel_stride]
    const int32_t* n_sel;        // [n_sessions]
    __nv_bfloat16* view_k;
    __nv_bfloat16* view_v;
    int32_t* status;
    int session_first, sel_stride, max_bps, max_blocks;
    int LG;                      // L * G
    int tile_elems;              // B * d
    int B;
    int cap_tokens;              // view capacity in tokens
    int d;
    size_t page_elems;
    // incremental view (Eq. "kvmem-working-set-delta"): the ids the view holds now; a slot whose block stays is skipped
    const int32_t* prev_ids;     // [n_sessions][sel_stride] or null
    const int32_t* n_prev;       // [n_sessions]
};

// page of selected block j of session s; -1 (flagged) if anything is out of range, -2 if the view's slot j holds the block already
__device__ __forceinline__ int lookup_page(const GatherArgs& a, int s, int j, int NB) {
    const int id = a.sel_ids[(size_t)s * a.sel_stride + j];
    if (a.prev_ids && j < a.n_prev[s] && a.prev_ids[(size_t)s * a.sel_stride + j] == id) return -2;   // the slot already holds this block
    if (id < 0 || id >= NB) { atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE); return -1; }
    const int pg = a.tables[(size_t)(a.session_first + s) * a.max_bps + id];
    if (pg < 0 || pg >= a.max_blocks) { atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE); return -1; }
    return pg;
}

// number of selected blocks that fit the view; flags the overflow once
__device__ __forceinline__ int usable_blocks(const GatherArgs& a, int s) {
    int n = a.n_sel[s];
    const int cap_blocks = a.cap_tokens / a.B;
    if (n > a.sel_stride || n > cap_blocks) {
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE);
        n = min(min(n, a.sel_stride), cap_blocks);
    }
    return max(n, 0);
}

__device__ __forceinline__ void tile_addresses(const GatherArgs& a, int s, long long tile, int page, const __nv_bfloat16*& src,
                                               __nv_bfloat16*& dst) {
    const int per_block = 2 * a.LG;
    const int j = (int)(tile / per_block), w = (int)(tile % per_block);
    const int kv = w / a.LG, lg = w % a.LG;
    src = a.pages + (size_t)page * a.page_elems + (size_t)w * a.tile_elems;
    __nv_bfloat16* view = kv ? a.view_v : a.view_k;
    dst = view + (((size_t)s * a.LG + lg) * a.cap_tokens + (size_t)j * a.B) * a.d;
}

template <int STAGES>
__global__ void __launch_bounds__(32)
gather_bulk_kernel(GatherArgs a) {
    pdl_wait();        // everything earlier in the stream is complete and visible from here on
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ uint64_t full[STAGES];
    const int s = blockIdx.y, lane = threadIdx.x;
    const int NB = a.nblocks_dev[a.session_first + s];
    const int n_blk = usable_blocks(a, s);
    const int per_block = 2 * a.LG;
    const long long n_tiles = (long long)n_blk * per_block;
    const long long t_begin = n_tiles * blockIdx.x / gridDim.x, t_end = n_tiles * (blockIdx.x + 1) / gridDim.x;
    const int n_mine = (int)(t_end - t_begin);
    if (n_mine <= 0) return;
    const uint32_t tile_bytes = (uint32_t)a.tile_elems * 2u;

    if (lane == 0) {
        for (int i = 0; i < STAGES; ++i) ptx::mbar_init(&full[i], 1);
        ptx::fence_mbar_init();
    }
    __syncwarp();

    // lane-parallel page lookups, 32 blocks at a time
    const int j_first = (int)(t_begin / per_block);
    int j_base = j_first;
    int my_page = (j_base + lane < n_blk) ? lookup_page(a, s, j_base + lane, NB) : -1;

    auto page_of = [&](int j) -> int {          // warp-uniform j, all lanes call
        if (j >= j_base + 32) {
            j_base = j;
            my_page = (j_base + lane < n_blk) ? lookup_page(a, s, j_base + lane, NB) : -1;
        }
        return __shfl_sync(0xffffffffu, my_page, j - j_base);
    };

    bool ok = true;
    uint32_t skip_mask = 0;                     // lane 0: stages whose tile belongs to a flagged id (nothing loaded, nothing stored)
    auto issue_load = [&](int i) {              // tile i of this CTA into stage i % STAGES
        const long long tile = t_begin + i;
        const int page = page_of((int)(tile / per_block));
        if (lane == 0) {
            const int st = i % STAGES;
            if (page < 0) {                     // flagged lookup: the tile is skipped, the status word reports it
                skip_mask |= 1u << st;
            } else {
                const __nv_bfloat16* src;
                __nv_bfloat16* dst;
                tile_addresses(a, s, tile, page, src, dst);
                ptx::mbar_expect_tx(&full[st], tile_bytes);
                ptx::bulk_g2s(smem + (size_t)st * tile_bytes, src, tile_bytes, &full[st]);
            }
        }
    };

    const int prologue = min(STAGES - 1, n_mine);
    for (int i = 0; i < prologue; ++i) issue_load(i);

    uint32_t phase_mask = 0;                    // lane 0: parity of the next completion of each stage's barrier
    for (int i = 0; i < n_mine; ++i) {
        const int st = i % STAGES;
        if (lane == 0) {
            if (skip_mask & (1u << st)) {
                skip_mask &= ~(1u << st);
                ptx::bulk_commit();             // an empty group keeps the group count of the refill logic in step
            } else if ((ok = ptx::mbar_wait(&full[st], (phase_mask >> st) & 1u))) {
                phase_mask ^= 1u << st;
                const __nv_bfloat16* src;
                __nv_bfloat16* dst;
                tile_addresses(a, s, t_begin + i, 0, src, dst);
                ptx::bulk_s2g(dst, smem + (size_t)st * tile_bytes, tile_bytes);
                ptx::bulk_commit();
            }
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        // refill the stage whose store was committed one iteration ago
        const int nxt = i + STAGES - 1;
        if (nxt < n_mine) {
            if (lane == 0) ptx::bulk_wait_read<1>();   // all but the newest store have left shared memory
            __syncwarp();
            issue_load(nxt);
        }
    }
    if (lane == 0) {
        ptx::bulk_wait<0>();
        if (!ok) atomicExch(a.status, (int)KVMEM_E_TIMEOUT);
    }
}

__global__ void __launch_bounds__(256)
gather_ldst_kernel(GatherArgs a) {
    pdl_wait();        // everything earlier in the stream is complete and visible from here on
    const int s = blockIdx.y;
    const int NB = a.nblocks_dev[a.session_first + s];
    const int n_blk = usable_blocks(a, s);
    const int per_block = 2 * a.LG;
    const long long n_tiles = (long long)n_blk * per_block;
    const long long t_begin = n_tiles * blockIdx.x / gridDim.x, t_end = n_tiles * (blockIdx.x + 1) / gridDim.x;
    const int vec_per_tile = a.tile_elems / 8;
    int cached_j = -1, page = -1;
    for (long long tile = t_begin; tile < t_end; ++tile) {
        const int j = (int)(tile / per_block);
        if (j != cached_j) { page = lookup_page(a, s, j, NB); cached_j = j; }
        if (page < 0) continue;
        const __nv_bfloat16* src;
        __nv_bfloat16* dst;
        tile_addresses(a, s, tile, page, src, dst);
        const uint4* s4 = reinterpret_cast<const uint4*>(src);
        uint4* d4 = reinterpret_cast<uint4*>(dst);
        for (int v = threadIdx.x; v < vec_per_tile; v += 4 * 256) {
            uint4 r[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (v + u * 256 < vec_per_tile) r[u] = __ldg(s4 + v + u * 256);
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (v + u * 256 < vec_per_tile) d4[v + u * 256] = r[u];
        }
    }
}

Option g_pdl{1};           // programmatic dependent launch of the step's kernels
Option g_gather_ctas{0};    // 0: as many single-warp CTAs as fit; > 0: at most this many (kernel-variant switch)
Option g_gather_mode{1};   // 1: TMA bulk ring, 0: ld/st

// Per session: how many slots of the new view keep their block, receive a retained block that sat elsewhere, receive an
// incoming block (the counts of the working-set delta, Eq. "kvmem-working-set-delta").  One CTA per session.
__global__ void __launch_bounds__(256)
view_delta_stats_kernel(const int32_t* __restrict__ prev_ids, const int32_t* __restrict__ n_prev, const int32_t* __restrict__ sel_ids,
                        const int32_t* __restrict__ n_sel, int sel_stride, int32_t* __restrict__ stats) {
    pdl_wait();
    __shared__ int cnt[3];
    const int s = blockIdx.x;
    if (threadIdx.x < 3) cnt[threadIdx.x] = 0;
    __syncthreads();
    const int np = min(max(n_prev[s], 0), sel_stride), nn = min(max(n_sel[s], 0), sel_stride);
    const int32_t* prev = prev_ids + (size_t)s * sel_stride;
    const int32_t* next = sel_ids + (size_t)s * sel_stride;
    int mine[3] = {0, 0, 0};
    for (int j = threadIdx.x; j < nn; j += blockDim.x) {
        const int id = next[j];
        int act = 2;
        if (j < np && prev[j] == id) act = 0;
        else {
            int lo = 0, hi = np - 1;                         // prev is ascending: binary search
            while (lo <= hi) {
                const int mid = (lo + hi) >> 1, v = prev[mid];
                if (v == id) { act = 1; break; }
                if (v < id) lo = mid + 1; else hi = mid - 1;
            }
        }
        mine[act] += 1;
    }
#pragma unroll
    for (int i = 0; i < 3; ++i)
        if (mine[i]) atomicAdd(&cnt[i], mine[i]);
    __syncthreads();
    if (threadIdx.x < 3) stats[(size_t)s * 3 + threadIdx.x] = cnt[threadIdx.x];
}

cudaError_t launch_gather(const kvmem_pool& p, int session_first, int n_sessions, const int32_t* sel_ids,
                          int sel_stride, const int32_t* n_sel, __nv_bfloat16* view_k, __nv_bfloat16* view_v,
                          int view_cap_tokens, cudaStream_t st, const int32_t* prev_ids, const int32_t* n_prev, int32_t* delta_stats) {
    const Geometry& g = p.geo;
    if (prev_ids && delta_stats) {
        launch_pdl(view_delta_stats_kernel, dim3((unsigned)n_sessions), dim3(256), 0, st, prev_ids, n_prev, sel_ids, n_sel, sel_stride, delta_stats);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    GatherArgs a{};
    a.prev_ids = prev_ids; a.n_prev = n_prev;
    a.pages = p.pages; a.tables = p.tables; a.nblocks_dev = p.nblocks_dev;
    a.sel_ids = sel_ids; a.n_sel = n_sel; a.view_k = view_k; a.view_v = view_v; a.status = p.status_dev;
    a.session_first = session_first; a.sel_stride = sel_stride; a.max_bps = g.max_bps; a.max_blocks = g.max_blocks;
    a.LG = g.L * g.G; a.tile_elems = g.B * g.d; a.B = g.B; a.cap_tokens = view_cap_tokens; a.d = g.d;
    a.page_elems = p.lay.page_elems;
    const size_t tile_bytes = (size_t)a.tile_elems * 2;
    if (g_gather_mode == 1 && tile_bytes % 16 == 0 && tile_bytes * 4 <= 200 * 1024) {
        constexpr int STAGES = 4;
        const size_t smem = tile_bytes * STAGES;
        static PerDeviceOnce attr_done;
        if (attr_done.pending(p.cfg.device)) {
            cudaError_t e = cudaFuncSetAttribute(gather_bulk_kernel<STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 200 * 1024);
            if (e != cudaSuccess) return e;
            attr_done.mark(p.cfg.device);
        }
        // as many single-warp CTAs as fit the shared memory of every SM, split evenly over the sessions
        const int per_sm = std::max(1, (int)((220 * 1024) / (smem + 1024)));
        // Measured on this part: the copy is fastest with about 12 MiB in flight over all SMs (185 CTAs of 64 KiB at
        // 16 KiB tiles: 98.7 % of the copy peak); with every CTA that fits (444) it loses 4-5 % to read/write turn-arounds.
        const int fit = p.sm_count * per_sm;
        int total = g_gather_ctas > 0 ? g_gather_ctas : std::max(p.sm_count, (int)((12u << 20) / smem));
        total = std::min(total, fit);
        const int ctas = std::max(1, total / n_sessions);
        dim3 grid((unsigned)ctas, (unsigned)n_sessions);
        launch_pdl(gather_bulk_kernel<STAGES>, dim3(grid), dim3(32), smem, st, a);
    } else {
        const int ctas = std::max(1, p.sm_count * 8 / n_sessions);
        dim3 grid((unsigned)ctas, (unsigned)n_sessions);
        launch_pdl(gather_ldst_kernel, dim3(grid), dim3(256), 0, st, a);
    }
    return cudaGetLastError();
}

}  // namespace kvmem
