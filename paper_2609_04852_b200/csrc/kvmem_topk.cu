// Selector (Sec. 4.3: reserve sink and recent blocks, fill the rest of the budget with the largest
// R_b, restore chronological order; budget from Eq. "active_budget" / Eq. "active_capacity").
//
// One CTA per session.  Scores are non-negative fp32, so their bit patterns order like unsigned
// integers.  MSB-first 8-bit radix passes over the non-reserved candidates, starting at the highest
// bit in which two candidates differ, narrow down the value T of the k'-th largest score and how many
// candidates are strictly larger (histograms in shared memory, 8 copies to spread the atomics).  The
// passes stop as soon as the bin that holds the k'-th largest is needed whole, or holds at most 32
// candidates, which one warp then ranks directly.  A final ascending sweep over block ids flags reserved
// blocks, every candidate above T, and the first (k' - above) ones equal to T, i.e. equal scores go to
// the lower id, compacts the flagged ids with a block-wide prefix sum into shared memory and writes
// them out coalesced: the output is chronological without a sort, and identical from run to run.
#include <algorithm>

#include <cooperative_groups.h>

#include "kvmem_internal.cuh"

namespace kvmem {

constexpr int kTopkThreads = 1024;
constexpr int kItems = 16;                                  // consecutive block ids per thread and tile
constexpr int kTopkTile = kTopkThreads * kItems;            // 16,384 ids per sweep

constexpr int kHistCopies = 8;                              // warp w adds into copy w % 8: 8x less same-address contention

struct TopkShared {
    unsigned int hist[kHistCopies][256];
    unsigned int warp_tot[32];
    unsigned int warp_min[32], warp_max[32];
    unsigned int bin_tot[256];
    unsigned int small[32];                     // the candidates of the boundary bin, once there are at most 32
    unsigned int prefix, remaining, bin_count, n_small;
};

// exclusive prefix of `val` over the CTA (thread order) and the CTA total; two barriers
__device__ __forceinline__ unsigned block_exclusive_scan(unsigned val, TopkShared& sh, unsigned& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned inc = val;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) sh.warp_tot[warp] = inc;
    __syncthreads();
    const unsigned wt = sh.warp_tot[lane];                  // kTopkThreads / 32 == 32 warps
    unsigned winc = wt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += t;
    }
    const unsigned warp_off = __shfl_sync(0xffffffffu, winc - wt, warp);
    total = __shfl_sync(0xffffffffu, winc, 31);
    __syncthreads();
    return warp_off + inc - val;
}

// REG = true (sessions of at most 1,024 * ITEMS blocks): the scores are loaded once and then live in registers,
// ITEMS consecutive ids per thread, for every later pass (ITEMS = 16: staged through shared memory so that the
// global loads stay coalesced; fewer: each thread loads its own 4 to 32 contiguous bytes).  The kernel is bound by
// instruction issue and barrier latency on its one SM, so a short session takes the instantiation with the
// fewest items per thread that covers it.
// REG = false: any length; every pass re-reads the scores from global memory.
constexpr int kStagePitch = kItems + 4;                     // floats per thread in the staging buffer: conflict-free 128-bit reads

template <bool REG, int ITEMS>
__global__ void __launch_bounds__(kTopkThreads)
topk_kernel(const float* __restrict__ scores, int scores_stride, const int32_t* __restrict__ nblocks_dev,
            int session_first, int B, kvmem_select_params_t prm, int32_t* __restrict__ sel_ids, int sel_stride,
            int32_t* __restrict__ n_sel, int32_t* __restrict__ status) {
    pdl_wait();        // everything earlier in the stream is complete and visible from here on
    pdl_trigger();     // the next kernel's CTAs may take their places; they wait in the same way
    __shared__ TopkShared sh;
    extern __shared__ __align__(16) unsigned int stage[];   // [kTopkThreads][kStagePitch] score staging (REG), then kTopkTile output ids
    const int s = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    // The session's block count and its scores are requested together: the vector reads below are bounded by the row
    // length (readable whatever the count is) and masked by the count afterwards, one memory round trip instead of two.
    const int NB = nblocks_dev[session_first + s];
    const int row_len = scores_stride;
    const unsigned int* bits = reinterpret_cast<const unsigned int*>(scores + (size_t)s * scores_stride);
    int32_t* out = sel_ids + (size_t)s * sel_stride;
    constexpr int kItems = ITEMS, kTopkTile = kTopkThreads * ITEMS;      // shadow the file-scope values of the 16-item layout
    unsigned int vreg[kItems];
    if constexpr (REG && ITEMS < 16) {
        if (ITEMS % 4 == 0 && (reinterpret_cast<uintptr_t>(bits) & 15u) == 0) {
#pragma unroll
            for (int j = 0; j < ITEMS / 4; ++j) {
                const int g4 = tid * (ITEMS / 4) + j;                      // ids 4*g4 .. 4*g4 + 3
                uint4 u = make_uint4(0u, 0u, 0u, 0u);
                if (4 * g4 + 3 < row_len) {
                    u = *reinterpret_cast<const uint4*>(bits + 4 * g4);
                } else if (4 * g4 < row_len) {
                    u.x = bits[4 * g4];
                    if (4 * g4 + 1 < row_len) u.y = bits[4 * g4 + 1];
                    if (4 * g4 + 2 < row_len) u.z = bits[4 * g4 + 2];
                }
                vreg[(4 * j) % ITEMS] = u.x; vreg[(4 * j + 1) % ITEMS] = u.y; vreg[(4 * j + 2) % ITEMS] = u.z; vreg[(4 * j + 3) % ITEMS] = u.w;
            }
#pragma unroll
            for (int i = 0; i < ITEMS; ++i) vreg[i] = tid * ITEMS + i < NB ? vreg[i] : 0u;
        } else {
#pragma unroll
            for (int i = 0; i < ITEMS; ++i) {
                const int idx = tid * ITEMS + i;
                vreg[i] = idx < NB ? bits[idx] : 0u;
            }
        }
    } else if constexpr (REG) {
        if ((reinterpret_cast<uintptr_t>(bits) & 15u) == 0) {
            // coalesced 128-bit global reads, all of a thread's loads in flight before the first use
            uint4 u[kItems / 4];
#pragma unroll
            for (int j = 0; j < kItems / 4; ++j) {
                const int g4 = j * kTopkThreads + tid;                     // group of ids 4*g4 .. 4*g4 + 3
                u[j] = make_uint4(0u, 0u, 0u, 0u);
                if (4 * g4 + 3 < row_len) {
                    u[j] = *reinterpret_cast<const uint4*>(bits + 4 * g4);
                } else if (4 * g4 < row_len) {
                    u[j].x = bits[4 * g4];
                    if (4 * g4 + 1 < row_len) u[j].y = bits[4 * g4 + 1];
                    if (4 * g4 + 2 < row_len) u[j].z = bits[4 * g4 + 2];
                }
            }
#pragma unroll
            for (int j = 0; j < kItems / 4; ++j) {
                const int g4 = j * kTopkThreads + tid;
                u[j].x = 4 * g4 < NB ? u[j].x : 0u;
                u[j].y = 4 * g4 + 1 < NB ? u[j].y : 0u;
                u[j].z = 4 * g4 + 2 < NB ? u[j].z : 0u;
                u[j].w = 4 * g4 + 3 < NB ? u[j].w : 0u;
                *reinterpret_cast<uint4*>(&stage[(g4 / (kItems / 4)) * kStagePitch + (g4 % (kItems / 4)) * 4]) = u[j];
            }
        } else {
            for (int idx = tid; idx < kTopkTile; idx += kTopkThreads)      // coalesced 32-bit reads
                stage[(idx / kItems) * kStagePitch + (idx % kItems)] = idx < NB ? bits[idx] : 0u;
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kItems; i += 4) {
            const uint4 u = *reinterpret_cast<const uint4*>(&stage[tid * kStagePitch + i]);
            vreg[i] = u.x; vreg[i + 1] = u.y; vreg[i + 2] = u.z; vreg[i + 3] = u.w;
        }
    }
    // score bits of id (base + tid * kItems + i)
#define KVMEM_TOPK_VAL(base, i) (REG ? vreg[i] : bits[(base) + tid * kItems + (i)])

    // budget clamp
    long long room = (long long)prm.max_view_tokens - (long long)prm.mandatory_tokens;
    long long kk = room <= 0 ? 0 : room <= 0x7fffffffll ? (long long)((int)room / B) : room / B;   // 32-bit division on the usual path
    if (prm.budget_blocks < kk) kk = prm.budget_blocks;
    if (NB < kk) kk = NB;
    if (kk < 0) kk = 0;
    if (kk > sel_stride) {                      // the host checked this against its own block counts
        if (tid == 0) atomicExch(status, (int)KVMEM_E_DEVICE_RANGE);
        kk = sel_stride;
    }
    const int k = (int)kk;
    if (k == 0) {
        if (tid == 0) n_sel[s] = 0;
        return;
    }
    // reserved ranges: sinks [0, n_sink), recents [recent_lo, NB)
    const int n_sink = min(prm.n_sink_blocks, k);
    int recent_lo = max(NB - prm.n_recent_blocks, n_sink);
    recent_lo = max(recent_lo, NB - (k - n_sink));
    recent_lo = min(max(recent_lo, 0), NB);
    const int n_cand = recent_lo - n_sink;
    const int kc = k - n_sink - (NB - recent_lo);          // slots left for scored candidates
    unsigned int T = 0xffffffffu, need_eq = 0;             // defaults: nothing from the candidates

    if (kc > 0 && kc >= n_cand) {
        T = 0u; need_eq = 0xffffffffu;                     // every candidate is kept
    } else if (kc > 0) {
        // range of the candidates' bit patterns: bits above the highest differing bit are common to all
        unsigned int lo = 0xffffffffu, hi = 0u;
        for (int base = 0; base < NB; base += kTopkTile) {
            const int b0 = base + tid * kItems;
#pragma unroll
            for (int i = 0; i < kItems; ++i) {
                const int b = b0 + i;
                if (b >= n_sink && b < recent_lo) { const unsigned int v = KVMEM_TOPK_VAL(base, i); lo = min(lo, v); hi = max(hi, v); }
            }
        }
        lo = __reduce_min_sync(0xffffffffu, lo);
        hi = __reduce_max_sync(0xffffffffu, hi);
        if (lane == 0) { sh.warp_min[tid >> 5] = lo; sh.warp_max[tid >> 5] = hi; }
        __syncthreads();
        lo = __reduce_min_sync(0xffffffffu, sh.warp_min[lane]);
        hi = __reduce_max_sync(0xffffffffu, sh.warp_max[lane]);
        if (lo == hi) {
            T = lo; need_eq = (unsigned)kc;                // all candidates tie: the lowest ids win
        } else {
            const int hb = 31 - __clz(lo ^ hi);            // highest bit in which two candidates differ
            unsigned int known = hb >= 31 ? 0u : ~((2u << hb) - 1u);
            if (tid == 0) { sh.prefix = hi & known; sh.remaining = (unsigned)kc; sh.n_small = 0u; }
            for (int i = tid; i < kHistCopies * 256; i += kTopkThreads) (&sh.hist[0][0])[i] = 0u;
            __syncthreads();
            int shift = max(hb - 7, 0);
            while (true) {
                const unsigned int prefix = sh.prefix;
                unsigned int* my_hist = sh.hist[(tid >> 5) % kHistCopies];
                for (int base = 0; base < NB; base += kTopkTile) {
                    const int b0 = base + tid * kItems;
#pragma unroll
                    for (int i = 0; i < kItems; ++i) {
                        const int b = b0 + i;
                        unsigned int v = 0;
                        bool live = b >= n_sink && b < recent_lo;
                        if (live) { v = KVMEM_TOPK_VAL(base, i); live = (v & known) == prefix; }
                        if (live) atomicAdd(&my_hist[(v >> shift) & 255u], 1u);
                    }
                }
                __syncthreads();
                if (tid < 256) {
                    // thread t adds the copies of bin t (conflict-free) and leaves them zeroed for the next pass
                    unsigned int t = 0;
#pragma unroll
                    for (int k2 = 0; k2 < kHistCopies; ++k2) { t += sh.hist[k2][tid]; sh.hist[k2][tid] = 0u; }
                    sh.bin_tot[tid] = t;
                }
                __syncthreads();
                if (tid < 32) {
                    // warp 0 walks the 256 bins from the top: lane i owns bins [255 - 8i - 7, 255 - 8i]
                    const unsigned int rem = sh.remaining;
                    unsigned int c[8], mine = 0;
#pragma unroll
                    for (int j = 0; j < 8; ++j) { c[j] = sh.bin_tot[255 - 8 * lane - j]; mine += c[j]; }
                    unsigned int inc = mine;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const unsigned int t = __shfl_up_sync(0xffffffffu, inc, o);
                        if (lane >= o) inc += t;
                    }
                    const unsigned int before = inc - mine;            // candidates in bins above this lane's
                    const bool here = before < rem && rem <= inc;      // the k-th largest falls into my bins
                    // (if the counts were inconsistent nobody would claim it; the last lane then takes bin 0)
                    const unsigned int claim = __ballot_sync(0xffffffffu, here);
                    if (here || (claim == 0u && lane == 31)) {
                        unsigned int left = rem - before;
                        int bin = 255 - 8 * lane, j = 0;
                        for (; j < 7; ++j) {
                            if (c[j] >= left) break;
                            left -= c[j];
                            --bin;
                        }
                        sh.prefix = (prefix & ~(255u << shift)) | ((unsigned)bin << shift);
                        sh.remaining = left;                           // how many of this digit are still needed
                        sh.bin_count = c[j];                           // how many candidates carry this digit
                    }
                }
                __syncthreads();
                known |= 255u << shift;
                const unsigned int left = sh.remaining, in_bin = sh.bin_count;
                if (shift == 0) { T = sh.prefix; need_eq = left; break; }
                if (in_bin <= left) {
                    // the whole bin is needed: everything at or above its lowest possible value is kept
                    T = sh.prefix; need_eq = 0xffffffffu;
                    break;
                }
                if (in_bin <= 32u) {
                    // few candidates left: collect them (order does not matter) and let one warp rank them
                    const unsigned int pfx = sh.prefix;
                    for (int base = 0; base < NB; base += kTopkTile) {
                        const int b0 = base + tid * kItems;
#pragma unroll
                        for (int i = 0; i < kItems; ++i) {
                            const int b = b0 + i;
                            if (b >= n_sink && b < recent_lo) {
                                const unsigned int v = KVMEM_TOPK_VAL(base, i);
                                if ((v & known) == pfx) {
                                    const unsigned int slot = atomicAdd(&sh.n_small, 1u);
                                    if (slot < 32u) sh.small[slot] = v;
                                }
                            }
                        }
                    }
                    __syncthreads();
                    if (tid < 32) {
                        const unsigned int n = min(sh.n_small, 32u);
                        const unsigned int mine = lane < n ? sh.small[lane] : 0u;
                        unsigned int gt = 0, eq = 0;
                        for (unsigned int j = 0; j < n; ++j) {
                            const unsigned int o = __shfl_sync(0xffffffffu, mine, (int)j);
                            gt += o > mine;
                            eq += o == mine;
                        }
                        if (lane < n && gt < left && left <= gt + eq) { sh.prefix = mine; sh.remaining = left - gt; }
                    }
                    __syncthreads();
                    T = sh.prefix; need_eq = sh.remaining;
                    break;
                }
                shift = max(shift - 8, 0);
            }
        }
    }

    // ascending sweep: each thread owns kItems consecutive ids, so thread order is id order
    unsigned carry_eq = 0, carry_sel = 0;
    for (int base = 0; base < NB; base += kTopkTile) {
        const int b0 = base + tid * kItems;
        unsigned flags_res = 0, flags_gt = 0, flags_eq = 0;
#pragma unroll
        for (int i = 0; i < kItems; ++i) {
            const int b = b0 + i;
            if (b < NB) {
                if (b < n_sink || b >= recent_lo) flags_res |= 1u << i;
                else if (kc > 0) {
                    const unsigned int v = KVMEM_TOPK_VAL(base, i);
                    if (v > T) flags_gt |= 1u << i;
                    else if (v == T) flags_eq |= 1u << i;
                }
            }
        }
        // one scan of (kept for sure | equal to T) counts, 16 bits each (a sweep covers 16,384 ids); the
        // equal ones are kept in id order until need_eq of them are in
        const unsigned sure = flags_res | flags_gt;
        unsigned tot_packed;
        const unsigned ex = block_exclusive_scan((unsigned)__popc(sure) | ((unsigned)__popc(flags_eq) << 16), sh, tot_packed);
        unsigned eq_rank = carry_eq + (ex >> 16);
        const unsigned tot_eq = tot_packed >> 16;
        const unsigned eq_left_before = need_eq > carry_eq ? need_eq - carry_eq : 0u;     // equal ones this sweep may still take
        const unsigned tot_sel = (tot_packed & 0xffffu) + min(tot_eq, eq_left_before);
        unsigned rel = (ex & 0xffffu) + min(ex >> 16, eq_left_before);
        unsigned take = sure;
#pragma unroll
        for (int i = 0; i < kItems; ++i)
            if (flags_eq & (1u << i)) { if (eq_rank < need_eq) take |= 1u << i; ++eq_rank; }
        // compact into shared memory (scattered 4-byte writes are cheap there), then write out coalesced
        int* outbuf = reinterpret_cast<int*>(stage);                   // at most kTopkTile ids per sweep
#pragma unroll
        for (int i = 0; i < kItems; ++i)
            if (take & (1u << i)) outbuf[rel++] = b0 + i;
        __syncthreads();
        for (unsigned i = tid; i < tot_sel; i += kTopkThreads)
            if (carry_sel + i < (unsigned)sel_stride) out[carry_sel + i] = outbuf[i];
        __syncthreads();
        carry_eq += tot_eq;
        carry_sel += tot_sel;
    }
    if (tid == 0) n_sel[s] = (int32_t)min(carry_sel, (unsigned)sel_stride);
#undef KVMEM_TOPK_VAL
}

// ---------------------------------------------------------------------------------------------------
// Sessions of more than 16,384 blocks: the same selection by a thread-block cluster.  Tile t (16,384
// consecutive ids) belongs to CTA t mod 8 of the cluster.  Every radix pass builds its histogram per CTA,
// the eight histograms are added through distributed shared memory, and every CTA takes the same
// decision from the same totals; the final sweep ranks the tiles through per-tile counts published the
// same way.  All cluster-wide steps are hardware cluster barriers (no spinning), and every CTA meets
// the same barriers because every branch between them depends on cluster-wide values only.
constexpr int kTopkCluster = 8;
constexpr int kTopkMaxOwnTiles = 64;             // tiles per CTA: 8 * 64 * 16,384 blocks per session at most

struct TopkClusterShared {
    unsigned int hist[kHistCopies][256];
    unsigned int bin_tot[256];                   // this CTA's bin totals of the current pass (read by the others)
    unsigned int all_tot[256];                   // the cluster's totals
    unsigned int warp_tot[32];
    unsigned int warp_min[32], warp_max[32];
    unsigned int cta_min, cta_max;               // (read by the others)
    unsigned int small[32], n_small;             // this CTA's candidates of a small boundary bin (read by the others)
    unsigned int tile_counts[kTopkMaxOwnTiles];  // per own tile: kept for sure | equal to T << 16 (read by the others)
    unsigned int prefix, remaining, bin_count;
    unsigned int carry_sel, carry_eq;
};

__device__ __forceinline__ unsigned cluster_block_scan(unsigned val, unsigned int* warp_tot, unsigned& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned inc = val;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    const unsigned wt = warp_tot[lane];
    unsigned winc = wt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += t;
    }
    const unsigned warp_off = __shfl_sync(0xffffffffu, winc - wt, warp);
    total = __shfl_sync(0xffffffffu, winc, 31);
    __syncthreads();
    return warp_off + inc - val;
}

__global__ void __launch_bounds__(kTopkThreads)
topk_cluster_kernel(const float* __restrict__ scores, int scores_stride, const int32_t* __restrict__ nblocks_dev,
                    int session_first, int B, kvmem_select_params_t prm, int32_t* __restrict__ sel_ids, int sel_stride,
                    int32_t* __restrict__ n_sel, int32_t* __restrict__ status) {
    pdl_wait();
    pdl_trigger();
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    __shared__ TopkClusterShared sh;
    extern __shared__ __align__(16) unsigned int stage[];   // [kTopkThreads][kStagePitch] scores of a tile, then its output ids
    const int rank = (int)cluster.block_rank();
    const int s = blockIdx.x / kTopkCluster, tid = threadIdx.x, lane = tid & 31;
    const int NB = nblocks_dev[session_first + s];
    const unsigned int* bits = reinterpret_cast<const unsigned int*>(scores + (size_t)s * scores_stride);
    int32_t* out = sel_ids + (size_t)s * sel_stride;
    const int n_tiles = (NB + kTopkTile - 1) / kTopkTile;
    auto remote = [&](int r) { return cluster.map_shared_rank(&sh, r); };

    long long room = (long long)prm.max_view_tokens - (long long)prm.mandatory_tokens;
    long long kk = room <= 0 ? 0 : room <= 0x7fffffffll ? (long long)((int)room / B) : room / B;
    if (prm.budget_blocks < kk) kk = prm.budget_blocks;
    if (NB < kk) kk = NB;
    if (kk < 0) kk = 0;
    if (kk > sel_stride) {
        if (tid == 0 && rank == 0) atomicExch(status, (int)KVMEM_E_DEVICE_RANGE);
        kk = sel_stride;
    }
    const int k = (int)kk;
    if (k == 0) {                                // cluster-uniform: nobody waits for anybody
        if (tid == 0 && rank == 0) n_sel[s] = 0;
        return;
    }
    const int n_sink = min(prm.n_sink_blocks, k);
    int recent_lo = max(NB - prm.n_recent_blocks, n_sink);
    recent_lo = max(recent_lo, NB - (k - n_sink));
    recent_lo = min(max(recent_lo, 0), NB);
    const int n_cand = recent_lo - n_sink;
    const int kc = k - n_sink - (NB - recent_lo);
    unsigned int T = 0xffffffffu, need_eq = 0;
    if (tid == 0) sh.n_small = 0u;

    if (kc > 0 && kc >= n_cand) {
        T = 0u; need_eq = 0xffffffffu;
    } else if (kc > 0) {
        unsigned int lo = 0xffffffffu, hi = 0u;
        // order does not matter in the counting passes: consecutive lanes read consecutive ids
        for (int t = rank; t < n_tiles; t += kTopkCluster) {
#pragma unroll
            for (int i = 0; i < kItems; ++i) {
                const int b = t * kTopkTile + i * kTopkThreads + tid;
                if (b >= n_sink && b < recent_lo) { const unsigned int v = bits[b]; lo = min(lo, v); hi = max(hi, v); }
            }
        }
        lo = __reduce_min_sync(0xffffffffu, lo);
        hi = __reduce_max_sync(0xffffffffu, hi);
        if (lane == 0) { sh.warp_min[tid >> 5] = lo; sh.warp_max[tid >> 5] = hi; }
        __syncthreads();
        if (tid < 32) {
            lo = __reduce_min_sync(0xffffffffu, sh.warp_min[lane]);
            hi = __reduce_max_sync(0xffffffffu, sh.warp_max[lane]);
            if (lane == 0) { sh.cta_min = lo; sh.cta_max = hi; }
        }
        cluster.sync();
        lo = 0xffffffffu; hi = 0u;
        for (int r = 0; r < kTopkCluster; ++r) { lo = min(lo, remote(r)->cta_min); hi = max(hi, remote(r)->cta_max); }
        if (lo == hi) {
            T = lo; need_eq = (unsigned)kc;
        } else {
            const int hb = 31 - __clz(lo ^ hi);
            unsigned int known = hb >= 31 ? 0u : ~((2u << hb) - 1u);
            unsigned int prefix = hi & known, remaining = (unsigned)kc;      // identical in every thread of the cluster
            for (int i = tid; i < kHistCopies * 256; i += kTopkThreads) (&sh.hist[0][0])[i] = 0u;
            __syncthreads();
            int shift = max(hb - 7, 0);
            while (true) {
                unsigned int* my_hist = sh.hist[(tid >> 5) % kHistCopies];
                for (int t = rank; t < n_tiles; t += kTopkCluster) {
#pragma unroll
                    for (int i = 0; i < kItems; ++i) {
                        const int b = t * kTopkTile + i * kTopkThreads + tid;
                        if (b >= n_sink && b < recent_lo) {
                            const unsigned int v = bits[b];
                            if ((v & known) == prefix) atomicAdd(&my_hist[(v >> shift) & 255u], 1u);
                        }
                    }
                }
                __syncthreads();
                if (tid < 256) {
                    unsigned int t = 0;
#pragma unroll
                    for (int k2 = 0; k2 < kHistCopies; ++k2) { t += sh.hist[k2][tid]; sh.hist[k2][tid] = 0u; }
                    sh.bin_tot[tid] = t;
                }
                cluster.sync();                              // every CTA's bin totals are in place
                if (tid < 256) {
                    unsigned int t = 0;
                    for (int r = 0; r < kTopkCluster; ++r) t += remote(r)->bin_tot[tid];
                    sh.all_tot[tid] = t;
                }
                __syncthreads();
                if (tid < 32) {
                    unsigned int c[8], mine = 0;
#pragma unroll
                    for (int j = 0; j < 8; ++j) { c[j] = sh.all_tot[255 - 8 * lane - j]; mine += c[j]; }
                    unsigned int inc = mine;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const unsigned int t = __shfl_up_sync(0xffffffffu, inc, o);
                        if (lane >= o) inc += t;
                    }
                    const unsigned int before = inc - mine;
                    const bool here = before < remaining && remaining <= inc;
                    const unsigned int claim = __ballot_sync(0xffffffffu, here);
                    if (here || (claim == 0u && lane == 31)) {
                        unsigned int left = remaining - before;
                        int bin = 255 - 8 * lane, j = 0;
                        for (; j < 7; ++j) {
                            if (c[j] >= left) break;
                            left -= c[j];
                            --bin;
                        }
                        sh.prefix = (prefix & ~(255u << shift)) | ((unsigned)bin << shift);
                        sh.remaining = left;
                        sh.bin_count = c[j];
                    }
                }
                __syncthreads();
                cluster.sync();                              // everybody has read everybody's totals: they may be rewritten
                known |= 255u << shift;
                prefix = sh.prefix; remaining = sh.remaining;
                const unsigned int in_bin = sh.bin_count;
                if (shift == 0) { T = prefix; need_eq = remaining; break; }
                if (in_bin <= remaining) { T = prefix; need_eq = 0xffffffffu; break; }
                if (in_bin <= 32u) {
                    for (int t = rank; t < n_tiles; t += kTopkCluster) {
#pragma unroll
                        for (int i = 0; i < kItems; ++i) {
                            const int b = t * kTopkTile + i * kTopkThreads + tid;
                            if (b >= n_sink && b < recent_lo) {
                                const unsigned int v = bits[b];
                                if ((v & known) == prefix) {
                                    const unsigned int slot = atomicAdd(&sh.n_small, 1u);
                                    if (slot < 32u) sh.small[slot] = v;
                                }
                            }
                        }
                    }
                    cluster.sync();                          // every CTA's short list is complete
                    if (tid < 32) {
                        // lane i takes the i-th candidate of the cluster (ranks in order, then slots in order)
                        unsigned int mine = 0, n = 0;
                        for (int r = 0; r < kTopkCluster; ++r) {
                            const unsigned int nr = min(remote(r)->n_small, 32u);
                            if ((unsigned)lane >= n && (unsigned)lane < n + nr) mine = remote(r)->small[lane - n];
                            n += nr;
                        }
                        n = min(n, 32u);
                        unsigned int gt = 0, eq = 0;
                        for (unsigned int j = 0; j < n; ++j) {
                            const unsigned int o = __shfl_sync(0xffffffffu, mine, (int)j);
                            gt += o > mine;
                            eq += o == mine;
                        }
                        if ((unsigned)lane < n && gt < remaining && remaining <= gt + eq) { sh.prefix = mine; sh.remaining = remaining - gt; }
                    }
                    __syncthreads();
                    T = sh.prefix; need_eq = sh.remaining;
                    break;
                }
                shift = max(shift - 8, 0);
            }
        }
    }

    // per-tile counts of what is kept for sure and of what equals T, published to the cluster
    int n_own = 0;
    for (int t = rank; t < n_tiles; t += kTopkCluster, ++n_own) {
        unsigned cnt = 0;
#pragma unroll
        for (int i = 0; i < kItems; ++i) {
            const int b = t * kTopkTile + i * kTopkThreads + tid;
            if (b < NB) {
                if (b < n_sink || b >= recent_lo) cnt += 1u;
                else if (kc > 0) {
                    const unsigned int v = bits[b];
                    if (v > T) cnt += 1u;
                    else if (v == T) cnt += 1u << 16;
                }
            }
        }
        unsigned total;
        cluster_block_scan(cnt, sh.warp_tot, total);
        if (tid == 0 && n_own < kTopkMaxOwnTiles) sh.tile_counts[n_own] = total;
    }
    cluster.sync();
    // the ascending sweep over this CTA's tiles
    for (int t = rank; t < n_tiles; t += kTopkCluster) {
        if (tid == 0) {
            // what the tiles before t keep (sequential: an equal score is kept only while need_eq lasts)
            unsigned cs = 0, ce = 0;
            for (int u = 0; u < t; ++u) {
                const unsigned pc = remote(u % kTopkCluster)->tile_counts[u / kTopkCluster];
                const unsigned eqs = pc >> 16, left = need_eq > ce ? need_eq - ce : 0u;
                cs += (pc & 0xffffu) + min(eqs, left);
                ce += eqs;
            }
            sh.carry_sel = cs; sh.carry_eq = ce;
        }
        __syncthreads();
        const unsigned carry_sel = sh.carry_sel, carry_eq = sh.carry_eq;
        const int b0 = t * kTopkTile + tid * kItems;
        // the sweep needs id order inside a thread: coalesced loads into shared memory, then 16 consecutive ids each
        unsigned int vreg[kItems];
        for (int idx = tid; idx < kTopkTile; idx += kTopkThreads) {
            const int b = t * kTopkTile + idx;
            stage[(idx / kItems) * kStagePitch + (idx % kItems)] = b < NB ? bits[b] : 0u;
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kItems; i += 4) {
            const uint4 u = *reinterpret_cast<const uint4*>(&stage[tid * kStagePitch + i]);
            vreg[i] = u.x; vreg[i + 1] = u.y; vreg[i + 2] = u.z; vreg[i + 3] = u.w;
        }
        __syncthreads();                                    // the buffer becomes the output buffer below
        unsigned flags_res = 0, flags_gt = 0, flags_eq = 0;
#pragma unroll
        for (int i = 0; i < kItems; ++i) {
            const int b = b0 + i;
            if (b < NB) {
                if (b < n_sink || b >= recent_lo) flags_res |= 1u << i;
                else if (kc > 0) {
                    const unsigned int v = vreg[i];
                    if (v > T) flags_gt |= 1u << i;
                    else if (v == T) flags_eq |= 1u << i;
                }
            }
        }
        const unsigned sure = flags_res | flags_gt;
        unsigned tot_packed;
        const unsigned ex = cluster_block_scan((unsigned)__popc(sure) | ((unsigned)__popc(flags_eq) << 16), sh.warp_tot, tot_packed);
        unsigned eq_rank = carry_eq + (ex >> 16);
        const unsigned tot_eq = tot_packed >> 16;
        const unsigned eq_left_before = need_eq > carry_eq ? need_eq - carry_eq : 0u;
        const unsigned tot_sel = (tot_packed & 0xffffu) + min(tot_eq, eq_left_before);
        unsigned rel = (ex & 0xffffu) + min(ex >> 16, eq_left_before);
        unsigned take = sure;
#pragma unroll
        for (int i = 0; i < kItems; ++i)
            if (flags_eq & (1u << i)) { if (eq_rank < need_eq) take |= 1u << i; ++eq_rank; }
        int* outbuf = reinterpret_cast<int*>(stage);
#pragma unroll
        for (int i = 0; i < kItems; ++i)
            if (take & (1u << i)) outbuf[rel++] = b0 + i;
        __syncthreads();
        for (unsigned i = tid; i < tot_sel; i += kTopkThreads)
            if (carry_sel + i < (unsigned)sel_stride) out[carry_sel + i] = outbuf[i];
        __syncthreads();
    }
    if (tid == 0 && rank == 0) {
        unsigned cs = 0, ce = 0;
        for (int u = 0; u < n_tiles; ++u) {
            const unsigned pc = remote(u % kTopkCluster)->tile_counts[u / kTopkCluster];
            const unsigned eqs = pc >> 16, left = need_eq > ce ? need_eq - ce : 0u;
            cs += (pc & 0xffffu) + min(eqs, left);
            ce += eqs;
        }
        n_sel[s] = (int32_t)min(cs, (unsigned)sel_stride);
    }
    cluster.sync();                                          // nobody leaves while its shared memory may still be read
}

Option g_topk_items{0};     // 0: fewest items per thread that cover the session; 2..16: at least this many (kernel-variant switch)
Option g_topk_cluster{1};   // sessions above 16,384 blocks: 1 = cluster of 8 CTAs, 0 = one CTA re-reading the scores

cudaError_t launch_topk(const kvmem_pool& p, int session_first, int n_sessions, const float* scores,
                        int scores_stride, const kvmem_select_params_t& prm, int32_t* sel_ids, int sel_stride,
                        int32_t* n_sel, cudaStream_t st) {
    int max_nb = 0;
    for (int s = session_first; s < session_first + n_sessions; ++s) max_nb = std::max(max_nb, p.sess_blocks[s]);
    const size_t smem = (size_t)kTopkThreads * kStagePitch * sizeof(unsigned int);
    static_assert(kTopkThreads * kStagePitch >= kTopkTile, "the staging buffer doubles as the output buffer of one sweep");
    static PerDeviceOnce attr_done;
    if (attr_done.pending(p.cfg.device)) {
        cudaError_t e = cudaFuncSetAttribute(topk_kernel<true, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(topk_kernel<false, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_done.mark(p.cfg.device);
    }
    const int max_tiles = (max_nb + kTopkTile - 1) / kTopkTile;
    if (max_nb > kTopkTile && g_topk_cluster && max_tiles <= kTopkCluster * kTopkMaxOwnTiles) {
        // long sessions: one cluster of 8 CTAs per session
        static PerDeviceOnce cattr_done;
        if (cattr_done.pending(p.cfg.device)) {
            cudaError_t e = cudaFuncSetAttribute(topk_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            cattr_done.mark(p.cfg.device);
        }
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)(kTopkCluster * n_sessions));
        cfg.blockDim = dim3(kTopkThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = kTopkCluster;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, topk_cluster_kernel, scores, scores_stride, (const int32_t*)p.nblocks_dev, session_first,
                                  p.geo.B, prm, sel_ids, sel_stride, n_sel, p.status_dev);
    }
#define KVMEM_TOPK_LAUNCH(REG, ITEMS, BYTES)                                                                            \
    launch_pdl(topk_kernel<REG, ITEMS>, dim3(n_sessions), dim3(kTopkThreads), (size_t)(BYTES), st, scores, scores_stride, \
               p.nblocks_dev, session_first, p.geo.B, prm, sel_ids, sel_stride, n_sel, p.status_dev)
    // the shortest instantiation that holds the longest session in registers; its dynamic shared memory is the
    // output buffer of one sweep (1,024 * ITEMS ids)
    const int items = g_topk_items > 0 ? g_topk_items : 1;
    if (max_nb <= kTopkThreads * 1 && items <= 1) KVMEM_TOPK_LAUNCH(true, 1, kTopkThreads * 1 * 4);
    else if (max_nb <= kTopkThreads * 2 && items <= 2) KVMEM_TOPK_LAUNCH(true, 2, kTopkThreads * 2 * 4);
    else if (max_nb <= kTopkThreads * 4 && items <= 4) KVMEM_TOPK_LAUNCH(true, 4, kTopkThreads * 4 * 4);
    else if (max_nb <= kTopkThreads * 8 && items <= 8) KVMEM_TOPK_LAUNCH(true, 8, kTopkThreads * 8 * 4);
    else if (max_nb <= kTopkTile) KVMEM_TOPK_LAUNCH(true, 16, smem);
    else KVMEM_TOPK_LAUNCH(false, 16, smem);
#undef KVMEM_TOPK_LAUNCH
    return cudaGetLastError();
}

}  // namespace kvmem
