// Selector (Sec. 4.3: reserve sink and recent blocks, fill the rest of the budget with the largest
// R_b, restore chronological order; budget from Eq. "active_budget" / Eq. "active_capacity").
//
// One CTA per session.  Scores are non-negative fp32, so their bit patterns order like unsigned
// integers.  MSB-first 8-bit radix passes over the non-reserved candidates, starting at the highest
// bit in which two candidates differ, find the value T of the k'-th largest score and how many
// candidates are strictly larger (histograms in shared memory, 8 copies to spread the atomics).  A final ascending sweep
// over block ids flags reserved blocks, every candidate above T, and the first (k' - above) ones
// equal to T, i.e. equal scores go to the lower id, and compacts the flagged ids with a block-wide
// prefix sum: the output is chronological without a sort, and identical from run to run.
#include <algorithm>

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
    unsigned int prefix, remaining;
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

// REG = true (sessions of at most 16,384 blocks): the scores are staged once through shared memory with
// coalesced loads and then live in registers, 16 consecutive ids per thread, for every later pass.
// REG = false: any length; every pass re-reads the scores from global memory.
constexpr int kStagePitch = kItems + 4;                     // floats per thread in the staging buffer: conflict-free 128-bit reads

template <bool REG>
__global__ void __launch_bounds__(kTopkThreads)
topk_kernel(const float* __restrict__ scores, int scores_stride, const int32_t* __restrict__ nblocks_dev,
            int session_first, int B, kvmem_select_params_t prm, int32_t* __restrict__ sel_ids, int sel_stride,
            int32_t* __restrict__ n_sel, int32_t* __restrict__ status) {
    __shared__ TopkShared sh;
    extern __shared__ __align__(16) unsigned int stage[];   // REG only: [kTopkThreads][kStagePitch]
    const int s = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    const int NB = nblocks_dev[session_first + s];
    const unsigned int* bits = reinterpret_cast<const unsigned int*>(scores + (size_t)s * scores_stride);
    int32_t* out = sel_ids + (size_t)s * sel_stride;
    unsigned int vreg[kItems];
    if (REG) {
        for (int idx = tid; idx < kTopkTile; idx += kTopkThreads)          // coalesced global reads
            stage[(idx / kItems) * kStagePitch + (idx % kItems)] = idx < NB ? bits[idx] : 0u;
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
    long long kk = room > 0 ? room / B : 0;
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
            if (tid == 0) { sh.prefix = hi & known; sh.remaining = (unsigned)kc; }
            int shift = max(hb - 7, 0);
            while (true) {
                for (int i = tid; i < kHistCopies * 256; i += kTopkThreads) (&sh.hist[0][0])[i] = 0u;
                __syncthreads();
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
                if (tid < 32) {
                    // warp 0 walks the 256 bins from the top: lane i owns bins [255 - 8i - 7, 255 - 8i]
                    const unsigned int rem = sh.remaining;
                    unsigned int c[8], mine = 0;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        unsigned int t = 0;
#pragma unroll
                        for (int k2 = 0; k2 < kHistCopies; ++k2) t += sh.hist[k2][255 - 8 * lane - j];
                        c[j] = t; mine += t;
                    }
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
                        int bin = 255 - 8 * lane;
#pragma unroll
                        for (int j = 0; j < 7; ++j) {
                            if (c[j] >= left) break;
                            left -= c[j];
                            --bin;
                        }
                        sh.prefix = (prefix & ~(255u << shift)) | ((unsigned)bin << shift);
                        sh.remaining = left;                           // how many of this digit are still needed
                    }
                }
                __syncthreads();
                known |= 255u << shift;
                if (shift == 0) break;
                shift = max(shift - 8, 0);
            }
            T = sh.prefix;
            need_eq = sh.remaining;
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
        unsigned tot_eq, tot_sel;
        unsigned eq_rank = carry_eq + block_exclusive_scan(__popc(flags_eq), sh, tot_eq);
        unsigned take = flags_res | flags_gt;
#pragma unroll
        for (int i = 0; i < kItems; ++i)
            if (flags_eq & (1u << i)) { if (eq_rank < need_eq) take |= 1u << i; ++eq_rank; }
        unsigned pos = carry_sel + block_exclusive_scan(__popc(take), sh, tot_sel);
#pragma unroll
        for (int i = 0; i < kItems; ++i)
            if (take & (1u << i)) { if (pos < (unsigned)sel_stride) out[pos] = b0 + i; ++pos; }
        carry_eq += tot_eq;
        carry_sel += tot_sel;
    }
    if (tid == 0) n_sel[s] = (int32_t)min(carry_sel, (unsigned)sel_stride);
#undef KVMEM_TOPK_VAL
}

cudaError_t launch_topk(const kvmem_pool& p, int session_first, int n_sessions, const float* scores,
                        int scores_stride, const kvmem_select_params_t& prm, int32_t* sel_ids, int sel_stride,
                        int32_t* n_sel, cudaStream_t st) {
    int max_nb = 0;
    for (int s = session_first; s < session_first + n_sessions; ++s) max_nb = std::max(max_nb, p.sess_blocks[s]);
    if (max_nb <= kTopkTile) {
        const size_t smem = (size_t)kTopkThreads * kStagePitch * sizeof(unsigned int);
        static bool attr_done = false;
        if (!attr_done) {
            cudaError_t e = cudaFuncSetAttribute(topk_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            attr_done = true;
        }
        topk_kernel<true><<<n_sessions, kTopkThreads, smem, st>>>(scores, scores_stride, p.nblocks_dev, session_first,
                                                                  p.geo.B, prm, sel_ids, sel_stride, n_sel, p.status_dev);
    } else {
        topk_kernel<false><<<n_sessions, kTopkThreads, 0, st>>>(scores, scores_stride, p.nblocks_dev, session_first,
                                                                p.geo.B, prm, sel_ids, sel_stride, n_sel, p.status_dev);
    }
    return cudaGetLastError();
}

}  // namespace kvmem
