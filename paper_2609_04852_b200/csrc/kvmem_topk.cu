// Selector (Sec. 4.3: reserve sink and recent blocks, fill the rest of the budget with the largest
// R_b, restore chronological order; budget from Eq. "active_budget" / Eq. "active_capacity").
//
// One CTA per session.  Scores are non-negative fp32, so their bit patterns order like unsigned
// integers.  Four MSB-first 8-bit radix passes over the non-reserved candidates find the value T of
// the k'-th largest score and how many candidates are strictly larger.  A final ascending sweep
// over block ids flags reserved blocks, every candidate above T, and the first (k' - above) ones
// equal to T, i.e. equal scores go to the lower id, and compacts the flagged ids with a block-wide
// prefix sum: the output is chronological without a sort, and identical from run to run.
#include "kvmem_internal.cuh"

namespace kvmem {

constexpr int kTopkThreads = 1024;
constexpr int kItems = 16;                                  // consecutive block ids per thread and tile
constexpr int kTopkTile = kTopkThreads * kItems;            // 16,384 ids per sweep

struct TopkShared {
    unsigned int hist[256];
    unsigned int warp_tot[32];
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

__global__ void __launch_bounds__(kTopkThreads)
topk_kernel(const float* __restrict__ scores, int scores_stride, const int32_t* __restrict__ nblocks_dev,
            int session_first, int B, kvmem_select_params_t prm, int32_t* __restrict__ sel_ids, int sel_stride,
            int32_t* __restrict__ n_sel, int32_t* __restrict__ status) {
    __shared__ TopkShared sh;
    const int s = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    const int NB = nblocks_dev[session_first + s];
    const unsigned int* bits = reinterpret_cast<const unsigned int*>(scores + (size_t)s * scores_stride);
    int32_t* out = sel_ids + (size_t)s * sel_stride;

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
        if (tid == 0) { sh.prefix = 0u; sh.remaining = (unsigned)kc; }
        for (int shift = 24; shift >= 0; shift -= 8) {
            if (tid < 256) sh.hist[tid] = 0u;
            __syncthreads();
            const unsigned int prefix = sh.prefix;
            const unsigned int mask = (shift == 24) ? 0u : (0xffffffffu << (shift + 8));
            for (int base = 0; base < NB; base += kTopkTile) {
                const int b0 = base + tid * kItems;
#pragma unroll 4
                for (int i = 0; i < kItems; ++i) {
                    const int b = b0 + i;
                    unsigned int v = 0;
                    bool live = b >= n_sink && b < recent_lo;
                    if (live) { v = bits[b]; live = (v & mask) == prefix; }
                    // one shared-memory atomic per distinct digit in the warp
                    const unsigned int digit = live ? ((v >> shift) & 255u) : 256u;
                    const unsigned int peers = __match_any_sync(0xffffffffu, digit);
                    if (live && lane == __ffs(peers) - 1) atomicAdd(&sh.hist[digit], (unsigned)__popc(peers));
                }
            }
            __syncthreads();
            if (tid < 32) {
                // warp 0 walks the 256 bins from the top: lane i owns bins [255 - 8i - 7, 255 - 8i]
                const unsigned int rem = sh.remaining;
                unsigned int c[8], mine = 0;
#pragma unroll
                for (int j = 0; j < 8; ++j) { c[j] = sh.hist[255 - 8 * lane - j]; mine += c[j]; }
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
                    sh.prefix = prefix | ((unsigned)bin << shift);
                    sh.remaining = left;                           // how many of this digit are still needed
                }
            }
            __syncthreads();
        }
        T = sh.prefix;
        need_eq = sh.remaining;
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
                    const unsigned int v = bits[b];
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
}

cudaError_t launch_topk(const kvmem_pool& p, int session_first, int n_sessions, const float* scores,
                        int scores_stride, const kvmem_select_params_t& prm, int32_t* sel_ids, int sel_stride,
                        int32_t* n_sel, cudaStream_t st) {
    topk_kernel<<<n_sessions, kTopkThreads, 0, st>>>(scores, scores_stride, p.nblocks_dev, session_first, p.geo.B, prm,
                                                     sel_ids, sel_stride, n_sel, p.status_dev);
    return cudaGetLastError();
}

}  // namespace kvmem
