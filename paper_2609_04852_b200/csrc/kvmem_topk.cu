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

struct TopkShared {
    unsigned int hist[256];
    unsigned int warp_a[32], warp_b[32];
    unsigned int prefix, remaining, carry_eq, carry_sel;
};

// exclusive scan of two flags across the CTA; returns (rank_a, rank_b) and adds the totals to the carries
__device__ __forceinline__ void block_scan2(bool fa, bool fb, TopkShared& sh, unsigned& ra, unsigned& rb,
                                            unsigned& tot_a, unsigned& tot_b) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned ba = __ballot_sync(0xffffffffu, fa), bb = __ballot_sync(0xffffffffu, fb);
    const unsigned lt = (1u << lane) - 1u;
    if (lane == 0) { sh.warp_a[warp] = __popc(ba); sh.warp_b[warp] = __popc(bb); }
    __syncthreads();
    unsigned oa = 0, ob = 0, ta = 0, tb = 0;
    for (int w = 0; w < kTopkThreads / 32; ++w) {
        const unsigned ca = sh.warp_a[w], cb = sh.warp_b[w];
        if (w < warp) { oa += ca; ob += cb; }
        ta += ca; tb += cb;
    }
    ra = oa + __popc(ba & lt);
    rb = ob + __popc(bb & lt);
    tot_a = ta; tot_b = tb;
    __syncthreads();
}

__global__ void __launch_bounds__(kTopkThreads)
topk_kernel(const float* __restrict__ scores, int scores_stride, const int32_t* __restrict__ nblocks_dev,
            int session_first, int B, kvmem_select_params_t prm, int32_t* __restrict__ sel_ids, int sel_stride,
            int32_t* __restrict__ n_sel, int32_t* __restrict__ status) {
    __shared__ TopkShared sh;
    const int s = blockIdx.x, tid = threadIdx.x;
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
            for (int b = n_sink + tid; b < recent_lo; b += kTopkThreads) {
                const unsigned int v = bits[b];
                if ((v & mask) == prefix) atomicAdd(&sh.hist[(v >> shift) & 255u], 1u);
            }
            __syncthreads();
            if (tid == 0) {
                unsigned int rem = sh.remaining;
                int bin = 255;
                for (; bin > 0; --bin) {
                    const unsigned int c = sh.hist[bin];
                    if (c >= rem) break;
                    rem -= c;
                }
                sh.prefix = prefix | ((unsigned)bin << shift);
                sh.remaining = rem;                        // how many of value-prefix "bin" are still needed
            }
            __syncthreads();
        }
        T = sh.prefix;
        need_eq = sh.remaining;
    }
    if (tid == 0) { sh.carry_eq = 0u; sh.carry_sel = 0u; }
    __syncthreads();

    for (int base = 0; base < NB; base += kTopkThreads) {
        const int b = base + tid;
        bool reserved = false, eq = false, gt = false;
        if (b < NB) {
            reserved = (b < n_sink) || (b >= recent_lo);
            if (!reserved && kc > 0) {
                const unsigned int v = bits[b];
                gt = v > T;
                eq = v == T;
            }
        }
        const unsigned carry_eq = sh.carry_eq, carry_sel = sh.carry_sel;
        unsigned r_eq, r_dummy, t_eq, t_dummy;
        block_scan2(eq, false, sh, r_eq, r_dummy, t_eq, t_dummy);
        const bool take = reserved || gt || (eq && (carry_eq + r_eq) < need_eq);
        unsigned r_sel, t_sel;
        block_scan2(take, false, sh, r_sel, r_dummy, t_sel, t_dummy);
        if (take) {
            const unsigned pos = carry_sel + r_sel;
            if (pos < (unsigned)sel_stride) out[pos] = b;
        }
        if (tid == 0) { sh.carry_eq = carry_eq + t_eq; sh.carry_sel = carry_sel + t_sel; }
        __syncthreads();
    }
    if (tid == 0) n_sel[s] = (int32_t)min(sh.carry_sel, (unsigned)sel_stride);
}

cudaError_t launch_topk(const kvmem_pool& p, int session_first, int n_sessions, const float* scores,
                        int scores_stride, const kvmem_select_params_t& prm, int32_t* sel_ids, int sel_stride,
                        int32_t* n_sel, cudaStream_t st) {
    topk_kernel<<<n_sessions, kTopkThreads, 0, st>>>(scores, scores_stride, p.nblocks_dev, session_first, p.geo.B, prm,
                                                     sel_ids, sel_stride, n_sel, p.status_dev);
    return cudaGetLastError();
}

}  // namespace kvmem
