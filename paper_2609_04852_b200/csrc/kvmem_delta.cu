// Working-set delta (Eq. "kvmem-working-set-delta", Sec. 4.4): R = W_next n W_prev (retained),
// L = W_next \ W_prev (incoming), E = W_prev \ W_next (outgoing), from the chronological id lists of
// two consecutive steps.  One CTA per session.  Membership is a binary search in the other (ascending)
// list; the three outputs are compacted with block-wide prefix sums, so they come out in ascending id
// order and identical from run to run.  A retained block carries its old and new slot: the position
// change (new - old) * B is what a delta re-RoPE of its resident keys needs.
#include "kvmem_internal.cuh"

namespace kvmem {

constexpr int kDeltaThreads = 1024;

// exclusive prefix of `val` over the CTA (thread order) and the CTA total; two barriers
__device__ __forceinline__ unsigned delta_scan(unsigned val, unsigned* warp_tot, unsigned& total) {
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

// index of `id` in the ascending list a[0..n), or -1
__device__ __forceinline__ int find_sorted(const int32_t* __restrict__ a, int n, int id) {
    int lo = 0, hi = n;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (a[mid] < id) lo = mid + 1; else hi = mid;
    }
    return (lo < n && a[lo] == id) ? lo : -1;
}

__global__ void __launch_bounds__(kDeltaThreads)
working_set_delta_kernel(const int32_t* __restrict__ prev_ids, const int32_t* __restrict__ n_prev,
                         const int32_t* __restrict__ next_ids, const int32_t* __restrict__ n_next, int stride,
                         int32_t* __restrict__ retained, int32_t* __restrict__ incoming, int32_t* __restrict__ outgoing,
                         int32_t* __restrict__ counts, int32_t* __restrict__ status) {
    __shared__ unsigned warp_tot[32];
    const int s = blockIdx.x, tid = threadIdx.x;
    int np = n_prev[s], nn = n_next[s];
    if (np < 0 || np > stride || nn < 0 || nn > stride) {
        if (tid == 0) atomicExch(status, (int)KVMEM_E_DEVICE_RANGE);
        np = min(max(np, 0), stride); nn = min(max(nn, 0), stride);
    }
    const int32_t* prev = prev_ids + (size_t)s * stride;
    const int32_t* next = next_ids + (size_t)s * stride;
    int32_t* ret = retained + (size_t)s * stride * 3;
    int32_t* inc = incoming + (size_t)s * stride * 2;
    int32_t* out = outgoing + (size_t)s * stride;
    unsigned nR = 0, nL = 0, nE = 0;
    for (int base = 0; base < nn; base += kDeltaThreads) {       // next -> retained | incoming
        const int j = base + tid;
        int id = 0, old = -1;
        if (j < nn) { id = next[j]; old = find_sorted(prev, np, id); }
        unsigned tR, tL;
        const unsigned pR = nR + delta_scan(j < nn && old >= 0, warp_tot, tR);
        const unsigned pL = nL + delta_scan(j < nn && old < 0, warp_tot, tL);
        if (j < nn) {
            if (old >= 0) { ret[3 * pR] = id; ret[3 * pR + 1] = old; ret[3 * pR + 2] = j; }
            else { inc[2 * pL] = id; inc[2 * pL + 1] = j; }
        }
        nR += tR; nL += tL;
    }
    for (int base = 0; base < np; base += kDeltaThreads) {       // prev -> outgoing
        const int i = base + tid;
        int id = 0;
        bool gone = false;
        if (i < np) { id = prev[i]; gone = find_sorted(next, nn, id) < 0; }
        unsigned tE;
        const unsigned pE = nE + delta_scan(gone, warp_tot, tE);
        if (gone) out[pE] = id;
        nE += tE;
    }
    if (tid == 0) { counts[3 * s] = (int32_t)nR; counts[3 * s + 1] = (int32_t)nL; counts[3 * s + 2] = (int32_t)nE; }
}

cudaError_t launch_working_set_delta(const kvmem_pool& p, int n_sessions, const int32_t* prev_ids, const int32_t* n_prev,
                                     const int32_t* next_ids, const int32_t* n_next, int stride, int32_t* retained,
                                     int32_t* incoming, int32_t* outgoing, int32_t* counts, cudaStream_t st) {
    working_set_delta_kernel<<<n_sessions, kDeltaThreads, 0, st>>>(prev_ids, n_prev, next_ids, n_next, stride, retained,
                                                                   incoming, outgoing, counts, p.status_dev);
    return cudaGetLastError();
}

}  // namespace kvmem
