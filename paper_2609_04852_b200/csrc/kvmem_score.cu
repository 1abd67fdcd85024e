// Query-conditioned block scoring for decode-sized queries (Eq. "kvmem-block-score", Sec. 4.3):
//   R_b = sum_m (1/(L*H)) sum_{l,h} softmax_{b'}( q[l][m][h] . kbar[l][b'][g(h)] / sqrt(d) )_b
//
// The index is streamed once.  A CTA owns 128 consecutive blocks of one (session, layer, KV
// head); a half-warp owns one Mean-K vector (16 lanes x one 128-bit load = 256 B), so a warp reads
// 512 contiguous bytes per step.  The M*r query rows that share this KV head sit in registers as
// fp32; every lane forms its 8-dimension partial dot product for all rows, and a transposing
// butterfly (15 shuffles for 16 rows) leaves lane i of the half-warp with the finished logit of
// row i.  Logits (already multiplied by log2(e)/sqrt(d)) are staged in shared memory, written out
// coalesced, and each CTA records per-row (max, sum-exp) of its tile: the cross-tile softmax
// statistics that Sec. 5.2 describes for tiled scoring.  A second small kernel merges the tile
// statistics per row and reduces rows in a fixed order, so results are run-to-run identical.
#include <math.h>

#include "kvmem_internal.cuh"

namespace kvmem {

constexpr int kChunk = 128;       // blocks per CTA tile
constexpr int kScoreThreads = 256;
constexpr int kMaxDecodeTokens = 16;

ScoreWorkspace plan_score_workspace(const kvmem_pool_config_t& c, int n_sessions, int n_q_tokens, char* base) {
    ScoreWorkspace w{};
    const int r = c.n_q_heads / c.n_kv_heads;
    w.rows = n_q_tokens * r;
    w.rows_pad = (w.rows + 15) / 16 * 16;
    w.nb_pad = (c.max_blocks_per_session + kChunk - 1) / kChunk * kChunk;
    w.n_chunks = w.nb_pad / kChunk;
    const size_t lg = (size_t)c.n_layers * c.n_kv_heads;
    const int rows_store = n_q_tokens <= kMaxDecodeTokens ? w.rows_pad : 16;
    w.logits_bytes = align_up((size_t)n_sessions * lg * rows_store * w.nb_pad * sizeof(float), 256);
    w.partials_bytes = align_up((size_t)n_sessions * lg * rows_store * w.n_chunks * sizeof(float2), 256);
    w.scores_bytes = align_up((size_t)n_sessions * c.max_blocks_per_session * sizeof(float), 256);
    w.total = w.logits_bytes + w.partials_bytes + w.scores_bytes;
    if (base) {
        w.logits = reinterpret_cast<float*>(base);
        w.partials = reinterpret_cast<float2*>(base + w.logits_bytes);
        w.scores = reinterpret_cast<float*>(base + w.logits_bytes + w.partials_bytes);
    }
    return w;
}

// Sum N per-lane partials across the 16 lanes of a half-warp.  While more than one value is live,
// each step keeps half of them (chosen by one lane-id bit) and hands the other half to the partner
// lane; afterwards it is a plain butterfly.  On return v[0] holds the total of value
// (hl >> (4 - log2 N)), hl = lane id within the half-warp.
template <int N>
__device__ __forceinline__ void halfwarp_transpose_reduce(float (&v)[N], int hl) {
    int n = N;
#pragma unroll
    for (int o = 8; o >= 1; o >>= 1) {
        if (n > 1) {
            const int half = n >> 1;
            const bool up = (hl & o) != 0;
#pragma unroll
            for (int i = 0; i < N / 2; ++i) {
                if (i < half) {
                    const float keep = up ? v[i + half] : v[i];
                    const float send = up ? v[i] : v[i + half];
                    v[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                }
            }
            n = half;
        } else {
            v[0] += __shfl_xor_sync(0xffffffffu, v[0], o);
        }
    }
}

__device__ __forceinline__ void unpack8(const uint4& u, float (&f)[8]) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

template <int RP>
__global__ void __launch_bounds__(kScoreThreads, 1)
score_logits_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ index,
                    const int32_t* __restrict__ nblocks_dev, int session_first, int M, int L, int H, int G,
                    int max_bps, size_t index_elems_per_session, float* __restrict__ logits,
                    float2* __restrict__ partials, int rows, int rows_pad, int nb_pad, int n_chunks,
                    float scale_log2e) {
    constexpr int SH = (RP == 16) ? 0 : (RP == 8) ? 1 : 2;   // lanes per finished row = 1 << SH
    __shared__ float slog[RP][kChunk + 4];

    const int s = blockIdx.z, lg = blockIdx.y, chunk = blockIdx.x;
    const int l = lg / G, g = lg % G, r = H / G;
    const int NB = nblocks_dev[session_first + s];
    const int b0 = chunk * kChunk;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int hl = lane & 15, hw = tid >> 4;               // lane in half-warp, half-warp in CTA (0..15)
    const size_t slab = ((size_t)s * L * G + lg) * rows_pad;  // first row of this (s, l, g)

    const __nv_bfloat16* idx_lg =
        index + (size_t)(session_first + s) * index_elems_per_session + (size_t)lg * max_bps * 128;

    for (int pass = 0; pass * RP < rows_pad; ++pass) {
        const int row0 = pass * RP;
        if (row0 >= rows && pass > 0) break;
        // query rows of this pass, dims [8*hl, 8*hl + 8), as fp32 registers
        float qr[RP][8];
#pragma unroll
        for (int j = 0; j < RP; ++j) {
            const int row = row0 + j;
            if (row < rows) {
                const int m = row / r, hr = row % r;
                const uint4 u = *reinterpret_cast<const uint4*>(
                    q + ((((size_t)s * M + m) * L + l) * H + (size_t)g * r + hr) * 128 + hl * 8);
                unpack8(u, qr[j]);
            } else {
#pragma unroll
                for (int c = 0; c < 8; ++c) qr[j][c] = 0.0f;
            }
        }
        if (b0 < NB) {
#pragma unroll 2
            for (int it = 0; it < kChunk / 16; ++it) {
                const int col = it * 16 + hw;
                const int blk = b0 + col;
                const bool valid = blk < NB;
                uint4 u = make_uint4(0, 0, 0, 0);
                if (valid) u = __ldg(reinterpret_cast<const uint4*>(idx_lg + (size_t)blk * 128 + hl * 8));
                float kf[8];
                unpack8(u, kf);
                float acc[RP];
#pragma unroll
                for (int j = 0; j < RP; ++j) {
                    float a = 0.0f;
#pragma unroll
                    for (int c = 0; c < 8; ++c) a = fmaf(qr[j][c], kf[c], a);
                    acc[j] = a;
                }
                halfwarp_transpose_reduce<RP>(acc, hl);
                if ((hl & ((1 << SH) - 1)) == 0) slog[hl >> SH][col] = valid ? acc[0] * scale_log2e : -INFINITY;
            }
        }
        __syncthreads();
        // per-row statistics of this tile and coalesced logit store
        for (int j = warp; j < RP; j += kScoreThreads / 32) {
            const int row = row0 + j;
            float mx = -INFINITY, v[kChunk / 32];
#pragma unroll
            for (int i = 0; i < kChunk / 32; ++i) {
                v[i] = (b0 < NB) ? slog[j][lane + 32 * i] : -INFINITY;
                mx = fmaxf(mx, v[i]);
            }
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            float sum = 0.0f;
            if (mx > -INFINITY) {
#pragma unroll
                for (int i = 0; i < kChunk / 32; ++i) sum += exp2f(v[i] - mx);
            }
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (row < rows_pad) {
                if (lane == 0) partials[(slab + row) * n_chunks + chunk] = make_float2(mx, sum);
                float* dst = logits + (slab + row) * (size_t)nb_pad + b0;
#pragma unroll
                for (int i = 0; i < kChunk / 32; ++i) dst[lane + 32 * i] = v[i];
            }
        }
        __syncthreads();
    }
}

// Merge the tile statistics of every row, then R_b = (1/(L*H)) sum_rows exp2(logit - max_row) / Z_row.
__global__ void __launch_bounds__(256)
score_finish_kernel(const float* __restrict__ logits, const float2* __restrict__ partials,
                    const int32_t* __restrict__ nblocks_dev, int session_first, int LG, int rows, int rows_pad,
                    int nb_pad, int n_chunks, float inv_LH, float* __restrict__ scores, int scores_stride) {
    extern __shared__ float2 rowstat[];   // [LG * rows] : (max, 1/Z)
    const int s = blockIdx.y;
    const int NB = nblocks_dev[session_first + s];
    if ((int)(blockIdx.x * blockDim.x) >= NB) return;
    const int live_chunks = min(n_chunks, (NB + kChunk - 1) / kChunk);
    for (int i = threadIdx.x; i < LG * rows; i += blockDim.x) {
        const int lg = i / rows, j = i % rows;
        const float2* p = partials + (((size_t)s * LG + lg) * rows_pad + j) * n_chunks;
        float mx = -INFINITY;
        for (int c = 0; c < live_chunks; ++c) mx = fmaxf(mx, p[c].x);
        float z = 0.0f;
        for (int c = 0; c < live_chunks; ++c) {
            const float2 t = p[c];
            if (t.x > -INFINITY) z += t.y * exp2f(t.x - mx);
        }
        rowstat[i] = make_float2(mx, 1.0f / z);
    }
    __syncthreads();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= NB) return;
    float total = 0.0f;
    for (int lg = 0; lg < LG; ++lg) {
        const float* base = logits + (((size_t)s * LG + lg) * rows_pad) * (size_t)nb_pad + b;
        float part = 0.0f;
        for (int j = 0; j < rows; ++j) {
            const float2 st = rowstat[lg * rows + j];
            part += exp2f(base[(size_t)j * nb_pad] - st.x) * st.y;
        }
        total += part;
    }
    scores[(size_t)s * scores_stride + b] = total * inv_LH;
}

cudaError_t launch_score_decode(const kvmem_pool& p, int session_first, int n_sessions, const __nv_bfloat16* q,
                                int M, const ScoreWorkspace& ws, float* scores, int scores_stride, cudaStream_t st) {
    const Geometry& g = p.geo;
    if (M > kMaxDecodeTokens) return cudaErrorNotSupported;
    const float scale_log2e = 1.4426950408889634f / sqrtf((float)g.d);
    int max_nb = 0;
    for (int s = session_first; s < session_first + n_sessions; ++s) max_nb = std::max(max_nb, p.sess_blocks[s]);
    if (max_nb == 0) return cudaSuccess;
    const int chunks = (max_nb + kChunk - 1) / kChunk;
    dim3 grid((unsigned)chunks, (unsigned)(g.L * g.G), (unsigned)n_sessions);
#define KVMEM_SCORE_ARGS                                                                                           \
    q, p.index, p.nblocks_dev, session_first, M, g.L, g.H, g.G, g.max_bps, p.lay.index_elems_per_session, ws.logits, \
        ws.partials, ws.rows, ws.rows_pad, ws.nb_pad, ws.n_chunks, scale_log2e
    if (ws.rows <= 4)
        score_logits_kernel<4><<<grid, kScoreThreads, 0, st>>>(KVMEM_SCORE_ARGS);
    else if (ws.rows <= 8)
        score_logits_kernel<8><<<grid, kScoreThreads, 0, st>>>(KVMEM_SCORE_ARGS);
    else
        score_logits_kernel<16><<<grid, kScoreThreads, 0, st>>>(KVMEM_SCORE_ARGS);
#undef KVMEM_SCORE_ARGS
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int LG = g.L * g.G;
    const size_t smem = (size_t)LG * ws.rows * sizeof(float2);
    if (smem > 48 * 1024) {
        e = cudaFuncSetAttribute(score_finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    dim3 fgrid((unsigned)((max_nb + 255) / 256), (unsigned)n_sessions);
    score_finish_kernel<<<fgrid, 256, smem, st>>>(ws.logits, ws.partials, p.nblocks_dev, session_first, LG, ws.rows,
                                                  ws.rows_pad, ws.nb_pad, ws.n_chunks, 1.0f / (float)(g.L * g.H),
                                                  scores, scores_stride);
    return cudaGetLastError();
}

}  // namespace kvmem
