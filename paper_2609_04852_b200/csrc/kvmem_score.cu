// Query-conditioned block scoring for decode-sized queries (Eq. "kvmem-block-score", Sec. 4.3):
//   R_b = sum_m (1/(L*H)) sum_{l,h} softmax_{b'}( q[l][m][h] . kbar[l][b'][g(h)] / sqrt(d) )_b
//
// The index is streamed once.  About one persistent CTA per SM owns a contiguous range of
// 128-block tiles of one (session, layer, KV head); tiles (32 KiB, contiguous in the index) arrive
// through a ring of shared-memory stages filled by 1-D TMA bulk copies (mbarrier completion, bounded
// waits).  A half-warp owns one Mean-K vector (16 lanes x one 128-bit shared-memory load = 256 B).  The M*r query rows that share this KV head sit in registers as
// fp32; every lane forms its 8-dimension partial dot product for all rows, and a transposing
// butterfly (15 shuffles for 16 rows) leaves lane i of the half-warp with the finished logit of
// row i.  Logits (already multiplied by log2(e)/sqrt(d)) are staged in shared memory, written out
// coalesced, and each CTA carries per-row (max, sum-exp) across its tiles: the cross-tile softmax
// statistics that Sec. 5.2 describes for tiled scoring.  A second small kernel merges the tile
// statistics per row and reduces rows in a fixed order, so results are run-to-run identical.
#include <cudaTypedefs.h>
#include <math.h>

#include <algorithm>

#include "kvmem_internal.cuh"
#include "kvmem_ptx.cuh"

namespace kvmem {

constexpr int kChunk = 128;       // blocks per CTA tile
constexpr int kScoreThreads = 256;
constexpr int kScoreStages = 3;   // 32 KiB index tiles in flight per CTA (two CTAs of the tensor-core kernel share an SM)
constexpr int kMaxScoreParts = 64;

ScoreWorkspace plan_score_workspace(const kvmem_pool_config_t& c, int n_sessions, int n_q_tokens, char* base) {
    ScoreWorkspace w{};
    const int r = c.n_q_heads / c.n_kv_heads;
    w.rows = n_q_tokens * r;
    w.rows_pad = (w.rows + 15) / 16 * 16;
    w.nb_pad = (c.max_blocks_per_session + kChunk - 1) / kChunk * kChunk;
    w.n_chunks = w.nb_pad / kChunk;
    const size_t lg = (size_t)c.n_layers * c.n_kv_heads;
    const int rows_store = w.rows_pad;
    w.logits_bytes = align_up((size_t)n_sessions * lg * rows_store * w.nb_pad * sizeof(float), 256);
    w.partials_bytes = align_up((size_t)n_sessions * lg * rows_store * kMaxScoreParts * sizeof(float2), 256);
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
                    float2* __restrict__ partials, int rows, int rows_pad, int nb_pad, int n_parts,
                    float scale_log2e, int32_t* __restrict__ status) {
    pdl_wait();        // everything earlier in the stream is complete and visible from here on
    pdl_trigger();     // the next kernel's CTAs may take their places; they wait in the same way
    constexpr int SH = (RP == 16) ? 0 : (RP == 8) ? 1 : 2;   // lanes per finished row = 1 << SH
    constexpr int RPW = (RP + 7) / 8;                        // rows whose statistics one warp carries
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ uint64_t full_bar[kScoreStages];
    __shared__ float slog[RP][kChunk + 4];
    uint4* stage_mem = reinterpret_cast<uint4*>(smem_raw);   // [kScoreStages][kChunk][16] x 16 B

    const int s = blockIdx.z, lg = blockIdx.y, part = blockIdx.x;
    const int l = lg / G, g = lg % G, r = H / G;
    const int NB = nblocks_dev[session_first + s];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int hl = lane & 15, hw = tid >> 4;               // lane in half-warp, half-warp in CTA (0..15)
    const size_t slab = ((size_t)s * L * G + lg) * rows_pad;  // first row of this (s, l, g)
    const __nv_bfloat16* idx_lg =
        index + (size_t)(session_first + s) * index_elems_per_session + (size_t)lg * max_bps * 128;

    // this CTA's contiguous range of 128-block chunks
    const int n_chunks = (NB + kChunk - 1) / kChunk;
    const int c_begin = (int)((long long)n_chunks * part / n_parts), c_end = (int)((long long)n_chunks * (part + 1) / n_parts);
    const int n_mine = c_end - c_begin;

    if (tid == 0) {
        for (int i = 0; i < kScoreStages; ++i) ptx::mbar_init(&full_bar[i], 1);
        ptx::fence_mbar_init();
    }
    __syncthreads();

    int issued = 0, waited = 0;                            // running counts over all passes (barrier phases)
    auto issue = [&](int chunk) {                          // thread 0 only
        const int st = issued % kScoreStages;
        const int b0 = chunk * kChunk;
        const uint32_t bytes = (uint32_t)min(kChunk, NB - b0) * 256u;
        ptx::mbar_expect_tx(&full_bar[st], bytes);
        ptx::bulk_g2s(stage_mem + (size_t)st * kChunk * 16, idx_lg + (size_t)b0 * 128, bytes, &full_bar[st]);
    };

    for (int pass = 0; pass * RP < rows; ++pass) {
        const int row0 = pass * RP;
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
        float run_m[RPW], run_l[RPW];
#pragma unroll
        for (int i = 0; i < RPW; ++i) { run_m[i] = -INFINITY; run_l[i] = 0.0f; }

        if (tid == 0) {
            for (int i = 0; i < min(kScoreStages - 1, n_mine); ++i) { issue(c_begin + i); ++issued; }
        }
        for (int i = 0; i < n_mine; ++i) {
            const int chunk = c_begin + i, b0 = chunk * kChunk;
            const int st = waited % kScoreStages;
            const bool ok = ptx::mbar_wait(&full_bar[st], (uint32_t)((waited / kScoreStages) & 1));
            ++waited;
            if (__syncthreads_or(!ok)) {                  // CTA-uniform: somebody gave up
                if (tid == 0) atomicExch(status, (int)KVMEM_E_TIMEOUT);
                return;
            }
            // stage (i - 1) was released by the barrier above: refill it
            if (tid == 0 && i + kScoreStages - 1 < n_mine) { issue(chunk + kScoreStages - 1); ++issued; }
            const uint4* tile = stage_mem + (size_t)st * kChunk * 16;
#pragma unroll 2
            for (int it = 0; it < kChunk / 16; ++it) {
                const int col = it * 16 + hw;
                const bool valid = b0 + col < NB;
                uint4 u = make_uint4(0, 0, 0, 0);
                if (valid) u = tile[col * 16 + hl];
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
            __syncthreads();
            // per-row statistics of this tile (folded into the running pair) and coalesced logit store
#pragma unroll
            for (int jj = 0; jj < RPW; ++jj) {
                const int j = warp + 8 * jj;
                if (j < RP) {
                    float mx = -INFINITY, v[kChunk / 32];
#pragma unroll
                    for (int t = 0; t < kChunk / 32; ++t) {
                        v[t] = slog[j][lane + 32 * t];
                        mx = fmaxf(mx, v[t]);
                    }
#pragma unroll
                    for (int o = 16; o >= 1; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                    const float mn = fmaxf(run_m[jj], mx);      // finite: a chunk holds at least one block
                    float sum = 0.0f;
#pragma unroll
                    for (int t = 0; t < kChunk / 32; ++t) sum += exp2f(v[t] - mn);
#pragma unroll
                    for (int o = 16; o >= 1; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
                    run_l[jj] = run_l[jj] * exp2f(run_m[jj] - mn) + sum;
                    run_m[jj] = mn;
                    float* dst = logits + (slab + row0 + j) * (size_t)nb_pad + b0;
#pragma unroll
                    for (int t = 0; t < kChunk / 32; ++t) dst[lane + 32 * t] = v[t];
                }
            }
            __syncthreads();
        }
#pragma unroll
        for (int jj = 0; jj < RPW; ++jj) {
            const int j = warp + 8 * jj;
            if (j < RP && lane == 0) partials[(slab + row0 + j) * n_parts + part] = make_float2(run_m[jj], run_l[jj]);
        }
    }
}

// Same contract as score_logits_kernel, with the dot products on the tensor cores: the M*r <= 16 query
// rows of a pass form one m16 MMA tile (bf16 mma.sync, fp32 accumulate), each warp takes 16 of the
// tile's 128 Mean-K vectors.  Index tiles arrive by tiled TMA with the 128-byte swizzle, so the
// ldmatrix reads are conflict-free.  This removes the fp32-ALU bound of the shuffle kernel (16 rows
// x 128 dims = 2,048 FMAs per 256-byte vector) and leaves the kernel bound by the index stream.
__global__ void __launch_bounds__(kScoreThreads, 2)
score_logits_mma_kernel(const __grid_constant__ CUtensorMap map_idx, const __nv_bfloat16* __restrict__ q,
                        const int32_t* __restrict__ nblocks_dev, int session_first, int M, int L, int H, int G,
                        int max_bps, float* __restrict__ logits, float2* __restrict__ partials, int rows, int rows_pad,
                        int nb_pad, int n_parts, float scale_log2e, int32_t* __restrict__ status,
                        int nb_override, int col_off, int part_stride, int part_off) {
    // nb_override >= 0: the tensor map covers one staged tile of a host-resident index (nb_override blocks per head,
    // max_bps rows apart); its logits go to columns col_off.. and its statistics to slots part_off.. of part_stride
    pdl_wait();        // everything earlier in the stream is complete and visible from here on
    pdl_trigger();     // the next kernel's CTAs may take their places; they wait in the same way
    constexpr int RP = 16;
    extern __shared__ unsigned char smem_dyn[];
    __shared__ uint64_t full_bar[kScoreStages];
    __shared__ float slog[RP][kChunk + 4];
    unsigned char* stage_mem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    constexpr uint32_t kHalf = kChunk * 128;                 // one 64-dim half of a tile: 128 rows x 128 B
    constexpr uint32_t kStage = 2 * kHalf;

    const int s = blockIdx.z, lg = blockIdx.y, part = blockIdx.x;
    const int l = lg / G, g = lg % G, r = H / G;
    const int NB = nb_override >= 0 ? nb_override : nblocks_dev[session_first + s];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const size_t slab = ((size_t)s * L * G + lg) * rows_pad;
    const int row_base = ((session_first + s) * L * G + lg) * max_bps;     // first index row of this (session, l, g)

    const int n_chunks = (NB + kChunk - 1) / kChunk;
    const int c_begin = (int)((long long)n_chunks * part / n_parts), c_end = (int)((long long)n_chunks * (part + 1) / n_parts);
    const int n_mine = c_end - c_begin;

    if (tid == 0) {
        for (int i = 0; i < kScoreStages; ++i) ptx::mbar_init(&full_bar[i], 1);
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&map_idx);
    }
    __syncthreads();

    int issued = 0, waited = 0;
    auto issue = [&](int chunk) {                          // thread 0 only
        const int st = issued % kScoreStages;
        unsigned char* dst = stage_mem + (size_t)st * kStage;
        ptx::mbar_expect_tx(&full_bar[st], kStage);
        ptx::tma_load_2d(dst, &map_idx, 0, row_base + chunk * kChunk, &full_bar[st]);
        ptx::tma_load_2d(dst + kHalf, &map_idx, 64, row_base + chunk * kChunk, &full_bar[st]);
    };
    const uint32_t stage0 = ptx::smem_u32(stage_mem);
    const int mj = lane >> 3, mr = lane & 7;               // ldmatrix: matrix index and row within it

    for (int pass = 0; pass * RP < rows; ++pass) {
        const int row0 = pass * RP;
        // Q fragments (A operand, m16k16 x 8 k-steps): row j = m * r + hr -> q[s][m][l][g*r + hr]
        uint32_t qf[8][4];
        {
            const int ra = row0 + (lane >> 2), rb = ra + 8;
            const __nv_bfloat16* qa = nullptr;
            const __nv_bfloat16* qb = nullptr;
            if (ra < rows) qa = q + ((((size_t)s * M + ra / r) * L + l) * H + (size_t)g * r + ra % r) * 128;
            if (rb < rows) qb = q + ((((size_t)s * M + rb / r) * L + l) * H + (size_t)g * r + rb % r) * 128;
            const int kq = 2 * (lane & 3);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                qf[ks][0] = qa ? *reinterpret_cast<const uint32_t*>(qa + ks * 16 + kq) : 0u;
                qf[ks][1] = qb ? *reinterpret_cast<const uint32_t*>(qb + ks * 16 + kq) : 0u;
                qf[ks][2] = qa ? *reinterpret_cast<const uint32_t*>(qa + ks * 16 + kq + 8) : 0u;
                qf[ks][3] = qb ? *reinterpret_cast<const uint32_t*>(qb + ks * 16 + kq + 8) : 0u;
            }
        }
        float run_m[2] = {-INFINITY, -INFINITY}, run_l[2] = {0.0f, 0.0f};

        if (tid == 0) {
            for (int i = 0; i < min(kScoreStages - 1, n_mine); ++i) { issue(c_begin + i); ++issued; }
        }
        for (int i = 0; i < n_mine; ++i) {
            const int chunk = c_begin + i, b0 = chunk * kChunk;
            const int st = waited % kScoreStages;
            const bool ok = ptx::mbar_wait(&full_bar[st], (uint32_t)((waited / kScoreStages) & 1));
            ++waited;
            if (__syncthreads_or(!ok)) {                  // CTA-uniform: somebody gave up
                if (tid == 0) atomicExch(status, (int)KVMEM_E_TIMEOUT);
                return;
            }
            if (tid == 0 && i + kScoreStages - 1 < n_mine) { issue(chunk + kScoreStages - 1); ++issued; }
            const uint32_t tile = stage0 + (uint32_t)st * kStage;
            // S = Q Kbar^T for this warp's 16 vectors: 2 n-tiles x 8 k-steps
            float sc[2][4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) { sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.0f; }
#pragma unroll
            for (int kp = 0; kp < 4; ++kp) {
                const int cg = kp * 4 + mj;
                const uint32_t half_off = (uint32_t)(cg >> 3) * kHalf;
                const int c = cg & 7;
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    const int rowi = warp * 16 + nt * 8 + mr;
                    const uint32_t addr = tile + half_off + (uint32_t)rowi * 128u + (uint32_t)((c ^ (rowi & 7)) << 4);
                    uint32_t b0r, b1r, b2r, b3r;
                    ptx::ldmatrix_x4(addr, b0r, b1r, b2r, b3r);
                    ptx::mma_bf16_16816(sc[nt], qf[2 * kp], b0r, b1r);
                    ptx::mma_bf16_16816(sc[nt], qf[2 * kp + 1], b2r, b3r);
                }
            }
            {
                const int ra = lane >> 2, rb = ra + 8;
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    const int col = warp * 16 + nt * 8 + 2 * (lane & 3);
                    const bool v0 = b0 + col < NB, v1 = b0 + col + 1 < NB;
                    slog[ra][col] = v0 ? sc[nt][0] * scale_log2e : -INFINITY;
                    slog[ra][col + 1] = v1 ? sc[nt][1] * scale_log2e : -INFINITY;
                    slog[rb][col] = v0 ? sc[nt][2] * scale_log2e : -INFINITY;
                    slog[rb][col + 1] = v1 ? sc[nt][3] * scale_log2e : -INFINITY;
                }
            }
            __syncthreads();
            // per-row statistics of this tile (folded into the running pair) and coalesced logit store
#pragma unroll
            for (int jj = 0; jj < 2; ++jj) {
                const int j = warp + 8 * jj;
                float mx = -INFINITY, v[kChunk / 32];
#pragma unroll
                for (int t = 0; t < kChunk / 32; ++t) {
                    v[t] = slog[j][lane + 32 * t];
                    mx = fmaxf(mx, v[t]);
                }
#pragma unroll
                for (int o = 16; o >= 1; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                const float mn = fmaxf(run_m[jj], mx);      // finite: a chunk holds at least one block
                float sum = 0.0f;
#pragma unroll
                for (int t = 0; t < kChunk / 32; ++t) sum += exp2f(v[t] - mn);
#pragma unroll
                for (int o = 16; o >= 1; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
                run_l[jj] = run_l[jj] * exp2f(run_m[jj] - mn) + sum;
                run_m[jj] = mn;
                float* dst = logits + (slab + row0 + j) * (size_t)nb_pad + col_off + b0;
#pragma unroll
                for (int t = 0; t < kChunk / 32; ++t) dst[lane + 32 * t] = v[t];
            }
            __syncthreads();
        }
#pragma unroll
        for (int jj = 0; jj < 2; ++jj) {
            const int j = warp + 8 * jj;
            if (lane == 0) partials[(slab + row0 + j) * part_stride + part_off + part] = make_float2(run_m[jj], run_l[jj]);
        }
    }
}

// Merge the per-CTA statistics of every row, then R_b = (1/(L*H)) sum_rows exp2(logit - max_row) / Z_row.
// A CTA owns 32 consecutive blocks.  The session's (max, sum-exp) pairs are contiguous: they are staged
// in shared memory by one flat 128-bit copy (all loads independent) and merged there by a group of
// threads per row (fixed tree order).  Then thread (lgs, bl) sums the rows of heads lgs, lgs + 8, ...
// for block bl (independent coalesced loads), and the 8 partial sums are added in a fixed order.
constexpr int kFinishBlocks = 32;
__global__ void __launch_bounds__(256)
score_finish_kernel(const float* __restrict__ logits, const float2* __restrict__ partials,
                    const int32_t* __restrict__ nblocks_dev, int session_first, int LG, int rows, int rows_pad,
                    int nb_pad, int n_parts, float inv_LH, float* __restrict__ scores, int scores_stride, int stage_parts,
                    int nb_override) {
    pdl_wait();        // everything earlier in the stream is complete and visible from here on
    pdl_trigger();     // the next kernel's CTAs may take their places; they wait in the same way
    extern __shared__ float2 fin_smem[];  // rowstat [LG * rows_pad] : (max, 1/Z); then staged partials [LG * rows_pad][n_parts]
    float2* rowstat = fin_smem;
    float2* staged = fin_smem + LG * rows_pad;
    __shared__ float red[8][kFinishBlocks];
    const int s = blockIdx.y;
    const int n_slots = LG * rows_pad;                        // rows incl. padding: slot = lg * rows_pad + j
    const float2* sess_parts = partials + (size_t)s * n_slots * n_parts;
    // The kernel is a chain of memory round trips with little data behind them, so the first loads of every kind are
    // requested together: the session's block count, the logits of this thread's first head (the logit rows are
    // nb_pad long, so a column below nb_pad is readable whatever the count turns out to be) and the statistics.
    const int bl = threadIdx.x & 31, lgs = threadIdx.x >> 5;
    const int b0 = blockIdx.x * kFinishBlocks + bl;
    float pre[16];
    const bool have_pre = rows <= 16 && b0 < nb_pad && lgs < LG;
    if (have_pre) {
        const float* base = logits + (((size_t)s * LG + lgs) * rows_pad) * (size_t)nb_pad + b0;
#pragma unroll
        for (int j = 0; j < 16; ++j) pre[j] = j < rows ? base[(size_t)j * nb_pad] : 0.0f;
    }
    const int NB = nb_override >= 0 ? nb_override : nblocks_dev[session_first + s];
    if ((int)(blockIdx.x * kFinishBlocks) >= NB) return;
    if (stage_parts) {
        const int n16 = n_slots * n_parts / 2;                // rows_pad is a multiple of 16: an even number of pairs
        const uint4* src = reinterpret_cast<const uint4*>(sess_parts);
        uint4* dst = reinterpret_cast<uint4*>(staged);
#pragma unroll 4
        for (int i = threadIdx.x; i < n16; i += 256) dst[i] = src[i];
        __syncthreads();
    }
    // tpr threads per row (a power of two, at most 32): each merges a strided share of the parts, then a butterfly
    int tpr = 1;
    while (tpr < 32 && tpr * 2 * n_slots <= 256 && tpr * 2 <= n_parts) tpr *= 2;
    for (int base = 0; base < n_slots; base += 256 / tpr) {
        const int slot = base + (int)threadIdx.x / tpr, sub = (int)threadIdx.x % tpr;
        const bool live = slot < n_slots && (slot % rows_pad) < rows;
        float mx = -INFINITY, z = 0.0f;
        if (live) {
            const float2* pr = stage_parts ? staged + (size_t)slot * n_parts : sess_parts + (size_t)slot * n_parts;
            for (int c = sub; c < n_parts; c += tpr) mx = fmaxf(mx, pr[c].x);
            for (int c = sub; c < n_parts; c += tpr) {
                const float2 t = pr[c];
                if (t.x > -INFINITY) z += t.y * exp2f(t.x - mx);
            }
        }
        for (int o = 1; o < tpr; o <<= 1) {
            const float om = __shfl_xor_sync(0xffffffffu, mx, o), oz = __shfl_xor_sync(0xffffffffu, z, o);
            const float nm = fmaxf(mx, om);
            const float za = mx > -INFINITY ? z * exp2f(mx - nm) : 0.0f, zb = om > -INFINITY ? oz * exp2f(om - nm) : 0.0f;
            // the same operand order on both partners, so every thread of the group ends with identical bits
            z = (sub & o) ? zb + za : za + zb;
            mx = nm;
        }
        if (live && sub == 0) rowstat[slot] = make_float2(mx, 1.0f / z);
    }
    __syncthreads();
    float part = 0.0f;
    if (b0 < NB) {
        for (int lg = lgs; lg < LG; lg += 8) {
            const float* base = logits + (((size_t)s * LG + lg) * rows_pad) * (size_t)nb_pad + b0;
            float sub = 0.0f;
            if (have_pre && lg == lgs) {
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    if (j < rows) {
                        const float2 st = rowstat[lg * rows_pad + j];
                        sub += exp2f(pre[j] - st.x) * st.y;
                    }
                }
            } else {
#pragma unroll 16
                for (int j = 0; j < rows; ++j) {
                    const float2 st = rowstat[lg * rows_pad + j];
                    sub += exp2f(base[(size_t)j * nb_pad] - st.x) * st.y;
                }
            }
            part += sub;
        }
    }
    red[lgs][bl] = part;
    __syncthreads();
    if (threadIdx.x < kFinishBlocks) {
        const int b = blockIdx.x * kFinishBlocks + threadIdx.x;
        if (b < NB) {
            float total = 0.0f;
#pragma unroll
            for (int i = 0; i < 8; ++i) total += red[i][threadIdx.x];
            scores[(size_t)s * scores_stride + b] = total * inv_LH;
        }
    }
}

Option g_score_mode{1};   // 1: tensor-core dot products (default), 0: fp32 ALU + warp-shuffle kernel

// index [max_sessions * L * G * max_bps rows][128] bf16 as a 2-D tensor; box = 64 dims x 128 rows, 128-byte swizzle
static bool make_score_index_map(CUtensorMap* map, const __nv_bfloat16* index, long long index_rows) {
    static PFN_cuTensorMapEncodeTiled_v12000 enc = nullptr;
    if (!enc) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return false;
        enc = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(ptr);
    }
    cuuint64_t dims[2] = {128, (cuuint64_t)index_rows};
    cuuint64_t strides[1] = {256};
    cuuint32_t box[2] = {64, (cuuint32_t)kChunk};
    cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(index), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaError_t launch_score_decode(const kvmem_pool& p, int session_first, int n_sessions, const __nv_bfloat16* q,
                                int M, const ScoreWorkspace& ws, float* scores, int scores_stride, float score_scale, cudaStream_t st) {
    const Geometry& g = p.geo;
    if (M > kMaxDecodeTokens) return cudaErrorNotSupported;
    const float scale_log2e = 1.4426950408889634f / sqrtf((float)g.d);
    int max_nb = 0;
    for (int s = session_first; s < session_first + n_sessions; ++s) max_nb = std::max(max_nb, p.sess_blocks[s]);
    if (max_nb == 0) return cudaSuccess;
    const int LG = g.L * g.G;
    // One session: its block count is known here (the host's copy, which sized the grid anyway) and is handed to the
    // kernels as an argument, which spares each of them a dependent read of the device copy before its first load.
    const int nb_known = n_sessions == 1 ? max_nb : -1;
    const int chunks = (max_nb + kChunk - 1) / kChunk;
    // persistent CTAs: about one per SM, each streaming a contiguous range of chunks of one (session, l, g)
    // Two CTAs of the tensor-core kernel fit on an SM.  The second one is used only while the row statistics stay
    // short (many sessions or heads: at most 4 partials per row); a long single session is fastest with one CTA per
    // SM and half as many partials to merge (measured at 1M: 18 parts 38.6 us, 36 parts 41.7 us for the select stage).
    const int heads = std::max(1, LG * n_sessions);
    const int fit1 = p.sm_count / heads, fit2 = g_score_mode == 1 ? 2 * p.sm_count / heads : fit1;
    const int n_parts = std::max(1, std::min({chunks, kMaxScoreParts, fit2 <= 4 ? fit2 : fit1}));
    const size_t smem = (size_t)kScoreStages * kChunk * 256;
    dim3 grid((unsigned)n_parts, (unsigned)LG, (unsigned)n_sessions);
    cudaError_t e;
    const long long index_rows = (long long)g.max_sessions * g.L * g.G * g.max_bps;
    if (g_score_mode == 1 && index_rows <= 0x7fffffffll) {     // TMA row coordinates are 32-bit
        CUtensorMap map_idx;
        if (!make_score_index_map(&map_idx, p.index, index_rows)) return cudaErrorInvalidValue;
        static PerDeviceOnce attr_done;
        if (attr_done.pending(p.cfg.device)) {
            e = cudaFuncSetAttribute(score_logits_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(smem + 1024));
            if (e != cudaSuccess) return e;
            attr_done.mark(p.cfg.device);
        }
        launch_pdl(score_logits_mma_kernel, dim3(grid), dim3(kScoreThreads), smem + 1024, st, 
            map_idx, q, p.nblocks_dev, session_first, M, g.L, g.H, g.G, g.max_bps, ws.logits, ws.partials, ws.rows,
            ws.rows_pad, ws.nb_pad, n_parts, scale_log2e, p.status_dev, nb_known, 0, n_parts, 0);
    } else {
#define KVMEM_SCORE_LAUNCH(RP)                                                                                         \
    do {                                                                                                               \
        static PerDeviceOnce attr_done;                                                                                 \
        if (attr_done.pending(p.cfg.device)) {                                                                                              \
            e = cudaFuncSetAttribute(score_logits_kernel<RP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
            if (e != cudaSuccess) return e;                                                                            \
            attr_done.mark(p.cfg.device);                                                                                          \
        }                                                                                                              \
        launch_pdl(score_logits_kernel<RP>, dim3(grid), dim3(kScoreThreads), smem, st,                                                     \
            q, p.index, p.nblocks_dev, session_first, M, g.L, g.H, g.G, g.max_bps, p.lay.index_elems_per_session,      \
            ws.logits, ws.partials, ws.rows, ws.rows_pad, ws.nb_pad, n_parts, scale_log2e, p.status_dev);              \
    } while (0)
        if (ws.rows <= 4) KVMEM_SCORE_LAUNCH(4);
        else if (ws.rows <= 8) KVMEM_SCORE_LAUNCH(8);
        else KVMEM_SCORE_LAUNCH(16);
#undef KVMEM_SCORE_LAUNCH
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    size_t fsmem = (size_t)LG * ws.rows_pad * sizeof(float2);
    const size_t stage_bytes = fsmem * n_parts;
    const int stage_parts = fsmem + stage_bytes <= 96 * 1024 ? 1 : 0;       // stage the pairs when they fit
    if (stage_parts) fsmem += stage_bytes;
    if (fsmem > 48 * 1024) {
        e = cudaFuncSetAttribute(score_finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fsmem);
        if (e != cudaSuccess) return e;
    }
    dim3 fgrid((unsigned)((max_nb + kFinishBlocks - 1) / kFinishBlocks), (unsigned)n_sessions);
    launch_pdl(score_finish_kernel, dim3(fgrid), dim3(256), fsmem, st, ws.logits, ws.partials, p.nblocks_dev, session_first, LG, ws.rows,
                                                   ws.rows_pad, ws.nb_pad, n_parts, score_scale / (float)(g.L * g.H),
                                                   scores, scores_stride, stage_parts, nb_known);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------
// Scoring against an index that lives in HOST memory (Sec. 5.2: the index is streamed to the GPU in
// tiles and the softmax statistics are carried across tiles).  Tiles of tile_blocks blocks per (layer,
// KV head) are copied into one of two device staging buffers on the pool's copy stream while the
// previous tile is scored on the caller's stream (events in both directions, no device-wide
// synchronisation).  Every tile adds its per-row (max, sum-exp) pairs to the partials array; the logits
// of all blocks stay on the device (fp32, [rows][NB]); after the last tile the pairs are merged per row
// in a fixed order and the finish kernel normalises, exactly as for an index in device memory.

// (max, sum-exp) pairs of one row -> one pair, in slot order
__global__ void __launch_bounds__(128)
score_merge_partials_kernel(const float2* __restrict__ partials, float2* __restrict__ merged, int n_rows, int n_parts) {
    const int row = blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= n_rows) return;
    const float2* p = partials + (size_t)row * n_parts;
    float mx = -INFINITY;
    for (int c = 0; c < n_parts; ++c) mx = fmaxf(mx, p[c].x);
    float z = 0.0f;
    for (int c = 0; c < n_parts; ++c) {
        const float2 t = p[c];
        if (t.x > -INFINITY) z += t.y * exp2f(t.x - mx);
    }
    merged[row] = make_float2(mx, z);
}

HostScorePlan plan_host_score(const kvmem_pool_config_t& c, int n_blocks, int n_q_tokens, int tile_blocks, int sm_count, char* base) {
    HostScorePlan w{};
    const int r = c.n_q_heads / c.n_kv_heads, LG = c.n_layers * c.n_kv_heads;
    w.rows = n_q_tokens * r;
    w.rows_pad = (w.rows + 15) / 16 * 16;
    w.nb_pad = (n_blocks + kChunk - 1) / kChunk * kChunk;
    w.n_tiles = (n_blocks + tile_blocks - 1) / tile_blocks;
    w.parts_per_tile = std::max(1, std::min({tile_blocks / kChunk, kMaxScoreParts, sm_count / std::max(1, LG)}));
    w.part_stride = w.n_tiles * w.parts_per_tile;
    w.logits_bytes = align_up((size_t)LG * w.rows_pad * w.nb_pad * sizeof(float), 256);
    w.partials_bytes = align_up((size_t)LG * w.rows_pad * w.part_stride * sizeof(float2), 256);
    w.merged_bytes = align_up((size_t)LG * w.rows_pad * sizeof(float2), 256);
    w.total = w.logits_bytes + w.partials_bytes + w.merged_bytes;
    w.staging_bytes = 2 * align_up((size_t)LG * tile_blocks * 256, 256);
    if (base) {
        w.logits = reinterpret_cast<float*>(base);
        w.partials = reinterpret_cast<float2*>(base + w.logits_bytes);
        w.merged = reinterpret_cast<float2*>(base + w.logits_bytes + w.partials_bytes);
    }
    return w;
}

cudaError_t launch_score_host_index(kvmem_pool& p, const __nv_bfloat16* index_host, int n_blocks, int stride_blocks,
                                    const __nv_bfloat16* q, int M, int tile_blocks, void* staging, const HostScorePlan& ws,
                                    float* scores, cudaStream_t st) {
    const Geometry& g = p.geo;
    const int LG = g.L * g.G;
    cudaError_t e;
    if (!p.copy_stream) {                                  // created on first use, destroyed with the pool
        e = cudaStreamCreateWithFlags(&p.copy_stream, cudaStreamNonBlocking);
        if (e != cudaSuccess) return e;
        for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
            e = cudaEventCreateWithFlags(&p.ev_ready[i], cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p.ev_free[i], cudaEventDisableTiming);
        }
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p.ev_start, cudaEventDisableTiming);
        if (e != cudaSuccess) return e;
    }
    static PerDeviceOnce attr_done;
    const size_t smem = (size_t)kScoreStages * kChunk * 256 + 1024;
    if (attr_done.pending(p.cfg.device)) {
        e = cudaFuncSetAttribute(score_logits_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_done.mark(p.cfg.device);
    }
    const size_t buf_bytes = align_up((size_t)LG * tile_blocks * 256, 256);
    const float scale_log2e = 1.4426950408889634f / sqrtf((float)g.d);
    // whatever the caller's stream did with the staging buffers before (an earlier call) is finished first
    if ((e = cudaEventRecord(p.ev_start, st)) != cudaSuccess) return e;
    if ((e = cudaStreamWaitEvent(p.copy_stream, p.ev_start, 0)) != cudaSuccess) return e;
    for (int i = 0; i < ws.n_tiles; ++i) {
        const int b0 = i * tile_blocks, nb = std::min(tile_blocks, n_blocks - b0), buf = i & 1;
        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(reinterpret_cast<char*>(staging) + (size_t)buf * buf_bytes);
        if (i >= 2 && (e = cudaStreamWaitEvent(p.copy_stream, p.ev_free[buf], 0)) != cudaSuccess) return e;
        // one strided copy: nb * 256 bytes of each of the L*G heads
        e = cudaMemcpy2DAsync(dst, (size_t)tile_blocks * 256, index_host + (size_t)b0 * g.d, (size_t)stride_blocks * 256,
                              (size_t)nb * 256, (size_t)LG, cudaMemcpyHostToDevice, p.copy_stream);
        if (e != cudaSuccess) return e;
        if ((e = cudaEventRecord(p.ev_ready[buf], p.copy_stream)) != cudaSuccess) return e;
        if ((e = cudaStreamWaitEvent(st, p.ev_ready[buf], 0)) != cudaSuccess) return e;
        CUtensorMap map_idx;
        if (!make_score_index_map(&map_idx, dst, (long long)LG * tile_blocks)) return cudaErrorInvalidValue;
        dim3 grid((unsigned)ws.parts_per_tile, (unsigned)LG, 1);
        score_logits_mma_kernel<<<grid, kScoreThreads, smem, st>>>(map_idx, q, p.nblocks_dev, 0, M, g.L, g.H, g.G, tile_blocks,
                                                                  ws.logits, ws.partials, ws.rows, ws.rows_pad, ws.nb_pad,
                                                                  ws.parts_per_tile, scale_log2e, p.status_dev, nb, b0,
                                                                  ws.part_stride, i * ws.parts_per_tile);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        if ((e = cudaEventRecord(p.ev_free[buf], st)) != cudaSuccess) return e;
    }
    const int n_rows = LG * ws.rows_pad;
    score_merge_partials_kernel<<<(n_rows + 127) / 128, 128, 0, st>>>(ws.partials, ws.merged, n_rows, ws.part_stride);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    const size_t fsmem = 2 * (size_t)LG * ws.rows_pad * sizeof(float2);
    if (fsmem > 48 * 1024) {
        e = cudaFuncSetAttribute(score_finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fsmem);
        if (e != cudaSuccess) return e;
    }
    dim3 fgrid((unsigned)((n_blocks + kFinishBlocks - 1) / kFinishBlocks), 1);
    score_finish_kernel<<<fgrid, 256, fsmem, st>>>(ws.logits, ws.merged, nullptr, 0, LG, ws.rows, ws.rows_pad, ws.nb_pad, 1,
                                                   1.0f / (float)(g.L * g.H), scores, n_blocks, 1, n_blocks);
    return cudaGetLastError();
}

}  // namespace kvmem
