// Decode-sized block scoring in ONE kernel (Eq. "kvmem-block-score", Sec. 4.3; the softmax kept global
// across tiles, Sec. 5.2):
//   R_b = sum_m (1/(L*H)) sum_{l,h} softmax_{b'}( q[l][m][h] . kbar[l][b'][g(h)] / sqrt(d) )_b
//
// The three-kernel form (logits to global memory, a finish kernel that merges the row statistics and
// normalises, then the selection) spends most of its time between kernels.  Here a CTA owns a range of
// blocks of one session for ALL (layer, KV head) pairs, keeps the logits of its range in shared memory,
// publishes its per-row (max, sum-exp) pairs, meets the other CTAs at one grid-wide barrier, merges the
// pairs of its session (every CTA in the same fixed order, so all arrive at the same statistics) and
// writes R for its own blocks: no logit ever leaves the SM and the sum over heads is formed in a fixed
// order inside one CTA, so the scores are identical from run to run.
//
// Index tiles arrive by tiled TMA (128-byte swizzle) through a ring of 32 KiB stages; a stage holds 128
// Mean-K vectors = (128 / C) heads x C blocks, C in {16, 32, 64, 128} chosen so that short sessions still
// spread over the SMs.  The <= 16 query rows of a KV head are one m16 MMA tile (bf16 mma.sync, fp32
// accumulate); each warp takes 16 vectors of a stage.
//
// The grid barrier needs every CTA resident at once: the launcher sizes the grid to at most one CTA per SM
// and falls back to the three-kernel form otherwise.  The wait at the barrier is bounded like every other
// wait in this library: a CTA that gives up records KVMEM_E_TIMEOUT and returns.
#include <cudaTypedefs.h>
#include <math.h>

#include <algorithm>

#include "kvmem_internal.cuh"
#include "kvmem_ptx.cuh"

namespace kvmem {

constexpr int kFsThreads = 256;
constexpr int kFsStages = 3;
constexpr int kFsStageVecs = 128;                       // Mean-K vectors per stage
constexpr uint32_t kFsHalf = kFsStageVecs * 128;        // one 64-dim half of a stage: 128 rows x 128 B
constexpr uint32_t kFsStage = 2 * kFsHalf;              // 32 KiB
constexpr int kFsRows = 16;                             // query rows per KV head (one m16 tile)
constexpr int kFsMaxLG = 16;
constexpr int kFsQBytes = kFsRows * 256;                // one head's query tile in shared memory

struct FusedScoreArgs {
    const __nv_bfloat16* q;
    const int32_t* nblocks_dev;
    float2* partials;            // [n_sessions][parts][LG * 16]: (max, sum-exp) of every row over one CTA's blocks
    float* scores;
    int32_t* status;
    unsigned int* bar;           // bar[0]: arrivals, bar[16]: generation (own 64-byte lines inside the pool's status area)
    int scores_stride, session_first, M, L, H, G, r, rows, max_bps;
    int C;                       // blocks per chunk
    int parts;                   // CTAs per session
    int n_ctas;                  // parts * n_sessions
    int max_chunks;              // chunks a CTA has logit room for
    float scale_log2e, out_scale;
};

// One arrival per CTA (thread 0, after a CTA barrier and a fence).  The last arrival re-arms the counter and advances
// the generation the others wait for.  false: the wait ran out.
__device__ __forceinline__ bool grid_barrier_bounded(unsigned int* count, unsigned int* gen, unsigned int n) {
    unsigned int g;
    asm volatile("ld.acquire.gpu.u32 %0, [%1];" : "=r"(g) : "l"(gen) : "memory");
    __threadfence();
    const unsigned int old = atomicAdd(count, 1u);
    if (old == n - 1u) {
        atomicExch(count, 0u);
        __threadfence();
        asm volatile("st.release.gpu.u32 [%0], %1;" ::"l"(gen), "r"(g + 1u) : "memory");
        return true;
    }
    uint64_t t0 = 0;
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        unsigned int now_g;
        asm volatile("ld.acquire.gpu.u32 %0, [%1];" : "=r"(now_g) : "l"(gen) : "memory");
        if (now_g != g) return true;
        if ((i & 63u) == 63u) {
            const uint64_t now = ptx::globaltimer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitLimitNs) return false;
        }
    }
    return false;
}

__global__ void __launch_bounds__(kFsThreads, 1)
score_fused_kernel(const __grid_constant__ CUtensorMap map_idx, FusedScoreArgs a) {
    extern __shared__ unsigned char smem_dyn[];
    __shared__ uint64_t full_bar[kFsStages];
    __shared__ int barrier_ok;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int part = blockIdx.x, s = blockIdx.y;
    const int LG = a.L * a.G, C = a.C, rows = a.rows;

    unsigned char* stage_mem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    unsigned char* qsm = stage_mem + (size_t)kFsStages * kFsStage;                  // [LG][16 rows][256 B], 16-byte chunks XOR-ed with row & 7
    float2* rowstat = reinterpret_cast<float2*>(qsm + (size_t)LG * kFsQBytes);      // [LG * 16]: (max, 1 / Z)
    float* slog = reinterpret_cast<float*>(rowstat + LG * kFsRows);                 // [chunk][lg][row < rows][C] logits (exp2 domain)

    if (tid == 0) {
        for (int i = 0; i < kFsStages; ++i) ptx::mbar_init(&full_bar[i], 1);
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&map_idx);
    }
    __syncthreads();
    pdl_wait();        // everything earlier in the stream is complete and visible from here on
    pdl_trigger();     // the next kernel's CTAs may take their places; they wait in the same way

    const int NB = a.nblocks_dev[a.session_first + s];
    const int n_chunks = (NB + C - 1) / C;
    const int c_begin = (int)((long long)n_chunks * part / a.parts);
    int n_mine = (int)((long long)n_chunks * (part + 1) / a.parts) - c_begin;
    if (n_mine > a.max_chunks) {            // the host sized the logit room from its own block counts
        if (tid == 0) atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE);
        n_mine = a.max_chunks;
    }
    const int hps = kFsStageVecs / C;                         // heads per stage
    const int spc = (LG + hps - 1) / hps;                     // stages per chunk
    const int n_st = n_mine * spc;

    // the query rows of every head: row j = m * r + hr  ->  q[s][m][l][g*r + hr]; rows past `rows` are zero
    for (int i = tid; i < LG * kFsRows * 16; i += kFsThreads) {
        const int lg = i >> 8, row = (i >> 4) & 15, ch = i & 15;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (row < rows) {
            const int l = lg / a.G, g = lg % a.G;
            v = *reinterpret_cast<const uint4*>(a.q + ((((size_t)s * a.M + row / a.r) * a.L + l) * a.H + (size_t)g * a.r + row % a.r) * 128 + ch * 8);
        }
        *reinterpret_cast<uint4*>(qsm + (size_t)lg * kFsQBytes + row * 256 + ((ch ^ (row & 7)) << 4)) = v;
    }

    auto issue = [&](int i) {                                 // thread 0 only: stage i of this CTA
        const int st = i % kFsStages, ci = i / spc, lg0 = (i % spc) * hps;
        const int n_sub = min(hps, LG - lg0);
        const int b0 = (c_begin + ci) * C;
        unsigned char* dst = stage_mem + (size_t)st * kFsStage;
        ptx::mbar_expect_tx(&full_bar[st], (uint32_t)n_sub * (uint32_t)C * 256u);
        for (int j = 0; j < n_sub; ++j) {
            const int row = ((a.session_first + s) * LG + lg0 + j) * a.max_bps + b0;
            ptx::tma_load_2d(dst + (size_t)j * C * 128, &map_idx, 0, row, &full_bar[st]);
            ptx::tma_load_2d(dst + kFsHalf + (size_t)j * C * 128, &map_idx, 64, row, &full_bar[st]);
        }
    };
    if (tid == 0)
        for (int i = 0; i < min(kFsStages - 1, n_st); ++i) issue(i);
    __syncthreads();                                          // the query tiles are in place

    const uint32_t stage0 = ptx::smem_u32(stage_mem), q0 = ptx::smem_u32(qsm);
    const int mj = lane >> 3, mr = lane & 7;                  // ldmatrix: matrix index and row within it
    bool alive = true;
    for (int i = 0; i < n_st; ++i) {
        const int st = i % kFsStages;
        const bool ok = ptx::mbar_wait(&full_bar[st], (uint32_t)((i / kFsStages) & 1));
        if (__syncthreads_or(!ok)) {                          // CTA-uniform: somebody gave up
            if (tid == 0) atomicExch(a.status, (int)KVMEM_E_TIMEOUT);
            alive = false;
            break;
        }
        // the stage consumed in iteration i - 1 was released by the barrier above: refill it
        if (tid == 0 && i + kFsStages - 1 < n_st) issue(i + kFsStages - 1);
        const int ci = i / spc, lg0 = (i % spc) * hps;
        const int j = (warp * 16) / C, off = (warp * 16) % C;  // this warp's head within the stage and block offset within the chunk
        const int lg = lg0 + j;
        if (lg < LG) {
            const uint32_t tile = stage0 + (uint32_t)st * kFsStage;
            const int qrow = mr + 8 * (mj & 1);
            const uint32_t qaddr = q0 + (uint32_t)lg * kFsQBytes + (uint32_t)qrow * 256u;
            float sc[2][4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) { sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.0f; }
#pragma unroll
            for (int kp = 0; kp < 4; ++kp) {
                const int cg = kp * 4 + mj;
                const uint32_t half_off = (uint32_t)(cg >> 3) * kFsHalf;
                const int c = cg & 7;
                uint32_t qa[2][4];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int ks = 2 * kp + h;
                    ptx::ldmatrix_x4(qaddr + (uint32_t)(((ks * 2 + (mj >> 1)) ^ (qrow & 7)) << 4), qa[h][0], qa[h][1], qa[h][2], qa[h][3]);
                }
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    const int rowi = warp * 16 + nt * 8 + mr;
                    const uint32_t addr = tile + half_off + (uint32_t)rowi * 128u + (uint32_t)((c ^ (rowi & 7)) << 4);
                    uint32_t b0r, b1r, b2r, b3r;
                    ptx::ldmatrix_x4(addr, b0r, b1r, b2r, b3r);
                    ptx::mma_bf16_16816(sc[nt], qa[0], b0r, b1r);
                    ptx::mma_bf16_16816(sc[nt], qa[1], b2r, b3r);
                }
            }
            const int ra = lane >> 2, rb = ra + 8;
            const int bbase = (c_begin + ci) * C;
            float* la = slog + ((size_t)(ci * LG + lg) * rows + ra) * C;
            float* lb = slog + ((size_t)(ci * LG + lg) * rows + rb) * C;
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
                const int col = off + nt * 8 + 2 * (lane & 3);
                const bool v0 = bbase + col < NB, v1 = bbase + col + 1 < NB;
                if (ra < rows) *reinterpret_cast<float2*>(la + col) = make_float2(v0 ? sc[nt][0] * a.scale_log2e : -INFINITY, v1 ? sc[nt][1] * a.scale_log2e : -INFINITY);
                if (rb < rows) *reinterpret_cast<float2*>(lb + col) = make_float2(v0 ? sc[nt][2] * a.scale_log2e : -INFINITY, v1 ? sc[nt][3] * a.scale_log2e : -INFINITY);
            }
        }
    }
    __syncthreads();

    // per-row statistics of this CTA's blocks: warp-strided over the (head, row) pairs, lane-strided over the blocks
    float2* my_parts = a.partials + ((size_t)s * a.parts + part) * (LG * kFsRows);
    for (int p = warp; p < LG * kFsRows; p += kFsThreads / 32) {
        const int lg = p >> 4, row = p & 15;
        float mx = -INFINITY, sum = 0.0f;
        if (row < rows && alive) {
            for (int ci = 0; ci < n_mine; ++ci) {
                const float* src = slog + ((size_t)(ci * LG + lg) * rows + row) * C;
                for (int c = lane; c < C; c += 32) mx = fmaxf(mx, src[c]);
            }
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            if (mx > -INFINITY) {
                for (int ci = 0; ci < n_mine; ++ci) {
                    const float* src = slog + ((size_t)(ci * LG + lg) * rows + row) * C;
                    for (int c = lane; c < C; c += 32) sum += exp2f(src[c] - mx);
                }
            }
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        }
        if (lane == 0) my_parts[p] = make_float2(mx, sum);
    }
    __syncthreads();
    if (tid == 0) {
        const bool ok = grid_barrier_bounded(a.bar, a.bar + 16, (unsigned int)a.n_ctas);
        if (!ok) atomicExch(a.status, (int)KVMEM_E_TIMEOUT);
        __threadfence();
        barrier_ok = ok ? 1 : 0;
    }
    __syncthreads();
    if (!barrier_ok || !alive) return;

    // merge the session's pairs per row, every CTA in the same order (part 0, 1, ...): identical statistics everywhere
    if (tid < LG * kFsRows) {
        float m = -INFINITY, z = 0.0f;
        if ((tid & 15) < rows) {
            const float2* src = a.partials + (size_t)s * a.parts * (LG * kFsRows) + tid;
            for (int pt = 0; pt < a.parts; ++pt) {
                const float2 t = __ldcg(src + (size_t)pt * (LG * kFsRows));
                if (t.x > -INFINITY) {
                    const float nm = fmaxf(m, t.x);
                    z = z * exp2f(m - nm) + t.y * exp2f(t.x - nm);
                    m = nm;
                }
            }
        }
        rowstat[tid] = make_float2(m, z > 0.0f ? 1.0f / z : 0.0f);
    }
    __syncthreads();

    // R for this CTA's blocks: eight lanes share a block, lane `sub` adds the (head, row) terms sub, sub + 8, ...;
    // the eight partial sums meet in a butterfly, i.e. in a fixed order
    const int n_own = n_mine * C, T = LG * rows;
    for (int base = 0; base < n_own; base += kFsThreads / 8) {
        const int bl = base + (tid >> 3), sub = tid & 7;
        float acc = 0.0f;
        if (bl < n_own) {
            const int ci = bl / C, col = bl % C;
            for (int t = sub; t < T; t += 8) {
                const int lg = t / rows, row = t % rows;
                const float2 st = rowstat[lg * kFsRows + row];
                acc += exp2f(slog[((size_t)(ci * LG + lg) * rows + row) * C + col] - st.x) * st.y;
            }
        }
        acc += __shfl_xor_sync(0xffffffffu, acc, 1);
        acc += __shfl_xor_sync(0xffffffffu, acc, 2);
        acc += __shfl_xor_sync(0xffffffffu, acc, 4);
        const int b = c_begin * C + bl;
        if (sub == 0 && bl < n_own && b < NB) a.scores[(size_t)s * a.scores_stride + b] = acc * a.out_scale;
    }
}

int g_score_fused = 1;    // 1: one-kernel scoring where it fits (default), 0: logits kernel + finish kernel

static bool make_fused_index_map(CUtensorMap* map, const __nv_bfloat16* index, long long index_rows, int box_rows) {
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
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(index), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// *launched = false: the shape does not fit the one-kernel form (too many rows, heads or blocks per CTA); nothing was enqueued
cudaError_t launch_score_fused(const kvmem_pool& p, int session_first, int n_sessions, const __nv_bfloat16* q, int M,
                               const ScoreWorkspace& ws, float* scores, int scores_stride, float score_scale, cudaStream_t st,
                               bool* launched) {
    *launched = false;
    const Geometry& g = p.geo;
    const int LG = g.L * g.G, rows = M * g.r;
    if (!g_score_fused || g_score_mode != 1 || rows > kFsRows || LG > kFsMaxLG || n_sessions > p.sm_count) return cudaSuccess;
    const long long index_rows = (long long)g.max_sessions * LG * g.max_bps;
    if (index_rows > 0x7fffffffll) return cudaSuccess;
    int max_nb = 0;
    for (int s = session_first; s < session_first + n_sessions; ++s) max_nb = std::max(max_nb, p.sess_blocks[s]);
    if (max_nb == 0) { *launched = true; return cudaSuccess; }
    // the largest chunk that still spreads the sessions over most of the SMs
    int C = 16;
    for (int c : {128, 64, 32}) {
        if ((long long)n_sessions * ((max_nb + c - 1) / c) * 4 >= 3ll * p.sm_count) { C = c; break; }
    }
    const int chunks = (max_nb + C - 1) / C;
    const int parts = std::max(1, std::min(chunks, p.sm_count / n_sessions));
    const int max_chunks = (chunks + parts - 1) / parts;
    const size_t smem = 1024 + (size_t)kFsStages * kFsStage + (size_t)LG * kFsQBytes + (size_t)LG * kFsRows * sizeof(float2) +
                        (size_t)max_chunks * LG * rows * C * sizeof(float);
    if (smem > 227 * 1024) return cudaSuccess;
    if (parts > kFusedScoreMaxParts || (size_t)n_sessions * parts * LG * kFsRows * sizeof(float2) > ws.partials_bytes) return cudaSuccess;
    CUtensorMap map_idx;
    if (!make_fused_index_map(&map_idx, p.index, index_rows, C)) return cudaErrorInvalidValue;
    static PerDeviceOnce attr_done;
    if (attr_done.pending(p.cfg.device)) {
        cudaError_t e = cudaFuncSetAttribute(score_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        attr_done.mark(p.cfg.device);
    }
    FusedScoreArgs a{};
    a.q = q; a.nblocks_dev = p.nblocks_dev; a.partials = ws.partials; a.scores = scores; a.status = p.status_dev;
    a.bar = reinterpret_cast<unsigned int*>(p.status_dev) + 16;          // 64 bytes into the status area
    a.scores_stride = scores_stride; a.session_first = session_first; a.M = M; a.L = g.L; a.H = g.H; a.G = g.G; a.r = g.r;
    a.rows = rows; a.max_bps = g.max_bps; a.C = C; a.parts = parts; a.n_ctas = parts * n_sessions; a.max_chunks = max_chunks;
    a.scale_log2e = 1.4426950408889634f / sqrtf((float)g.d);
    a.out_scale = score_scale / (float)(g.L * g.H);
    launch_pdl(score_fused_kernel, dim3((unsigned)parts, (unsigned)n_sessions), dim3(kFsThreads), smem, st, map_idx, a);
    *launched = true;
    return cudaGetLastError();
}

}  // namespace kvmem
