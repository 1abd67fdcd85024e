// Block scoring for a multi-token query chunk (Eq. "kvmem-block-score", Sec. 4.3) as a dense
// contraction on the 5th-generation tensor cores.
//
// Per (session, layer, KV head): logits S = Q_g K̄_g^T with Q_g the M*(H/G) query rows of the head
// group (2,048 x 128 for a 512-token chunk) and K̄_g the head's Mean-K index (NB x 128).  The
// 2,048 x 16,384 logit matrix (1 GiB in fp32 over 8 heads) is never stored; the exact softmax needs
// row statistics before column sums, so the contraction runs twice:
//   pass 1 (S   = Q K̄^T): per query row, running max and sum-exp over all blocks -> rowstat (max, log2 Z)
//   pass 2 (S^T = K̄ Q^T): p = exp2(s - max - log2 Z) summed over all query rows    -> headsum[l][g][b]
// and a small kernel adds the heads in a fixed order: R_b = (1/(L*H)) sum_{l,g} headsum.
// tcgen05.ld hands each epilogue thread one accumulator row (one TMEM lane).  Pass 1 puts query rows
// on the lanes, so the row statistics are thread-local; pass 2 swaps the operands and puts blocks on
// the lanes, so the sum over query rows is thread-local too: no shuffles, no atomics, and the
// per-row shifts -(max + log2 Z) are broadcast reads from shared memory.
//
// Both passes: UMMA M = 128, N = 256, K = 128 (8 instructions of K = 16), bf16 in, fp32 accumulate.
// Warp 0 is the TMA producer (stationary operand once per work item, streamed operand through a
// shared-memory ring, 128-byte swizzle), one thread of warp 1 issues tcgen05.mma into two 256-column
// TMEM accumulators, warps 2-17 are the epilogue (four per TMEM lane quarter, a quarter of a tile's columns each).  The epilogue of tile t overlaps the MMAs of tile
// t + 1.  Pass 1: one CTA per 128-row query panel, sweeping all blocks.  Pass 2: persistent CTAs, one
// work item = 128 blocks of one head, sweeping that head's query rows.  All mbarrier waits are bounded.
#include <cudaTypedefs.h>
#include <math.h>

#include <algorithm>

#include "kvmem_internal.cuh"
#include "kvmem_ptx.cuh"

namespace kvmem {

constexpr int kCkBM = 128;                    // accumulator rows (UMMA M): one TMEM lane each
constexpr int kCkBN = 256;                    // accumulator columns per tile (UMMA N): the largest N halves the
                                              // MMA instructions per flop, which one issuing thread must sustain
constexpr int kCkAccs = 2;                    // TMEM accumulators of 256 columns in flight
constexpr int kCkStages1 = 3;                 // streamed tiles in flight, pass 1
constexpr int kCkStages2 = 2;                 // streamed tiles in flight, pass 2 (two stationary panels + shifts also live in smem)
constexpr int kCkEpiWarps = 16;               // four per TMEM lane quarter, each takes a quarter of a tile's columns
constexpr int kCkSplit = kCkEpiWarps / 4;     // column slices per tile
constexpr int kCkThreads = 64 + 32 * kCkEpiWarps;   // TMA warp, MMA warp, epilogue warps
constexpr int kCkHalfCols = kCkBN / kCkSplit; // columns per epilogue warp and tile
constexpr int kCkChunks = kCkHalfCols / 32;   // 32-column register chunks per epilogue warp and tile
constexpr int kCkAHalf = kCkBM * 128;         // bytes of one 64-dim half of the 128-row operand tile (16 KiB)
constexpr int kCkBHalf = kCkBN * 128;         // bytes of one 64-dim half of the 256-row operand tile (32 KiB)
constexpr int kCkTmemCols = kCkAccs * kCkBN;  // 512: all of tensor memory
constexpr size_t kCkSmem = 2 * kCkAHalf + (size_t)kCkStages1 * 2 * kCkBHalf + 1024;

namespace t5 {   // tcgen05 wrappers

__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(ptx::smem_u32(dst_smem)), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate, one CTA
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// mbarrier arrives once all MMAs issued so far by this thread have completed
__device__ __forceinline__ void commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(ptx::smem_u32(bar)) : "memory");
}
// issue the load of 32 columns without waiting for it
__device__ __forceinline__ void ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes, 8-row groups
// 1,024 bytes apart.  Only the low word depends on the address; advancing K by 16 elements (32 bytes,
// inside the swizzle span) adds 2 to it, and the second 64-dim half adds half_bytes / 16.
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);   // SBO, descriptor version 1, SWIZZLE_128B
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr) { return (addr & 0x3ffffu) >> 4; }
__device__ __forceinline__ uint64_t make_desc(uint32_t lo) { return ((uint64_t)kDescHi << 32) | (uint64_t)lo; }

}  // namespace t5

__device__ __forceinline__ void tma_load_4d(void* dst_smem, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::
            "r"(ptx::smem_u32(dst_smem)),
        "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(ptx::smem_u32(bar))
        : "memory");
}

struct ChunkArgs {
    const int32_t* nblocks_dev;
    float2* rowstat;      // [ns][LG][n_chunks][kCkSplit][rows_pad]  (max, sum-exp) of every query row over one run of block tiles and one slice of the tile columns, log2 domain
    float* shift;         // [ns][LG][shift_stride]                  -(max + log2 Z) per query row
    float* headsum;       // [ns][LG][kCkSplit][nb_pad]              per column slice: sum over the head's query rows of the softmax weights
    int32_t* status;
    int session_first, n_sessions, M, L, G, r, rows, rows_pad, nb_pad, n_bpanels, n_panels, n_chunks, shift_stride;
    float scale_log2e;
};

// fp32 accumulate, bf16 x bf16, both operands K-major, N = 256, M = 128
__device__ __forceinline__ uint32_t chunk_idesc() {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kCkBN >> 3) << 17) | ((uint32_t)(kCkBM >> 4) << 24);
}

// one 128 x 256 x 128 tile: 8 MMAs of K = 16
__device__ __forceinline__ void issue_tile_mma(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo) {
    const uint32_t idesc = chunk_idesc();
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const uint32_t ka = (uint32_t)(k >> 2) * (kCkAHalf >> 4) + (uint32_t)(k & 3) * 2u;
        const uint32_t kb = (uint32_t)(k >> 2) * (kCkBHalf >> 4) + (uint32_t)(k & 3) * 2u;
        t5::mma_bf16(d_tmem, t5::make_desc(a_lo + ka), t5::make_desc(b_lo + kb), idesc, k > 0 ? 1u : 0u);
    }
}

// Packed fp32 arithmetic (two lanes per instruction, operands in 64-bit register pairs): the scale-and-
// shift, the accumulation and the polynomial below cost half the issue slots of their scalar forms, which
// matters because the epilogue is bounded by the special-function unit first and by issue slots second.
namespace f2 {
__device__ __forceinline__ uint64_t pk(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ uint64_t pk(uint32_t lo, uint32_t hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpk(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ void unpk(uint64_t v, uint32_t& lo, uint32_t& hi) { asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
}  // namespace f2

// 2^x for a pair, on the FMA and integer pipes: the share of the exponentials that the special-function
// unit (16 results per clock and SM, the limiter of both passes) is spared.  x = n + f with n the nearest
// integer and |f| <= 1/2; 2^f by a degree-4 polynomial (relative error below 3e-6), 2^n by adding n to
// the exponent field.  Arguments below -125 (including -inf) return about 2^-125 instead of 0, which
// is immaterial next to weights that sum to one per query row.
__device__ __forceinline__ uint64_t ex2_poly2(uint64_t x2) {
    float x0, x1;
    f2::unpk(x2, x0, x1);
    const uint64_t x = f2::pk(fmaxf(x0, -125.0f), fmaxf(x1, -125.0f));
    const uint64_t t = f2::add(x, f2::pk(12582912.0f, 12582912.0f));         // 1.5 * 2^23: n sits in the low mantissa bits
    const uint64_t n = f2::add(t, f2::pk(-12582912.0f, -12582912.0f));
    const uint64_t f = f2::fma(n, f2::pk(-1.0f, -1.0f), x);                   // exact
    uint64_t p = f2::fma(f2::pk(0.009570100344717503f, 0.009570100344717503f), f, f2::pk(0.05591785907745361f, 0.05591785907745361f));
    p = f2::fma(p, f, f2::pk(0.240247443318367f, 0.240247443318367f));
    p = f2::fma(p, f, f2::pk(0.6931217908859253f, 0.6931217908859253f));
    p = f2::fma(p, f, f2::pk(0.9999992847442627f, 0.9999992847442627f));
    uint32_t p0, p1, t0, t1;
    f2::unpk(p, p0, p1);
    f2::unpk(t, t0, t1);
    return f2::pk(p0 + (t0 << 23), p1 + (t1 << 23));
}

// pair number `pidx` of a 32-column chunk takes the polynomial when every POLY-th pair of exponentials
// is moved off the special-function unit (POLY = 0: none)
template <int POLY>
__device__ __forceinline__ uint64_t ex2_pair(uint64_t x2, int pidx) {
    if (POLY > 0 && pidx % POLY == POLY - 1) return ex2_poly2(x2);
    float x0, x1;
    f2::unpk(x2, x0, x1);
    return f2::pk(t5::ex2(x0), t5::ex2(x1));
}

// Fold 32 raw logits of one query row into its running (max, sum-exp), exp2 domain.  `live` (ragged
// tiles only) is how many of the 32 columns are real blocks.
template <bool RAGGED, int POLY>
__device__ __forceinline__ void rowstat_chunk(const uint32_t (&raw)[32], int live, float scale_log2e, float& run_m, float& run_z) {
    if (RAGGED) {
        // rare (the last tile of a session): scalar, every exponential on the special-function unit so
        // that a switched-off column contributes exactly 0
        float v[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = i >= live ? -INFINITY : __uint_as_float(raw[i]);
        float mx = v[0];
#pragma unroll
        for (int i = 1; i < 32; ++i) mx = fmaxf(mx, v[i]);
        const float mn = fmaxf(run_m, mx * scale_log2e);
        if (!(mn > -INFINITY)) return;
        float sum = 0.0f;
#pragma unroll
        for (int i = 0; i < 32; ++i) sum += t5::ex2(fmaf(v[i], scale_log2e, -mn));
        run_z = run_z * t5::ex2(run_m - mn) + sum;
        run_m = mn;
        return;
    }
    // maximum of the raw logits by a tree of three-input maxima (the scale is positive, so it commutes with max)
    float m[11];
#pragma unroll
    for (int i = 0; i < 10; ++i)
        m[i] = f2::max3(__uint_as_float(raw[3 * i]), __uint_as_float(raw[3 * i + 1]), __uint_as_float(raw[3 * i + 2]));
    m[10] = fmaxf(__uint_as_float(raw[30]), __uint_as_float(raw[31]));
    const float mx = f2::max3(f2::max3(f2::max3(m[0], m[1], m[2]), f2::max3(m[3], m[4], m[5]), f2::max3(m[6], m[7], m[8])), m[9], m[10]);
    const float mn = fmaxf(run_m, mx * scale_log2e);
    const uint64_t sc2 = f2::pk(scale_log2e, scale_log2e), nm2 = f2::pk(-mn, -mn);
    uint64_t acc0 = f2::pk(0.0f, 0.0f), acc1 = acc0;
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
        acc0 = f2::add(acc0, ex2_pair<POLY>(f2::fma(f2::pk(raw[i], raw[i + 1]), sc2, nm2), i >> 1));
        acc1 = f2::add(acc1, ex2_pair<POLY>(f2::fma(f2::pk(raw[i + 2], raw[i + 3]), sc2, nm2), (i >> 1) + 1));
    }
    float s0, s1, s2, s3;
    f2::unpk(acc0, s0, s1);
    f2::unpk(acc1, s2, s3);
    run_z = run_z * t5::ex2(run_m - mn) + ((s0 + s1) + (s2 + s3));
    run_m = mn;
}

// ---------------------------------------------------------------------------------------------------
// Pass 1.  Persistent CTAs; work item = (session, layer x KV head, 128-row query panel, run of
// kCkChunkTiles block tiles), run index fastest, a contiguous range of items per CTA: the panel in
// shared memory changes at most a few times per CTA and all SMs carry the same number of tiles to
// within one item.  TMEM lane = query row.
constexpr int kCkChunkTiles = 8;

template <int POLY>
__global__ void __launch_bounds__(kCkThreads, 1)
score_chunk_rowstat_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_idx,
                           ChunkArgs a) {
    pdl_wait();        // everything earlier in the stream is complete and visible from here on
    pdl_trigger();     // the next kernel's CTAs may take their places; they wait in the same way
    extern __shared__ unsigned char smem_dyn[];
    __shared__ uint64_t a_full, a_empty, b_full[kCkStages1], b_empty[kCkStages1], acc_full[kCkAccs], acc_empty[kCkAccs];
    __shared__ uint32_t tmem_base_slot;

    unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    unsigned char* smem_a = base;                              // Q panel: 2 halves x 16 KiB
    unsigned char* smem_b = base + 2 * kCkAHalf;               // index tiles: stages x 2 halves x 32 KiB

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int LG = a.L * a.G;
    const int n_items = a.n_sessions * LG * a.n_panels * a.n_chunks;
    const int item_begin = (int)((long long)n_items * blockIdx.x / gridDim.x);
    const int item_end = (int)((long long)n_items * (blockIdx.x + 1) / gridDim.x);

    if (tid == 0) {
        ptx::mbar_init(&a_full, 1);
        ptx::mbar_init(&a_empty, 1);
        for (int i = 0; i < kCkStages1; ++i) { ptx::mbar_init(&b_full[i], 1); ptx::mbar_init(&b_empty[i], 1); }
        for (int i = 0; i < kCkAccs; ++i) { ptx::mbar_init(&acc_full[i], 1); ptx::mbar_init(&acc_empty[i], kCkEpiWarps); }
        ptx::fence_mbar_init();
    }
    if (warp == 1) {                     // one warp allocates the tensor memory for the whole CTA
        t5::tmem_alloc(&tmem_base_slot, kCkTmemCols);
        t5::tmem_relinquish();
    }
    t5::fence_before();
    __syncthreads();
    t5::fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    // every role walks the same item sequence and skips the same (empty) items; t0..t1 are the item's tiles
    auto item_live = [&](int item, int& s, int& lg, int& panel, int& chunk, int& t0, int& t1, int& NB) {
        chunk = item % a.n_chunks;
        panel = (item / a.n_chunks) % a.n_panels;
        lg = (item / (a.n_chunks * a.n_panels)) % LG;
        s = item / (a.n_chunks * a.n_panels * LG);
        NB = a.nblocks_dev[a.session_first + s];
        const int n_tiles = (NB + kCkBN - 1) / kCkBN;
        t0 = chunk * kCkChunkTiles;
        t1 = min(t0 + kCkChunkTiles, n_tiles);
        return t0 < t1;
    };

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            ptx::prefetch_tensormap(&map_q);
            ptx::prefetch_tensormap(&map_idx);
            int la = 0, tt = 0, cur_panel = -1;
            bool ok = true;
            for (int item = item_begin; ok && item < item_end; ++item) {
                int s, lg, panel, chunk, t0, t1, NB;
                if (!item_live(item, s, lg, panel, chunk, t0, t1, NB)) continue;
                const int l = lg / a.G, g = lg % a.G;
                if (item / a.n_chunks != cur_panel) {
                    // Q panel: rows j = m * r + hr of this KV head; 128 rows = 128 / r tokens x r heads.
                    // The previous panel must have been consumed by every MMA that reads it.
                    cur_panel = item / a.n_chunks;
                    if (la >= 1) ok = ptx::mbar_wait_suspended(&a_empty, (uint32_t)((la - 1) & 1));
                    if (!ok) break;
                    const int m0 = s * a.M + panel * (kCkBM / a.r);
                    ptx::mbar_expect_tx(&a_full, 2 * kCkAHalf);
                    tma_load_4d(smem_a, &map_q, 0, g * a.r, l, m0, &a_full);
                    tma_load_4d(smem_a + kCkAHalf, &map_q, 64, g * a.r, l, m0, &a_full);
                    ++la;
                }
                const int z = ((a.session_first + s) * a.L + l) * a.G + g;
                for (int t = t0; t < t1; ++t, ++tt) {
                    const int st = tt % kCkStages1;
                    if (tt >= kCkStages1) ok = ptx::mbar_wait_suspended(&b_empty[st], (uint32_t)(((tt / kCkStages1) & 1) ^ 1));
                    if (!ok) break;
                    unsigned char* dst = smem_b + (size_t)st * 2 * kCkBHalf;
                    ptx::mbar_expect_tx(&b_full[st], 2 * kCkBHalf);
                    ptx::tma_load_3d(dst, &map_idx, 0, t * kCkBN, z, &b_full[st]);
                    ptx::tma_load_3d(dst + kCkBHalf, &map_idx, 64, t * kCkBN, z, &b_full[st]);
                }
            }
            if (!ok) atomicExch(a.status, (int)KVMEM_E_TIMEOUT);
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t a_lo = t5::desc_lo(ptx::smem_u32(smem_a)), b_lo0 = t5::desc_lo(ptx::smem_u32(smem_b));
            int la = 0, tt = 0, cur_panel = -1;
            bool ok = true;
            for (int item = item_begin; ok && item < item_end; ++item) {
                int s, lg, panel, chunk, t0, t1, NB;
                if (!item_live(item, s, lg, panel, chunk, t0, t1, NB)) continue;
                if (item / a.n_chunks != cur_panel) {
                    cur_panel = item / a.n_chunks;
                    if (la >= 1) t5::commit(&a_empty);     // arrives once every MMA on the old panel is done
                    ok = ptx::mbar_wait_suspended(&a_full, (uint32_t)(la & 1));
                    ++la;
                }
                for (int t = t0; ok && t < t1; ++t, ++tt) {
                    const int st = tt % kCkStages1, acc = tt % kCkAccs;
                    ok = ptx::mbar_wait_suspended(&b_full[st], (uint32_t)((tt / kCkStages1) & 1));
                    if (ok && tt >= kCkAccs) ok = ptx::mbar_wait_suspended(&acc_empty[acc], (uint32_t)(((tt / kCkAccs) & 1) ^ 1));
                    if (!ok) break;
                    t5::fence_after();
                    issue_tile_mma(tmem_base + (uint32_t)acc * kCkBN, a_lo, b_lo0 + (uint32_t)st * (2 * kCkBHalf >> 4));
                    t5::commit(&b_empty[st]);                  // the index tile may be overwritten
                    t5::commit(&acc_full[acc]);                // the accumulator may be read
                }
            }
            if (!ok) atomicExch(a.status, (int)KVMEM_E_TIMEOUT);
        }
    } else {
        // ------------------------------------------------ epilogue: warp -> (TMEM lane quarter, column slice)
        const int quarter = warp & 3;                      // warps 2..17 -> quarters 2,3,0,1,...
        const int half = (warp - 2) >> 2;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(half * kCkHalfCols);
        int tt = 0;
        bool failed = false;
        for (int item = item_begin; !failed && item < item_end; ++item) {
            int s, lg, panel, chunk, t0, t1, NB;
            if (!item_live(item, s, lg, panel, chunk, t0, t1, NB)) continue;
            const int row = panel * kCkBM + quarter * 32 + lane;   // row of this (session, l, g): m * r + hr
            float run_m = -INFINITY, run_z = 0.0f;
            for (int t = t0; t < t1; ++t, ++tt) {
                const int acc = tt % kCkAccs;
                const bool arrived = ptx::mbar_wait_suspended(&acc_full[acc], (uint32_t)((tt / kCkAccs) & 1));
                if (!__all_sync(0xffffffffu, arrived)) {
                    if (lane == 0) atomicExch(a.status, (int)KVMEM_E_TIMEOUT);
                    failed = true;
                    break;
                }
                t5::fence_after();
                const int col0 = t * kCkBN + half * kCkHalfCols;
                const bool ragged = col0 + kCkHalfCols > NB;
#pragma unroll
                for (int c = 0; c < kCkChunks; ++c) {
                    // 32 columns at a time: fewer live registers leave the compiler room to overlap the exponentials
                    uint32_t buf[32];
                    t5::ld32_issue(lane_addr + (uint32_t)(acc * kCkBN + c * 32), buf);
                    t5::ld_wait();
                    if (c == kCkChunks - 1) {           // the whole slice has been read: hand the accumulator back
                        t5::fence_before();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(&acc_empty[acc]);
                    }
                    if (!ragged) rowstat_chunk<false, POLY>(buf, 0, a.scale_log2e, run_m, run_z);
                    else rowstat_chunk<true, POLY>(buf, NB - (col0 + c * 32), a.scale_log2e, run_m, run_z);
                }
            }
            if (!failed && row < a.rows)
                a.rowstat[((((size_t)s * LG + lg) * a.n_chunks + chunk) * kCkSplit + half) * a.rows_pad + row] = make_float2(run_m, run_z);
        }
    }

    t5::fence_before();
    __syncthreads();
    if (warp == 1) {
        t5::fence_after();
        t5::tmem_dealloc(tmem_base, kCkTmemCols);
    }
}

// Between the passes: shift = -(max + log2 Z) of every query row, merging the row statistics of all
// tile runs and column slices; -inf switches a padding row off in pass 2.  A CTA takes 32 consecutive rows: a lane is a
// row (the partials of neighbouring rows are neighbours in memory, so every load of a warp is one coalesced 256 bytes; a
// warp per row read one 32-byte sector per 8-byte pair), the eight warps share out the partials (a long history has
// hundreds per row), eight of a warp's loads are in flight at a time, and the eight partial results are merged in warp
// order: fixed order throughout, so the same bits from run to run.
constexpr int kCkShiftWarps = 8;
__global__ void __launch_bounds__(32 * kCkShiftWarps)
score_chunk_shift_kernel(ChunkArgs a) {
    pdl_wait();
    pdl_trigger();
    __shared__ float2 part[kCkShiftWarps][32];
    const int LG = a.L * a.G;
    const long long total = (long long)a.n_sessions * LG * a.shift_stride;      // shift_stride is a multiple of 32
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long e = (long long)blockIdx.x * 32 + lane;
    if ((long long)blockIdx.x * 32 >= total) return;
    const int j = (int)(e % a.shift_stride);
    const int head = (int)(e / a.shift_stride);
    const int NB = a.nblocks_dev[a.session_first + head / LG];
    const int n_tiles = (NB + kCkBN - 1) / kCkBN;
    const int live_chunks = (n_tiles + kCkChunkTiles - 1) / kCkChunkTiles;
    const bool live = e < total && j < a.rows && live_chunks > 0;
    float mx = -INFINITY, z = 0.0f;
    if (live) {
        const float2* rs = a.rowstat + ((size_t)head * a.n_chunks * kCkSplit) * a.rows_pad + j;
        const int n_part = live_chunks * kCkSplit;
        const int h_begin = (int)((long long)n_part * warp / kCkShiftWarps), h_end = (int)((long long)n_part * (warp + 1) / kCkShiftWarps);
        for (int h0 = h_begin; h0 < h_end; h0 += 8) {
            float2 pp[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) pp[u] = h0 + u < h_end ? rs[(size_t)(h0 + u) * a.rows_pad] : make_float2(-INFINITY, 0.0f);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (pp[u].x > -INFINITY) {
                    const float nm = fmaxf(mx, pp[u].x);
                    z = z * exp2f(mx - nm) + pp[u].y * exp2f(pp[u].x - nm);
                    mx = nm;
                }
            }
        }
    }
    part[warp][lane] = make_float2(mx, z);
    __syncthreads();
    if (warp == 0 && e < total) {
        float m = -INFINITY, zz = 0.0f;
#pragma unroll
        for (int w = 0; w < kCkShiftWarps; ++w) {
            const float2 p = part[w][lane];
            if (p.x > -INFINITY) {
                const float nm = fmaxf(m, p.x);
                zz = zz * exp2f(m - nm) + p.y * exp2f(p.x - nm);
                m = nm;
            }
        }
        a.shift[e] = live ? -(m + log2f(zz)) : -INFINITY;
    }
}

// ---------------------------------------------------------------------------------------------------
// Pass 2.  Persistent CTAs; work item = (session, layer x KV head, 128-block panel).  TMEM lane = block.
// Stationary operand: the panel's Mean-K vectors; streamed operand: the head's query rows, 256 at a time.
constexpr int kCkShiftMax = 4096;                // query rows per (session, l, g) the shift vector can hold
constexpr size_t kCkSmem2 = 2 * 2 * kCkAHalf + (size_t)kCkStages2 * 2 * kCkBHalf + kCkShiftMax * sizeof(float) + 1024;

template <int POLY>
__global__ void __launch_bounds__(kCkThreads, 1)
score_chunk_colsum_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_idx,
                          ChunkArgs a) {
    pdl_wait();        // everything earlier in the stream is complete and visible from here on
    pdl_trigger();     // the next kernel's CTAs may take their places; they wait in the same way
    extern __shared__ unsigned char smem_dyn[];
    __shared__ uint64_t a_full[2], a_empty[2], b_full[kCkStages2], b_empty[kCkStages2], acc_full[kCkAccs], acc_empty[kCkAccs];
    __shared__ uint32_t tmem_base_slot;

    unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    unsigned char* smem_a = base;                                  // index panels: 2 stages x 2 halves x 16 KiB
    unsigned char* smem_b = base + 2 * 2 * kCkAHalf;               // query tiles:  stages x 2 halves x 32 KiB
    float* shift = reinterpret_cast<float*>(smem_b + (size_t)kCkStages2 * 2 * kCkBHalf);  // [n_qtiles * 256]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int LG = a.L * a.G;
    const int n_items = a.n_sessions * LG * a.n_bpanels;           // panel index fastest: neighbours share a head's Q
    // a contiguous range of items per CTA: the head (and with it the shift vector) changes at most a few times
    const int item_begin = (int)((long long)n_items * blockIdx.x / gridDim.x);
    const int item_end = (int)((long long)n_items * (blockIdx.x + 1) / gridDim.x);
    const int n_qtiles = (a.rows + kCkBN - 1) / kCkBN;
    const int tokens_per_qtile = kCkBN / a.r;

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) { ptx::mbar_init(&a_full[i], 1); ptx::mbar_init(&a_empty[i], 1); }
        for (int i = 0; i < kCkAccs; ++i) { ptx::mbar_init(&acc_full[i], 1); ptx::mbar_init(&acc_empty[i], kCkEpiWarps); }
        for (int i = 0; i < kCkStages2; ++i) { ptx::mbar_init(&b_full[i], 1); ptx::mbar_init(&b_empty[i], 1); }
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        t5::tmem_alloc(&tmem_base_slot, kCkTmemCols);
        t5::tmem_relinquish();
    }
    t5::fence_before();
    __syncthreads();
    t5::fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    // every role walks the same item sequence and skips the same (empty) items
    auto item_live = [&](int item, int& s, int& lg, int& bp) {
        bp = item % a.n_bpanels;
        lg = (item / a.n_bpanels) % LG;
        s = item / (a.n_bpanels * LG);
        return bp * kCkBM < a.nblocks_dev[a.session_first + s];
    };

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            ptx::prefetch_tensormap(&map_q);
            ptx::prefetch_tensormap(&map_idx);
            int li = 0, tt = 0;
            bool ok = true;
            for (int item = item_begin; ok && item < item_end; ++item) {
                int s, lg, bp;
                if (!item_live(item, s, lg, bp)) continue;
                const int l = lg / a.G, g = lg % a.G;
                const int as = li & 1;
                if (li >= 2) ok = ptx::mbar_wait_suspended(&a_empty[as], (uint32_t)(((li >> 1) & 1) ^ 1));
                if (!ok) break;
                unsigned char* adst = smem_a + (size_t)as * 2 * kCkAHalf;
                const int z = ((a.session_first + s) * a.L + l) * a.G + g;
                ptx::mbar_expect_tx(&a_full[as], 2 * kCkAHalf);
                ptx::tma_load_3d(adst, &map_idx, 0, bp * kCkBM, z, &a_full[as]);
                ptx::tma_load_3d(adst + kCkAHalf, &map_idx, 64, bp * kCkBM, z, &a_full[as]);
                for (int qt = 0; qt < n_qtiles; ++qt, ++tt) {
                    const int st = tt % kCkStages2;
                    if (tt >= kCkStages2) ok = ptx::mbar_wait_suspended(&b_empty[st], (uint32_t)(((tt / kCkStages2) & 1) ^ 1));
                    if (!ok) break;
                    unsigned char* dst = smem_b + (size_t)st * 2 * kCkBHalf;
                    const int m0 = s * a.M + qt * tokens_per_qtile;
                    ptx::mbar_expect_tx(&b_full[st], 2 * kCkBHalf);
                    tma_load_4d(dst, &map_q, 0, g * a.r, l, m0, &b_full[st]);
                    tma_load_4d(dst + kCkBHalf, &map_q, 64, g * a.r, l, m0, &b_full[st]);
                }
                ++li;
            }
            if (!ok) atomicExch(a.status, (int)KVMEM_E_TIMEOUT);
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            int li = 0, tt = 0;
            bool ok = true;
            for (int item = item_begin; ok && item < item_end; ++item) {
                int s, lg, bp;
                if (!item_live(item, s, lg, bp)) continue;
                const int as = li & 1;
                ok = ptx::mbar_wait_suspended(&a_full[as], (uint32_t)((li >> 1) & 1));
                const uint32_t a_lo = t5::desc_lo(ptx::smem_u32(smem_a + (size_t)as * 2 * kCkAHalf));
                const uint32_t b_lo0 = t5::desc_lo(ptx::smem_u32(smem_b));
                for (int qt = 0; ok && qt < n_qtiles; ++qt, ++tt) {
                    const int st = tt % kCkStages2, acc = tt % kCkAccs;
                    ok = ptx::mbar_wait_suspended(&b_full[st], (uint32_t)((tt / kCkStages2) & 1));
                    if (ok && tt >= kCkAccs) ok = ptx::mbar_wait_suspended(&acc_empty[acc], (uint32_t)(((tt / kCkAccs) & 1) ^ 1));
                    if (!ok) break;
                    t5::fence_after();
                    issue_tile_mma(tmem_base + (uint32_t)acc * kCkBN, a_lo, b_lo0 + (uint32_t)st * (2 * kCkBHalf >> 4));
                    t5::commit(&b_empty[st]);
                    t5::commit(&acc_full[acc]);
                }
                if (ok) t5::commit(&a_empty[as]);          // the index panel may be overwritten
                ++li;
            }
            if (!ok) atomicExch(a.status, (int)KVMEM_E_TIMEOUT);
        }
    } else {
        // ------------------------------------------------ epilogue: warp -> (TMEM lane quarter, column half)
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(half * kCkHalfCols);
        const int et = tid - 64;                           // index among the epilogue threads
        int tt = 0, cur_head = -1;
        bool failed = false;                               // a warp that gave up still meets every named barrier
        for (int item = item_begin; item < item_end; ++item) {
            int s, lg, bp;
            if (!item_live(item, s, lg, bp)) continue;
            if (s * LG + lg != cur_head) {
                // shifts -(max + log2 Z) of this head's query rows (-inf on padding rows)
                cur_head = s * LG + lg;
                asm volatile("bar.sync 1, %0;" ::"n"(32 * kCkEpiWarps) : "memory");
                const float* gs = a.shift + (size_t)cur_head * a.shift_stride;
                for (int j = et; j < n_qtiles * kCkBN; j += 32 * kCkEpiWarps) shift[j] = gs[j];
                asm volatile("bar.sync 1, %0;" ::"n"(32 * kCkEpiWarps) : "memory");
            }
            float total = 0.0f;
            for (int qt = 0; qt < n_qtiles; ++qt, ++tt) {
                if (failed) continue;
                const int acc = tt % kCkAccs;
                const bool arrived = ptx::mbar_wait_suspended(&acc_full[acc], (uint32_t)((tt / kCkAccs) & 1));
                if (!__all_sync(0xffffffffu, arrived)) {
                    if (lane == 0) atomicExch(a.status, (int)KVMEM_E_TIMEOUT);
                    failed = true;
                    continue;
                }
                t5::fence_after();
                const float4* sh4 = reinterpret_cast<const float4*>(shift + qt * kCkBN + half * kCkHalfCols);
                const uint64_t sc2 = f2::pk(a.scale_log2e, a.scale_log2e);
                uint64_t acc0 = f2::pk(0.0f, 0.0f), acc1 = acc0;
#pragma unroll
                for (int c = 0; c < kCkChunks; ++c) {
                    // 32 columns at a time: fewer live registers leave the compiler room to overlap the exponentials
                    uint32_t buf[32];
                    t5::ld32_issue(lane_addr + (uint32_t)(acc * kCkBN + c * 32), buf);
                    t5::ld_wait();
                    if (c == kCkChunks - 1) {           // the whole slice has been read: hand the accumulator back
                        t5::fence_before();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(&acc_empty[acc]);
                    }
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        const float4 sh = sh4[c * 8 + (i >> 2)];            // same address in every lane: broadcast
                        acc0 = f2::add(acc0, ex2_pair<POLY>(f2::fma(f2::pk(buf[i], buf[i + 1]), sc2, f2::pk(sh.x, sh.y)), i >> 1));
                        acc1 = f2::add(acc1, ex2_pair<POLY>(f2::fma(f2::pk(buf[i + 2], buf[i + 3]), sc2, f2::pk(sh.z, sh.w)), (i >> 1) + 1));
                    }
                }
                float s0, s1, s2, s3;
                f2::unpk(acc0, s0, s1);
                f2::unpk(acc1, s2, s3);
                total += (s0 + s1) + (s2 + s3);
            }
            const int b = bp * kCkBM + quarter * 32 + lane;
            if (!failed && b < a.nblocks_dev[a.session_first + s])
                a.headsum[(((size_t)s * LG + lg) * kCkSplit + half) * a.nb_pad + b] = total;
        }
    }

    t5::fence_before();
    __syncthreads();
    if (warp == 1) {
        t5::fence_after();
        t5::tmem_dealloc(tmem_base, kCkTmemCols);
    }
}

// R_b = (1/(L*H)) * sum over (layer, KV head, column half) of the head sums, in a fixed order.
__global__ void __launch_bounds__(256)
score_chunk_finish_kernel(const float* __restrict__ headsum, const int32_t* __restrict__ nblocks_dev, int session_first,
                          int LG, int nb_pad, float inv_LH, float* __restrict__ scores, int scores_stride) {
    pdl_wait();        // everything earlier in the stream is complete and visible from here on
    pdl_trigger();     // the next kernel's CTAs may take their places; they wait in the same way
    const int s = blockIdx.y;
    const int NB = nblocks_dev[session_first + s];
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= NB) return;
    const float* p = headsum + (size_t)s * LG * nb_pad + b;
    float total = 0.0f;
    for (int i = 0; i < LG; ++i) total += p[(size_t)i * nb_pad];
    scores[(size_t)s * scores_stride + b] = total * inv_LH;
}

static PFN_cuTensorMapEncodeTiled_v12000 get_encode_fn() {
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(ptr);
    }
    return fn;
}

ChunkWorkspace plan_chunk_workspace(const kvmem_pool_config_t& c, int n_sessions, int n_q_tokens, char* base) {
    ChunkWorkspace w{};
    const int r = c.n_q_heads / c.n_kv_heads;
    w.rows = n_q_tokens * r;
    w.n_panels = (w.rows + kCkBM - 1) / kCkBM;
    w.rows_pad = w.n_panels * kCkBM;
    w.nb_pad = (c.max_blocks_per_session + 255) / 256 * 256;
    w.n_chunks = std::max(1, (w.nb_pad / kCkBN + kCkChunkTiles - 1) / kCkChunkTiles);
    w.shift_stride = (w.rows + kCkBN - 1) / kCkBN * kCkBN;
    const size_t lg = (size_t)c.n_layers * c.n_kv_heads;
    w.rowstat_bytes = align_up((size_t)n_sessions * lg * w.n_chunks * kCkSplit * w.rows_pad * sizeof(float2), 256);
    w.shift_bytes = align_up((size_t)n_sessions * lg * w.shift_stride * sizeof(float), 256);
    w.colsum_bytes = align_up((size_t)n_sessions * lg * kCkSplit * w.nb_pad * sizeof(float), 256);
    w.scores_bytes = align_up((size_t)n_sessions * c.max_blocks_per_session * sizeof(float), 256);
    w.total = w.rowstat_bytes + w.shift_bytes + w.colsum_bytes + w.scores_bytes;
    if (base) {
        w.rowstat = reinterpret_cast<float2*>(base);
        w.shift = reinterpret_cast<float*>(base + w.rowstat_bytes);
        w.colsum = reinterpret_cast<float*>(base + w.rowstat_bytes + w.shift_bytes);
        w.scores = reinterpret_cast<float*>(base + w.rowstat_bytes + w.shift_bytes + w.colsum_bytes);
    }
    return w;
}

bool chunked_scoring_supported(const kvmem_pool_config_t& c, int n_q_tokens) {
    const int r = c.n_q_heads / c.n_kv_heads;
    return c.head_dim == 128 && r >= 1 && kCkBM % r == 0 && (long long)n_q_tokens * r <= kCkShiftMax;
}

// q [ns*M][L][H][128] as a 4-D tensor; box = 64 dims x r heads x 1 layer x (rows / r) tokens = `rows` rows of 128 B
static bool make_q_map(PFN_cuTensorMapEncodeTiled_v12000 enc, CUtensorMap* map, const __nv_bfloat16* q, const Geometry& g,
                       int n_tokens_total, int rows) {
    cuuint64_t dims[4] = {128, (cuuint64_t)g.H, (cuuint64_t)g.L, (cuuint64_t)n_tokens_total};
    cuuint64_t strides[3] = {256, (cuuint64_t)g.H * 256, (cuuint64_t)g.L * g.H * 256};
    cuuint32_t box[4] = {64, (cuuint32_t)g.r, 1, (cuuint32_t)(rows / g.r)};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<__nv_bfloat16*>(q), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// index [max_sessions * L * G][max_bps][128]; box = 64 dims x `rows` blocks x 1
static bool make_index_map(PFN_cuTensorMapEncodeTiled_v12000 enc, CUtensorMap* map, const kvmem_pool& p, int rows) {
    const Geometry& g = p.geo;
    cuuint64_t dims[3] = {128, (cuuint64_t)g.max_bps, (cuuint64_t)g.max_sessions * g.L * g.G};
    cuuint64_t strides[2] = {256, (cuuint64_t)g.max_bps * 256};
    cuuint32_t box[3] = {64, (cuuint32_t)rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, p.index, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

Option g_chunk_poly{4};   // every n-th exponential of the chunked passes on the FMA pipe; 0: none

cudaError_t launch_score_chunked(const kvmem_pool& p, int session_first, int n_sessions, const __nv_bfloat16* q, int M,
                                 const ChunkWorkspace& ws, float* scores, int scores_stride, float score_scale, cudaStream_t st) {
    const Geometry& g = p.geo;
    PFN_cuTensorMapEncodeTiled_v12000 enc = get_encode_fn();
    if (!enc) return cudaErrorNotSupported;
    int max_nb = 0;
    for (int s = session_first; s < session_first + n_sessions; ++s) max_nb = std::max(max_nb, p.sess_blocks[s]);
    if (max_nb == 0) return cudaSuccess;

    CUtensorMap q_panel, q_tile, idx_tile, idx_panel;      // 128- and 256-row boxes of each operand
    if (!make_q_map(enc, &q_panel, q, g, n_sessions * M, kCkBM) || !make_q_map(enc, &q_tile, q, g, n_sessions * M, kCkBN) ||
        !make_index_map(enc, &idx_tile, p, kCkBN) || !make_index_map(enc, &idx_panel, p, kCkBM))
        return cudaErrorInvalidValue;
    ChunkArgs a{};
    a.nblocks_dev = p.nblocks_dev; a.rowstat = ws.rowstat; a.shift = ws.shift; a.headsum = ws.colsum; a.status = p.status_dev;
    a.session_first = session_first; a.n_sessions = n_sessions; a.M = M; a.L = g.L; a.G = g.G; a.r = g.r;
    a.rows = ws.rows; a.rows_pad = ws.rows_pad; a.nb_pad = ws.nb_pad; a.n_panels = ws.n_panels;
    a.n_bpanels = (max_nb + kCkBM - 1) / kCkBM;
    a.n_chunks = ((max_nb + kCkBN - 1) / kCkBN + kCkChunkTiles - 1) / kCkChunkTiles;
    a.shift_stride = ws.shift_stride;
    a.scale_log2e = 1.4426950408889634f / sqrtf((float)g.d);
    const int LG = g.L * g.G;
    const int n_items1 = n_sessions * LG * a.n_panels * a.n_chunks;
    const int n_items2 = n_sessions * LG * a.n_bpanels;
    const int grid1 = std::min(n_items1, p.sm_count), grid2 = std::min(n_items2, p.sm_count);
    const long long n_shift = (long long)n_sessions * LG * a.shift_stride;
    const int sgrid = (int)((n_shift + 31) / 32);                    // 32 rows per CTA
    cudaError_t e = cudaSuccess;
#define KVMEM_CHUNK_PASSES(POLY)                                                                                              \
    do {                                                                                                                      \
        static PerDeviceOnce attr_done;                                                                                        \
        if (attr_done.pending(p.cfg.device)) {                                                                                                     \
            e = cudaFuncSetAttribute(score_chunk_rowstat_kernel<POLY>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCkSmem); \
            if (e == cudaSuccess)                                                                                             \
                e = cudaFuncSetAttribute(score_chunk_colsum_kernel<POLY>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCkSmem2); \
            if (e != cudaSuccess) return e;                                                                                   \
            attr_done.mark(p.cfg.device);                                                                                                 \
        }                                                                                                                     \
        launch_pdl(score_chunk_rowstat_kernel<POLY>, dim3(grid1), dim3(kCkThreads), kCkSmem, st, q_panel, idx_tile, a);                           \
        e = cudaGetLastError();                                                                                               \
        if (e != cudaSuccess) return e;                                                                                       \
        launch_pdl(score_chunk_shift_kernel, dim3(sgrid), dim3(32 * kCkShiftWarps), 0, st, a);                                                                   \
        e = cudaGetLastError();                                                                                               \
        if (e != cudaSuccess) return e;                                                                                       \
        launch_pdl(score_chunk_colsum_kernel<POLY>, dim3(grid2), dim3(kCkThreads), kCkSmem2, st, q_tile, idx_panel, a);                           \
        e = cudaGetLastError();                                                                                               \
        if (e != cudaSuccess) return e;                                                                                       \
    } while (0)
    switch (g_chunk_poly) {
        case 2: KVMEM_CHUNK_PASSES(2); break;
        case 3: KVMEM_CHUNK_PASSES(3); break;
        case 4: KVMEM_CHUNK_PASSES(4); break;
        case 5: KVMEM_CHUNK_PASSES(5); break;
        default: KVMEM_CHUNK_PASSES(0); break;
    }
#undef KVMEM_CHUNK_PASSES
    dim3 fgrid((unsigned)((max_nb + 255) / 256), (unsigned)n_sessions);
    launch_pdl(score_chunk_finish_kernel, dim3(fgrid), dim3(256), 0, st, ws.colsum, p.nblocks_dev, session_first, kCkSplit * LG, ws.nb_pad,
                                                     score_scale / (float)(g.L * g.H), scores, scores_stride);
    return cudaGetLastError();
}

}  // namespace kvmem
