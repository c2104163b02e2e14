// Dense contractions of chunked prefill on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// C[m, n] = sum_k X[m, k] W[n, k] for hundreds to thousands of token rows m: a real dense
// contraction, unlike the decode-sized streams.  A persistent CTA per SM walks 128 x 256 output tiles:
//   warp 0 (one lane)  TMA producer: per 64-wide K stage the hi plane and the lo plane of 128
//                      activation rows and four 64-row boxes of weights, 128-byte swizzle, into a
//                      3-stage ring (mbarrier full/empty pairs) that runs on across tile boundaries;
//   warp 1 (one lane)  issues tcgen05.mma (M 128, N 256, K 16, bf16 x bf16 -> fp32 in TMEM): per
//                      stage four K steps for the hi plane and four for the lo plane, all into the
//                      same accumulator, then tcgen05.commit to release the stage; tiles alternate
//                      between two accumulators (2 x 256 TMEM columns);
//   warps 2..5         epilogue: wait for an accumulator, tcgen05.ld (each warp its 32-lane
//                      quarter of TMEM), then either store fp32 rows or apply SwiGLU to the
//                      (gate, up) column halves and store (hi, lo) bf16 pairs, and hand the
//                      accumulator back -- all while the next tile's MMAs run.
// Activations are (hi, lo) bf16 pairs stored [row][2][K]; a 3-D tensor map (K, plane, row) picks a
// plane of 128 rows as one box.  For the experts the rows are expert slots (tokens gathered in
// expert order) and a tile is one entry of the permute kernel's group list.
// Every wait is bounded: a wait that gives up sets the device status word, the CTA stops issuing,
// frees its TMEM columns and returns.
#include "common.cuh"
#include "kernels.h"

namespace mars {

static int g_umma_sms = 0;     // SMs of the device (set by init_umma_kernels)

constexpr int kUmStages = 3;
constexpr int kUmTileM = 128, kUmTileN = 256, kUmStageK = 64;
constexpr int kUmTileBytes = kUmTileM * kUmStageK * 2;              // 16 KB: 128 rows x 128 B
constexpr int kUmBBytes = kUmTileN * kUmStageK * 2;                 // 32 KB: 256 weight rows x 128 B
constexpr int kUmStageBytes = 2 * kUmTileBytes + kUmBBytes;         // A hi, A lo, B
constexpr int kUmThreads = 192;
constexpr uint32_t kUmSpin = 1u << 22;

__device__ __forceinline__ void um_mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void um_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Bounded wait on an mbarrier phase: at most `limit` polls, then false (the caller sets the status
// word, stops issuing, frees its tensor memory and returns).
__device__ __forceinline__ bool um_wait_n(uint64_t* bar, uint32_t parity, uint32_t limit) {
    for (uint32_t i = 0; i < limit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ bool um_wait(uint64_t* bar, uint32_t parity) { return um_wait_n(bar, parity, kUmSpin); }
__device__ __forceinline__ void um_tma_2d(void* dst, const CUtensorMap* tm, int x, int y, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(dst)), "l"((uint64_t)tm), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void um_tma_3d(void* dst, const CUtensorMap* tm, int x, int y, int z, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(smem_u32(dst)), "l"((uint64_t)tm), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar)) : "memory");
}

// Shared-memory matrix descriptor of a K-major tile written by TMA with the 128-byte swizzle:
// rows of 128 bytes, groups of 8 rows 1024 bytes apart (stride byte offset), descriptor version 1,
// layout type 2 (128-byte swizzle); the leading byte offset is unused for swizzled K-major tiles.
__device__ __forceinline__ uint64_t um_smem_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3fffu);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, N = 256, M = 128.
constexpr uint32_t kUmIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kUmTileN >> 3) << 17) |
                              ((uint32_t)(kUmTileM >> 4) << 24);

__device__ __forceinline__ void um_mma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(kUmIdesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void um_mma_idesc(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void um_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void um_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

struct UmmaParams {
    int K;                    // contraction length, multiple of 64
    int m_rows;               // rows of A (tokens or slots)
    const int32_t* groups;    // null: tile y covers rows 128 y ..; else tile y = group y (expert, first slot, rows, 0)
    const int32_t* n_groups;
    int b_rows_per_expert;    // rows of B per expert (grouped calls)
    int n_cols;               // output columns (store mode) or expert_inter (SwiGLU mode)
    int swiglu;               // 0: out[m][n_cols] fp32; 1: act[m][2][n_cols] from (gate, up) column halves;
                              // 2: per-row softmax statistics of the tile's columns (scoring pass, see below);
                              // 3: QKV projection with norm, RoPE and the cache append in the epilogue
    float* out;               // mode 2: optional copy of the raw logits [m][n_cols], or null
    __nv_bfloat16* act;
    int32_t* err;
    // mode 2: the columns are vocabulary entries; z = logit * inv_temp.  Column tile x writes, for each of
    // its rows, (max z, sum exp(z - max)) to score_ml[x * m_rows + row]; the tile that holds column
    // targets[row] also writes that z to score_tgt[row].
    const int32_t* targets;
    float inv_temp;
    float2* score_ml;
    float* score_tgt;
    int tiles_x;              // column tiles per row tile (mode 1: 128 output columns each, else 256)
    int use_lo;               // 1: accumulate the lo plane of the activations as well (hi + lo = ~16 mantissa bits)
    QkvEpilogue qkv;          // mode 3: the tile's columns are whole heads of the QKV projection (kernels.h)
    int out_lo;               // mode 1: 1 = write the lo plane of the activations too (the consumer reads it)
};

template <int D>
__device__ __forceinline__ void qkv_head_epilogue(const QkvEpilogue& e, uint32_t taddr, int head, int t) {
    constexpr int HALF = D / 2;
    float v[D];
#pragma unroll
    for (int c = 0; c < D; c += 32) {
        uint32_t raw[32];
        um_ld32(taddr + c, raw);
#pragma unroll
        for (int j = 0; j < 32; ++j) v[c + j] = __uint_as_float(raw[j]);
    }
    if (t < 0) return;                                    // row past the call's tokens: the loads above are warp-wide
    const bool is_q = head < e.nq, is_k = !is_q && head < e.nq + e.nkv;
    const int pos = e.tok_pos[t];
    __nv_bfloat16* cache_row = nullptr;
    if (!is_q) {
        const int page = e.block_table[(size_t)e.tok_seq[t] * e.max_pages_per_seq + pos / e.page_size];
        const int hk = is_k ? head - e.nq : head - e.nq - e.nkv;
        cache_row = (is_k ? e.k_pool : e.v_pool) +
                    ((((size_t)e.layer * e.n_pages + page) * e.nkv + hk) * e.page_size + pos % e.page_size) * D;
    }
    if (is_q || is_k) {
        if (e.qk_norm) {
            float ss = 0.f;
#pragma unroll
            for (int i = 0; i < D; ++i) ss += v[i] * v[i];
            const float r = rsqrtf(ss / (float)D + e.eps);
            const __nv_bfloat16* g = is_q ? e.q_gain : e.k_gain;
#pragma unroll
            for (int i = 0; i < D; i += 8) {
                const uint4 gv = *reinterpret_cast<const uint4*>(g + i);
                const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w};
#pragma unroll
                for (int q = 0; q < 4; ++q) { v[i + 2 * q] *= r * bf16_lo(gw[q]); v[i + 2 * q + 1] *= r * bf16_hi(gw[q]); }
            }
        }
        const float2* cs = e.rope + (size_t)t * HALF;
#pragma unroll
        for (int i = 0; i < HALF; i += 2) {
            const float4 c2 = *reinterpret_cast<const float4*>(cs + i);      // (cos, sin) of i and i + 1
            const float a0 = v[i] * c2.x - v[i + HALF] * c2.y, b0 = v[i + HALF] * c2.x + v[i] * c2.y;
            const float a1 = v[i + 1] * c2.z - v[i + 1 + HALF] * c2.w, b1 = v[i + 1 + HALF] * c2.z + v[i + 1] * c2.w;
            v[i] = a0; v[i + HALF] = b0; v[i + 1] = a1; v[i + 1 + HALF] = b1;
        }
    }
    if (is_q) {
        __nv_bfloat16* dq = e.q_out + (size_t)t * 2 * e.nq * D + (size_t)head * D;
#pragma unroll
        for (int i = 0; i < D; i += 8) {
            uint32_t hi[4], lo[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                hi[q] = pack_bf16(v[i + 2 * q], v[i + 2 * q + 1]);
                lo[q] = pack_bf16(v[i + 2 * q] - bf16_lo(hi[q]), v[i + 2 * q + 1] - bf16_hi(hi[q]));
            }
            *reinterpret_cast<uint4*>(dq + i) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            *reinterpret_cast<uint4*>(dq + (size_t)e.nq * D + i) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
    } else {
#pragma unroll
        for (int i = 0; i < D; i += 8)
            *reinterpret_cast<uint4*>(cache_row + i) = make_uint4(pack_bf16(v[i], v[i + 1]), pack_bf16(v[i + 2], v[i + 3]),
                                                                  pack_bf16(v[i + 4], v[i + 5]), pack_bf16(v[i + 6], v[i + 7]));
    }
}

// The kernel is persistent: CTA c computes tiles c, c + gridDim.x, ... (column tile fastest, so that
// CTAs running side by side share the row tile's activations and, for grouped calls, an expert's
// weights through the L2).  Tensor memory holds TWO accumulators (2 x 256 columns): while the four
// epilogue warps drain tile t, the MMA lane already accumulates tile t + 1, and the TMA producer runs
// ahead through the ring across tile boundaries, so the tensor pipe only idles at the very start.
struct UmTile { int m0, m_valid, b_row0, b_row1, col0, x; };

__device__ __forceinline__ UmTile um_tile(const UmmaParams& p, int tile) {
    UmTile t;
    const int y = tile / p.tiles_x;
    t.x = tile - y * p.tiles_x;
    if (p.groups) {
        const int4 g = reinterpret_cast<const int4*>(p.groups)[y];
        t.m0 = g.y; t.m_valid = g.z;
        const int base = g.x * p.b_rows_per_expert;
        if (p.swiglu) { t.col0 = t.x * 128; t.b_row0 = base + t.col0; t.b_row1 = base + p.n_cols + t.col0; }
        else { t.col0 = t.x * kUmTileN; t.b_row0 = base + t.col0; t.b_row1 = t.b_row0 + 128; }
    } else {
        t.m0 = y * kUmTileM; t.m_valid = min(kUmTileM, p.m_rows - t.m0);
        t.col0 = t.x * kUmTileN; t.b_row0 = t.col0; t.b_row1 = t.col0 + 128;
    }
    return t;
}

__device__ __forceinline__ void um_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__global__ void __launch_bounds__(kUmThreads, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b, UmmaParams p) {
    extern __shared__ unsigned char um_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)um_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t full_bar[kUmStages], empty_bar[kUmStages], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ volatile int dead;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int i = 0; i < kUmStages; ++i) { um_mbar_init(&full_bar[i], 1); um_mbar_init(&empty_bar[i], 1); }
        for (int i = 0; i < 2; ++i) { um_mbar_init(&acc_full[i], 1); um_mbar_init(&acc_empty[i], 4); }
        dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 2) {   // one warp allocates the TMEM columns: two fp32 accumulators of 128 lanes x 256 columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                     "r"(2 * kUmTileN));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = tmem_slot;
    pdl_wait();      // the group list and the activations come from earlier kernels

    const int nk = p.K / kUmStageK;
    const int n_y = p.groups ? *p.n_groups : (p.m_rows + kUmTileM - 1) / kUmTileM;
    const int n_tiles = n_y * p.tiles_x;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;                                         // ring stages produced so far
            for (int tile = blockIdx.x; tile < n_tiles && !dead; tile += gridDim.x) {
                const UmTile t = um_tile(p, tile);
                for (int ks = 0; ks < nk && !dead; ++ks, ++it) {
                    const int s = it % kUmStages;
                    if (!um_wait(&empty_bar[s], ((it / kUmStages) & 1) ^ 1)) {   // passes at once in the first round
                        dead = 1; atomicOr(p.err, kErrTimeout); break;
                    }
                    unsigned char* st = smem + (size_t)s * kUmStageBytes;
                    um_expect_tx(&full_bar[s], p.use_lo ? kUmStageBytes : kUmStageBytes - kUmTileBytes);
                    um_tma_3d(st, &tm_a, ks * kUmStageK, 0, t.m0, &full_bar[s]);
                    if (p.use_lo) um_tma_3d(st + kUmTileBytes, &tm_a, ks * kUmStageK, 1, t.m0, &full_bar[s]);
                    unsigned char* sb = st + 2 * kUmTileBytes;        // four boxes of 64 weight rows (8 KB each)
                    um_tma_2d(sb, &tm_b, ks * kUmStageK, t.b_row0, &full_bar[s]);
                    um_tma_2d(sb + 8192, &tm_b, ks * kUmStageK, t.b_row0 + 64, &full_bar[s]);
                    um_tma_2d(sb + 16384, &tm_b, ks * kUmStageK, t.b_row1, &full_bar[s]);
                    um_tma_2d(sb + 24576, &tm_b, ks * kUmStageK, t.b_row1 + 64, &full_bar[s]);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            uint32_t it = 0;
            int local = 0;                                           // tiles of this CTA so far
            for (int tile = blockIdx.x; tile < n_tiles && !dead; tile += gridDim.x, ++local) {
                const int buf = local & 1;
                // the epilogue must have drained this accumulator (two tiles ago)
                if (!um_wait(&acc_empty[buf], ((local >> 1) & 1) ^ 1)) { dead = 1; atomicOr(p.err, kErrTimeout); break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t acc = tmem_d + (uint32_t)(buf * kUmTileN);
                for (int ks = 0; ks < nk && !dead; ++ks, ++it) {
                    const int s = it % kUmStages;
                    if (!um_wait(&full_bar[s], (it / kUmStages) & 1)) { dead = 1; atomicOr(p.err, kErrTimeout); break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_hi = smem_u32(smem + (size_t)s * kUmStageBytes);
                    const uint64_t d_hi = um_smem_desc(a_hi), d_lo = um_smem_desc(a_hi + kUmTileBytes),
                                   d_b = um_smem_desc(a_hi + 2 * kUmTileBytes);
#pragma unroll
                    for (int kk = 0; kk < kUmStageK / 16; ++kk) {   // 32 bytes along K per step: +2 in the address field
                        um_mma(acc, d_hi + 2 * kk, d_b + 2 * kk, (ks | kk) != 0);
                        if (p.use_lo) um_mma(acc, d_lo + 2 * kk, d_b + 2 * kk, 1u);
                    }
                    um_commit(&empty_bar[s]);                        // the stage is free once these MMAs retire
                }
                um_commit(&acc_full[buf]);
            }
        }
    } else {
        // epilogue: a warp may touch the TMEM lanes 32 (warp % 4) .. +31
        const int quarter = warp & 3;
        const int r = quarter * 32 + lane;                           // row of the tile = TMEM lane
        int local = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++local) {
            const int buf = local & 1;
            const UmTile t = um_tile(p, tile);
            const int m0 = t.m0, m_valid = t.m_valid, col0 = t.col0;
            if (lane == 0 && !dead && !um_wait(&acc_full[buf], (local >> 1) & 1)) { dead = 1; atomicOr(p.err, kErrTimeout); }
            __syncwarp();
            if (!__all_sync(0xffffffffu, !dead)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t lane_base = tmem_d + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * kUmTileN);
            if (!p.swiglu) {
#pragma unroll 1
                for (int c = 0; c < kUmTileN; c += 32) {
                    uint32_t v[32];
                    um_ld32(lane_base + c, v);
                    if (r < m_valid) {
                        float* dst = p.out + (size_t)(m0 + r) * p.n_cols + col0 + c;
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            if (col0 + c + j < p.n_cols)
                                *reinterpret_cast<float4*>(dst + j) =
                                    make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]),
                                                __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                    }
                }
            } else if (p.swiglu == 3) {
                const QkvEpilogue& e = p.qkv;
                const int t = r < m_valid ? m0 + r : -1;
                const int n_heads = e.nq + 2 * e.nkv;
                if (e.head_dim == 128) {
#pragma unroll 1
                    for (int hh = 0; hh < kUmTileN / 128; ++hh)
                        if (col0 / 128 + hh < n_heads) qkv_head_epilogue<128>(e, lane_base + hh * 128, col0 / 128 + hh, t);
                } else {
#pragma unroll 1
                    for (int hh = 0; hh < kUmTileN / 64; ++hh)
                        if (col0 / 64 + hh < n_heads) qkv_head_epilogue<64>(e, lane_base + hh * 64, col0 / 64 + hh, t);
                }
            } else if (p.swiglu == 2) {
                const bool live = r < m_valid;
                const int tgt = live ? p.targets[m0 + r] : -1;
                float mx = -INFINITY, sum = 0.f, zt = 0.f;
#pragma unroll 1
                for (int c = 0; c < kUmTileN; c += 32) {
                    uint32_t v[32];
                    um_ld32(lane_base + c, v);
                    const int cbase = col0 + c;
                    if (live && cbase < p.n_cols) {
                        float cm = -INFINITY;
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (cbase + j < p.n_cols) cm = fmaxf(cm, __uint_as_float(v[j]) * p.inv_temp);
                        const float nm = fmaxf(mx, cm);
                        float add = 0.f;
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (cbase + j < p.n_cols) {
                                const float z = __uint_as_float(v[j]) * p.inv_temp;
                                add += __expf(z - nm);
                                if (cbase + j == tgt) zt = z;
                            }
                        sum = sum * __expf(mx - nm) + add;     // exp(-inf) = 0 on the first chunk
                        mx = nm;
                        if (p.out) {
                            float* dst = p.out + (size_t)(m0 + r) * p.n_cols + cbase;
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (cbase + j < p.n_cols) dst[j] = __uint_as_float(v[j]);
                        }
                    }
                }
                if (live) {
                    p.score_ml[(size_t)t.x * p.m_rows + m0 + r] = make_float2(mx, sum);
                    if (tgt >= col0 && tgt < col0 + kUmTileN && tgt < p.n_cols) p.score_tgt[m0 + r] = zt;
                }
            } else {
#pragma unroll 1
                for (int c = 0; c < 128; c += 32) {
                    uint32_t gt[32], up[32];
                    um_ld32(lane_base + c, gt);
                    um_ld32(lane_base + 128 + c, up);
                    if (r < m_valid) {
                        // expert_inter is a multiple of 64: a run of 8 columns is inside or outside as a whole
                        __nv_bfloat16* dst = p.act + (size_t)(m0 + r) * 2 * p.n_cols + col0 + c;
#pragma unroll
                        for (int j = 0; j < 32; j += 8)
                            if (col0 + c + j < p.n_cols) {
                                uint32_t hi[4], lo[4];
#pragma unroll
                                for (int q = 0; q < 4; ++q) {
                                    float a[2];
#pragma unroll
                                    for (int e = 0; e < 2; ++e) {
                                        const float gte = __uint_as_float(gt[j + 2 * q + e]);
                                        a[e] = gte / (1.f + expf(-gte)) * __uint_as_float(up[j + 2 * q + e]);
                                    }
                                    hi[q] = pack_bf16(a[0], a[1]);
                                    lo[q] = pack_bf16(a[0] - bf16_lo(hi[q]), a[1] - bf16_hi(hi[q]));
                                }
                                *reinterpret_cast<uint4*>(dst + j) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                                if (p.out_lo) *reinterpret_cast<uint4*>(dst + p.n_cols + j) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                            }
                    }
                }
            }
            // this warp has read its lanes of the accumulator: hand it back to the MMA lane
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) um_arrive(&acc_empty[buf]);
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    __syncthreads();
    if (warp == 2) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(2 * kUmTileN));
    }
}

// ---------------------------------------------------------------------------------------------
// Decode-sized dense projections (QKV, output projection, lm_head) on the same tensor cores with the
// operands swapped: 128 WEIGHT rows sit on the TMEM lanes and up to 256 token columns on N, so the
// kernel streams each weight once from HBM (TMA ring; two CTAs per SM at <= 64 tokens) while the hi and
// lo activation planes of the K range are re-read from L2.  With 64 tokens carried as (hi, lo) pairs these projections
// are tensor-bound on the mma.sync path (128 columns per weight row); here they are HBM streams again.
// gridDim.y splits K; every split writes an fp32 partial [split][token][row] that the consumer adds
// in a fixed order.
// NB = 1 .. 4 boxes of 64 token rows per activation plane: 64 .. 256 token columns per pass.
constexpr int kSwABytes = 128 * kUmStageK * 2;                       // 16 KB of weights per stage
constexpr int kSwBoxBytes = 64 * kUmStageK * 2;                      // 8 KB: one box of 64 token rows
template <int NB>
struct SwCfg {
    static constexpr int kTok = 64 * NB;
    static constexpr int kPlaneBytes = NB * kSwBoxBytes;
    static constexpr int kStageBytes = kSwABytes + 2 * kPlaneBytes;
    static constexpr int kStages = NB == 4 ? 2 : 3;                  // 96 / 144 / 192 / 160 KB of ring
    // A tcgen05.mma of M 128, K 16 occupies the tensor pipe for ~108 clk whatever N <= 128 is (160 clk at N = 256;
    // measured), so with up to 128 tokens the hi and the lo plane, which lie next to each other in a stage, are ONE
    // operand of 2 x kTok columns: half as many instructions per stage, and the stream of 16 KB weight stages is no
    // longer held to 8 x 108 clk each.  The two halves of the accumulator are added in the epilogue.
    static constexpr bool kFusePlanes = NB <= 2;
    static constexpr int kAccCols = kFusePlanes ? 2 * kTok : kTok;
    static constexpr int kTmemCols = NB == 3 ? 256 : kAccCols;       // allocations are powers of two
    static constexpr int kCtasPerSm = NB == 1 ? 2 : 1;
    static constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kAccCols >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
    static constexpr size_t smem_bytes() { return (size_t)kStages * kStageBytes + 1024; }
};

struct SwapParams {
    int rows, n_tok, k_per_split;      // weight rows, token columns (<= 64), K range of one split (multiple of 64)
    float* out;                        // [splits][n_tok][rows]
    int32_t* err;
};

template <int NB>
__global__ void __launch_bounds__(kUmThreads, SwCfg<NB>::kCtasPerSm)
umma_swap_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x, SwapParams p) {
    constexpr int kSwStages = SwCfg<NB>::kStages, kSwTok = SwCfg<NB>::kTok, kSwStageBytes = SwCfg<NB>::kStageBytes;
    constexpr int kSwBBytes = SwCfg<NB>::kPlaneBytes;
    constexpr uint32_t kSwIdesc = SwCfg<NB>::kIdesc;
    extern __shared__ unsigned char um_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)um_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t full_bar[kSwStages], empty_bar[kSwStages], accum_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ volatile int dead;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int row0 = blockIdx.x * 128, k0 = blockIdx.y * p.k_per_split;
    const int nk = p.k_per_split / kUmStageK;

    if (tid == 0) {
        for (int i = 0; i < kSwStages; ++i) { um_mbar_init(&full_bar[i], 1); um_mbar_init(&empty_bar[i], 1); }
        um_mbar_init(&accum_bar, 1);
        dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                     "r"(SwCfg<NB>::kTmemCols));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // The weights are constants of the step: the first ring-full of weight tiles is requested
            // before the previous kernel has finished; the activations it produces only after pdl_wait().
            const int pre = nk < kSwStages ? nk : kSwStages;
            for (int ks = 0; ks < pre; ++ks) {
                unsigned char* st = smem + (size_t)ks * kSwStageBytes;
                const int k = k0 + ks * kUmStageK;
                um_expect_tx(&full_bar[ks], kSwStageBytes);
                um_tma_2d(st, &tm_w, k, row0, &full_bar[ks]);
                um_tma_2d(st + 8192, &tm_w, k, row0 + 64, &full_bar[ks]);
            }
            pdl_wait();
            for (int ks = 0; ks < pre; ++ks) {
                unsigned char* st = smem + (size_t)ks * kSwStageBytes;
                const int k = k0 + ks * kUmStageK;
#pragma unroll
                for (int bx = 0; bx < NB; ++bx) {
                    um_tma_3d(st + kSwABytes + bx * kSwBoxBytes, &tm_x, k, 0, 64 * bx, &full_bar[ks]);
                    um_tma_3d(st + kSwABytes + kSwBBytes + bx * kSwBoxBytes, &tm_x, k, 1, 64 * bx, &full_bar[ks]);
                }
            }
            for (int ks = pre; ks < nk && !dead; ++ks) {
                const int s = ks % kSwStages;
                if (!um_wait(&empty_bar[s], ((ks / kSwStages) - 1) & 1)) {
                    dead = 1; atomicOr(p.err, kErrTimeout); break;
                }
                unsigned char* st = smem + (size_t)s * kSwStageBytes;
                const int k = k0 + ks * kUmStageK;
                um_expect_tx(&full_bar[s], kSwStageBytes);
                um_tma_2d(st, &tm_w, k, row0, &full_bar[s]);
                um_tma_2d(st + 8192, &tm_w, k, row0 + 64, &full_bar[s]);
#pragma unroll
                for (int bx = 0; bx < NB; ++bx) {
                    um_tma_3d(st + kSwABytes + bx * kSwBoxBytes, &tm_x, k, 0, 64 * bx, &full_bar[s]);
                    um_tma_3d(st + kSwABytes + kSwBBytes + bx * kSwBoxBytes, &tm_x, k, 1, 64 * bx, &full_bar[s]);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            for (int ks = 0; ks < nk && !dead; ++ks) {
                const int s = ks % kSwStages;
                if (!um_wait(&full_bar[s], (ks / kSwStages) & 1)) { dead = 1; atomicOr(p.err, kErrTimeout); break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a = smem_u32(smem + (size_t)s * kSwStageBytes);
                const uint64_t d_w = um_smem_desc(a), d_hi = um_smem_desc(a + kSwABytes),
                               d_lo = um_smem_desc(a + kSwABytes + kSwBBytes);
#pragma unroll
                for (int kk = 0; kk < kUmStageK / 16; ++kk) {
                    um_mma_idesc(tmem_d, d_w + 2 * kk, d_hi + 2 * kk, kSwIdesc, (ks | kk) != 0);   // fused: hi and lo rows in one operand
                    if (!SwCfg<NB>::kFusePlanes) um_mma_idesc(tmem_d, d_w + 2 * kk, d_lo + 2 * kk, kSwIdesc, 1u);
                }
                um_commit(&empty_bar[s]);
            }
            um_commit(&accum_bar);
        }
    } else {
        const int quarter = warp & 3;
        const int row = row0 + quarter * 32 + lane;                  // weight row = TMEM lane
        if (lane == 0 && !um_wait(&accum_bar, 0)) { dead = 1; atomicOr(p.err, kErrTimeout); }
        __syncwarp();
        const bool ok = __all_sync(0xffffffffu, !dead);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok) {
            const uint32_t lane_base = tmem_d + ((uint32_t)(quarter * 32) << 16);
            float* out = p.out + (size_t)blockIdx.y * p.n_tok * p.rows;
#pragma unroll 1
            for (int c = 0; c < kSwTok && c < p.n_tok; c += 32) {
                uint32_t v[32];
                um_ld32(lane_base + c, v);
                if (SwCfg<NB>::kFusePlanes) {                        // columns kSwTok.. hold the lo plane's share
                    uint32_t w[32];
                    um_ld32(lane_base + kSwTok + c, w);
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(w[j]));
                }
                if (row < p.rows) {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (c + j < p.n_tok) out[(size_t)(c + j) * p.rows + row] = __uint_as_float(v[j]);
                }
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    __syncthreads();
    if (warp == 2) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(SwCfg<NB>::kTmemCols));
    }
}

// out[split][t][row] for t < n_tok <= 256; K = splits * k_per_split.
int launch_umma_swap(const CUtensorMap& tm_w, const CUtensorMap& tm_x, int rows, int n_tok, int K, int splits, float* out,
                     int32_t* err, cudaStream_t st) {
    SwapParams p{rows, n_tok, K / splits, out, err};
    const dim3 grid((rows + 127) / 128, splits);
    if (n_tok <= 64)
        launch_chained(umma_swap_kernel<1>, grid, dim3(kUmThreads), SwCfg<1>::smem_bytes(), st, tm_w, tm_x, p);
    else if (n_tok <= 128)
        launch_chained(umma_swap_kernel<2>, grid, dim3(kUmThreads), SwCfg<2>::smem_bytes(), st, tm_w, tm_x, p);
    else if (n_tok <= 192)
        launch_chained(umma_swap_kernel<3>, grid, dim3(kUmThreads), SwCfg<3>::smem_bytes(), st, tm_w, tm_x, p);
    else
        launch_chained(umma_swap_kernel<4>, grid, dim3(kUmThreads), SwCfg<4>::smem_bytes(), st, tm_w, tm_x, p);
    return 1;
}
int umma_swap_max_tokens() { return 256; }

// Number of K splits of a swap-AB projection: as many as divide the 64-wide K stages evenly (at least 8
// stages each, at most K / 256 splits: the partial buffers are sized for that) while all CTAs still run
// in one wave.
int umma_swap_splits(int rows, int n_tok, int K) {
    const int tiles = (rows + 127) / 128, stages = K / kUmStageK;
    const int slots = g_umma_sms * (n_tok <= 64 ? 2 : 1);
    int best = 1;
    for (int s = 1; s <= K / 256; s *= 2)
        if (stages % s == 0 && stages / s >= 8 && tiles * s <= slots) best = s;
    return best;
}

// Rows of the normalised activations gathered into expert-slot order: xperm[slot] = h[slot_token[slot]]
// (the hi plane, and the lo plane when the contraction uses it), so that a group's rows are one contiguous TMA box.
__global__ void __launch_bounds__(256) gather_rows_kernel(Buffers b, int H, int n_slots, int planes) {
    pdl_wait();
    const int slot = blockIdx.x;
    if (slot >= n_slots) return;
    const uint4* src = reinterpret_cast<const uint4*>(b.h + (size_t)b.slot_token[slot] * 2 * H);
    uint4* dst = reinterpret_cast<uint4*>(b.xperm + (size_t)slot * 2 * H);
    for (int i = threadIdx.x; i < planes * H / 8; i += blockDim.x) dst[i] = src[i];
}

static size_t umma_smem_bytes() { return (size_t)kUmStages * kUmStageBytes + 1024; }

// Persistent grid: one CTA per SM, or fewer when there are fewer tiles.
static int umma_grid(int tiles) { return tiles < g_umma_sms ? (tiles < 1 ? 1 : tiles) : g_umma_sms; }

int launch_umma_dense(const CUtensorMap& tm_a, const CUtensorMap& tm_b, int m_rows, int n_cols, int K, float* out,
                      int32_t* err, int use_lo, cudaStream_t st) {
    const int tx = (n_cols + kUmTileN - 1) / kUmTileN, ty = (m_rows + kUmTileM - 1) / kUmTileM;
    UmmaParams p{K, m_rows, nullptr, nullptr, 0, n_cols, 0, out, nullptr, err, nullptr, 0.f, nullptr, nullptr, tx, use_lo, QkvEpilogue{}};
    launch_chained(umma_gemm_kernel, dim3(umma_grid(tx * ty)), dim3(kUmThreads), umma_smem_bytes(), st, tm_a, tm_b, p);
    return 1;
}

// QKV projection of a prefill-sized call with the per-head norm, RoPE and cache append in its epilogue.
int launch_umma_qkv(const CUtensorMap& tm_a, const CUtensorMap& tm_b, int m_rows, int n_cols, int K, const QkvEpilogue& ep,
                    int32_t* err, int use_lo, cudaStream_t st) {
    const int tx = (n_cols + kUmTileN - 1) / kUmTileN, ty = (m_rows + kUmTileM - 1) / kUmTileM;
    UmmaParams p{K, m_rows, nullptr, nullptr, 0, n_cols, 3, nullptr, nullptr, err, nullptr, 0.f, nullptr, nullptr, tx, use_lo, ep};
    launch_chained(umma_gemm_kernel, dim3(umma_grid(tx * ty)), dim3(kUmThreads), umma_smem_bytes(), st, tm_a, tm_b, p);
    return 1;
}

int launch_umma_experts(const Shape& s, const Buffers& b, const CUtensorMap& tm_xperm, const CUtensorMap& tm_wgu,
                        const CUtensorMap& tm_act, const CUtensorMap& tm_wdown, int n_tok, int gate_up_lo, int down_lo, cudaStream_t st) {
    const int n_slots = n_tok * s.k;
    const int max_groups = s.E + (n_slots + kUmTileM - 1) / kUmTileM;
    launch_chained(gather_rows_kernel, dim3(n_slots), dim3(256), 0, st, b, s.H, n_slots, gate_up_lo ? 2 : 1);
    const int gx = (s.I + 127) / 128, dx = (s.H + kUmTileN - 1) / kUmTileN;
    UmmaParams gu{s.H, n_slots, b.groups, b.n_groups, 2 * s.I, s.I, 1, nullptr, b.act, b.err, nullptr, 0.f, nullptr, nullptr, gx, gate_up_lo, QkvEpilogue{}};
    gu.out_lo = down_lo;
    launch_chained(umma_gemm_kernel, dim3(umma_grid(gx * max_groups)), dim3(kUmThreads), umma_smem_bytes(), st, tm_xperm,
                   tm_wgu, gu);
    UmmaParams dn{s.I, n_slots, b.groups, b.n_groups, s.H, s.H, 0, b.y, nullptr, b.err, nullptr, 0.f, nullptr, nullptr, dx, down_lo, QkvEpilogue{}};
    launch_chained(umma_gemm_kernel, dim3(umma_grid(dx * max_groups)), dim3(kUmThreads), umma_smem_bytes(), st, tm_act,
                   tm_wdown, dn);
    return 3;
}

// ---------------------------------------------------------------------------------------------
// Teacher-forced scoring: log pi(target | prefix) = z_target - logsumexp(z) over the vocabulary, for
// every token row, without materialising the logits.  The contraction above leaves one (max, sum)
// pair per row and 256-column vocabulary tile; a warp per row merges them in a fixed order.
__global__ void __launch_bounds__(256) score_combine_kernel(const float2* __restrict__ ml, const float* __restrict__ zt,
                                                            const int32_t* __restrict__ targets, int n_rows, int n_tiles,
                                                            int vocab, float* __restrict__ out, int32_t* err) {
    pdl_wait();
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= n_rows) return;
    const int tgt = targets[row];
    if (tgt < 0 || tgt >= vocab) {             // negative: no target at this position; too large: reported
        if (lane == 0) {
            out[row] = 0.f;
            if (tgt >= vocab) atomicOr(err, kErrBadToken);
        }
        return;
    }
    float m = -INFINITY, l = 0.f;
    for (int t = lane; t < n_tiles; t += 32) {
        const float2 p = ml[(size_t)t * n_rows + row];
        const float nm = fmaxf(m, p.x);
        l = l * __expf(m - nm) + p.y * __expf(p.x - nm);
        m = nm;
    }
    const float M = warp_max(m);
    l = warp_sum(m == -INFINITY ? 0.f : l * __expf(m - M));
    if (lane == 0) out[row] = zt[row] - (M + logf(l));
}

int launch_umma_score(const CUtensorMap& tm_h, const CUtensorMap& tm_lm, int n_rows, int vocab, int K,
                      const int32_t* targets, float inv_temp, float2* score_ml, float* score_tgt, float* logits_tap,
                      float* out_logprobs, int32_t* err, cudaStream_t st) {
    const int n_tiles = (vocab + kUmTileN - 1) / kUmTileN;
    UmmaParams p{K, n_rows, nullptr, nullptr, 0, vocab, 2, logits_tap, nullptr, err, targets, inv_temp, score_ml, score_tgt,
                 n_tiles, 1, QkvEpilogue{}};
    launch_chained(umma_gemm_kernel, dim3(umma_grid(n_tiles * ((n_rows + kUmTileM - 1) / kUmTileM))), dim3(kUmThreads),
                   umma_smem_bytes(), st, tm_h, tm_lm, p);
    launch_chained(score_combine_kernel, dim3((n_rows + 7) / 8), dim3(256), 0, st, score_ml, score_tgt, targets, n_rows, n_tiles, vocab,
                                                            out_logprobs, err);
    return 2;
}

int score_vocab_tiles(int vocab) { return (vocab + kUmTileN - 1) / kUmTileN; }

// ---------------------------------------------------------------------------------------------
// Self-test of the give-up path that every bounded wait above takes.  One CTA with the same roles as
// the contraction kernels: a warp allocates tensor-memory columns, a consumer lane waits on an
// mbarrier with um_wait_n, a producer lane arrives on it -- or, when `arrive` is 0, does not, so that
// the wait runs out after `limit` polls.  The consumer then sets the timeout bit of the status word,
// the CTA frees its tensor memory and the kernel returns normally; nothing traps, spins on or faults.
__global__ void __launch_bounds__(96) wait_probe_kernel(int32_t* err, int arrive, uint32_t limit) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        um_mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(32));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    pdl_wait();
    if (warp == 1 && lane == 0 && arrive) um_arrive(&bar);
    if (warp == 0 && lane == 0 && !um_wait_n(&bar, 0, limit)) atomicOr(err, kErrTimeout);
    __syncthreads();
    if (warp == 2) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_slot), "r"(32));
    }
}

int launch_wait_probe(int32_t* err, int arrive, uint32_t limit, cudaStream_t st) {
    launch_chained(wait_probe_kernel, dim3(1), dim3(96), 0, st, err, arrive, limit);
    return 1;
}

cudaError_t init_umma_kernels() {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&g_umma_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(umma_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)umma_smem_bytes());
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(umma_swap_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SwCfg<1>::smem_bytes());
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(umma_swap_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SwCfg<2>::smem_bytes());
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(umma_swap_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SwCfg<3>::smem_bytes());
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(umma_swap_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SwCfg<4>::smem_bytes());
}

}  // namespace mars
