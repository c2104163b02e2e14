// Causal attention of chunked prefill on the 5th-generation tensor cores (tcgen05 + TMEM), for the
// head shape head_dim 128 with 8 query heads per KV head.
//
// A work item is a block of up to 16 consecutive prompt tokens of one request; a unit is (item, KV
// head).  The 16 tokens x 8 query heads of the KV head are the 128 rows of one MMA tile (row =
// 8 * token + head), so one pass over the keys serves 128 query rows and the diagonal block of the
// causal mask is only 16 tokens wide.  A persistent CTA per SM walks units; per unit
//   warp 8 (one lane)   TMA producer: the Q tile (hi and lo planes, two 64-wide halves of head_dim,
//                       through a 4-D tensor map (d, head, plane, token)), then the K and V page
//                       tiles of 128 cached tokens each through two-stage rings;
//   warp 10 (one lane)  S issuer: S = Q K^T (M 128, N 128, K 128; hi and lo planes of Q accumulate
//                       into the same fp32 tile in TMEM, two S buffers);
//   warp 9 (one lane)   P V issuer: once the softmax warps have written P, O_tile = P V (M 128, N 128,
//                       K 128; hi and lo planes of P), with P read as the A operand from TENSOR MEMORY and
//                       V as an MN-major operand straight from the [token][d] page tile.  (One lane can
//                       issue a tcgen05.mma only every ~108 clk, whatever N <= 128 is: hence tiles as wide
//                       as tensor memory allows and two issuing lanes.)
//   warps 0..7          softmax: two threads share row r (TMEM lane r; warp w reads lanes 32 (w % 4) ..,
//                       warps 0..3 the first half of the columns, warps 4..7 the second): each reads
//                       its 64 scores with tcgen05.ld, masks by the row's causal length, the two
//                       exchange their maxima through shared memory, each writes its part of
//                       P = exp2(s - m) as (hi, lo) bf16 pairs back into tensor memory with tcgen05.st,
//                       over the scores it came from (two tokens per column: hi plane in the first half
//                       of the S buffer's columns, lo plane in the second), and adds its 64 columns of
//                       O_tile into fp32 output registers after rescaling them (the output accumulator
//                       lives in registers, so no TMEM round trip is needed when the running max moves).
//                       Eight warps, two per scheduler, hide each other's instruction latencies; four
//                       ran at half the speed, sixteen were slower again.
// While the softmax warps work on tile j the tensor pipe already computes S of tile j + 1; S of tile
// j + 2 waits for P V of tile j, whose P operand occupies the same columns.
// Tensor memory: S / P buffers at columns 0 and 128, O_tile buffers at 256 and 384.
//
// SHARED mode (decode): the 16 "tokens" of a block are decode rows of DIFFERENT sequences that list the
// same pages for a span of cached tokens (members of a rollout group forked from one prompt).  An
// item is (first cached token, tokens, rows <= 16, 0, token row x 16, partial slot x 16); the query
// tile is assembled from one-token TMA boxes, every row sees the whole span, and each row's (max,
// sum, unnormalised O) goes to its partial slot for the span merge.
// Every wait is bounded: a wait that gives up sets the device status word, all roles stop, the CTA
// frees its TMEM columns and returns.
#include "common.cuh"
#include "kernels.h"

namespace mars {

constexpr int kFaQ = 16;                   // query tokens per block
constexpr int kFaHeads = 8;                // query heads per KV head
constexpr int kFaRows = kFaQ * kFaHeads;   // 128 rows of the MMA tile
constexpr int kFaD = 128;
constexpr int kFaKv = 128;                 // cached tokens per tile.  A tcgen05.mma of M 128, K 16 occupies the tensor pipe for
                                            // ~108 clk whatever N <= 128 is (measured), so the tile is as wide as tensor memory
                                            // allows: half as many S instructions per key as with 64
constexpr int kFaKStages = 2;               // K tiles in flight (free as soon as S is computed)
constexpr int kFaVStages = 2;               // V tiles in flight (free after P V)
constexpr int kFaQTile = kFaRows * 128;    // one (plane, half) tile of Q: 128 rows x 128 B = 16 KB
constexpr int kFaQBytes = 4 * kFaQTile;    // hi/lo x two halves of head_dim
constexpr int kFaHalf = kFaKv * 128;       // one 64-wide half (of head_dim) of a K or V tile: 128 tokens x 128 B = 16 KB
constexpr int kFaTile = 2 * kFaHalf;        // a K or a V tile: two halves
constexpr int kFaSmem = kFaQBytes + (kFaKStages + kFaVStages) * kFaTile;
constexpr int kFaParts = 2;                 // threads per row of the tile (each a quarter of the score / output columns)
constexpr int kFaSoftmaxWarps = 4 * kFaParts;
constexpr int kFaSoftmaxThreads = 32 * kFaSoftmaxWarps;
constexpr int kFaThreads = kFaSoftmaxThreads + 96;   // softmax warps, producer warp, two MMA warps (P V and S)
constexpr int kFaTmemCols = 512;           // S buffers (P over them) at columns 0 and 128, O_tile buffers at 256 and 384
constexpr int kFaOCol = 2 * kFaKv;          // first O_tile column
static_assert(kFaOCol + 2 * kFaD <= kFaTmemCols, "tensor memory layout");
constexpr uint32_t kFaSpin = 1u << 22;

constexpr int kFaShItem = 4 + 2 * kFaQ;   // words of a shared item

struct FaParams {
    const int32_t* step;
    StepLayout lay;
    const int32_t* block_table;
    __nv_bfloat16* o_out;      // [n_tok][2][nq * D]
    float* part_o;             // [slots][nq][D] (shared mode)
    float2* part_ml;           // [slots][nq]
    int32_t* err;
    int max_pages_per_seq, n_pages, page_size, box_rows, nkv, nq, layer;
    float scale_log2;
};

__device__ __forceinline__ void fa_mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void fa_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void fa_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool fa_wait(uint64_t* bar, uint32_t parity) {
    for (uint32_t i = 0; i < kFaSpin; ++i) {
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
__device__ __forceinline__ void fa_tma_2d(void* dst, const CUtensorMap* tm, int x, int y, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(dst)), "l"((uint64_t)tm), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void fa_tma_4d(void* dst, const CUtensorMap* tm, int x, int y, int z, int w, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(smem_u32(dst)), "l"((uint64_t)tm), "r"(x), "r"(y), "r"(z), "r"(w), "r"(smem_u32(bar)) : "memory");
}

// Shared-memory matrix descriptors (descriptor version 1, 128-byte swizzle), see the PTX ISA.
// K-major tile (rows of 128 B, 8-row groups 1024 B apart): Q, K and P.
__device__ __forceinline__ uint64_t fa_desc_kmajor(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3fffu);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// MN-major tile: a row of 128 B holds 64 consecutive N elements (head_dim) of one K index (token);
// 8-token groups are 1024 B apart (stride offset), the next 64 N elements `lbo` bytes further
// (leading offset): the V page tile exactly as TMA writes it.
__device__ __forceinline__ uint64_t fa_desc_mnmajor(uint32_t addr, uint32_t lbo) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3fffu);
    d |= (uint64_t)((lbo >> 4) & 0x3fffu) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptors: fp32 accumulator, bf16 operands; bit 16 = B is MN-major.
constexpr uint32_t kFaIdescS = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kFaKv >> 3) << 17) | ((uint32_t)(kFaRows >> 4) << 24);
constexpr uint32_t kFaIdescO = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(kFaD >> 3) << 17) |
                               ((uint32_t)(kFaRows >> 4) << 24);

__device__ __forceinline__ void fa_mma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void fa_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void fa_ld32(uint32_t taddr, uint32_t (&r)[32]) {
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

// 16 consecutive TMEM columns of this thread's lane (the mirror image of the load above).
__device__ __forceinline__ void fa_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
// D += A B with the A operand in tensor memory: 128 lanes (rows) x 8 columns, two bf16 per column, per K step of 16.
__device__ __forceinline__ void fa_mma_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t db, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %6, %7, %8}, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
        : "memory");
}

__device__ __forceinline__ float fa_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct FaUnit { int row0, start, len, nq_blk, hk, n_tiles; const int32_t* bt; const int32_t* it; };

template <bool SHARED>
__device__ __forceinline__ FaUnit fa_unit(const FaParams& p, int u) {
    FaUnit c;
    const int item = u / p.nkv;
    c.hk = u - item * p.nkv;
    if (SHARED) {
        c.it = p.step + p.lay.sh_items + kFaShItem * item;
        c.start = c.it[0]; c.len = c.it[1]; c.nq_blk = c.it[2]; c.row0 = c.it[4];
    } else {
        const int4 it = reinterpret_cast<const int4*>(p.step + p.lay.items)[p.step[H_PF_FIRST] + item];
        c.it = nullptr;
        c.row0 = it.x; c.start = 0; c.len = it.z; c.nq_blk = it.w;  // len: keys visible to the LAST query of the block
    }
    c.n_tiles = (c.len + kFaKv - 1) / kFaKv;
    c.bt = p.block_table + (size_t)p.step[p.lay.tok_seq + c.row0] * p.max_pages_per_seq;
    return c;
}

template <bool SHARED>
__global__ void __launch_bounds__(kFaThreads, 1)
fattn_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                     const __grid_constant__ CUtensorMap tm_v, FaParams p) {
    extern __shared__ unsigned char fa_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)fa_raw + 1023) & ~(uintptr_t)1023);
    unsigned char* q_smem = smem;                                   // [plane][half][128 rows][128 B]
    unsigned char* k_smem = smem + kFaQBytes;                       // [stage][half][128 tokens][128 B]
    unsigned char* v_smem = k_smem + kFaKStages * kFaTile;          // [stage][half][128 tokens][128 B]
    __shared__ __align__(8) uint64_t q_full, q_free, k_full[kFaKStages], k_empty[kFaKStages], v_full[kFaVStages],
        v_empty[kFaVStages], s_ready[2], p_ready[2], o_ready[2], pv_done[2];
    __shared__ uint32_t tmem_slot;
    __shared__ volatile int dead;
    __shared__ float xmax[2][kFaParts][kFaRows];                     // [tile parity][column part][row]
    __shared__ float xsum[kFaParts][kFaRows];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        fa_mbar_init(&q_full, 1); fa_mbar_init(&q_free, 1);
        for (int i = 0; i < kFaKStages; ++i) { fa_mbar_init(&k_full[i], 1); fa_mbar_init(&k_empty[i], 1); }
        for (int i = 0; i < kFaVStages; ++i) { fa_mbar_init(&v_full[i], 1); fa_mbar_init(&v_empty[i], 1); }
        for (int i = 0; i < 2; ++i) { fa_mbar_init(&s_ready[i], 1); fa_mbar_init(&p_ready[i], kFaSoftmaxWarps); fa_mbar_init(&o_ready[i], 1); fa_mbar_init(&pv_done[i], 1); }
        dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == kFaSoftmaxWarps) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                     "r"(kFaTmemCols));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_slot;
    pdl_wait();

    const int n_units = p.step[SHARED ? H_SH_ITEMS : H_PF_ITEMS] * p.nkv;

    if (warp == kFaSoftmaxWarps) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t g = 0;                                          // tiles requested so far (ring positions)
            int local = 0;
            for (int u = blockIdx.x; u < n_units && !dead; u += gridDim.x, ++local) {
                const FaUnit c = fa_unit<SHARED>(p, u);
                // tile j of this unit: K into its ring, V into its ring (separate lifetimes: K is free once
                // S is computed, V only after P V)
                auto load_tile = [&](int j) -> bool {
                    const int ks = g % kFaKStages, vs = g % kFaVStages;
                    if (!fa_wait(&k_empty[ks], ((g / kFaKStages) & 1) ^ 1)) return false;
                    if (!fa_wait(&v_empty[vs], ((g / kFaVStages) & 1) ^ 1)) return false;
                    unsigned char* kd = k_smem + (size_t)ks * kFaTile;
                    unsigned char* vd = v_smem + (size_t)vs * kFaTile;
                    const int n_valid = min(kFaKv, c.len - j * kFaKv);
                    const int n_boxes = (n_valid + p.box_rows - 1) / p.box_rows;
                    fa_expect_tx(&k_full[ks], (uint32_t)(n_boxes * p.box_rows * 128 * 2));
                    fa_expect_tx(&v_full[vs], (uint32_t)(n_boxes * p.box_rows * 128 * 2));
                    for (int bi = 0; bi < n_boxes; ++bi) {
                        const int tok = c.start + j * kFaKv + bi * p.box_rows;
                        const int page = c.bt[tok / p.page_size];
                        const int y = (((p.layer * p.n_pages + page) * p.nkv + c.hk) * p.page_size) + tok % p.page_size;
                        const int off = bi * p.box_rows * 128;
#pragma unroll
                        for (int hf = 0; hf < 2; ++hf) fa_tma_2d(kd + hf * kFaHalf + off, &tm_k, hf * 64, y, &k_full[ks]);
#pragma unroll
                        for (int hf = 0; hf < 2; ++hf) fa_tma_2d(vd + hf * kFaHalf + off, &tm_v, hf * 64, y, &v_full[vs]);
                    }
                    ++g;
                    return true;
                };
                // the first tiles may be requested while the previous unit still uses the Q tile
                const int early = min(c.n_tiles, kFaKStages);
                bool ok = true;
                for (int j = 0; j < early && ok; ++j) ok = load_tile(j);
                if (ok) ok = fa_wait(&q_free, (local & 1) ^ 1);
                if (ok && SHARED) {
                    // one-token boxes (8 heads x 128 B = 1 KB each): row i of the block is token row it[4 + i]
                    fa_expect_tx(&q_full, (uint32_t)c.nq_blk * 4096u);
                    for (int i = 0; i < c.nq_blk; ++i)
#pragma unroll
                        for (int pl = 0; pl < 2; ++pl)
#pragma unroll
                            for (int hf = 0; hf < 2; ++hf)
                                fa_tma_4d(q_smem + (pl * 2 + hf) * kFaQTile + i * 1024, &tm_q, hf * 64, c.hk * kFaHeads, pl,
                                          c.it[4 + i], &q_full);
                } else if (ok) {
                    fa_expect_tx(&q_full, kFaQBytes);
#pragma unroll
                    for (int pl = 0; pl < 2; ++pl)
#pragma unroll
                        for (int hf = 0; hf < 2; ++hf)
                            fa_tma_4d(q_smem + (pl * 2 + hf) * kFaQTile, &tm_q, hf * 64, c.hk * kFaHeads, pl, c.row0, &q_full);
                }
                for (int j = early; j < c.n_tiles && ok; ++j) ok = load_tile(j);
                if (!ok) { dead = 1; atomicOr(p.err, kErrTimeout); }
            }
        }
    } else if (warp == kFaSoftmaxWarps + 1) {
        // ------------------------------------------------------------------ MMA issuer
        // P V issuer: O_tile(g) = P(g) V(g) as soon as the softmax warps have written P(g) (into tensor memory, over S(g))
        if (lane == 0) {
            uint32_t g = 0;                                          // tiles consumed so far
            for (int u = blockIdx.x; u < n_units && !dead; u += gridDim.x) {
                const FaUnit c = fa_unit<SHARED>(p, u);
                bool ok = true;
                for (int j = 0; j < c.n_tiles && ok; ++j, ++g) {
                    const int vs = g % kFaVStages;
                    ok = fa_wait(&p_ready[g & 1], (g >> 1) & 1) && fa_wait(&v_full[vs], (g / kFaVStages) & 1);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint64_t dv = fa_desc_mnmajor(smem_u32(v_smem + (size_t)vs * kFaTile), kFaHalf);
                    const uint32_t acc = tmem + kFaOCol + (g & 1) * kFaD;
                    const uint32_t pt = tmem + (g & 1) * kFaKv;
#pragma unroll
                    for (int pl = 0; pl < 2; ++pl)
#pragma unroll
                        for (int kk = 0; kk < kFaKv / 16; ++kk)
                            fa_mma_ts(acc, pt + pl * (kFaKv / 2) + kk * 8, dv + 128 * kk, kFaIdescO, (pl | kk) != 0);
                    fa_commit(&o_ready[g & 1]);
                    fa_commit(&v_empty[vs]);
                    fa_commit(&pv_done[g & 1]);                      // P(g) has been consumed: its columns may take S(g + 2)
                }
                if (!ok) { dead = 1; atomicOr(p.err, kErrTimeout); break; }
            }
        }
    } else if (warp == kFaSoftmaxWarps + 2) {
        // S issuer, a lane of its own (one lane issues a tcgen05.mma only every ~108 clk): S(g) = Q K(g)^T into S
        // buffer g & 1 once P V(g - 2), which reads P(g - 2) out of the same columns, has retired.
        if (lane == 0) {
            uint32_t g = 0;
            int local = 0;
            const uint32_t q_addr = smem_u32(q_smem);
            for (int u = blockIdx.x; u < n_units && !dead; u += gridDim.x, ++local) {
                const FaUnit c = fa_unit<SHARED>(p, u);
                bool ok = fa_wait(&q_full, local & 1);
                for (int j = 0; j < c.n_tiles && ok; ++j, ++g) {
                    const int ks = g % kFaKStages;
                    if (g >= 2) ok = fa_wait(&pv_done[g & 1], ((g - 2) >> 1) & 1);
                    if (ok) ok = fa_wait(&k_full[ks], (g / kFaKStages) & 1);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t k_addr = smem_u32(k_smem + (size_t)ks * kFaTile);
                    const uint32_t acc = tmem + (g & 1) * kFaKv;
#pragma unroll
                    for (int pl = 0; pl < 2; ++pl)
#pragma unroll
                        for (int hf = 0; hf < 2; ++hf) {
                            const uint64_t da = fa_desc_kmajor(q_addr + (pl * 2 + hf) * kFaQTile);
                            const uint64_t db = fa_desc_kmajor(k_addr + hf * kFaHalf);
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk) fa_mma(acc, da + 2 * kk, db + 2 * kk, kFaIdescS, (pl | hf | kk) != 0);
                        }
                    fa_commit(&s_ready[g & 1]);
                    fa_commit(&k_empty[ks]);                         // the K tile is free once these MMAs retire
                }
                if (!ok) { dead = 1; atomicOr(p.err, kErrTimeout); break; }
                fa_commit(&q_free);                                  // every MMA that reads this unit's Q has been issued
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax warps
        const int quarter = warp & 3, half = warp >> 2;           // half: which part of the columns (0 .. kFaParts - 1)
        const int r = quarter * 32 + lane;                           // row of the tile = TMEM lane
        const int q_tok = r >> 3, head = r & 7;
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
        constexpr int SC = kFaKv / kFaParts, OC = kFaD / kFaParts;   // score and output columns of this thread
        uint32_t g = 0;
        for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
            const FaUnit c = fa_unit<SHARED>(p, u);
            // keys visible to this row's query; rows past the block's last token are computed but never stored
            const int my_len = SHARED ? c.len : min(c.len, c.len - (c.nq_blk - 1 - q_tok));
            float o[OC];
#pragma unroll
            for (int i = 0; i < OC; ++i) o[i] = 0.f;
            float m_run = -INFINITY, l_run = 0.f;                    // l_run: sum over this thread's columns only
            float alpha_prev = 0.f;                                  // rescale factor of the tile whose O_tile is still to be added
            // adds O_tile of tile gt (its P V has been issued) into the output registers
            auto accumulate = [&](uint32_t gt, float alpha) {
                if (lane == 0 && !dead && !fa_wait(&o_ready[gt & 1], (gt >> 1) & 1)) { dead = 1; atomicOr(p.err, kErrTimeout); }
                __syncwarp();
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                for (int cb = 0; cb < OC; cb += 32) {
                    uint32_t v[32];
                    fa_ld32(lane_base + kFaOCol + (gt & 1) * kFaD + half * OC + cb, v);
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[cb + i] = fmaf(o[cb + i], alpha, __uint_as_float(v[i]));
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            };
            // No early exit from these loops: the eight warps meet at a named barrier in every tile, so a
            // warp must never leave while others still go there.  After a wait has given up (`dead`),
            // the remaining iterations run without waiting (their results are garbage and the status
            // word says so).
            for (int j = 0; j < c.n_tiles; ++j, ++g) {
                if (lane == 0 && !dead && !fa_wait(&s_ready[g & 1], (g >> 1) & 1)) { dead = 1; atomicOr(p.err, kErrTimeout); }
                __syncwarp();
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                // this thread's 64 scores of the row
                const int kv0 = j * kFaKv + half * SC;
                float sv[SC];
                float mx = -INFINITY;
#pragma unroll
                for (int cb = 0; cb < SC; cb += 32) {
                    uint32_t v[32];
                    fa_ld32(lane_base + (g & 1) * kFaKv + half * SC + cb, v);
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        sv[cb + i] = kv0 + cb + i < my_len ? __uint_as_float(v[i]) * p.scale_log2 : -INFINITY;
                        mx = fmaxf(mx, sv[cb + i]);
                    }
                }
                xmax[g & 1][half][r] = mx;
                asm volatile("bar.sync 1, %0;" ::"n"(kFaSoftmaxThreads) : "memory");
                float mo = mx;
#pragma unroll
                for (int q = 0; q < kFaParts; ++q) mo = fmaxf(mo, xmax[g & 1][q][r]);
                const float m_new = fmaxf(m_run, mo);
                const float m_use = m_new == -INFINITY ? 0.f : m_new;
                const float alpha = fa_exp2(m_run - m_use);
                float sum = 0.f;
                // P as (hi, lo) bf16 planes goes back into tensor memory, over this tile's scores (every thread of
                // the row has read them: the barrier above): the A operand of P V is row = lane, two tokens per
                // column, so this thread's 64 tokens are 32 columns of the hi plane (first half of the S buffer's
                // columns) and 32 of the lo plane (second half).  No shared-memory round trip, no proxy fence.
#pragma unroll
                for (int cb = 0; cb < SC; cb += 32) {
                    uint32_t hi[16], lo[16];
#pragma unroll
                    for (int q = 0; q < 16; ++q) {
                        const float a = fa_exp2(sv[cb + 2 * q] - m_use), b2 = fa_exp2(sv[cb + 2 * q + 1] - m_use);
                        sum += a + b2;
                        hi[q] = pack_bf16(a, b2);
                        lo[q] = pack_bf16(a - bf16_lo(hi[q]), b2 - bf16_hi(hi[q]));
                    }
                    const uint32_t pt = lane_base + (g & 1) * kFaKv + (half * SC + cb) / 2;
                    fa_st16(pt, hi);
                    fa_st16(pt + kFaKv / 2, lo);
                }
                l_run = l_run * alpha + sum;
                m_run = m_new;
                // the last tile may reach past the request's tokens: those value rows hold whatever the page
                // holds, and 0 * NaN is NaN, so they are cleared (whole rows: the swizzle permutes within a row)
                const int n_valid = min(kFaKv, c.len - j * kFaKv);
                if (n_valid < kFaKv) {
                    const int vs = g % kFaVStages;
                    if (lane == 0 && !dead && !fa_wait(&v_full[vs], (g / kFaVStages) & 1)) { dead = 1; atomicOr(p.err, kErrTimeout); }
                    __syncwarp();
                    unsigned char* vt = v_smem + (size_t)vs * kFaTile;
                    for (int i = tid; i < (kFaKv - n_valid) * 16; i += kFaSoftmaxThreads) {
                        const int row = n_valid + (i >> 4), piece = i & 15;
                        *reinterpret_cast<uint4*>(vt + (piece >> 3) * kFaHalf + row * 128 + (piece & 7) * 16) = make_uint4(0, 0, 0, 0);
                    }
                }
                // P must have landed in tensor memory, and cleared value rows must be visible to the tensor core's
                // reads: hand over to the MMA lane
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                if (n_valid < kFaKv) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) fa_arrive(&p_ready[g & 1]);
                // while P V of this tile runs, add the previous tile's O_tile
                if (j > 0) accumulate(g - 1, alpha_prev);
                alpha_prev = alpha;
            }
            accumulate(g - 1, alpha_prev);
            // the row's sum: both threads of the row saw the same sequence of maxima, so their sums add
            xsum[half][r] = l_run;
            asm volatile("bar.sync 1, %0;" ::"n"(kFaSoftmaxThreads) : "memory");
            float l_row = 0.f;                                       // the same order in every thread of the row
#pragma unroll
            for (int q = 0; q < kFaParts; ++q) l_row += xsum[q][r];
            if (SHARED) {
                if (q_tok < c.nq_blk) {
                    const size_t ph = (size_t)c.it[4 + kFaQ + q_tok] * p.nq + c.hk * kFaHeads + head;
                    float* dst = p.part_o + ph * kFaD + half * OC;
#pragma unroll
                    for (int i = 0; i < OC; i += 4) *reinterpret_cast<float4*>(dst + i) = make_float4(o[i], o[i + 1], o[i + 2], o[i + 3]);
                    if (half == 0) p.part_ml[ph] = make_float2(m_run, l_row);
                }
            } else if (q_tok < c.nq_blk) {
                const float inv = 1.f / l_row;
                __nv_bfloat16* dst = p.o_out + (size_t)(c.row0 + q_tok) * 2 * p.nq * kFaD + (size_t)(c.hk * kFaHeads + head) * kFaD +
                                     half * OC;
#pragma unroll
                for (int i = 0; i < OC; i += 8) {
                    uint32_t hi[4], lo[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float a = o[i + 2 * q] * inv, b2 = o[i + 2 * q + 1] * inv;
                        hi[q] = pack_bf16(a, b2);
                        lo[q] = pack_bf16(a - bf16_lo(hi[q]), b2 - bf16_hi(hi[q]));
                    }
                    *reinterpret_cast<uint4*>(dst + i) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                    *reinterpret_cast<uint4*>(dst + (size_t)p.nq * kFaD + i) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                }
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    __syncthreads();
    if (warp == kFaSoftmaxWarps) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kFaTmemCols));
    }
}

bool fattn_supported(const Shape& s) { return s.D == kFaD && s.nq / s.nkv == kFaHeads; }
int fattn_block_tokens() { return kFaQ; }

static FaParams fa_params(const Shape& s, const Buffers& b, const StepLayout& lay, const KvView& kv, int layer) {
    FaParams p;
    p.step = b.step; p.lay = lay; p.block_table = kv.block_table; p.o_out = b.o; p.part_o = b.part_o; p.part_ml = b.part_ml;
    p.err = b.err;
    p.max_pages_per_seq = kv.max_pages_per_seq; p.n_pages = kv.n_pages; p.page_size = kv.page_size;
    p.box_rows = kv.page_size < 64 ? kv.page_size : 64;   // rows of a box of the cache pools' tensor maps
    p.nkv = s.nkv; p.nq = s.nq; p.layer = layer;
    p.scale_log2 = (float)(1.4426950408889634 / sqrt((double)s.D));
    return p;
}

int launch_fattn_prefill(const Shape& s, const Buffers& b, const StepLayout& lay, const KvView& kv, const CUtensorMap& tm_q,
                         const CUtensorMap& tm_k, const CUtensorMap& tm_v, int layer, int n_items, int sm_count,
                         cudaStream_t st) {
    const FaParams p = fa_params(s, b, lay, kv, layer);
    int grid = n_items * s.nkv;
    if (grid > sm_count) grid = sm_count;
    if (grid < 1) grid = 1;
    launch_chained(fattn_kernel<false>, dim3(grid), dim3(kFaThreads), (size_t)kFaSmem + 1024, st, tm_q, tm_k, tm_v, p);
    return 1;
}

// Shared spans of decode rows: tm_q1 is the query map with one-token boxes.
int fattn_shared_rows() { return kFaQ; }
int fattn_shared_item_words() { return kFaShItem; }
int launch_fattn_shared(const Shape& s, const Buffers& b, const StepLayout& lay, const KvView& kv, const CUtensorMap& tm_q1,
                        const CUtensorMap& tm_k, const CUtensorMap& tm_v, int layer, int n_items, int sm_count,
                        cudaStream_t st) {
    const FaParams p = fa_params(s, b, lay, kv, layer);
    int grid = n_items * s.nkv;
    if (grid > sm_count) grid = sm_count;
    if (grid < 1) grid = 1;
    launch_chained(fattn_kernel<true>, dim3(grid), dim3(kFaThreads), (size_t)kFaSmem + 1024, st, tm_q1, tm_k, tm_v, p);
    return 1;
}

cudaError_t init_fattn_kernels() {
    cudaError_t e = cudaFuncSetAttribute(fattn_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFaSmem + 1024);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(fattn_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFaSmem + 1024);
}

}  // namespace mars
