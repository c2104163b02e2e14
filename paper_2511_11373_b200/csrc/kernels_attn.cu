// Split-K paged grouped-query attention for decode-shaped queries (one query position per work
// item), and the merge of the per-span partial results.
//
// A work item is (token row, span of cached tokens); a unit is (item, KV head).  A persistent CTA
// walks units; for each it streams the span's K and V page tiles into shared memory with TMA
// (128-byte swizzle, 3-stage ring, one mbarrier per stage), computes S = Q K^T for the g query
// heads of the KV head with the heads on the MMA M axis and 8 tokens per N tile, keeps an online
// softmax per warp (row statistics reduced with warp shuffles), accumulates O = P V from the same
// tiles (ldmatrix.trans), and finally merges its four warps and writes (max, sum, unnormalised O).
#include "common.cuh"
#include "kernels.h"

namespace mars {

constexpr int kAttnWarps = 4;
constexpr int kAttnStages = 3;
constexpr int kStageTok = 64;
constexpr uint32_t kSpinLimit = 1u << 26;

struct AttnParams {
    const __nv_bfloat16* q;  // [n_tok, 2, nq, D]: hi rows, lo rows
    float* part_o;           // [items, nq, D]
    float2* part_ml;         // [items, nq]
    const int32_t* step;
    StepLayout lay;
    const int32_t* block_table;
    int32_t* err;
    int max_pages_per_seq, n_pages, page_size, box_rows, nkv, nq, g, layer;
    float scale_log2;
};

__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls and reports it.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

// One 2-D tile (64 elements x box rows) global -> shared, completion counted on `bar`.
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, int x, int y, uint64_t* bar, uint64_t pol) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(smem_u32(dst)), "l"((uint64_t)tm), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(pol)
        : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

// Byte offset of (token row r, 16-byte piece `piece` of the 128-byte half `half`) inside a tile
// that TMA wrote with the 128-byte swizzle: [half][64 rows][128 B], piece index XOR (row mod 8).
__device__ __forceinline__ uint32_t tile_off(int half, int r, int piece) {
    return (uint32_t)(half * (kStageTok * 128) + r * 128 + ((piece ^ (r & 7)) << 4));
}

template <int D>
__global__ void __launch_bounds__(kAttnWarps * 32, 2)
attn_decode_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, AttnParams p) {
    constexpr int TILE_BYTES = kStageTok * D * 2;
    constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    constexpr int HALVES = D / 64;
    constexpr int KSTEPS = D / 16;
    constexpr int NTILES = D / 8;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t full_bar[kAttnStages];
    __shared__ volatile int dead;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gid = lane >> 2, tig = lane & 3;
    if (tid == 0) {
        for (int i = 0; i < kAttnStages; ++i) mbar_init(&full_bar[i], 1);
        dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    pdl_wait();

    const int32_t* hdr = p.step;
    const int n_units = hdr[H_NITEMS] * p.nkv;
    const int4* items = reinterpret_cast<const int4*>(p.step + p.lay.items);
    const uint64_t pol = l2_evict_first_policy();
    uint32_t gs = 0;  // stages consumed so far by this CTA (ring position and parity)

    // A unit's first ring stages are requested while the previous unit is still in its epilogue
    // (warp merge, partial store, span merge), so the stream into the SM does not pause between units.
    struct Unit { int row, start, len, slot_out, hk, n_st; const int32_t* bt; };
    auto load_unit = [&](int u) {
        Unit c;
        const int item = u / p.nkv;
        c.hk = u - item * p.nkv;
        const int4 it = items[item];
        c.row = it.x; c.start = it.y; c.len = it.z; c.slot_out = it.w;
        c.n_st = (c.len + kStageTok - 1) / kStageTok;
        c.bt = p.block_table + (size_t)p.step[p.lay.tok_seq + c.row] * p.max_pages_per_seq;
        return c;
    };
    auto issue = [&](const Unit& c, int j, uint32_t g_stage) {
        const int slot = g_stage % kAttnStages;
        unsigned char* kdst = smem + (size_t)slot * STAGE_BYTES;
        unsigned char* vdst = kdst + TILE_BYTES;
        const int n_valid = min(kStageTok, c.len - j * kStageTok);
        const int n_boxes = (n_valid + p.box_rows - 1) / p.box_rows;
        mbar_expect_tx(&full_bar[slot], (uint32_t)(n_boxes * p.box_rows * D * 2 * 2));
        for (int bi = 0; bi < n_boxes; ++bi) {
            const int tok = c.start + j * kStageTok + bi * p.box_rows;
            const int page = c.bt[tok / p.page_size];
            const int y = (((p.layer * p.n_pages + page) * p.nkv + c.hk) * p.page_size) + tok % p.page_size;
#pragma unroll
            for (int hf = 0; hf < HALVES; ++hf) {
                const int off = hf * (kStageTok * 128) + bi * p.box_rows * 128;
                tma_load_2d(kdst + off, &tm_k, hf * 64, y, &full_bar[slot], pol);
                tma_load_2d(vdst + off, &tm_v, hf * 64, y, &full_bar[slot], pol);
            }
        }
    };
    auto prefetch = [&](const Unit& c, uint32_t g0) {
        const int pre = min(kAttnStages - 1, c.n_st);
        for (int j = 0; j < pre; ++j) issue(c, j, g0 + j);
    };

    int u = blockIdx.x;
    bool have = u < n_units;
    Unit cur;
    if (have) {
        cur = load_unit(u);
        if (tid == 0) prefetch(cur, gs);
    }
    while (have) {
        const int row = cur.row, len = cur.len, slot_out = cur.slot_out, hk = cur.hk, n_st = cur.n_st;

        // Query fragments.  The group has at most 8 heads, so MMA rows 0..7 carry the hi part of head
        // gid and rows 8..15 its lo part: S = d0 + d2 (d1 + d3) costs no extra tensor work.
        uint32_t qa[KSTEPS][4];
        {
            const __nv_bfloat16* qhi = p.q + (size_t)row * 2 * p.nq * D + (size_t)(hk * p.g + gid) * D;
            const __nv_bfloat16* qlo = qhi + (size_t)p.nq * D;
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
                qa[ks][0] = qa[ks][1] = qa[ks][2] = qa[ks][3] = 0u;
                if (gid < p.g) {
                    qa[ks][0] = *reinterpret_cast<const uint32_t*>(qhi + ks * 16 + 2 * tig);
                    qa[ks][1] = *reinterpret_cast<const uint32_t*>(qlo + ks * 16 + 2 * tig);
                    qa[ks][2] = *reinterpret_cast<const uint32_t*>(qhi + ks * 16 + 8 + 2 * tig);
                    qa[ks][3] = *reinterpret_cast<const uint32_t*>(qlo + ks * 16 + 8 + 2 * tig);
                }
            }
        }

        float oacc[NTILES][4];
#pragma unroll
        for (int c = 0; c < NTILES; ++c) oacc[c][0] = oacc[c][1] = oacc[c][2] = oacc[c][3] = 0.f;
        float m_run = -INFINITY, l_run = 0.f;

        for (int j = 0; j < n_st; ++j) {
            if (tid == 0 && !dead && j + kAttnStages - 1 < n_st) issue(cur, j + kAttnStages - 1, gs + j + kAttnStages - 1);
            const uint32_t g_stage = gs + j;
            const int slot = g_stage % kAttnStages;
            // Every lane polls; the outcome is made warp-uniform before any .sync instruction.
            int my_ok = 1;
            if (dead) {
                my_ok = 0;
            } else if (!mbar_wait(&full_bar[slot], (g_stage / kAttnStages) & 1)) {
                my_ok = 0;
                dead = 1;
                atomicOr(p.err, kErrTimeout);
            }
            const bool ok = __all_sync(0xffffffffu, my_ok);
            const int n_valid = min(kStageTok, len - j * kStageTok);
            const int w0 = warp * 16;
            if (w0 < n_valid && ok) {
                const uint32_t kbase = smem_u32(smem + (size_t)slot * STAGE_BYTES);
                const uint32_t vbase = kbase + TILE_BYTES;
                if (n_valid < w0 + 16) {
                    // ragged tail: rows past the end hold whatever the page holds; P is zero there, but
                    // 0 * NaN is NaN, so the value rows are cleared.
                    unsigned char* vt = smem + (size_t)slot * STAGE_BYTES + TILE_BYTES;
                    for (int i = lane; i < (w0 + 16 - n_valid) * HALVES * 8; i += 32) {
                        const int r = n_valid + i / (HALVES * 8), rem = i % (HALVES * 8);
                        *reinterpret_cast<uint4*>(vt + (rem / 8) * (kStageTok * 128) + r * 128 + (rem % 8) * 16) =
                            make_uint4(0, 0, 0, 0);
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                }
                // S = Q K^T for this warp's 16 tokens (two N tiles)
                float sacc[2][4];
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f;
                    const int r = w0 + nt * 8 + (lane & 7);
#pragma unroll
                    for (int kk = 0; kk < D / 32; ++kk) {
                        uint32_t kb[4];
                        ldmatrix_x4(kb, kbase + tile_off(kk >> 1, r, (kk & 1) * 4 + (lane >> 3)));
                        mma_16816(sacc[nt], qa[2 * kk][0], qa[2 * kk][1], qa[2 * kk][2], qa[2 * kk][3], kb[0], kb[1]);
                        mma_16816(sacc[nt], qa[2 * kk + 1][0], qa[2 * kk + 1][1], qa[2 * kk + 1][2], qa[2 * kk + 1][3],
                                  kb[2], kb[3]);
                    }
                }
                // online softmax over the tokens of row gid (log2 domain)
                float sv[4];
                float mx = -INFINITY;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int tl = w0 + (i >> 1) * 8 + 2 * tig + (i & 1);
                    sv[i] = tl < n_valid ? (sacc[i >> 1][i & 1] + sacc[i >> 1][2 + (i & 1)]) * p.scale_log2 : -INFINITY;
                    mx = fmaxf(mx, sv[i]);
                }
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                const float m_new = fmaxf(m_run, mx);
                const float alpha = exp2f(m_run - m_new);
                float pv[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) pv[i] = exp2f(sv[i] - m_new);
                l_run = l_run * alpha + (pv[0] + pv[1] + pv[2] + pv[3]);
                m_run = m_new;
                // P as (hi, lo) pairs: hi on rows 0..7, lo on rows 8..15 of the A operand
                float pl[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) pl[i] = pv[i] - __bfloat162float(__float2bfloat16_rn(pv[i]));
                const uint32_t pa0 = pack_bf16(pv[0], pv[1]), pa2 = pack_bf16(pv[2], pv[3]);
                const uint32_t pa1 = pack_bf16(pl[0], pl[1]), pa3 = pack_bf16(pl[2], pl[3]);
                // O = alpha O + P V
#pragma unroll
                for (int c = 0; c < NTILES; c += 2) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) { oacc[c][i] *= alpha; oacc[c + 1][i] *= alpha; }
                    const int mi = lane >> 3;
                    const int r = w0 + (mi & 1) * 8 + (lane & 7);
                    const int ch = c + (mi >> 1);
                    uint32_t vb[4];
                    ldmatrix_x4_trans(vb, vbase + tile_off(ch >> 3, r, ch & 7));
                    mma_16816(oacc[c], pa0, pa1, pa2, pa3, vb[0], vb[1]);
                    mma_16816(oacc[c + 1], pa0, pa1, pa2, pa3, vb[2], vb[3]);
                }
            }
            __syncthreads();
        }
        gs += n_st;

        // the next unit's first stages go into ring slots gs, gs + 1; the slot after them stays free
        // until that unit's main loop, and serves as scratch for the epilogue below
        const int un = u + gridDim.x;
        const bool have_next = un < n_units;
        Unit nxt = cur;
        if (have_next) {
            nxt = load_unit(un);
            if (tid == 0 && !dead) prefetch(nxt, gs);
        }
        unsigned char* scratch = smem + (size_t)((gs + kAttnStages - 1) % kAttnStages) * STAGE_BYTES;

        // merge the four warps
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
        float* mo = reinterpret_cast<float*>(scratch);              // [warps][8][D]
        float* mm = mo + kAttnWarps * 8 * D;                        // [warps][8]
        float* ml = mm + kAttnWarps * 8;                            // [warps][8]
#pragma unroll
        for (int c = 0; c < NTILES; ++c) {
            mo[(warp * 8 + gid) * D + c * 8 + 2 * tig] = oacc[c][0] + oacc[c][2];       // hi rows + lo rows
            mo[(warp * 8 + gid) * D + c * 8 + 2 * tig + 1] = oacc[c][1] + oacc[c][3];
        }
        if (tig == 0) { mm[warp * 8 + gid] = m_run; ml[warp * 8 + gid] = l_run; }
        __syncthreads();
        for (int idx = tid; idx < p.g * D; idx += kAttnWarps * 32) {
            const int hh = idx / D, d = idx - hh * D;
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < kAttnWarps; ++w) M = fmaxf(M, mm[w * 8 + hh]);
            float L = 0.f, o = 0.f;
#pragma unroll
            for (int w = 0; w < kAttnWarps; ++w) {
                const float sc = exp2f(mm[w * 8 + hh] - M);
                L += ml[w * 8 + hh] * sc;
                o += mo[(w * 8 + hh) * D + d] * sc;
            }
            const size_t ph = (size_t)slot_out * p.nq + hk * p.g + hh;
            p.part_o[ph * D + d] = o;
            if (d == 0) p.part_ml[ph] = make_float2(M, L);
        }
        // the generic-proxy writes above must be ordered before the next TMA write to this memory
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
        cur = nxt; u = un; have = have_next;
    }
}

// ---------------------------------------------------------------------------------------------
// Attention of a BLOCK of up to kPfQueries query rows that read the same cached tokens, so that every
// K/V tile is fetched once for the block.  A unit is (item, KV head); the tiles stream through the
// same TMA ring as in the decode kernel, and warp w owns query w of the block: it scores all 64
// tokens of every stage (four 16-token blocks) and keeps its own online softmax and accumulator.
//
// SHARED == false: causal attention of chunked prefill.  An item is a run of consecutive prompt
//   tokens of one request (items: first token row, 0, keys visible to the LAST query, number of
//   queries); every warp masks by its own causal length.  Nothing is split along the keys, so the
//   normalised output goes straight to b.o as (hi, lo) pairs.
// SHARED == true: decode rows of DIFFERENT sequences whose block tables list the same pages for a
//   span of cached tokens (members of a rollout group forked from one prompt).  An item is (first
//   cached token, tokens, rows, 0, token row x 4, partial slot x 4); all rows see the whole span, and
//   each writes (max, sum, unnormalised O) to its own partial slot for the span merge.
constexpr int kPfQueries = 4;

template <int D>
__device__ __forceinline__ void attend16(uint32_t kbase, uint32_t vbase, int w0, int n_valid, const uint32_t (&qa)[D / 16][4],
                                         float (&oacc)[D / 8][4], float& m_run, float& l_run, float scale_log2, int lane) {
    constexpr int NTILES = D / 8;
    const int tig = lane & 3;
    float sacc[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
        sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f;
        const int r = w0 + nt * 8 + (lane & 7);
#pragma unroll
        for (int kk = 0; kk < D / 32; ++kk) {
            uint32_t kb[4];
            ldmatrix_x4(kb, kbase + tile_off(kk >> 1, r, (kk & 1) * 4 + (lane >> 3)));
            mma_16816(sacc[nt], qa[2 * kk][0], qa[2 * kk][1], qa[2 * kk][2], qa[2 * kk][3], kb[0], kb[1]);
            mma_16816(sacc[nt], qa[2 * kk + 1][0], qa[2 * kk + 1][1], qa[2 * kk + 1][2], qa[2 * kk + 1][3], kb[2], kb[3]);
        }
    }
    float sv[4];
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int tl = w0 + (i >> 1) * 8 + 2 * tig + (i & 1);
        sv[i] = tl < n_valid ? (sacc[i >> 1][i & 1] + sacc[i >> 1][2 + (i & 1)]) * scale_log2 : -INFINITY;
        mx = fmaxf(mx, sv[i]);
    }
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float m_new = fmaxf(m_run, mx);
    const float alpha = exp2f(m_run - m_new);
    float pv[4], pl[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        pv[i] = exp2f(sv[i] - m_new);
        pl[i] = pv[i] - __bfloat162float(__float2bfloat16_rn(pv[i]));
    }
    l_run = l_run * alpha + (pv[0] + pv[1] + pv[2] + pv[3]);
    m_run = m_new;
    const uint32_t pa0 = pack_bf16(pv[0], pv[1]), pa2 = pack_bf16(pv[2], pv[3]);
    const uint32_t pa1 = pack_bf16(pl[0], pl[1]), pa3 = pack_bf16(pl[2], pl[3]);
#pragma unroll
    for (int c = 0; c < NTILES; c += 2) {
#pragma unroll
        for (int i = 0; i < 4; ++i) { oacc[c][i] *= alpha; oacc[c + 1][i] *= alpha; }
        const int mi = lane >> 3;
        const int r = w0 + (mi & 1) * 8 + (lane & 7);
        const int ch = c + (mi >> 1);
        uint32_t vb[4];
        ldmatrix_x4_trans(vb, vbase + tile_off(ch >> 3, r, ch & 7));
        mma_16816(oacc[c], pa0, pa1, pa2, pa3, vb[0], vb[1]);
        mma_16816(oacc[c + 1], pa0, pa1, pa2, pa3, vb[2], vb[3]);
    }
}

template <int D, bool SHARED>
__global__ void __launch_bounds__(kPfQueries * 32, 2)
attn_block_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, AttnParams p,
                    __nv_bfloat16* o_out) {
    constexpr int TILE_BYTES = kStageTok * D * 2;
    constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    constexpr int HALVES = D / 64;
    constexpr int KSTEPS = D / 16;
    constexpr int NTILES = D / 8;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t full_bar[kAttnStages];
    __shared__ volatile int dead;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gid = lane >> 2, tig = lane & 3;
    if (tid == 0) {
        for (int i = 0; i < kAttnStages; ++i) mbar_init(&full_bar[i], 1);
        dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    pdl_wait();

    const int n_units = p.step[SHARED ? H_SH_ITEMS : H_PF_ITEMS] * p.nkv;
    const int4* items = reinterpret_cast<const int4*>(p.step + p.lay.items) + p.step[H_PF_FIRST];
    const uint64_t pol = l2_evict_first_policy();
    uint32_t gs = 0;

    for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
        const int item = u / p.nkv, hk = u - item * p.nkv;
        int row0, start, len, nq_blk, my_row, my_slot = 0;
        if (SHARED) {
            const int32_t* it = p.step + p.lay.sh_items + 12 * item;
            start = it[0]; len = it[1]; nq_blk = it[2];
            const int w = min(warp, nq_blk - 1);
            row0 = it[4]; my_row = it[4 + w]; my_slot = it[8 + w];
        } else {
            const int4 it = items[item];
            row0 = it.x; start = 0; len = it.z; nq_blk = it.w;    // len: keys visible to the last query
            my_row = row0 + min(warp, nq_blk - 1);
        }
        const int seq = p.step[p.lay.tok_seq + row0];
        const int n_st = (len + kStageTok - 1) / kStageTok;
        const int32_t* bt = p.block_table + (size_t)seq * p.max_pages_per_seq;
        const bool has_q = warp < nq_blk;
        const int my_len = SHARED ? len : len - (nq_blk - 1 - warp);   // keys visible to this warp's query

        auto issue = [&](int j, uint32_t g_stage) {
            const int slot = g_stage % kAttnStages;
            unsigned char* kdst = smem + (size_t)slot * STAGE_BYTES;
            unsigned char* vdst = kdst + TILE_BYTES;
            const int n_valid = min(kStageTok, len - j * kStageTok);
            const int n_boxes = (n_valid + p.box_rows - 1) / p.box_rows;
            mbar_expect_tx(&full_bar[slot], (uint32_t)(n_boxes * p.box_rows * D * 2 * 2));
            for (int bi = 0; bi < n_boxes; ++bi) {
                const int tok = start + j * kStageTok + bi * p.box_rows;
                const int page = bt[tok / p.page_size];
                const int y = (((p.layer * p.n_pages + page) * p.nkv + hk) * p.page_size) + tok % p.page_size;
#pragma unroll
                for (int hf = 0; hf < HALVES; ++hf) {
                    const int off = hf * (kStageTok * 128) + bi * p.box_rows * 128;
                    tma_load_2d(kdst + off, &tm_k, hf * 64, y, &full_bar[slot], pol);
                    tma_load_2d(vdst + off, &tm_v, hf * 64, y, &full_bar[slot], pol);
                }
            }
        };
        if (tid == 0 && !dead) {
            const int pre = min(kAttnStages - 1, n_st);
            for (int j = 0; j < pre; ++j) issue(j, gs + j);
        }

        uint32_t qa[KSTEPS][4];
        {
            const __nv_bfloat16* qhi = p.q + (size_t)my_row * 2 * p.nq * D + (size_t)(hk * p.g + gid) * D;
            const __nv_bfloat16* qlo = qhi + (size_t)p.nq * D;
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
                qa[ks][0] = qa[ks][1] = qa[ks][2] = qa[ks][3] = 0u;
                if (gid < p.g && has_q) {
                    qa[ks][0] = *reinterpret_cast<const uint32_t*>(qhi + ks * 16 + 2 * tig);
                    qa[ks][1] = *reinterpret_cast<const uint32_t*>(qlo + ks * 16 + 2 * tig);
                    qa[ks][2] = *reinterpret_cast<const uint32_t*>(qhi + ks * 16 + 8 + 2 * tig);
                    qa[ks][3] = *reinterpret_cast<const uint32_t*>(qlo + ks * 16 + 8 + 2 * tig);
                }
            }
        }
        float oacc[NTILES][4];
#pragma unroll
        for (int c = 0; c < NTILES; ++c) oacc[c][0] = oacc[c][1] = oacc[c][2] = oacc[c][3] = 0.f;
        float m_run = -INFINITY, l_run = 0.f;

        for (int j = 0; j < n_st; ++j) {
            if (tid == 0 && !dead && j + kAttnStages - 1 < n_st) issue(j + kAttnStages - 1, gs + j + kAttnStages - 1);
            const uint32_t g_stage = gs + j;
            const int slot = g_stage % kAttnStages;
            int my_ok = 1;
            if (dead) {
                my_ok = 0;
            } else if (!mbar_wait(&full_bar[slot], (g_stage / kAttnStages) & 1)) {
                my_ok = 0;
                dead = 1;
                atomicOr(p.err, kErrTimeout);
            }
            const bool ok = __all_sync(0xffffffffu, my_ok);
            const int blk_valid = min(kStageTok, len - j * kStageTok);       // rows that hold this request's tokens
            if (blk_valid < kStageTok) {
                // last stage: clear the value rows past the end (0 * NaN), all warps read all rows
                unsigned char* vt = smem + (size_t)slot * STAGE_BYTES + TILE_BYTES;
                for (int i = tid; i < (kStageTok - blk_valid) * HALVES * 8; i += kPfQueries * 32) {
                    const int r = blk_valid + i / (HALVES * 8), rem = i % (HALVES * 8);
                    *reinterpret_cast<uint4*>(vt + (rem / 8) * (kStageTok * 128) + r * 128 + (rem % 8) * 16) =
                        make_uint4(0, 0, 0, 0);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncthreads();
            }
            const int n_valid = min(kStageTok, my_len - j * kStageTok);      // causal: keys this query may see
            if (has_q && ok && n_valid > 0) {
                const uint32_t kbase = smem_u32(smem + (size_t)slot * STAGE_BYTES);
                const uint32_t vbase = kbase + TILE_BYTES;
                for (int w0 = 0; w0 < n_valid; w0 += 16)
                    attend16<D>(kbase, vbase, w0, n_valid, qa, oacc, m_run, l_run, p.scale_log2, lane);
            }
            __syncthreads();
        }
        gs += n_st;

        l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
        if (SHARED) {
            if (has_q && gid < p.g) {
                const size_t ph = (size_t)my_slot * p.nq + hk * p.g + gid;
                float* dst = p.part_o + ph * D;
#pragma unroll
                for (int c = 0; c < NTILES; ++c)
                    *reinterpret_cast<float2*>(dst + c * 8 + 2 * tig) =
                        make_float2(oacc[c][0] + oacc[c][2], oacc[c][1] + oacc[c][3]);      // hi rows + lo rows
                if (tig == 0) p.part_ml[ph] = make_float2(m_run, l_run);
            }
        } else if (has_q && gid < p.g) {
            const float inv = 1.f / l_run;
            __nv_bfloat16* dst = o_out + (size_t)my_row * 2 * p.nq * D + (size_t)(hk * p.g + gid) * D;
#pragma unroll
            for (int c = 0; c < NTILES; ++c)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int d = c * 8 + 2 * tig + e;
                    split_bf16((oacc[c][e] + oacc[c][2 + e]) * inv, dst[d], dst[(size_t)p.nq * D + d]);
                }
        }
    }
}

// Merge of the spans of one (token row, query head): log-sum-exp rule on (max, sum, O).  The span
// statistics are fetched in one round trip (one span per thread), then the partial outputs are
// read eight spans at a time.
template <int D>
__global__ void __launch_bounds__(D) attn_combine_kernel(Buffers b, StepLayout lay, int nq) {
    __shared__ float2 sml[D];
    pdl_wait();
    const int t = blockIdx.x, j = blockIdx.y, d = threadIdx.x;
    const int i0 = b.step[lay.tok_item_off + t], i1 = b.step[lay.tok_item_off + t + 1];
    float den = 0.f, o = 0.f;
    float M = -INFINITY;
    for (int c0 = i0; c0 < i1; c0 += D) {               // chunks of D spans (one chunk unless the context is huge)
        const int n = min(D, i1 - c0);
        __syncthreads();
        if (d < n) sml[d] = b.part_ml[(size_t)(c0 + d) * nq + j];
        __syncthreads();
        float Mc = M;
        for (int i = 0; i < n; ++i) Mc = fmaxf(Mc, sml[i].x);
        const float rescale = exp2f(M - Mc);            // 0 for the first chunk (M = -inf)
        den *= rescale; o *= rescale;
        M = Mc;
        for (int i = 0; i < n; i += 8) {
            float pv[8];
#pragma unroll
            for (int q = 0; q < 8; ++q)
                pv[q] = i + q < n ? b.part_o[((size_t)(c0 + i + q) * nq + j) * D + d] : 0.f;
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (i + q < n) {
                    const float sc = exp2f(sml[i + q].x - M);
                    den += sml[i + q].y * sc;
                    o += pv[q] * sc;
                }
        }
    }
    // (hi, lo) rows of the token: b.o is [n_tok][2][nq D]
    __nv_bfloat16* dst = b.o + (size_t)t * 2 * nq * D + (size_t)j * D + d;
    split_bf16(o / den, dst[0], dst[(size_t)nq * D]);
}

template <int D>
static size_t attn_smem_bytes() { return (size_t)kAttnStages * 2 * kStageTok * D * 2 + 1024; }

int launch_attention(const Shape& s, const Buffers& b, const StepLayout& lay, const KvView& kv, const CUtensorMap& tm_k,
                     const CUtensorMap& tm_v, int layer, int sm_count, cudaStream_t st) {
    AttnParams p;
    p.q = b.q; p.part_o = b.part_o; p.part_ml = b.part_ml; p.step = b.step; p.lay = lay;
    p.block_table = kv.block_table; p.err = b.err;
    p.max_pages_per_seq = kv.max_pages_per_seq; p.n_pages = kv.n_pages; p.page_size = kv.page_size;
    p.box_rows = kv.page_size < kStageTok ? kv.page_size : kStageTok;
    p.nkv = s.nkv; p.nq = s.nq; p.g = s.nq / s.nkv; p.layer = layer;
    p.scale_log2 = (float)(1.4426950408889634 / sqrt((double)s.D));
    const int grid = sm_count * 2;
    if (s.D == 128) launch_chained(attn_decode_kernel<128>, dim3(grid), dim3(kAttnWarps * 32), attn_smem_bytes<128>(), st, tm_k, tm_v, p);
    else launch_chained(attn_decode_kernel<64>, dim3(grid), dim3(kAttnWarps * 32), attn_smem_bytes<64>(), st, tm_k, tm_v, p);
    return 1;
}

int launch_attention_prefill(const Shape& s, const Buffers& b, const StepLayout& lay, const KvView& kv,
                             const CUtensorMap& tm_k, const CUtensorMap& tm_v, int layer, int sm_count, cudaStream_t st) {
    AttnParams p;
    p.q = b.q; p.part_o = b.part_o; p.part_ml = b.part_ml; p.step = b.step; p.lay = lay;
    p.block_table = kv.block_table; p.err = b.err;
    p.max_pages_per_seq = kv.max_pages_per_seq; p.n_pages = kv.n_pages; p.page_size = kv.page_size;
    p.box_rows = kv.page_size < kStageTok ? kv.page_size : kStageTok;
    p.nkv = s.nkv; p.nq = s.nq; p.g = s.nq / s.nkv; p.layer = layer;
    p.scale_log2 = (float)(1.4426950408889634 / sqrt((double)s.D));
    const int grid = sm_count * 2;
    if (s.D == 128) launch_chained(attn_block_kernel<128, false>, dim3(grid), dim3(kPfQueries * 32), attn_smem_bytes<128>(), st, tm_k, tm_v, p, b.o);
    else launch_chained(attn_block_kernel<64, false>, dim3(grid), dim3(kPfQueries * 32), attn_smem_bytes<64>(), st, tm_k, tm_v, p, b.o);
    return 1;
}

int launch_attention_shared(const Shape& s, const Buffers& b, const StepLayout& lay, const KvView& kv,
                            const CUtensorMap& tm_k, const CUtensorMap& tm_v, int layer, int n_items, int sm_count,
                            cudaStream_t st) {
    AttnParams p;
    p.q = b.q; p.part_o = b.part_o; p.part_ml = b.part_ml; p.step = b.step; p.lay = lay;
    p.block_table = kv.block_table; p.err = b.err;
    p.max_pages_per_seq = kv.max_pages_per_seq; p.n_pages = kv.n_pages; p.page_size = kv.page_size;
    p.box_rows = kv.page_size < kStageTok ? kv.page_size : kStageTok;
    p.nkv = s.nkv; p.nq = s.nq; p.g = s.nq / s.nkv; p.layer = layer;
    p.scale_log2 = (float)(1.4426950408889634 / sqrt((double)s.D));
    int grid = n_items * s.nkv;
    if (grid > sm_count * 2) grid = sm_count * 2;
    if (s.D == 128) launch_chained(attn_block_kernel<128, true>, dim3(grid), dim3(kPfQueries * 32), attn_smem_bytes<128>(), st, tm_k, tm_v, p, nullptr);
    else launch_chained(attn_block_kernel<64, true>, dim3(grid), dim3(kPfQueries * 32), attn_smem_bytes<64>(), st, tm_k, tm_v, p, nullptr);
    return 1;
}

int launch_attn_merge(const Shape& s, const Buffers& b, const StepLayout& lay, int n_tok, cudaStream_t st) {
    if (s.D == 128) launch_chained(attn_combine_kernel<128>, dim3(n_tok, s.nq), dim3(128), 0, st, b, lay, s.nq);
    else launch_chained(attn_combine_kernel<64>, dim3(n_tok, s.nq), dim3(64), 0, st, b, lay, s.nq);
    return 1;
}

cudaError_t init_attn_kernels() {
    cudaError_t e = cudaFuncSetAttribute(attn_decode_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)attn_smem_bytes<128>());
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_decode_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)attn_smem_bytes<64>());
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_block_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)attn_smem_bytes<128>());
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_block_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)attn_smem_bytes<64>());
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_block_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)attn_smem_bytes<128>());
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(attn_block_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)attn_smem_bytes<64>());
}

}  // namespace mars
