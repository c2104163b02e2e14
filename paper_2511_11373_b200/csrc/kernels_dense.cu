// Dense parts of the rollout step: step preparation, embedding, RMSNorm + QKV projection +
// per-head norm + RoPE + cache append, output projection + residual, lm_head.
#include "common.cuh"
#include "kernels.h"

namespace mars {

// ---------------------------------------------------------------------------------------------
// Step preparation: write the block-table entries of pages taken for this step and tabulate
// (cos, sin)(pos * theta_i) for every token row (fp64 angles: pos reaches 64k and beyond, where an
// fp32 product pos * theta_0 is already off by milliradians).
__global__ void prep_kernel(Buffers b, StepLayout lay, KvView kv, int half_d) {
    pdl_wait();
    const int32_t* hdr = b.step;
    const int n_tok = hdr[H_NTOK];
    if (blockIdx.x == 0) {
        const int n_up = hdr[H_NUPDATES];
        const int32_t* up = b.step + lay.updates;
        for (int i = threadIdx.x; i < n_up; i += blockDim.x)
            kv.block_table[(size_t)up[3 * i] * kv.max_pages_per_seq + up[3 * i + 1]] = up[3 * i + 2];
    }
    const int32_t* pos = b.step + lay.tok_pos;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_tok * half_d; i += gridDim.x * blockDim.x) {
        const int t = i / half_d, f = i - t * half_d;
        double sn, cs;
        sincos((double)pos[t] * b.inv_freq[f], &sn, &cs);
        b.rope[i] = make_float2((float)cs, (float)sn);
    }
}

int launch_prep(const Shape& s, const Buffers& b, const StepLayout& lay, const KvView& kv, int n_tok, cudaStream_t st) {
    const int total = n_tok * (s.D / 2);
    int grid = (total + 255) / 256;
    if (grid < 1) grid = 1;
    if (grid > 1024) grid = 1024;
    launch_chained(prep_kernel, dim3(grid), dim3(256), 0, st, b, lay, kv, s.D / 2);
    return 1;
}

// ---------------------------------------------------------------------------------------------
// RMSNorm of one fp32 row held in registers -> (hi, lo) bf16 rows (gain applied).  Called by every
// thread of the block; `vals` are this thread's elements c = tid + i * blockDim.  `out` points at
// the token's hi row; the lo row follows it.
template <int MAX_PER_THREAD>
__device__ __forceinline__ void rms_to_pair(const float (&vals)[MAX_PER_THREAD], int H, float eps,
                                            const __nv_bfloat16* gain, __nv_bfloat16* out, float* scratch) {
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < MAX_PER_THREAD; ++i) {
        const int c = threadIdx.x + i * blockDim.x;
        if (c < H) ss += vals[i] * vals[i];
    }
    ss = block_sum(ss, scratch);
    const float r = rsqrtf(ss / (float)H + eps);
#pragma unroll
    for (int i = 0; i < MAX_PER_THREAD; ++i) {
        const int c = threadIdx.x + i * blockDim.x;
        if (c < H) split_bf16(vals[i] * r * __bfloat162float(gain[c]), out[c], out[H + c]);
    }
}

constexpr int kRowThreads = 256;
constexpr int kRowMaxPer = 32;  // hidden <= 8192

// Embedding gather: x = embed[token] (fp32), h = rms(x) * gain of the first layer's attention norm.
__global__ void __launch_bounds__(kRowThreads) embed_kernel(Shape s, Buffers b, const __nv_bfloat16* embed,
                                                            const int32_t* tokens, const __nv_bfloat16* gain,
                                                            float* hidden_tap) {
    __shared__ float scratch[32];
    pdl_wait();
    const int t = blockIdx.x;
    int tok = tokens[t];
    if (tok < 0 || tok >= s.V) {
        if (threadIdx.x == 0) atomicOr(b.err, kErrBadToken);
        tok = 0;
    }
    float v[kRowMaxPer];
#pragma unroll
    for (int i = 0; i < kRowMaxPer; ++i) {
        const int c = threadIdx.x + i * kRowThreads;
        v[i] = c < s.H ? __bfloat162float(embed[(size_t)tok * s.H + c]) : 0.f;
    }
#pragma unroll
    for (int i = 0; i < kRowMaxPer; ++i) {
        const int c = threadIdx.x + i * kRowThreads;
        if (c < s.H) {
            b.x[(size_t)t * s.H + c] = v[i];
            if (hidden_tap) hidden_tap[(size_t)t * s.H + c] = v[i];
        }
    }
    rms_to_pair<kRowMaxPer>(v, s.H, s.eps, gain, b.h + (size_t)t * 2 * s.H, scratch);
}

int launch_embed(const Shape& s, const Buffers& b, const StepLayout&, const __nv_bfloat16* embed, const int32_t* tokens,
                 const __nv_bfloat16* first_gain, float* hidden_tap, int n_tok, cudaStream_t st) {
    launch_chained(embed_kernel, dim3(n_tok), dim3(kRowThreads), 0, st, s, b, embed, tokens, first_gain, hidden_tap);
    return 1;
}

// ---------------------------------------------------------------------------------------------
// Y^T = W X^T for up to 64 tokens per block: a CTA owns 128 weight rows (8 warps x 16) and a range
// of K.  The activations of that K range (hi/lo pairs = 128 columns) sit in shared memory, one
// phase of at most 512 elements at a time; the weights stream once from HBM through the per-warp
// cp.async rings and keep streaming while a phase's activations are swapped.  With split-K
// (gridDim.y > 1) every K range writes its own fp32 partial [ksplit][tokens][rows]; the consumer
// kernel adds the partials in a fixed order, so results do not depend on scheduling.
constexpr int kGemmMaxWarps = 10;   // 16 rows each; the CTA width is chosen per matrix (see launch_gemm)
constexpr int kGemmTok = 64;
constexpr int kGemmCols = 2 * kGemmTok;
constexpr int kGemmNT = kGemmCols / 8;
constexpr int kGemmMaxKS = 512;

struct GemmParams {
    const __nv_bfloat16* W;     // [rows, K]
    const __nv_bfloat16* X;     // [*, 2, K] (hi row, lo row per token)
    const int32_t* row_index;   // optional: X token of output token t is row_index[t]
    float* out;                 // [ksplit, n_tok, rows]
    int rows, K, n_tok;
    int ks;                     // K elements per phase (multiple of 64, <= 512)
    int phases;                 // phases per CTA; gridDim.y * phases * ks == K
};

static size_t gemm_smem_bytes(int ks, int warps) {
    return (size_t)kGemmCols * x_row_bytes(ks) + (size_t)warps * kRingWarpBytes;
}

__global__ void __launch_bounds__(kGemmMaxWarps * 32, 1) stream_gemm_kernel(GemmParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gid = lane >> 2, tig = lane & 3;
    const int xrow = x_row_bytes(p.ks);
    unsigned char* xt = smem;
    unsigned char* ring = smem + (size_t)kGemmCols * xrow + (size_t)warp * kRingWarpBytes;
    const int row_base = (blockIdx.x * (blockDim.x >> 5) + warp) * 16;
    const int tok0 = blockIdx.z * kGemmTok;
    const int n_here = min(kGemmTok, p.n_tok - tok0);
    const int k_begin = blockIdx.y * p.phases * p.ks;
    const int slices_per_phase = p.ks / 32;
    const int total_slices = p.phases * slices_per_phase;

    const int r0 = min(row_base + gid, p.rows - 1), r1 = min(row_base + gid + 8, p.rows - 1);
    const __nv_bfloat16* w0 = p.W + (size_t)r0 * p.K + k_begin + tig * 8;
    const __nv_bfloat16* w1 = p.W + (size_t)r1 * p.K + k_begin + tig * 8;

    // prime the ring: slices 0 .. kRing-1 (one commit group each, empty past the end)
#pragma unroll
    for (int i = 0; i < kRing; ++i) {
        if (i < total_slices) ring_issue(ring, i, lane, w0 + (size_t)i * 32, w1 + (size_t)i * 32);
        cp_async_commit();
    }

    float acc[kGemmNT][4];
#pragma unroll
    for (int n = 0; n < kGemmNT; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;

    // the weight ring above reads constants only; the activations come from the previous kernel
    pdl_wait();
    const int pieces = p.ks / 8;   // 16-byte pieces per activation row
    for (int ph = 0; ph < p.phases; ++ph) {
        if (ph > 0) __syncthreads();             // every warp is done with the previous phase's activations
        // activation rows of this phase by cp.async (columns past the last token repeat token 0: their
        // results are never stored)
        for (int i = threadIdx.x; i < kGemmCols * pieces; i += blockDim.x) {
            const int v = i / pieces, pc = i - v * pieces;     // v: column = 2 * token + plane
            const int t = (v >> 1) < n_here ? (v >> 1) : 0;
            const int src_tok = p.row_index ? p.row_index[tok0 + t] : tok0 + t;
            cp_async16(xt + (size_t)v * xrow + pc * 16,
                       p.X + ((size_t)src_tok * 2 + (v & 1)) * p.K + k_begin + (size_t)ph * p.ks + pc * 8);
        }
        cp_async_commit();
        // the activation group is the youngest: waiting for it also drains the ring, which costs one
        // memory round trip per phase
        cp_async_wait<0>();
        __syncthreads();
        const unsigned char* xs = xt + (size_t)gid * xrow + tig * 16;
        for (int sl = 0; sl < slices_per_phase; ++sl) {
            const int s = ph * slices_per_phase + sl;
            cp_async_wait<kRing - 1>();
            ring_consume<kGemmNT>(ring, s % kRing, lane, xs + (size_t)sl * 64, 8 * xrow, acc);
            const int nx = s + kRing;
            if (nx < total_slices) ring_issue(ring, s % kRing, lane, w0 + (size_t)nx * 32, w1 + (size_t)nx * 32);
            cp_async_commit();
        }
    }

    float* out = p.out + (size_t)blockIdx.y * p.n_tok * p.rows;
#pragma unroll
    for (int n = 0; n < kGemmNT; ++n)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            const int row = row_base + gid + hf * 8;
            const int t = n * 4 + tig;
            if (row < p.rows && t < n_here)
                out[(size_t)(tok0 + t) * p.rows + row] = acc[n][2 * hf] + acc[n][2 * hf + 1];   // hi + lo column
        }
}

// K range per phase and the number of K splits: split-K only pays (and only fits its partial
// buffer) for decode-sized token counts and matrices with few rows.
void gemm_plan(int K, int n_tok, bool many_rows, int* ks, int* ksplit, int* phases) {
    *ks = (K % kGemmMaxKS == 0) ? kGemmMaxKS : 256;      // K is a multiple of 256
    const int n_ph = K / *ks;
    if (n_tok <= kGemmTok && !many_rows) { *ksplit = n_ph; *phases = 1; }
    else { *ksplit = 1; *phases = n_ph; }
}

static int launch_gemm(GemmParams p, bool many_rows, int sm_count, cudaStream_t st) {
    int ksplit;
    gemm_plan(p.K, p.n_tok, many_rows, &p.ks, &ksplit, &p.phases);
    // CTA width: the number of 16-row warps that minimises waves x rows per CTA on this many SMs
    const int tok_tiles = (p.n_tok + kGemmTok - 1) / kGemmTok;
    int best_w = 8;
    long best_cost = -1;
    for (int w = 6; w <= kGemmMaxWarps; ++w) {
        const long ctas = (long)((p.rows + w * 16 - 1) / (w * 16)) * ksplit * tok_tiles;
        const long cost = ((ctas + sm_count - 1) / sm_count) * w;
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_w = w; }
    }
    dim3 grid((p.rows + best_w * 16 - 1) / (best_w * 16), ksplit, tok_tiles);
    launch_chained(stream_gemm_kernel, dim3(grid), dim3(best_w * 32), gemm_smem_bytes(p.ks, best_w), st, p);
    return 1;
}

// ---------------------------------------------------------------------------------------------
// Per-head RMS norm (optional), rotary embedding, cache append.  One block per token row, one
// warp per head in turn; lane l owns the rotation pairs (l + 32 i, l + 32 i + D/2).  Queries leave
// as (hi, lo) pairs: b.q is [n_tok][2][nq D]; keys and values are rounded to bf16 by the cache format.
template <int D>
__global__ void __launch_bounds__(128) qkv_post_kernel(Shape s, Buffers b, StepLayout lay, KvView kv,
                                                       const __nv_bfloat16* q_gain, const __nv_bfloat16* k_gain,
                                                       int layer, int ksplit, int n_tok) {
    constexpr int HALF = D / 2, PER = HALF / 32;
    pdl_wait();
    const int t = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_heads = s.nq + 2 * s.nkv;
    const int pos = b.step[lay.tok_pos + t], seq = b.step[lay.tok_seq + t];
    const int page = kv.block_table[(size_t)seq * kv.max_pages_per_seq + pos / kv.page_size];
    const int slot = pos % kv.page_size;
    const float* raw = b.qkv + (size_t)t * n_heads * D;
    for (int head = blockIdx.y * 4 + warp; head < n_heads; head += 4 * gridDim.y) {   // one head per warp
        const bool is_q = head < s.nq, is_k = !is_q && head < s.nq + s.nkv;
        float lo[PER], hi[PER];
        float ss = 0.f;
#pragma unroll
        for (int i = 0; i < PER; ++i) lo[i] = hi[i] = 0.f;
        // split-K partials, added in a fixed order; the loads of up to eight partials are issued before the
        // first add (one memory round trip, not one per partial)
        for (int sp0 = 0; sp0 < ksplit; sp0 += 8) {
            float pl[8][PER], ph[8][PER];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float* part = raw + (size_t)(sp0 + j) * n_tok * n_heads * D + head * D + lane;
#pragma unroll
                for (int i = 0; i < PER; ++i) {
                    pl[j][i] = sp0 + j < ksplit ? part[32 * i] : 0.f;
                    ph[j][i] = sp0 + j < ksplit ? part[32 * i + HALF] : 0.f;
                }
            }
#pragma unroll
            for (int j = 0; j < 8; ++j)
#pragma unroll
                for (int i = 0; i < PER; ++i) { lo[i] += pl[j][i]; hi[i] += ph[j][i]; }
        }
#pragma unroll
        for (int i = 0; i < PER; ++i) ss += lo[i] * lo[i] + hi[i] * hi[i];
        if (!is_q && !is_k) {  // value head: stored as is
            const int hk = head - s.nq - s.nkv;
            __nv_bfloat16* dst = kv.v_pool +
                ((((size_t)layer * kv.n_pages + page) * s.nkv + hk) * kv.page_size + slot) * D;
#pragma unroll
            for (int i = 0; i < PER; ++i) {
                dst[lane + 32 * i] = __float2bfloat16_rn(lo[i]);
                dst[lane + 32 * i + HALF] = __float2bfloat16_rn(hi[i]);
            }
            continue;
        }
        if (s.qk_norm) {
            ss = warp_sum(ss);
            const float r = rsqrtf(ss / (float)D + s.eps);
            const __nv_bfloat16* g = is_q ? q_gain : k_gain;
#pragma unroll
            for (int i = 0; i < PER; ++i) {
                lo[i] *= r * __bfloat162float(g[lane + 32 * i]);
                hi[i] *= r * __bfloat162float(g[lane + 32 * i + HALF]);
            }
        }
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const float2 cs = b.rope[(size_t)t * HALF + lane + 32 * i];
            const float a = lo[i] * cs.x - hi[i] * cs.y, c = hi[i] * cs.x + lo[i] * cs.y;
            if (is_q) {
                __nv_bfloat16* dq = b.q + (size_t)t * 2 * s.nq * D + head * D;
                split_bf16(a, dq[lane + 32 * i], dq[s.nq * D + lane + 32 * i]);
                split_bf16(c, dq[lane + 32 * i + HALF], dq[s.nq * D + lane + 32 * i + HALF]);
            } else {
                const int hk = head - s.nq;
                __nv_bfloat16* dk = kv.k_pool +
                    ((((size_t)layer * kv.n_pages + page) * s.nkv + hk) * kv.page_size + slot) * D;
                dk[lane + 32 * i] = __float2bfloat16_rn(a);
                dk[lane + 32 * i + HALF] = __float2bfloat16_rn(c);
            }
        }
    }
}

int launch_qkv(const Shape& s, const Buffers& b, const StepLayout& lay, const LayerW& w, const KvView& kv, int layer,
               int n_tok, int sm_count, cudaStream_t st) {
    GemmParams p{w.wqkv, b.h, nullptr, b.qkv, (s.nq + 2 * s.nkv) * s.D, s.H, n_tok, 0, 0};
    int n = launch_gemm(p, false, sm_count, st);
    int ks, ksplit, phases;
    gemm_plan(s.H, n_tok, false, &ks, &ksplit, &phases);
    return n + launch_qkv_post(s, b, lay, w, kv, layer, n_tok, ksplit, st);
}

int launch_qkv_post(const Shape& s, const Buffers& b, const StepLayout& lay, const LayerW& w, const KvView& kv, int layer,
                    int n_tok, int ksplit, cudaStream_t st) {
    const dim3 grid(n_tok, (s.nq + 2 * s.nkv + 3) / 4);
    if (s.D == 128)
        launch_chained(qkv_post_kernel<128>, dim3(grid), dim3(128), 0, st, s, b, lay, kv, w.q_norm, w.k_norm, layer, ksplit, n_tok);
    else
        launch_chained(qkv_post_kernel<64>, dim3(grid), dim3(128), 0, st, s, b, lay, kv, w.q_norm, w.k_norm, layer, ksplit, n_tok);
    return 1;
}

// Output projection: writes split-K partials of W_o o; the router kernel adds them to the residual.
int launch_oproj(const Shape& s, const Buffers& b, const LayerW& w, int n_tok, int sm_count, cudaStream_t st) {
    GemmParams p{w.wo, b.o, nullptr, b.opart, s.H, s.nq * s.D, n_tok, 0, 0};
    return launch_gemm(p, false, sm_count, st);
}

int launch_lm_head(const Shape& s, const Buffers& b, const StepLayout& lay, const __nv_bfloat16* lm_head, int n_emit,
                   int sm_count, cudaStream_t st) {
    GemmParams p{lm_head, b.h, b.step + lay.emit_rows, b.logits, s.V, s.H, n_emit, 0, 0};
    return launch_gemm(p, true, sm_count, st);
}

cudaError_t init_dense_kernels() {
    return cudaFuncSetAttribute(stream_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)gemm_smem_bytes(kGemmMaxKS, kGemmMaxWarps));
}

}  // namespace mars
