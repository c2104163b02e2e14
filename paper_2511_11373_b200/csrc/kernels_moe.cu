// Mixture-of-experts part of the rollout step: router (RMSNorm, fp32 gate logits, softmax, top-k,
// renormalise), token permutation by expert, grouped SwiGLU expert contraction for decode-sized
// groups (weights streamed once, swap-AB MMA tiles), weighted combine + residual + next norm.
#include "common.cuh"
#include "kernels.h"

namespace mars {

constexpr int kRouterThreads = 256;
constexpr int kRowMaxPer = 32;   // hidden <= 8192
constexpr int kMaxExperts = 1024;
constexpr int kMaxTopK = 32;

// ---------------------------------------------------------------------------------------------
// One block per token row.  h2 = rms(x) * g (kept in fp32 for the gate, stored as a (hi, lo) bf16
// pair for the experts); z_e = <W_r[e], h2> accumulated in fp32 in a fixed order; pi = softmax(z); the k largest
// pi (ties: lower index) and their renormalised weights.
__global__ void __launch_bounds__(kRouterThreads) router_kernel(Shape s, Buffers b, const __nv_bfloat16* gain,
                                                                const __nv_bfloat16* Wr, DebugTaps dbg, int layer,
                                                                int n_tok) {
    extern __shared__ float hs[];          // [H] normalised activations
    __shared__ float scratch[32];
    __shared__ float z[kMaxExperts];
    const int t = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int H = s.H, E = s.E, k = s.k;

    float ss = 0.f;
    for (int c = tid; c < H; c += kRouterThreads) {
        const float v = b.x[(size_t)t * H + c];
        hs[c] = v;
        ss += v * v;
    }
    ss = block_sum(ss, scratch);
    const float r = rsqrtf(ss / (float)H + s.eps);
    for (int c = tid; c < H; c += kRouterThreads) {
        const float v = hs[c] * r * __bfloat162float(gain[c]);
        hs[c] = v;
        split_bf16(v, b.h[(size_t)t * 2 * H + c], b.h[(size_t)t * 2 * H + H + c]);
    }
    __syncthreads();

    for (int e = warp; e < E; e += kRouterThreads / 32) {
        const __nv_bfloat16* w = Wr + (size_t)e * H;
        float acc = 0.f;
        for (int c = lane * 8; c < H; c += 256) {
            const uint4 v = *reinterpret_cast<const uint4*>(w + c);
            acc = fmaf(bf16_lo(v.x), hs[c], acc);     acc = fmaf(bf16_hi(v.x), hs[c + 1], acc);
            acc = fmaf(bf16_lo(v.y), hs[c + 2], acc); acc = fmaf(bf16_hi(v.y), hs[c + 3], acc);
            acc = fmaf(bf16_lo(v.z), hs[c + 4], acc); acc = fmaf(bf16_hi(v.z), hs[c + 5], acc);
            acc = fmaf(bf16_lo(v.w), hs[c + 6], acc); acc = fmaf(bf16_hi(v.w), hs[c + 7], acc);
        }
        acc = warp_sum(acc);
        if (lane == 0) z[e] = acc;
    }
    __syncthreads();

    if (warp == 0) {
        float mx = -INFINITY;
        for (int e = lane; e < E; e += 32) mx = fmaxf(mx, z[e]);
        mx = warp_max(mx);
        float sum = 0.f;
        for (int e = lane; e < E; e += 32) {
            const float ev = expf(z[e] - mx);
            z[e] = ev;
            sum += ev;
        }
        sum = warp_sum(sum);
        __syncwarp();
        for (int e = lane; e < E; e += 32) z[e] = z[e] / sum;   // pi
        __syncwarp();

        const int32_t* forced = dbg.forced_idx ? dbg.forced_idx + ((size_t)layer * n_tok + t) * k : nullptr;
        int my_idx = -1;        // lane j keeps the j-th selection
        float my_p = 0.f;
        if (forced) {
            if (lane < k) { my_idx = forced[lane]; my_p = z[my_idx]; }
        } else {
            for (int j = 0; j < k; ++j) {
                float best = -1.f;
                int bi = 0x7fffffff;
                for (int e = lane; e < E; e += 32) {
                    const float v = z[e];
                    if (v > best) { best = v; bi = e; }   // ascending e: the lower index wins ties
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const float ov = __shfl_xor_sync(0xffffffffu, best, o);
                    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                    if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
                }
                if (lane == j) { my_idx = bi; my_p = best; }
                if (lane == 0) z[bi] = -1.f;               // taken
                __syncwarp();
            }
        }
        float tot = lane < k ? my_p : 0.f;
        tot = warp_sum(tot);
        if (lane < k) {
            const float w = my_p / tot;
            b.route_idx[(size_t)t * k + lane] = my_idx;
            b.route_w[(size_t)t * k + lane] = w;
            if (dbg.router_idx) dbg.router_idx[((size_t)layer * n_tok + t) * k + lane] = my_idx;
            if (dbg.router_w) dbg.router_w[((size_t)layer * n_tok + t) * k + lane] = w;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Token permutation: histogram of expert ids, exclusive offsets, and for every expert the list of
// token rows it serves (slot order inside an expert is arbitrary: every (token, expert) product is
// computed independently of its slot).  Single block; also counts the distinct experts used.
__global__ void __launch_bounds__(1024) permute_kernel(Shape s, Buffers b, int layer, int n_pairs) {
    __shared__ int cnt[kMaxExperts];
    __shared__ int off[kMaxExperts + 1];
    const int tid = threadIdx.x, E = s.E;
    for (int e = tid; e < E; e += blockDim.x) cnt[e] = 0;
    __syncthreads();
    for (int i = tid; i < n_pairs; i += blockDim.x) atomicAdd(&cnt[b.route_idx[i]], 1);
    __syncthreads();
    if (tid == 0) {
        int acc = 0, active = 0;
        for (int e = 0; e < E; ++e) {
            off[e] = acc;
            acc += cnt[e];
            active += cnt[e] > 0;
        }
        off[E] = acc;
        b.active[layer] = active;
    }
    __syncthreads();
    for (int e = tid; e <= E; e += blockDim.x) b.expert_off[e] = off[e];
    for (int e = tid; e < E; e += blockDim.x) cnt[e] = 0;
    __syncthreads();
    for (int i = tid; i < n_pairs; i += blockDim.x) {
        const int e = b.route_idx[i];
        const int slot = off[e] + atomicAdd(&cnt[e], 1);
        b.slot_token[slot] = i / s.k;
        b.slot_of[i] = slot;
    }
}

// ---------------------------------------------------------------------------------------------
// Grouped SwiGLU, first half: act[slot, i] = silu(<W_gate[e, i], h>) * <W_up[e, i], h> for the
// tokens of expert e.  grid = (row blocks, experts); a warp owns 16 gate rows and the matching 16
// up rows and streams them once over the full K; the expert's activation rows sit in shared memory.
constexpr int kExpMaxWarps = 12;

template <int NT>
__device__ __forceinline__ void gate_up_tile(const __nv_bfloat16* Wg, const __nv_bfloat16* Wu, int H, int I,
                                             int row_base, const unsigned char* xs_base, int xrow, int m_here,
                                             __nv_bfloat16* act_out /* slot t0 of this expert, [slot][2][I] */,
                                             int lane) {
    const int gid = lane >> 2, tig = lane & 3;
    const __nv_bfloat16* wrow[2][2] = {
        {Wg + (size_t)(row_base + gid) * H + tig * 8, Wg + (size_t)(row_base + gid + 8) * H + tig * 8},
        {Wu + (size_t)(row_base + gid) * H + tig * 8, Wu + (size_t)(row_base + gid + 8) * H + tig * 8}};
    float acc[2][NT][4];
#pragma unroll
    for (int m = 0; m < 2; ++m)
#pragma unroll
        for (int n = 0; n < NT; ++n) acc[m][n][0] = acc[m][n][1] = acc[m][n][2] = acc[m][n][3] = 0.f;
    stream_mma<2, NT, 4>(wrow, H / 32, xs_base + (size_t)gid * xrow + tig * 16, 8 * xrow, acc);
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            const int row = row_base + gid + hf * 8;
            const int t = n * 4 + tig;                 // columns 2t (hi) and 2t+1 (lo) of token t
            if (t < m_here) {
                const float gte = acc[0][n][2 * hf] + acc[0][n][2 * hf + 1];
                const float up = acc[1][n][2 * hf] + acc[1][n][2 * hf + 1];
                __nv_bfloat16* dst = act_out + (size_t)t * 2 * I + row;
                split_bf16(gte / (1.f + expf(-gte)) * up, dst[0], dst[I]);
            }
        }
}

__global__ void __launch_bounds__(kExpMaxWarps * 32) expert_gate_up_kernel(Shape s, Buffers b, const __nv_bfloat16* Wgu,
                                                                        int tok_cap) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int e = blockIdx.y;
    const int o0 = b.expert_off[e], m = b.expert_off[e + 1] - o0;
    if (m == 0) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int H = s.H, I = s.I;
    const int row_base = (blockIdx.x * (blockDim.x >> 5) + warp) * 16;
    const bool row_ok = row_base < I;       // I is a multiple of 16
    const int xrow = x_row_bytes(H);
    const __nv_bfloat16* Wg = Wgu + (size_t)e * 2 * I * H;
    const __nv_bfloat16* Wu = Wg + (size_t)I * H;
    const int pieces = H / 8;
    for (int t0 = 0; t0 < m; t0 += tok_cap) {
        const int m_here = min(tok_cap, m - t0);
        const int cols_ld = (2 * m_here + 7) & ~7;      // column v = 2 * token + plane
        for (int i = threadIdx.x; i < cols_ld * pieces; i += blockDim.x) {
            const int v = i / pieces, pc = i - v * pieces;
            unsigned char* d = smem + (size_t)v * xrow + pc * 16;
            if ((v >> 1) < m_here)
                cp_async16(d, b.h + ((size_t)b.slot_token[o0 + t0 + (v >> 1)] * 2 + (v & 1)) * H + pc * 8);
            else *reinterpret_cast<uint4*>(d) = make_uint4(0, 0, 0, 0);
        }
        cp_async_commit();
        cp_async_wait<0>();
        __syncthreads();
        if (row_ok) {
            __nv_bfloat16* out = b.act + (size_t)(o0 + t0) * 2 * I;
            const int nt = (m_here + 3) >> 2;
            if (nt == 1) gate_up_tile<1>(Wg, Wu, H, I, row_base, smem, xrow, m_here, out, lane);
            else if (nt == 2) gate_up_tile<2>(Wg, Wu, H, I, row_base, smem, xrow, m_here, out, lane);
            else gate_up_tile<4>(Wg, Wu, H, I, row_base, smem, xrow, m_here, out, lane);
        }
        __syncthreads();
    }
}

// Second half: y[slot, r] = <W_down[e, r], act[slot]>.  A warp owns 32 output rows (two M tiles).
template <int NT>
__device__ __forceinline__ void down_tile(const __nv_bfloat16* Wd, int H, int I, int row_base,
                                          const unsigned char* xs_base, int xrow, int m_here, float* y_out, int lane) {
    const int gid = lane >> 2, tig = lane & 3;
    const __nv_bfloat16* wrow[2][2] = {
        {Wd + (size_t)(row_base + gid) * I + tig * 8, Wd + (size_t)(row_base + gid + 8) * I + tig * 8},
        {Wd + (size_t)(row_base + 16 + gid) * I + tig * 8, Wd + (size_t)(row_base + 24 + gid) * I + tig * 8}};
    float acc[2][NT][4];
#pragma unroll
    for (int m = 0; m < 2; ++m)
#pragma unroll
        for (int n = 0; n < NT; ++n) acc[m][n][0] = acc[m][n][1] = acc[m][n][2] = acc[m][n][3] = 0.f;
    stream_mma<2, NT, 4>(wrow, I / 32, xs_base + (size_t)gid * xrow + tig * 16, 8 * xrow, acc);
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int n = 0; n < NT; ++n)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const int row = row_base + mt * 16 + gid + hf * 8;
                const int t = n * 4 + tig;
                if (t < m_here) y_out[(size_t)t * H + row] = acc[mt][n][2 * hf] + acc[mt][n][2 * hf + 1];
            }
}

__global__ void __launch_bounds__(kExpMaxWarps * 32) expert_down_kernel(Shape s, Buffers b, const __nv_bfloat16* Wdn,
                                                                     int tok_cap) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int e = blockIdx.y;
    const int o0 = b.expert_off[e], m = b.expert_off[e + 1] - o0;
    if (m == 0) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int H = s.H, I = s.I;
    const int row_base = (blockIdx.x * (blockDim.x >> 5) + warp) * 32;
    const bool row_ok = row_base < H;       // H is a multiple of 32
    const int xrow = x_row_bytes(I);
    const __nv_bfloat16* Wd = Wdn + (size_t)e * H * I;
    const int pieces = I / 8;
    for (int t0 = 0; t0 < m; t0 += tok_cap) {
        const int m_here = min(tok_cap, m - t0);
        const int cols_ld = (2 * m_here + 7) & ~7;      // act rows are already (hi, lo) interleaved
        for (int i = threadIdx.x; i < cols_ld * pieces; i += blockDim.x) {
            const int v = i / pieces, pc = i - v * pieces;
            unsigned char* d = smem + (size_t)v * xrow + pc * 16;
            if ((v >> 1) < m_here) cp_async16(d, b.act + ((size_t)(o0 + t0) * 2 + v) * I + pc * 8);
            else *reinterpret_cast<uint4*>(d) = make_uint4(0, 0, 0, 0);
        }
        cp_async_commit();
        cp_async_wait<0>();
        __syncthreads();
        if (row_ok) {
            float* out = b.y + (size_t)(o0 + t0) * H;
            const int nt = (m_here + 3) >> 2;
            if (nt == 1) down_tile<1>(Wd, H, I, row_base, smem, xrow, m_here, out, lane);
            else if (nt == 2) down_tile<2>(Wd, H, I, row_base, smem, xrow, m_here, out, lane);
            else down_tile<4>(Wd, H, I, row_base, smem, xrow, m_here, out, lane);
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------------
// x += sum_j w_j y[slot(t, j)] (fixed order), optional hidden-state tap, then the RMSNorm that
// feeds the next projection (next layer's attention norm, or the final norm).
__global__ void __launch_bounds__(kRouterThreads) combine_kernel(Shape s, Buffers b, const __nv_bfloat16* next_gain,
                                                                 float* hidden_tap) {
    __shared__ float scratch[32];
    __shared__ int slots[kMaxTopK];
    __shared__ float ws[kMaxTopK];
    const int t = blockIdx.x, tid = threadIdx.x, H = s.H, k = s.k;
    if (tid < k) { slots[tid] = b.slot_of[(size_t)t * k + tid]; ws[tid] = b.route_w[(size_t)t * k + tid]; }
    __syncthreads();
    float v[kRowMaxPer];
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < kRowMaxPer; ++i) {
        const int c = tid + i * kRouterThreads;
        v[i] = 0.f;
        if (c < H) {
            float acc = b.x[(size_t)t * H + c];
            for (int j = 0; j < k; ++j) acc = fmaf(ws[j], b.y[(size_t)slots[j] * H + c], acc);
            v[i] = acc;
            b.x[(size_t)t * H + c] = acc;
            if (hidden_tap) hidden_tap[(size_t)t * H + c] = acc;
            ss += acc * acc;
        }
    }
    ss = block_sum(ss, scratch);
    const float r = rsqrtf(ss / (float)H + s.eps);
#pragma unroll
    for (int i = 0; i < kRowMaxPer; ++i) {
        const int c = tid + i * kRouterThreads;
        if (c < H)
            split_bf16(v[i] * r * __bfloat162float(next_gain[c]), b.h[(size_t)t * 2 * H + c],
                       b.h[(size_t)t * 2 * H + H + c]);
    }
}

// ---------------------------------------------------------------------------------------------
int launch_router(const Shape& s, const Buffers& b, const LayerW& w, const DebugTaps& dbg, int layer, int n_tok,
                  cudaStream_t st) {
    router_kernel<<<n_tok, kRouterThreads, s.H * sizeof(float), st>>>(s, b, w.mlp_norm, w.router, dbg, layer, n_tok);
    permute_kernel<<<1, 1024, 0, st>>>(s, b, layer, n_tok * s.k);
    return 2;
}

// Tokens held in shared memory per pass (4 per column tile); experts with more tokens loop and
// stream their weights again.  Small groups keep the footprint low enough for three CTAs of four
// warps per SM; larger ones use one wide CTA per SM so that enough loads stay in flight.
static void expert_plan(const Shape& s, int n_tok, int* cap, int* warps) {
    const double avg = (double)n_tok * s.k / s.E;
    *cap = avg <= 5.0 ? 8 : 16;
    *warps = *cap == 8 ? 4 : kExpMaxWarps;
    while ((size_t)*cap * 2 * x_row_bytes(s.H) > 200u * 1024u && *cap > 4) *cap /= 2;
}

int launch_gate_up(const Shape& s, const Buffers& b, const LayerW& w, int n_tok, cudaStream_t st) {
    int cap, warps;
    expert_plan(s, n_tok, &cap, &warps);
    dim3 g1((s.I / 16 + warps - 1) / warps, s.E);
    expert_gate_up_kernel<<<g1, warps * 32, (size_t)cap * 2 * x_row_bytes(s.H), st>>>(s, b, w.w_gate_up, cap);
    return 1;
}

int launch_down(const Shape& s, const Buffers& b, const LayerW& w, int n_tok, cudaStream_t st) {
    int cap, warps;
    expert_plan(s, n_tok, &cap, &warps);
    const int w2 = warps == kExpMaxWarps ? 8 : warps;
    dim3 g2((s.H / 32 + w2 - 1) / w2, s.E);
    expert_down_kernel<<<g2, w2 * 32, (size_t)cap * 2 * x_row_bytes(s.I), st>>>(s, b, w.w_down, cap);
    return 1;
}

int launch_combine(const Shape& s, const Buffers& b, const __nv_bfloat16* next_gain, float* hidden_tap, int n_tok,
                   cudaStream_t st) {
    combine_kernel<<<n_tok, kRouterThreads, 0, st>>>(s, b, next_gain, hidden_tap);
    return 1;
}

cudaError_t init_moe_kernels() {
    cudaError_t e = cudaFuncSetAttribute(expert_gate_up_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(expert_down_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(router_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
}

}  // namespace mars
