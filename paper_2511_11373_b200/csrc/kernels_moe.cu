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

// Softmax over the gate logits z[0..E) (shared memory, overwritten), the k largest probabilities
// (ties: lower index) or the forced experts, and their renormalised weights.  Executed by one warp.
__device__ void route_select(float* z, const Shape& s, const Buffers& b, const DebugTaps& dbg, int layer, int n_tok, int t,
                             int lane) {
    const int E = s.E, k = s.k;
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
            // across the lanes with two warp reductions instead of ten shuffles: probabilities are non-negative floats,
            // whose bit patterns order like the values (+1 keeps 0 for "nothing left in this lane"); among the lanes
            // that hold the maximum the lowest expert index wins
            const unsigned int key = best >= 0.f ? __float_as_uint(best) + 1u : 0u;
            const unsigned int top = __reduce_max_sync(0xffffffffu, key);
            bi = __reduce_min_sync(0xffffffffu, key == top ? bi : 0x7fffffff);
            best = __uint_as_float(top - 1u);
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

// ---------------------------------------------------------------------------------------------
// Token permutation: histogram of expert ids, exclusive offsets, and for every expert the list of
// token rows it serves (slot order inside an expert is arbitrary: every (token, expert) product is
// computed independently of its slot).  Run by ONE block of at least E threads; also counts the
// distinct experts used.
// `counted`: the per-expert counts were accumulated in b.perm_cnt by permute_count_kernel (large calls);
// then this block only scans them, writes the offsets, the group list and b.perm_cur, clears b.perm_cnt
// for the next use and leaves the slot assignment to permute_scatter_kernel.
// The routing indices are read with ld.global.cg: when the block runs at the end of the router kernel
// they were written by other blocks of the same grid.
struct PermuteSmem {
    int cnt[kMaxExperts];
    int off[kMaxExperts + 1];
    int wtot[3][32];
};

__device__ void permute_block(const Shape& s, const Buffers& b, int layer, int n_pairs, int tok_cap, int counted, PermuteSmem& sm) {
    int* cnt = sm.cnt;
    int* off = sm.off;
    const int tid = threadIdx.x, E = s.E;
    if (counted) {
        for (int e = tid; e < E; e += blockDim.x) { cnt[e] = b.perm_cnt[e]; b.perm_cnt[e] = 0; }
    } else {
        for (int e = tid; e < E; e += blockDim.x) cnt[e] = 0;
        __syncthreads();
        for (int i = tid; i < n_pairs; i += blockDim.x) atomicAdd(&cnt[__ldcg(b.route_idx + i)], 1);
    }
    __syncthreads();
    // one expert per thread (E <= 1024): exclusive scans of the token counts (slot offsets), of the
    // group counts (positions in the group list) and of "has tokens" (distinct experts)
    {
        const int lane = tid & 31, warp = tid >> 5;
        const int c = tid < E ? cnt[tid] : 0;
        int inc[3] = {c, (c + tok_cap - 1) / tok_cap, c > 0 ? 1 : 0};
        const int own[3] = {inc[0], inc[1], inc[2]};
#pragma unroll
        for (int q = 0; q < 3; ++q) {
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int nb = __shfl_up_sync(0xffffffffu, inc[q], o);
                if (lane >= o) inc[q] += nb;
            }
            if (lane == 31) sm.wtot[q][warp] = inc[q];
        }
        __syncthreads();
        int base[3] = {0, 0, 0}, tot[3] = {0, 0, 0};
        for (int w = 0; w < 32; ++w)
#pragma unroll
            for (int q = 0; q < 3; ++q) {
                if (w < warp) base[q] += sm.wtot[q][w];
                tot[q] += sm.wtot[q][w];
            }
        if (tid < E) {
            const int o0 = base[0] + inc[0] - own[0];
            off[tid] = o0;
            // token groups for the expert kernels: (expert, first slot, tokens <= tok_cap, 0)
            int ng = base[1] + inc[1] - own[1];
            for (int t0 = 0; t0 < c; t0 += tok_cap, ++ng)
                reinterpret_cast<int4*>(b.groups)[ng] = make_int4(tid, o0 + t0, min(tok_cap, c - t0), 0);
        }
        if (tid == 0) {
            off[E] = tot[0];
            *b.n_groups = tot[1];
            b.active[layer] = tot[2];
        }
    }
    __syncthreads();
    for (int e = tid; e <= E; e += blockDim.x) b.expert_off[e] = off[e];
    if (counted) {
        for (int e = tid; e < E; e += blockDim.x) b.perm_cur[e] = off[e];
        return;
    }
    for (int e = tid; e < E; e += blockDim.x) cnt[e] = 0;
    __syncthreads();
    for (int i = tid; i < n_pairs; i += blockDim.x) {
        const int e = __ldcg(b.route_idx + i);
        const int slot = off[e] + atomicAdd(&cnt[e], 1);
        b.slot_token[slot] = i / s.k;
        b.slot_of[i] = slot;
    }
}

__global__ void __launch_bounds__(1024) permute_kernel(Shape s, Buffers b, int layer, int n_pairs, int tok_cap, int counted) {
    __shared__ PermuteSmem sm;
    pdl_wait();
    permute_block(s, b, layer, n_pairs, tok_cap, counted, sm);
}

// ---------------------------------------------------------------------------------------------
// One block per token row.  h2 = rms(x) * g (kept in fp32 for the gate, stored as a (hi, lo) bf16
// pair for the experts); z_e = <W_r[e], h2> accumulated in fp32 in a fixed order; pi = softmax(z); the k largest
// pi (ties: lower index) and their renormalised weights.
constexpr int kRouterCta = 1024;
constexpr int kRouterPer = 8;    // hidden <= 8192
// perm_cap > 0: the block that finishes last (counted in b.n_groups[1], which is zero between kernels) also
// runs the token permutation with groups of perm_cap tokens, which saves a kernel boundary per layer.
__global__ void __launch_bounds__(kRouterCta) router_kernel(Shape s, Buffers b, const __nv_bfloat16* gain,
                                                            const __nv_bfloat16* Wr, DebugTaps dbg, int layer, int n_tok,
                                                            int o_ksplit, int perm_cap) {
    // one column tile of activations: row 0 = hi, row 1 = lo of this token, rows 2..7 zero
    extern __shared__ __align__(16) unsigned char xt[];
    __shared__ float scratch[32];
    __shared__ float z[kMaxExperts];
    __shared__ float zp[kMaxExperts];     // partial logits of the K quarters: [quarter][expert]
    pdl_wait();
    const int t = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gid = lane >> 2, tig = lane & 3;
    const int H = s.H, E = s.E, k = s.k;
    const int xrow = x_row_bytes(H);

    // residual: x += W_o o, delivered as split-K partials that are added here in a fixed order
    // (all loads of a partial are issued before any store, so that they overlap)
    float v[kRouterPer];
    float ss = 0.f;
    const float* __restrict__ xin = b.x + (size_t)t * H;
#pragma unroll
    for (int i = 0; i < kRouterPer; ++i) {
        const int c = tid + i * kRouterCta;
        v[i] = c < H ? xin[c] : 0.f;
    }
    // (per column the loads of up to eight partials are issued before the first add: one memory round trip, not eight)
    for (int sp0 = 0; sp0 < o_ksplit; sp0 += 8) {
#pragma unroll
        for (int i = 0; i < kRouterPer; ++i) {
            const int c = tid + i * kRouterCta;
            if (c < H) {
                float pv[8];
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    pv[j] = sp0 + j < o_ksplit ? b.opart[((size_t)(sp0 + j) * n_tok + t) * H + c] : 0.f;
#pragma unroll
                for (int j = 0; j < 8; ++j) v[i] += pv[j];
            }
        }
    }
#pragma unroll
    for (int i = 0; i < kRouterPer; ++i) {
        const int c = tid + i * kRouterCta;
        if (c < H) {
            b.x[(size_t)t * H + c] = v[i];
            ss += v[i] * v[i];
        }
    }
    ss = block_sum(ss, scratch);
    const float r = rsqrtf(ss / (float)H + s.eps);
#pragma unroll
    for (int i = 0; i < kRouterPer; ++i) {
        const int c = tid + i * kRouterCta;
        if (c < H) {
            __nv_bfloat16 hi, lo;
            split_bf16(v[i] * r * __bfloat162float(gain[c]), hi, lo);
            b.h[(size_t)t * 2 * H + c] = hi;
            b.h[(size_t)t * 2 * H + H + c] = lo;
            reinterpret_cast<__nv_bfloat16*>(xt)[c] = hi;
            reinterpret_cast<__nv_bfloat16*>(xt + xrow)[c] = lo;
        }
    }
    for (int i = tid; i < 6 * (H / 8); i += kRouterCta) {
        const int rw = 2 + i / (H / 8), pc = i % (H / 8);
        *reinterpret_cast<uint4*>(xt + (size_t)rw * xrow + pc * 16) = make_uint4(0, 0, 0, 0);
    }
    __syncthreads();

    // gate logits with the streaming contraction: a warp task is 16 experts x one quarter of K,
    // columns 0/1 = hi/lo.  The (hi, lo) pair carries ~16 mantissa bits of h2, sums are fp32 and
    // the K quarters are added in a fixed order.
    const int n_rb = (E + 15) / 16;
    const int kq = n_rb <= 8 ? 4 : (n_rb <= 16 ? 2 : 1);
    const int spq = (H / 32) / kq;                              // slices per quarter (H is a multiple of 256)
    for (int task = warp; task < n_rb * kq; task += kRouterCta / 32) {
        const int rb = task / kq, q = task - rb * kq;
        const int r0 = min(rb * 16 + gid, E - 1), r1 = min(rb * 16 + gid + 8, E - 1);
        const size_t koff = (size_t)q * spq * 32;
        const __nv_bfloat16* wrow[1][2] = {{Wr + (size_t)r0 * H + koff + tig * 8, Wr + (size_t)r1 * H + koff + tig * 8}};
        float acc[1][1][4] = {{{0.f, 0.f, 0.f, 0.f}}};
        stream_mma<1, 1, 8>(wrow, spq, xt + (size_t)gid * xrow + koff * 2 + tig * 16, 8 * xrow, acc);
        if (tig == 0) {
            if (rb * 16 + gid < E) zp[q * E + rb * 16 + gid] = acc[0][0][0] + acc[0][0][1];
            if (rb * 16 + gid + 8 < E) zp[q * E + rb * 16 + gid + 8] = acc[0][0][2] + acc[0][0][3];
        }
    }
    __syncthreads();
    for (int e = tid; e < E; e += kRouterCta) {
        float acc = zp[e];
        for (int q = 1; q < kq; ++q) acc += zp[q * E + e];
        z[e] = acc;
    }
    __syncthreads();

    if (warp == 0) {
        route_select(z, s, b, dbg, layer, n_tok, t, lane);
        __threadfence();                 // this token's routing is visible to the whole device before the count below
    }
    if (perm_cap <= 0) return;
    __shared__ int is_last;
    __shared__ PermuteSmem perm_sm;
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const int prev = atomicAdd(b.n_groups + 1, 1);
        is_last = prev == n_tok - 1;
        if (is_last) b.n_groups[1] = 0;  // every block has counted: ready for the next launch
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    permute_block(s, b, layer, n_tok * k, perm_cap, 0, perm_sm);
}

// Large calls (tens of thousands of (token, expert) pairs) count and hand out the slots with many
// blocks: every block histograms its chunk of pairs in shared memory and adds it to the global
// counts; after the scan above, every block reserves a run of slots per expert with one atomic
// per (block, expert) and places its pairs inside the run.  Which slot a pair gets depends on
// scheduling; the results do not (every pair's product is computed on its own and combined per
// token in a fixed order).
constexpr int kPermChunk = 1024;     // pairs per block
__global__ void __launch_bounds__(1024) permute_count_kernel(Shape s, Buffers b, int n_pairs) {
    __shared__ int cnt[kMaxExperts];
    pdl_wait();
    const int tid = threadIdx.x, E = s.E;
    for (int e = tid; e < E; e += blockDim.x) cnt[e] = 0;
    __syncthreads();
    const int i0 = blockIdx.x * kPermChunk, i1 = min(n_pairs, i0 + kPermChunk);
    for (int i = i0 + tid; i < i1; i += blockDim.x) atomicAdd(&cnt[b.route_idx[i]], 1);
    __syncthreads();
    for (int e = tid; e < E; e += blockDim.x)
        if (cnt[e]) atomicAdd(&b.perm_cnt[e], cnt[e]);
}

__global__ void __launch_bounds__(1024) permute_scatter_kernel(Shape s, Buffers b, int n_pairs) {
    __shared__ int cnt[kMaxExperts];
    __shared__ int base[kMaxExperts];
    pdl_wait();
    const int tid = threadIdx.x, E = s.E;
    for (int e = tid; e < E; e += blockDim.x) cnt[e] = 0;
    __syncthreads();
    const int i0 = blockIdx.x * kPermChunk, i1 = min(n_pairs, i0 + kPermChunk);
    for (int i = i0 + tid; i < i1; i += blockDim.x) atomicAdd(&cnt[b.route_idx[i]], 1);
    __syncthreads();
    for (int e = tid; e < E; e += blockDim.x) {
        base[e] = cnt[e] ? atomicAdd(&b.perm_cur[e], cnt[e]) : 0;
        cnt[e] = 0;
    }
    __syncthreads();
    for (int i = i0 + tid; i < i1; i += blockDim.x) {
        const int e = b.route_idx[i];
        const int slot = base[e] + atomicAdd(&cnt[e], 1);
        b.slot_token[slot] = i / s.k;
        b.slot_of[i] = slot;
    }
}

static int launch_permute(const Shape& s, const Buffers& b, int layer, int n_pairs, int cap, cudaStream_t st) {
    if (n_pairs < 4 * kPermChunk) {
        launch_chained(permute_kernel, dim3(1), dim3(1024), 0, st, s, b, layer, n_pairs, cap, 0);
        return 1;
    }
    const int blocks = (n_pairs + kPermChunk - 1) / kPermChunk;
    launch_chained(permute_count_kernel, dim3(blocks), dim3(1024), 0, st, s, b, n_pairs);
    launch_chained(permute_kernel, dim3(1), dim3(1024), 0, st, s, b, layer, n_pairs, cap, 1);
    launch_chained(permute_scatter_kernel, dim3(blocks), dim3(1024), 0, st, s, b, n_pairs);
    return 3;
}

// ---------------------------------------------------------------------------------------------
// Grouped SwiGLU, first half: act[slot, i] = silu(<W_gate[e, i], h>) * <W_up[e, i], h>.
//
// Work is cut into units of 8 gate rows + the matching 8 up rows of one token group (an expert and
// at most `cap` of its tokens, listed by the permute kernel).  A unit is one MMA row tile: gate rows
// on MMA rows 0..7, up rows on rows 8..15, so silu(gate) * up pairs up inside a thread.  The grid is
// persistent (one CTA per SM); CTA c owns the contiguous range [c U / G, (c+1) U / G) of the U
// units, i.e. parts of two or three groups, and walks it group by group: the group's activation
// rows are put in shared memory, then warp w takes the group's units w, w + W, ...  Each warp
// streams its weight rows through its own cp.async ring, and the ring keeps filling across unit
// and group boundaries, so the stream into an SM only pauses while a group's activations load.
constexpr int kGuMaxWarps = 16;
constexpr int kExpMaxWarps = 12;

struct GuCursor {               // position of a warp in its sequence of (group, unit, slice)
    int g, u, sl;
    const __nv_bfloat16 *p0, *p1;
};

template <int NT>
__device__ __forceinline__ void gate_up_epilogue(const float (&acc)[NT][4], int m_here, int row, int I,
                                                 __nv_bfloat16* act_out, int tig) {
#pragma unroll
    for (int n = 0; n < NT; ++n) {
        const int t = n * 4 + tig;                 // columns 2t (hi) and 2t+1 (lo) of token t
        if (t < m_here) {
            const float gte = acc[n][0] + acc[n][1], up = acc[n][2] + acc[n][3];
            __nv_bfloat16* dst = act_out + (size_t)t * 2 * I + row;
            split_bf16(gte / (1.f + expf(-gte)) * up, dst[0], dst[I]);
        }
    }
}

// cp.async.wait_group wants an immediate; after unrolling `pending` is a constant.
__device__ __forceinline__ void cp_async_wait_n(int pending) {
    switch (pending) {
        case 0: cp_async_wait<0>(); break;
        case 1: cp_async_wait<1>(); break;
        case 2: cp_async_wait<2>(); break;
        case 3: cp_async_wait<3>(); break;
        case 4: cp_async_wait<4>(); break;
        case 5: cp_async_wait<5>(); break;
        case 6: cp_async_wait<6>(); break;
        case 7: cp_async_wait<7>(); break;
        case 8: cp_async_wait<8>(); break;
        case 9: cp_async_wait<9>(); break;
        case 10: cp_async_wait<10>(); break;
        case 11: cp_async_wait<11>(); break;
        case 12: cp_async_wait<12>(); break;
        case 13: cp_async_wait<13>(); break;
        case 14: cp_async_wait<14>(); break;
        default: cp_async_wait<15>(); break;
    }
}

// One unit's K loop: kGuBatch slices are consumed, then kGuBatch slices are requested back to back, so
// that every weight row is asked for in runs of kGuBatch x 64 contiguous bytes (measured per launch on
// the 48-layer decode step: one slice at a time 156 us, two 153 us, four 142-145 us, eight 145 us; a
// deeper ring with fewer warps was slower).  n_slices = H / 32 is a multiple of 8.
constexpr int kGuBatch = 4;
constexpr int kGuRing = kRing;                                // slices in flight per warp
constexpr int kGuRingWarpBytes = kGuRing * kRingStageBytes;
static_assert(kGuBatch <= kGuRing && 8 % kGuBatch == 0, "the batch must divide the slice count");
template <int NT, typename Issue>
__device__ __forceinline__ void gu_stream(const unsigned char* ring, int& ccount, int lane, const unsigned char* xs, int xrow,
                                          int n_slices, float (&acc)[NT][4], Issue& issue_next) {
    for (int sl = 0; sl < n_slices; sl += kGuBatch) {
#pragma unroll
        for (int b = 0; b < kGuBatch; ++b) {
            cp_async_wait_n(kGuRing - 1 - b);
            ring_consume<NT>(ring, ccount % kGuRing, lane, xs + (size_t)(sl + b) * 64, 8 * xrow, acc);
            ++ccount;
        }
#pragma unroll
        for (int b = 0; b < kGuBatch; ++b) issue_next();
    }
}

__global__ void __launch_bounds__(kGuMaxWarps * 32, 1) expert_gate_up_kernel(Shape s, Buffers b, const __nv_bfloat16* Wgu,
                                                                          int tok_cap) {
    extern __shared__ __align__(128) unsigned char smem[];
    pdl_wait();      // the group list comes from the permute kernel
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gid = lane >> 2, tig = lane & 3;
    const int H = s.H, I = s.I;
    const int n_warps = blockDim.x >> 5;
    const int xrow = x_row_bytes(H);
    unsigned char* xt = smem;
    unsigned char* ring = smem + (size_t)2 * tok_cap * xrow + (size_t)warp * kGuRingWarpBytes;
    const int4* groups = reinterpret_cast<const int4*>(b.groups);
    const int n_groups = *b.n_groups;
    const int upe = I / 8;                                   // units per group
    const long long total = (long long)n_groups * upe;
    const int u_begin = (int)(total * blockIdx.x / gridDim.x), u_end = (int)(total * (blockIdx.x + 1) / gridDim.x);
    if (u_begin >= u_end) return;
    const int g_first = u_begin / upe, g_last = (u_end - 1) / upe;
    const int n_slices = H / 32;

    auto seg_lo = [&](int g) { return max(u_begin, g * upe); };
    auto seg_hi = [&](int g) { return min(u_end, (g + 1) * upe); };
    // move the cursor to the warp's next unit at or after (g, u) and set its weight row pointers
    auto settle = [&](GuCursor& c) {
        while (c.g <= g_last && c.u >= seg_hi(c.g)) {
            ++c.g;
            if (c.g <= g_last) c.u = seg_lo(c.g) + warp;
        }
        if (c.g <= g_last) {
            const int e = groups[c.g].x;
            const int row = (c.u - c.g * upe) * 8 + gid;
            c.p0 = Wgu + ((size_t)e * 2 * I + row) * H + tig * 8;
            c.p1 = c.p0 + (size_t)I * H;
        }
    };
    GuCursor ic;
    ic.g = g_first; ic.u = seg_lo(g_first) + warp; ic.sl = 0; ic.p0 = ic.p1 = nullptr;
    settle(ic);
    int icount = 0, ccount = 0;
    auto issue_next = [&]() {                                // one slice (or nothing) and one commit group
        if (ic.g <= g_last) {
            ring_issue(ring, icount % kGuRing, lane, ic.p0 + (size_t)ic.sl * 32, ic.p1 + (size_t)ic.sl * 32);
            if (++ic.sl == n_slices) {
                ic.sl = 0;
                ic.u += n_warps;
                settle(ic);
            }
        }
        cp_async_commit();
        ++icount;
    };
#pragma unroll 1
    for (int i = 0; i < kGuRing; ++i) issue_next();

    const int pieces = H / 8;
    for (int g = g_first; g <= g_last; ++g) {
        const int4 grp = groups[g];                          // (expert, first slot, tokens, 0)
        const int m_here = grp.z;
        if (g > g_first) __syncthreads();                    // everyone is done with the previous group's rows
        const int cols_ld = (2 * m_here + 7) & ~7;           // column v = 2 * token + plane
        for (int i = tid; i < cols_ld * pieces; i += blockDim.x) {
            const int v = i / pieces, pc = i - v * pieces;
            uint4 val = make_uint4(0, 0, 0, 0);
            if ((v >> 1) < m_here)
                val = *reinterpret_cast<const uint4*>(b.h + ((size_t)b.slot_token[grp.y + (v >> 1)] * 2 + (v & 1)) * H +
                                                      pc * 8);
            *reinterpret_cast<uint4*>(xt + (size_t)v * xrow + pc * 16) = val;
        }
        __syncthreads();
        const unsigned char* xs = xt + (size_t)gid * xrow + tig * 16;
        __nv_bfloat16* act_out = b.act + (size_t)grp.y * 2 * I;
        const int nt = (m_here + 3) >> 2;
        for (int u = seg_lo(g) + warp; u < seg_hi(g); u += n_warps) {
            const int row = (u - g * upe) * 8 + gid;
            if (nt == 1) {
                float acc[1][4] = {{0.f, 0.f, 0.f, 0.f}};
                gu_stream<1>(ring, ccount, lane, xs, xrow, n_slices, acc, issue_next);
                gate_up_epilogue<1>(acc, m_here, row, I, act_out, tig);
            } else if (nt == 2) {
                float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
                gu_stream<2>(ring, ccount, lane, xs, xrow, n_slices, acc, issue_next);
                gate_up_epilogue<2>(acc, m_here, row, I, act_out, tig);
            } else {
                float acc[4][4];
#pragma unroll
                for (int n = 0; n < 4; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
                gu_stream<4>(ring, ccount, lane, xs, xrow, n_slices, acc, issue_next);
                gate_up_epilogue<4>(acc, m_here, row, I, act_out, tig);
            }
        }
    }
    cp_async_wait<0>();
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
    pdl_wait();
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
    pdl_wait();
    const int t = blockIdx.x, tid = threadIdx.x, H = s.H, k = s.k;
    if (tid < k) { slots[tid] = b.slot_of[(size_t)t * k + tid]; ws[tid] = b.route_w[(size_t)t * k + tid]; }
    __syncthreads();
    // four columns per thread and visit; the k expert rows are fetched eight at a time so that the
    // loads are in flight together, and added in the order j = 0, 1, ...
    constexpr int kVec = kRowMaxPer / 4;
    float4 v[kVec];
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < kVec; ++i) {
        const int c = (tid + i * kRouterThreads) * 4;
        v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < H) {
            float4 acc = *reinterpret_cast<const float4*>(b.x + (size_t)t * H + c);
            for (int j0 = 0; j0 < k; j0 += 8) {
                float4 yv[8];
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    yv[j] = j0 + j < k ? *reinterpret_cast<const float4*>(b.y + (size_t)slots[j0 + j] * H + c)
                                       : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float wj = j0 + j < k ? ws[j0 + j] : 0.f;
                    acc.x = fmaf(wj, yv[j].x, acc.x); acc.y = fmaf(wj, yv[j].y, acc.y);
                    acc.z = fmaf(wj, yv[j].z, acc.z); acc.w = fmaf(wj, yv[j].w, acc.w);
                }
            }
            v[i] = acc;
            *reinterpret_cast<float4*>(b.x + (size_t)t * H + c) = acc;
            if (hidden_tap) *reinterpret_cast<float4*>(hidden_tap + (size_t)t * H + c) = acc;
            ss += acc.x * acc.x + acc.y * acc.y + acc.z * acc.z + acc.w * acc.w;
        }
    }
    ss = block_sum(ss, scratch);
    const float r = rsqrtf(ss / (float)H + s.eps);
#pragma unroll
    for (int i = 0; i < kVec; ++i) {
        const int c = (tid + i * kRouterThreads) * 4;
        if (c < H) {
            __nv_bfloat16* hi = b.h + (size_t)t * 2 * H + c;
            const float e[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
#pragma unroll
            for (int q = 0; q < 4; ++q) split_bf16(e[q] * r * __bfloat162float(next_gain[c + q]), hi[q], hi[H + q]);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Prefill-sized calls split the router in three: residual + RMSNorm here, the gate logits as one
// tensor-core contraction over all token rows, and the selection below.
__global__ void __launch_bounds__(kRouterThreads) resid_norm_kernel(Shape s, Buffers b, const __nv_bfloat16* gain, int n_tok,
                                                                   int o_ksplit) {
    __shared__ float scratch[32];
    pdl_wait();
    // four consecutive columns per thread and visit (hidden is a multiple of 256): 16-byte loads and stores
    constexpr int kVec = kRowMaxPer / 4;
    const int t = blockIdx.x, tid = threadIdx.x, H = s.H;
    float4 v[kVec];
    const float* __restrict__ xin = b.x + (size_t)t * H;
#pragma unroll
    for (int i = 0; i < kVec; ++i) {
        const int c = (tid + i * kRouterThreads) * 4;
        v[i] = c < H ? *reinterpret_cast<const float4*>(xin + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    // per column group the loads of up to eight partials are issued before the first add
    for (int sp0 = 0; sp0 < o_ksplit; sp0 += 8) {
#pragma unroll
        for (int i = 0; i < kVec; ++i) {
            const int c = (tid + i * kRouterThreads) * 4;
            if (c < H) {
                float4 pv[8];
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    pv[j] = sp0 + j < o_ksplit ? *reinterpret_cast<const float4*>(b.opart + ((size_t)(sp0 + j) * n_tok + t) * H + c)
                                               : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int j = 0; j < 8; ++j) { v[i].x += pv[j].x; v[i].y += pv[j].y; v[i].z += pv[j].z; v[i].w += pv[j].w; }
            }
        }
    }
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < kVec; ++i) {
        const int c = (tid + i * kRouterThreads) * 4;
        if (c < H) {
            *reinterpret_cast<float4*>(b.x + (size_t)t * H + c) = v[i];
            ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
        }
    }
    ss = block_sum(ss, scratch);
    const float r = rsqrtf(ss / (float)H + s.eps);
#pragma unroll
    for (int i = 0; i < kVec; ++i) {
        const int c = (tid + i * kRouterThreads) * 4;
        if (c < H) {
            const uint2 gw = *reinterpret_cast<const uint2*>(gain + c);
            const float e0 = v[i].x * r * bf16_lo(gw.x), e1 = v[i].y * r * bf16_hi(gw.x);
            const float e2 = v[i].z * r * bf16_lo(gw.y), e3 = v[i].w * r * bf16_hi(gw.y);
            const uint32_t h0 = pack_bf16(e0, e1), h1 = pack_bf16(e2, e3);
            const uint32_t l0 = pack_bf16(e0 - bf16_lo(h0), e1 - bf16_hi(h0)), l1 = pack_bf16(e2 - bf16_lo(h1), e3 - bf16_hi(h1));
            __nv_bfloat16* hrow = b.h + (size_t)t * 2 * H + c;
            *reinterpret_cast<uint2*>(hrow) = make_uint2(h0, h1);
            *reinterpret_cast<uint2*>(hrow + H) = make_uint2(l0, l1);
        }
    }
}

// One warp per token row: gate logits (fp32, from the contraction: n_parts split-K partials
// [part][n_tok][E], added in a fixed order) -> routing.  perm_cap > 0: the block that finishes last also
// runs the token permutation (as in router_kernel).
constexpr int kSelectWarps = 32;
__global__ void __launch_bounds__(kSelectWarps * 32) route_select_kernel(Shape s, Buffers b, DebugTaps dbg, int layer, int n_tok,
                                                                         int n_parts, int perm_cap) {
    extern __shared__ float zs[];     // [warps][E]
    pdl_wait();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int t = blockIdx.x * kSelectWarps + warp;
    if (t < n_tok) {
        float* z = zs + (size_t)warp * s.E;
        const size_t part_stride = (size_t)n_tok * s.E;
        for (int e0 = lane; e0 < s.E; e0 += 4 * 32) {       // four experts per lane and pass: their partials load together
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            for (int sp0 = 0; sp0 < n_parts; sp0 += 8) {
                float pv[8][4];
#pragma unroll
                for (int j = 0; j < 8; ++j)
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int e = e0 + 32 * q;
                        pv[j][q] = (sp0 + j < n_parts && e < s.E) ? b.rlogits[(size_t)(sp0 + j) * part_stride + (size_t)t * s.E + e] : 0.f;
                    }
#pragma unroll
                for (int j = 0; j < 8; ++j)
#pragma unroll
                    for (int q = 0; q < 4; ++q) acc[q] += pv[j][q];
            }
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (e0 + 32 * q < s.E) z[e0 + 32 * q] = acc[q];
        }
        __syncwarp();
        route_select(z, s, b, dbg, layer, n_tok, t, lane);
    }
    if (perm_cap <= 0) return;
    __shared__ int is_last;
    __shared__ PermuteSmem perm_sm;
    __syncthreads();                     // the block's routing has been written ...
    if (tid == 0) {
        __threadfence();                 // ... and is visible to the whole device before the count below
        const int prev = atomicAdd(b.n_groups + 1, 1);
        is_last = prev == (int)gridDim.x - 1;
        if (is_last) b.n_groups[1] = 0;  // every block has counted: ready for the next launch
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    permute_block(s, b, layer, n_tok * s.k, perm_cap, 0, perm_sm);
}

int launch_resid_norm(const Shape& s, const Buffers& b, const LayerW& w, int n_tok, int o_ksplit, cudaStream_t st) {
    launch_chained(resid_norm_kernel, dim3(n_tok), dim3(kRouterThreads), 0, st, s, b, w.mlp_norm, n_tok, o_ksplit);
    return 1;
}

static void expert_plan(const Shape& s, int n_tok, int* cap, int* warps);
int launch_route_select(const Shape& s, const Buffers& b, const DebugTaps& dbg, int layer, int n_tok, int group_cap, int n_parts,
                        cudaStream_t st) {
    int cap = group_cap;                                 // > 0: the tensor-core expert path wants one 128-row tile per group
    if (cap <= 0) {
        int warps;
        expert_plan(s, n_tok, &cap, &warps);
    }
    const bool fused = n_tok * s.k < 4 * kPermChunk;     // small permutations run in the selection's last block
    launch_chained(route_select_kernel, dim3((n_tok + kSelectWarps - 1) / kSelectWarps), dim3(kSelectWarps * 32),
                   (size_t)kSelectWarps * s.E * sizeof(float), st, s, b, dbg, layer, n_tok, n_parts, fused ? cap : 0);
    return fused ? 1 : 1 + launch_permute(s, b, layer, n_tok * s.k, cap, st);
}

// Tokens per group (4 per column tile); experts with more tokens are cut into several groups and
// stream their weights once per group.  `warps`: width of the gate/up CTA, limited by what is left
// of shared memory after the group's activation rows.
static void expert_plan(const Shape& s, int n_tok, int* cap, int* warps) {
    const double avg = (double)n_tok * s.k / s.E;
    *cap = avg <= 5.0 ? 8 : 16;
    while ((size_t)*cap * 2 * x_row_bytes(s.H) > 140u * 1024u && *cap > 4) *cap /= 2;
    const size_t left = 227u * 1024u - 1024u - (size_t)*cap * 2 * x_row_bytes(s.H);
    int w = (int)(left / kGuRingWarpBytes);
    *warps = w > kGuMaxWarps ? kGuMaxWarps : (w < 1 ? 1 : w);
}

// ---------------------------------------------------------------------------------------------
int launch_router(const Shape& s, const Buffers& b, const LayerW& w, const DebugTaps& dbg, int layer, int n_tok,
                  int group_cap, int o_ksplit, cudaStream_t st) {
    int cap, warps;
    expert_plan(s, n_tok, &cap, &warps);
    if (group_cap > 0) cap = group_cap;          // the tensor-core expert path wants one 128-row tile per group
    const bool fused = n_tok * s.k < 4 * kPermChunk;   // small permutations run in the router's last block
    launch_chained(router_kernel, dim3(n_tok), dim3(kRouterCta), 8 * x_row_bytes(s.H), st, s, b, w.mlp_norm, w.router, dbg, layer, n_tok,
                   o_ksplit, fused ? cap : 0);
    return fused ? 1 : 1 + launch_permute(s, b, layer, n_tok * s.k, cap, st);
}

int launch_gate_up(const Shape& s, const Buffers& b, const LayerW& w, int n_tok, int sm_count, cudaStream_t st) {
    int cap, warps;
    expert_plan(s, n_tok, &cap, &warps);
    const size_t smem = (size_t)cap * 2 * x_row_bytes(s.H) + (size_t)warps * kGuRingWarpBytes;
    launch_chained(expert_gate_up_kernel, dim3(sm_count), dim3(warps * 32), smem, st, s, b, w.w_gate_up, cap);
    return 1;
}

int launch_down(const Shape& s, const Buffers& b, const LayerW& w, int n_tok, cudaStream_t st) {
    int cap, warps;
    expert_plan(s, n_tok, &cap, &warps);
    const int w2 = cap > 8 ? 8 : 4;
    dim3 g2((s.H / 32 + w2 - 1) / w2, s.E);
    launch_chained(expert_down_kernel, dim3(g2), dim3(w2 * 32), (size_t)cap * 2 * x_row_bytes(s.I), st, s, b, w.w_down, cap);
    return 1;
}

int launch_combine(const Shape& s, const Buffers& b, const __nv_bfloat16* next_gain, float* hidden_tap, int n_tok,
                   cudaStream_t st) {
    launch_chained(combine_kernel, dim3(n_tok), dim3(kRouterThreads), 0, st, s, b, next_gain, hidden_tap);
    return 1;
}

cudaError_t init_moe_kernels() {
    cudaError_t e = cudaFuncSetAttribute(expert_gate_up_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(expert_down_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(route_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSelectWarps * kMaxExperts * (int)sizeof(float));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(router_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 8 * x_row_bytes(8192));
}

}  // namespace mars
