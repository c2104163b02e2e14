// log-softmax + greedy / nucleus sampling over one row of logits per emitting sequence.
//
// Nucleus selection needs no sort: the weights e_v = exp((l_v - max) / T) are positive floats, so
// their bit patterns order like the values.  A radix search (11 bits per pass over the key bits that
// differ between tokens) over per-bucket MASS histograms finds the weight of the token at which the
// descending cumulative mass reaches top_p; masses are accumulated in 2^-40 fixed point with integer
// atomics, which makes the result independent of the order in which threads add.  Tokens above that weight are in the
// nucleus, tokens equal to it enter in ascending id until the mass is reached.  The token is then
// drawn by inverting the cumulative distribution of the nucleus taken in ascending token id.
#include "common.cuh"
#include "kernels.h"

namespace mars {

constexpr int kSampleThreads = 1024;
constexpr int kBins = 2048;
constexpr double kFix = 1099511627776.0;  // 2^40

// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): first output word.
__device__ __forceinline__ uint32_t philox_first_word(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                                      uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t h0 = __umulhi(0xD2511F53u, c0), l0 = 0xD2511F53u * c0;
        const uint32_t h1 = __umulhi(0xCD9E8D57u, c2), l1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = h1 ^ c1 ^ k0, n2 = h0 ^ c3 ^ k1;
        c0 = n0; c1 = l1; c2 = n2; c3 = l0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return c0;
}

// floor(e * 2^40) for 0 <= e <= 1, in integer arithmetic: a float is mant * 2^(ex - 150), so the fixed-point
// value is the 24-bit mantissa shifted by ex - 110 (exactly what the conversion through fp64 would give).
__device__ __forceinline__ unsigned long long to_fix(float e) {
    const unsigned int key = __float_as_uint(e);
    const int ex = (int)(key >> 23);
    const unsigned long long mant = (key & 0x7fffffu) | (ex ? 0x800000u : 0u);
    const int sh = (ex ? ex : 1) - 110;
    return sh >= 0 ? mant << sh : (sh > -24 ? mant >> -sh : 0ull);
}

// Block-wide exclusive scan of one 64-bit value per thread (fixed order); returns this thread's
// exclusive prefix and writes the block total to *total.
__device__ __forceinline__ unsigned long long block_excl_scan(unsigned long long v, unsigned long long* warp_tot,
                                                              unsigned long long* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    __syncthreads();
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    unsigned long long base = 0, tot = 0;
    for (int w = 0; w < kSampleThreads / 32; ++w) {
        if (w < warp) base += warp_tot[w];
        tot += warp_tot[w];
    }
    *total = tot;
    return base + inc - v;
}

// Four consecutive logits starting at id i (a multiple of 4): one 16-byte load where the row allows it.
struct Quad { float x[4]; int n; };
__device__ __forceinline__ Quad load_quad(const float* l, int i, int V, bool vec) {
    Quad q;
    if (vec) {
        const float4 t = *reinterpret_cast<const float4*>(l + i);
        q.x[0] = t.x; q.x[1] = t.y; q.x[2] = t.z; q.x[3] = t.w; q.n = 4;
    } else {
        q.n = min(4, V - i);
#pragma unroll
        for (int j = 0; j < 4; ++j) q.x[j] = j < q.n ? l[i + j] : 0.f;
    }
    return q;
}

// fn(id, quad) for the quads at ids first, first + stride, ... below end; four loads are in flight per thread
// (a pass is otherwise bound by the latency of one L2 load per thread and iteration).
template <typename F>
__device__ __forceinline__ void sweep(const float* src, int V, bool vec, int first, int end, int stride, F&& fn) {
    int i = first;
    for (; i + 3 * stride < end; i += 4 * stride) {
        Quad q[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) q[u] = load_quad(src, i + u * stride, V, vec);
#pragma unroll
        for (int u = 0; u < 4; ++u) fn(i + u * stride, q[u]);
    }
    for (; i < end; i += stride) fn(i, load_quad(src, i, V, vec));
}

// ---- a row is shared by the C blocks of a cluster (C = 1 or 2): block r owns the r-th part of the ids, partial results
// cross through distributed shared memory, and both blocks take every decision from the same combined numbers.
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
template <int C>
__device__ __forceinline__ void cluster_sync() {       // also a barrier of the block
    if (C > 1) {
        asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    } else {
        __syncthreads();
    }
}
__device__ __forceinline__ uint32_t peer_smem(const void* p, uint32_t rank) {   // the same variable in block `rank`
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
    return r;
}
__device__ __forceinline__ uint32_t ld_peer_u32(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long ld_peer_u64(uint32_t a) {
    unsigned long long v;
    asm volatile("ld.shared::cluster.u64 %0, [%1];" : "=l"(v) : "r"(a) : "memory");
    return v;
}

// What a block shows its peer.
struct SampleXchg {
    float mx; int am;
    double zs;
    unsigned long long part;
    unsigned int k_or, k_and;
    unsigned long long w_above[32];
    unsigned int w_ties[32];
    int sel_token;
};

// CACHED: the weights e_v are written to b.expw in the pass that sums them and the later passes read them back
// (expf is a large part of a pass); otherwise every pass recomputes them from the logits.  Both give the same bits.
template <bool CACHED, int C>
__global__ void __launch_bounds__(kSampleThreads) sample_kernel(Shape s, Buffers b, StepLayout lay, int32_t* out_tokens,
                                                                float* out_logprobs, float* nucleus_mass) {
    // mass histogram of a radix pass as (low word, high word): 32-bit shared-memory atomics with an explicit carry
    __shared__ __align__(8) unsigned int hist_lo[kBins], hist_hi[kBins];
    __shared__ unsigned long long warp_tot[kSampleThreads / 32];
    __shared__ float red_f[32];
    __shared__ int red_i[32];
    __shared__ double red_d[32];
    __shared__ unsigned int red_u[2][32];
    __shared__ unsigned int sel_prefix;
    __shared__ unsigned long long sel_above;
    __shared__ SampleXchg xc;
    __shared__ unsigned long long all_above[32 * C];   // the warps' ranges of all blocks, in id order
    __shared__ unsigned int all_ties[32 * C];
    pdl_wait();

    const uint32_t rank = C > 1 ? cluster_rank() : 0u;
    const int row = blockIdx.x / C, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int V = s.V;
    const float* l = b.logits + (size_t)row * V;
    float* ew = CACHED ? b.expw + (size_t)row * V : nullptr;
    const bool vec = (V & 3) == 0 && (reinterpret_cast<uintptr_t>(l) & 15) == 0 &&
                     (!CACHED || (reinterpret_cast<uintptr_t>(ew) & 15) == 0);
    const int32_t* hdr = b.step;
    const bool greedy = hdr[H_GREEDY] != 0;
    const float T = greedy ? 1.f : __int_as_float(hdr[H_TEMPERATURE]);
    const float top_p = __int_as_float(hdr[H_TOP_P]);
    const float inv_t = 1.f / T;
    // this block's ids [id_lo, id_hi): whole groups of four
    const int groups = (V + 3) >> 2, gpc = (groups + C - 1) / C;
    const int id_lo = min(groups, (int)rank * gpc) * 4, id_hi = min(groups, ((int)rank + 1) * gpc) * 4;

    // max and argmax (lowest id on ties)
    float mx = -INFINITY;
    int am = 0x7fffffff;
    sweep(l, V, vec, id_lo + tid * 4, id_hi, kSampleThreads * 4, [&](int i, const Quad& q) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (j < q.n && q.x[j] > mx) { mx = q.x[j]; am = i + j; }
    });
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ox = __shfl_xor_sync(0xffffffffu, mx, o);
        const int oi = __shfl_xor_sync(0xffffffffu, am, o);
        if (ox > mx || (ox == mx && oi < am)) { mx = ox; am = oi; }
    }
    if (lane == 0) { red_f[warp] = mx; red_i[warp] = am; }
    __syncthreads();
    mx = red_f[0]; am = red_i[0];
    for (int w = 1; w < kSampleThreads / 32; ++w)
        if (red_f[w] > mx || (red_f[w] == mx && red_i[w] < am)) { mx = red_f[w]; am = red_i[w]; }
    if (C > 1) {
        if (tid == 0) { xc.mx = mx; xc.am = am; }
        cluster_sync<C>();
        const float ox = __uint_as_float(ld_peer_u32(peer_smem(&xc.mx, rank ^ 1u)));
        const int oi = (int)ld_peer_u32(peer_smem(&xc.am, rank ^ 1u));
        if (ox > mx || (ox == mx && oi < am)) { mx = ox; am = oi; }
    }

    // One pass for Z = sum exp((l - max) / T) (fp32 terms, fp64 sum in a fixed order), the total mass in fixed
    // point, and which key bits differ at all: near-flat logits share their sign, most of the exponent and
    // often some mantissa bits, and a radix digit taken from shared bits would send every token to the same
    // bucket (one hot shared-memory atomic).
    double zs = 0.0;
    unsigned long long part = 0;
    unsigned int k_or = 0u, k_and = 0xffffffffu;
    sweep(l, V, vec, id_lo + tid * 4, id_hi, kSampleThreads * 4, [&](int i, const Quad& q) {
        float ev[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            ev[j] = 0.f;
            if (j < q.n) {
                const float e = expf((q.x[j] - mx) * inv_t);
                ev[j] = e;
                zs += (double)e;
                part += to_fix(e);
                k_or |= __float_as_uint(e);
                k_and &= __float_as_uint(e);
            }
        }
        if (CACHED) {
            if (vec) *reinterpret_cast<float4*>(ew + i) = make_float4(ev[0], ev[1], ev[2], ev[3]);
            else
                for (int j = 0; j < q.n; ++j) ew[i + j] = ev[j];
        }
    });
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) zs += __shfl_xor_sync(0xffffffffu, zs, o);
    k_or = __reduce_or_sync(0xffffffffu, k_or);
    k_and = __reduce_and_sync(0xffffffffu, k_and);
    if (lane == 0) { red_d[warp] = zs; red_u[0][warp] = k_or; red_u[1][warp] = k_and; }
    unsigned long long z_fix;
    block_excl_scan(part, warp_tot, &z_fix);          // (its barriers also publish red_d and red_u)
    double Z = 0.0;
    for (int w = 0; w < kSampleThreads / 32; ++w) { Z += red_d[w]; k_or |= red_u[0][w]; k_and &= red_u[1][w]; }
    if (C > 1) {
        if (tid == 0) { xc.zs = Z; xc.part = z_fix; xc.k_or = k_or; xc.k_and = k_and; }
        cluster_sync<C>();
        const double oz = __longlong_as_double((long long)ld_peer_u64(peer_smem(&xc.zs, rank ^ 1u)));
        Z = rank == 0 ? Z + oz : oz + Z;               // block 0's part first, in both blocks
        z_fix += ld_peer_u64(peer_smem(&xc.part, rank ^ 1u));
        k_or |= ld_peer_u32(peer_smem(&xc.k_or, rank ^ 1u));
        k_and &= ld_peer_u32(peer_smem(&xc.k_and, rank ^ 1u));
    }
    const float log_z = (float)log(Z);

    if (greedy) {
        if (tid == 0 && rank == 0) {
            out_tokens[row] = am < V ? am : 0;   // (no logit compared greater than -inf: a row of NaN)
            out_logprobs[row] = -log_z;     // (l_max - max) / 1 - log Z
            if (nucleus_mass) nucleus_mass[row] = 1.f;
        }
        if (C > 1) cluster_sync<C>();       // the peer may still be reading this block's shared memory
        return;
    }

    // ---- nucleus threshold: radix search on the bit pattern of e_v, by mass
    const bool everything = top_p >= 1.f;
    unsigned long long target = (unsigned long long)((double)top_p * (double)z_fix);
    if (target < 1) target = 1;
    if (target > z_fix) target = z_fix;

    const unsigned int differ = k_or ^ k_and;
    int remaining = differ ? 32 - __clz(differ) : 0;  // low bits that vary (the sign bit never does: <= 31)
    unsigned int prefix = k_and >> remaining;          // the shared high bits
    unsigned long long above = 0;                      // mass of buckets strictly above the selected one
    if (!everything) {
        while (remaining > 0) {
            const int wd = remaining < 11 ? remaining : 11, sh = remaining - wd;
            for (int i = tid; i < kBins; i += kSampleThreads) { hist_lo[i] = 0u; hist_hi[i] = 0u; }
            if (tid == 0) { sel_prefix = prefix << wd; sel_above = above; }
            __syncthreads();
            sweep(CACHED ? ew : l, V, vec, id_lo + tid * 4, id_hi, kSampleThreads * 4, [&](int, const Quad& q) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float e = CACHED ? q.x[j] : expf((q.x[j] - mx) * inv_t);
                    const unsigned int key = __float_as_uint(e);
                    if (j < q.n && (key >> (sh + wd)) == prefix) {
                        const unsigned long long f = to_fix(e);
                        const unsigned int bin = (key >> sh) & ((1u << wd) - 1u), lo = (unsigned int)f;
                        unsigned int hi = (unsigned int)(f >> 32);
                        if (lo) hi += (unsigned int)(atomicAdd(&hist_lo[bin], lo) + lo < lo);   // the carry of this add
                        if (hi) atomicAdd(&hist_hi[bin], hi);
                    }
                }
            });
            cluster_sync<C>();
            // descending scan over the buckets of all blocks, two per thread
            const int b0 = kBins - 1 - 2 * tid;
            unsigned long long h0 = ((unsigned long long)hist_hi[b0] << 32) | hist_lo[b0];
            unsigned long long h1 = ((unsigned long long)hist_hi[b0 - 1] << 32) | hist_lo[b0 - 1];
            if (C > 1) {
                // bins b0 - 1 and b0 are adjacent words, b0 - 1 even: one 8-byte load per array
                const unsigned long long plo = ld_peer_u64(peer_smem(&hist_lo[b0 - 1], rank ^ 1u));
                const unsigned long long phi = ld_peer_u64(peer_smem(&hist_hi[b0 - 1], rank ^ 1u));
                h0 += ((phi >> 32) << 32) | (plo >> 32);
                h1 += ((phi & 0xffffffffull) << 32) | (plo & 0xffffffffull);
            }
            unsigned long long pass_total;
            const unsigned long long before = above + block_excl_scan(h0 + h1, warp_tot, &pass_total);
            if (before < target && before + h0 >= target) {
                sel_prefix = (prefix << wd) | (unsigned int)b0;
                sel_above = before;
            } else if (before + h0 < target && before + h0 + h1 >= target) {
                sel_prefix = (prefix << wd) | (unsigned int)(b0 - 1);
                sel_above = before + h0;
            }
            cluster_sync<C>();                          // the peer has read this block's histogram; sel_* are published
            prefix = sel_prefix;
            above = sel_above;
            remaining = sh;
            __syncthreads();
        }
    }
    // threshold weight: key == prefix.  Ties enter in ascending id until the mass is reached; with top_p >= 1
    // every token of positive weight is in (threshold key 0, no ties wanted).
    const unsigned int tkey = everything ? 0u : prefix;
    const unsigned long long q_fix = everything ? 0ull : to_fix(__uint_as_float(tkey));
    unsigned long long need_ties = 0;
    if (!everything) need_ties = q_fix > 0 ? (target - above + q_fix - 1) / q_fix : 0xffffffffull;

    // ---- the nucleus in ascending token id: every warp owns a contiguous range of ids, read in 512-byte slabs.  One
    // pass gives every warp the mass above the threshold and the number of ties in its range; ties all weigh
    // q_fix, so the range's nucleus mass follows from how many ties are still wanted when the range begins.
    const int g_first = id_lo >> 2, g_last = id_hi >> 2, gpw = (g_last - g_first + 31) >> 5;   // groups per warp
    const int g_begin = min(g_last, g_first + warp * gpw), g_end = min(g_last, g_begin + gpw);
    unsigned long long m_above = 0;
    unsigned int n_ties = 0;
    sweep(CACHED ? ew : l, V, vec, (g_begin + lane) * 4, g_end * 4, 128, [&](int, const Quad& q) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (j < q.n) {
                const float e = CACHED ? q.x[j] : expf((q.x[j] - mx) * inv_t);
                const unsigned int key = __float_as_uint(e);
                if (key > tkey) m_above += to_fix(e);
                n_ties += key == tkey;
            }
    });
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m_above += __shfl_xor_sync(0xffffffffu, m_above, o);
    n_ties = __reduce_add_sync(0xffffffffu, n_ties);
    if (lane == 0) { xc.w_above[warp] = m_above; xc.w_ties[warp] = n_ties; }
    if (tid == 0) xc.sel_token = -1;
    cluster_sync<C>();
    if (tid < 32 * C) {                                  // all ranges in id order: block 0's warps, then block 1's
        const uint32_t src = (uint32_t)tid >> 5;
        const int w = tid & 31;
        if (C == 1 || src == rank) {
            all_above[tid] = xc.w_above[w];
            all_ties[tid] = xc.w_ties[w];
        } else {
            all_above[tid] = ld_peer_u64(peer_smem(&xc.w_above[w], src));
            all_ties[tid] = ld_peer_u32(peer_smem(&xc.w_ties[w], src));
        }
    }
    __syncthreads();

    // uniform in (0, 1) from the counter-based generator
    const uint32_t slot = (uint32_t)b.step[lay.emit_slot + row];
    const uint32_t x0 = philox_first_word((uint32_t)hdr[H_STEP_LO], (uint32_t)hdr[H_STEP_HI], slot, 0u,
                                          (uint32_t)hdr[H_SEED_LO], (uint32_t)hdr[H_SEED_HI]);
    const double u = ((double)(x0 >> 8) + 0.5) * (1.0 / 16777216.0);

    // every thread: the ranges' nucleus masses in id order, the total, and where this warp's range starts
    unsigned long long mass_s = 0, my_base = 0, my_mass = 0, ties_seen = 0, my_tie_base = 0;
    const int my_range = (int)rank * 32 + warp;
    for (int w = 0; w < 32 * C; ++w) {
        const unsigned long long want = need_ties > ties_seen ? need_ties - ties_seen : 0ull;
        const unsigned long long m = all_above[w] + (want < all_ties[w] ? want : (unsigned long long)all_ties[w]) * q_fix;
        if (w == my_range) { my_base = mass_s; my_mass = m; my_tie_base = ties_seen; }
        mass_s += m;
        ties_seen += all_ties[w];
    }
    const double thr = u * (double)mass_s;     // first id whose cumulative mass exceeds thr

    if ((double)my_base <= thr && (double)(my_base + my_mass) > thr) {
        // this warp's range holds the token: walk it slab by slab with a warp-wide scan of the lanes' masses
        unsigned long long cum = my_base, rnk = my_tie_base;
        for (int g0 = g_begin; g0 < g_end; g0 += 32) {
            const int g = g0 + lane;
            Quad q;
            q.n = 0;
            if (g < g_end) q = load_quad(CACHED ? ew : l, g * 4, V, vec);
            unsigned long long fx[4];
            unsigned int tie_mask = 0, lane_ties = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                fx[j] = 0;
                if (j < q.n) {
                    const float e = CACHED ? q.x[j] : expf((q.x[j] - mx) * inv_t);
                    const unsigned int key = __float_as_uint(e);
                    if (key > tkey) fx[j] = to_fix(e);
                    else if (key == tkey) { tie_mask |= 1u << j; ++lane_ties; }
                }
            }
            // ranks of this lane's ties: ties of the lower lanes of the slab come first
            unsigned int tie_incl = lane_ties;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int n = __shfl_up_sync(0xffffffffu, tie_incl, o);
                if (lane >= o) tie_incl += n;
            }
            unsigned long long r = rnk + tie_incl - lane_ties, lane_mass = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (tie_mask >> j & 1) { if (r < need_ties) fx[j] = q_fix; ++r; }
                lane_mass += fx[j];
            }
            unsigned long long incl = lane_mass;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned long long n = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += n;
            }
            const unsigned int hit = __ballot_sync(0xffffffffu, (double)(cum + incl) > thr);
            if (hit) {
                if (lane == __ffs(hit) - 1) {
                    unsigned long long c = cum + incl - lane_mass;
                    int tok = -1;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {              // the first element whose cumulative mass crosses
                        c += fx[j];
                        if (tok < 0 && fx[j] > 0 && (double)c > thr) tok = g * 4 + j;
                    }
                    xc.sel_token = tok;
                }
                break;
            }
            cum += __shfl_sync(0xffffffffu, incl, 31);
            rnk += __shfl_sync(0xffffffffu, tie_incl, 31);
        }
    }
    cluster_sync<C>();
    if (tid == 0 && rank == 0) {
        int tok = xc.sel_token;
        if (C > 1 && tok < 0) tok = (int)ld_peer_u32(peer_smem(&xc.sel_token, 1u));
        if (tok < 0) tok = am;   // cannot happen while mass_s > 0; keeps the output defined
        if (tok < 0 || tok >= V) tok = 0;   // a row of NaN has no maximum either: stay inside the row
        out_tokens[row] = tok;
        out_logprobs[row] = (l[tok] - mx) * inv_t - log_z;
        if (nucleus_mass) nucleus_mass[row] = (float)((double)mass_s / (double)z_fix);
    }
    if (C > 1) cluster_sync<C>();           // block 0 may still be reading block 1's shared memory
}

// Launch with programmatic stream serialisation and, for C > 1, clusters of C blocks.
template <int C, typename K, typename... Args>
static cudaError_t launch_sample_cluster(K kernel, int n_emit, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_emit * C);
    cfg.blockDim = dim3(kSampleThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = C;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = C > 1 ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Args&&>(args)...);
}

int launch_sample(const Shape& s, const Buffers& b, const StepLayout& lay, int n_emit, int sm_count, int32_t* out_tokens,
                  float* out_logprobs, float* nucleus_mass, cudaStream_t st) {
    // two blocks per row while that still fits one wave (a pass is bound by what one SM can pull from L2)
    const bool pair = 2 * n_emit <= sm_count;
    if (b.expw) {
        if (pair) launch_sample_cluster<2>(sample_kernel<true, 2>, n_emit, st, s, b, lay, out_tokens, out_logprobs, nucleus_mass);
        else launch_sample_cluster<1>(sample_kernel<true, 1>, n_emit, st, s, b, lay, out_tokens, out_logprobs, nucleus_mass);
    } else {
        if (pair) launch_sample_cluster<2>(sample_kernel<false, 2>, n_emit, st, s, b, lay, out_tokens, out_logprobs, nucleus_mass);
        else launch_sample_cluster<1>(sample_kernel<false, 1>, n_emit, st, s, b, lay, out_tokens, out_logprobs, nucleus_mass);
    }
    return 1;
}

}  // namespace mars
