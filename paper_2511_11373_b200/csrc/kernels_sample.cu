// log-softmax + greedy / nucleus sampling over one row of logits per emitting sequence.
//
// Nucleus selection needs no sort: the weights e_v = exp((l_v - max) / T) are positive floats, so
// their bit patterns order like the values.  A three-pass radix search (11 + 10 + 10 bits) over
// per-bucket MASS histograms finds the weight of the token at which the descending cumulative mass
// reaches top_p; masses are accumulated in 2^-40 fixed point with integer atomics, which makes the
// result independent of the order in which threads add.  Tokens above that weight are in the
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

__device__ __forceinline__ unsigned long long to_fix(float e) { return (unsigned long long)((double)e * kFix); }

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

__global__ void __launch_bounds__(kSampleThreads) sample_kernel(Shape s, Buffers b, StepLayout lay, int32_t* out_tokens,
                                                                float* out_logprobs, float* nucleus_mass) {
    __shared__ unsigned long long hist[kBins];
    __shared__ unsigned long long warp_tot[kSampleThreads / 32];
    __shared__ float red_f[32];
    __shared__ int red_i[32];
    __shared__ double red_d[32];
    __shared__ unsigned int red_u[2][32];
    __shared__ unsigned int sel_prefix;
    __shared__ unsigned long long sel_above;
    __shared__ int sel_token;
    pdl_wait();

    const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int V = s.V;
    const float* l = b.logits + (size_t)row * V;
    const int32_t* hdr = b.step;
    const bool greedy = hdr[H_GREEDY] != 0;
    const float T = greedy ? 1.f : __int_as_float(hdr[H_TEMPERATURE]);
    const float top_p = __int_as_float(hdr[H_TOP_P]);
    const float inv_t = 1.f / T;

    // max and argmax (lowest id on ties)
    float mx = -INFINITY;
    int am = 0x7fffffff;
    for (int v = tid; v < V; v += kSampleThreads) {
        const float x = l[v];
        if (x > mx) { mx = x; am = v; }
    }
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

    // Z = sum exp((l - max) / T): fp32 terms, fp64 sum in a fixed order
    double zs = 0.0;
    for (int v = tid; v < V; v += kSampleThreads) zs += (double)expf((l[v] - mx) * inv_t);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) zs += __shfl_xor_sync(0xffffffffu, zs, o);
    if (lane == 0) red_d[warp] = zs;
    __syncthreads();
    double Z = 0.0;
    for (int w = 0; w < kSampleThreads / 32; ++w) Z += red_d[w];
    const float log_z = (float)log(Z);

    if (greedy) {
        if (tid == 0) {
            out_tokens[row] = am;
            out_logprobs[row] = -log_z;     // (l_max - max) / 1 - log Z
            if (nucleus_mass) nucleus_mass[row] = 1.f;
        }
        return;
    }

    // ---- nucleus threshold: radix search on the bit pattern of e_v, by mass
    // total mass in fixed point, and which key bits differ at all: near-flat logits share their sign,
    // most of the exponent and often some mantissa bits, and a radix digit taken from shared bits
    // would send every token to the same bucket (one hot shared-memory atomic).
    unsigned long long part = 0;
    unsigned int k_or = 0u, k_and = 0xffffffffu;
    for (int v = tid; v < V; v += kSampleThreads) {
        const float e = expf((l[v] - mx) * inv_t);
        part += to_fix(e);
        k_or |= __float_as_uint(e);
        k_and &= __float_as_uint(e);
    }
    k_or = __reduce_or_sync(0xffffffffu, k_or);
    k_and = __reduce_and_sync(0xffffffffu, k_and);
    if (lane == 0) { red_u[0][warp] = k_or; red_u[1][warp] = k_and; }
    unsigned long long z_fix;
    block_excl_scan(part, warp_tot, &z_fix);          // (its barriers also publish red_u)
    for (int w = 0; w < kSampleThreads / 32; ++w) { k_or |= red_u[0][w]; k_and &= red_u[1][w]; }
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
            for (int i = tid; i < kBins; i += kSampleThreads) hist[i] = 0ull;
            if (tid == 0) { sel_prefix = prefix << wd; sel_above = above; }
            __syncthreads();
            for (int v = tid; v < V; v += kSampleThreads) {
                const float e = expf((l[v] - mx) * inv_t);
                const unsigned int key = __float_as_uint(e);
                if ((key >> (sh + wd)) == prefix) atomicAdd(&hist[(key >> sh) & ((1u << wd) - 1u)], to_fix(e));
            }
            __syncthreads();
            // descending scan over the buckets, two per thread
            const int b0 = kBins - 1 - 2 * tid;
            const unsigned long long h0 = hist[b0], h1 = hist[b0 - 1];
            unsigned long long pass_total;
            const unsigned long long before = above + block_excl_scan(h0 + h1, warp_tot, &pass_total);
            if (before < target && before + h0 >= target) {
                sel_prefix = (prefix << wd) | (unsigned int)b0;
                sel_above = before;
            } else if (before + h0 < target && before + h0 + h1 >= target) {
                sel_prefix = (prefix << wd) | (unsigned int)(b0 - 1);
                sel_above = before + h0;
            }
            __syncthreads();
            prefix = sel_prefix;
            above = sel_above;
            remaining = sh;
            __syncthreads();
        }
    }
    // threshold weight: key == prefix.  Ties enter in ascending id until the mass is reached.
    const unsigned int tkey = prefix;
    const unsigned long long q = everything ? 1ull : to_fix(__uint_as_float(tkey));
    unsigned long long need_ties = 0;
    if (!everything) need_ties = q > 0 ? (target - above + q - 1) / q : 0xffffffffull;

    // ---- walk in ascending token id: contiguous chunk per thread
    const int chunk = (V + kSampleThreads - 1) / kSampleThreads;
    const int v0 = min(V, tid * chunk), v1 = min(V, v0 + chunk);
    unsigned long long my_ties = 0;
    if (!everything)
        for (int v = v0; v < v1; ++v) my_ties += __float_as_uint(expf((l[v] - mx) * inv_t)) == tkey;
    unsigned long long ties_total;
    const unsigned long long tie_base = everything ? 0ull : block_excl_scan(my_ties, warp_tot, &ties_total);
    unsigned long long my_mass = 0, tie_rank = tie_base;
    for (int v = v0; v < v1; ++v) {
        const float e = expf((l[v] - mx) * inv_t);
        const unsigned int key = __float_as_uint(e);
        bool in = everything || key > tkey;
        if (!everything && key == tkey) { in = tie_rank < need_ties; ++tie_rank; }
        if (in) my_mass += to_fix(e);
    }
    unsigned long long mass_s;
    const unsigned long long mass_base = block_excl_scan(my_mass, warp_tot, &mass_s);

    // uniform in (0, 1) from the counter-based generator
    const uint32_t slot = (uint32_t)b.step[lay.emit_slot + row];
    const uint32_t x0 = philox_first_word((uint32_t)hdr[H_STEP_LO], (uint32_t)hdr[H_STEP_HI], slot, 0u,
                                          (uint32_t)hdr[H_SEED_LO], (uint32_t)hdr[H_SEED_HI]);
    const double u = ((double)(x0 >> 8) + 0.5) * (1.0 / 16777216.0);
    const double thr = u * (double)mass_s;     // first id whose cumulative mass exceeds thr

    if (tid == 0) sel_token = -1;
    __syncthreads();
    if ((double)mass_base <= thr && (double)(mass_base + my_mass) > thr) {
        unsigned long long cum = mass_base, rank = tie_base;
        for (int v = v0; v < v1; ++v) {
            const float e = expf((l[v] - mx) * inv_t);
            const unsigned int key = __float_as_uint(e);
            bool in = everything || key > tkey;
            if (!everything && key == tkey) { in = rank < need_ties; ++rank; }
            if (in) {
                cum += to_fix(e);
                if ((double)cum > thr) { sel_token = v; break; }
            }
        }
    }
    __syncthreads();
    if (tid == 0) {
        int tok = sel_token;
        if (tok < 0) tok = am;   // cannot happen while mass_s > 0; keeps the output defined
        out_tokens[row] = tok;
        out_logprobs[row] = (l[tok] - mx) * inv_t - log_z;
        if (nucleus_mass) nucleus_mass[row] = (float)((double)mass_s / (double)z_fix);
    }
}

int launch_sample(const Shape& s, const Buffers& b, const StepLayout& lay, int n_emit, int32_t* out_tokens,
                  float* out_logprobs, float* nucleus_mass, cudaStream_t st) {
    launch_chained(sample_kernel, dim3(n_emit), dim3(kSampleThreads), 0, st, s, b, lay, out_tokens, out_logprobs, nucleus_mass);
    return 1;
}

}  // namespace mars
