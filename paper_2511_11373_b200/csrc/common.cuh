// Device-side helpers shared by the rollout-step kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "step.h"

namespace mars {

constexpr int kWarp = 32;

__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

// Two floats -> packed bf16x2 (round to nearest even), `lo` in the low half.
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
}
// v ~= hi + lo with both parts bf16: about 16 mantissa bits survive.  Activations travel between
// kernels as such pairs so that bf16 tensor-core contractions do not eat the error budget.
__device__ __forceinline__ void split_bf16(float v, __nv_bfloat16& hi, __nv_bfloat16& lo) {
    hi = __float2bfloat16_rn(v);
    lo = __float2bfloat16_rn(v - __bfloat162float(hi));
}
__device__ __forceinline__ uint16_t to_bf16_bits(float v) {
    __nv_bfloat16 t = __float2bfloat16_rn(v);
    return *reinterpret_cast<uint16_t*>(&t);
}

// 16-byte read-only streaming load: weights are read once per step, keep them out of L1.
__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col).  Fragment ownership, lane = 4*gid + tig:
//   A: a0 (row gid, k 2tig..2tig+1)  a1 (row gid+8, same k)  a2 (row gid, k 2tig+8..)  a3 (row gid+8, k 2tig+8..)
//   B: b0 (k 2tig..2tig+1, col gid)  b1 (k 2tig+8.., col gid)
//   D: d0,d1 (row gid, cols 2tig, 2tig+1)  d2,d3 (row gid+8, same cols)
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Sum over the block in a fixed order (deterministic).  `scratch` holds at least 32 floats.
__device__ __forceinline__ float block_sum(float v, float* scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float t = 0.f;
    for (int i = 0; i < nw; ++i) t += scratch[i];
    return t;
}

// Programmatic dependent launch.  Every kernel of the step is launched with the stream-serialisation
// attribute relaxed (launch_chained in kernels.h): its blocks are scheduled as soon as all blocks of
// the previous kernel of the stream have exited, without waiting for that grid's completion to be
// signalled, and pdl_wait() returns once the previous kernel has completed and its writes are visible.
// Rule kept by every kernel here: nothing produced by an earlier kernel is read, and no global memory
// is written, before pdl_wait(); only weights (constant during a step), shared memory, barriers and
// tensor memory are touched ahead of it.  Every kernel has at least one thread that executes
// pdl_wait() before the grid can end, so completion of a kernel implies completion of all kernels
// before it.  No kernel issues griddepcontrol.launch_dependents: measured on the 48-layer decode step
// (22.04 ms with plain launches), letting the next grid's blocks become resident early cost time
// (23.7 ms with the trigger at the top of every kernel, 21.6 ms with it in the small kernels only),
// while the implicit trigger at block exit gives 21.2 ms.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gsrc));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N)); }

// ----- the swap-AB streaming contraction --------------------------------------------------------
// Y^T[rows, tokens] = W[rows, K] * X^T: weight rows sit on the MMA M axis (16 per tile), tokens on
// the N axis (8 per tile), so a handful of tokens costs no more tensor work than one.  A fragments
// come straight from global memory with 16-byte loads: inside a 32-wide slice of K the thread
// (gid, tig) owns the 8 consecutive elements tig*8..tig*8+7 of rows gid and gid+8 and feeds them to
// two MMAs as k-columns {2tig, 2tig+1, 2tig+8, 2tig+9}.  The contraction does not care how k is
// numbered as long as B uses the same numbering, so the B fragment of token column gid is the same
// 16-byte slice of that token's activation row, read from shared memory.
//
// Activations are (hi, lo) bf16 pairs: token t occupies the two adjacent columns 2t (hi) and 2t+1
// (lo), which land in the same thread's accumulator pair, so the epilogue adds d0 + d1 (rows gid)
// and d2 + d3 (rows gid+8).  One 8-column tile therefore serves 4 tokens.
//
// MT: 16-row tiles per warp (each with its own pair of row pointers), NT: 8-token tiles, U: slices
// whose loads are issued before the first MMA (memory-level parallelism).
//   wrow[m][r]: pointer to W row (tile m, row gid + 8r), already offset by tig*8 elements
//   xs: shared-memory address of activation row `gid` of column tile 0, offset by tig*16 bytes
//   x_tile_stride: bytes between column tiles (8 rows), n_slices: K / 32
template <int MT, int NT, int U>
__device__ __forceinline__ void stream_mma(const __nv_bfloat16* const (&wrow)[MT][2], int n_slices,
                                           const unsigned char* xs, int x_tile_stride, float (&acc)[MT][NT][4]) {
    int s = 0;
    for (; s + U <= n_slices; s += U) {
        uint4 w[U][MT][2];
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int m = 0; m < MT; ++m)
#pragma unroll
                for (int r = 0; r < 2; ++r) w[u][m][r] = ldg_stream(wrow[m][r] + (size_t)(s + u) * 32);
#pragma unroll
        for (int u = 0; u < U; ++u) {
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                const uint4 x = *reinterpret_cast<const uint4*>(xs + (size_t)n * x_tile_stride + (size_t)(s + u) * 64);
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    mma_16816(acc[m][n], w[u][m][0].x, w[u][m][1].x, w[u][m][0].y, w[u][m][1].y, x.x, x.y);
                    mma_16816(acc[m][n], w[u][m][0].z, w[u][m][1].z, w[u][m][0].w, w[u][m][1].w, x.z, x.w);
                }
            }
        }
    }
    for (; s < n_slices; ++s) {
        uint4 w[MT][2];
#pragma unroll
        for (int m = 0; m < MT; ++m)
#pragma unroll
            for (int r = 0; r < 2; ++r) w[m][r] = ldg_stream(wrow[m][r] + (size_t)s * 32);
#pragma unroll
        for (int n = 0; n < NT; ++n) {
            const uint4 x = *reinterpret_cast<const uint4*>(xs + (size_t)n * x_tile_stride + (size_t)s * 64);
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                mma_16816(acc[m][n], w[m][0].x, w[m][1].x, w[m][0].y, w[m][1].y, x.x, x.y);
                mma_16816(acc[m][n], w[m][0].z, w[m][1].z, w[m][0].w, w[m][1].w, x.z, x.w);
            }
        }
    }
}

// ----- weight stream through a per-warp shared-memory ring ----------------------------------------
// The same contraction with the A operand staged by cp.async: every thread copies the two 16-byte
// pieces it will need for a K slice (its row of MMA rows 0..7 and its row of MMA rows 8..15) into a
// slot of its warp's ring and reads the same two pieces back kRing slices later.  The bytes in
// flight then live in shared memory instead of registers (a register-staged stream tops out near
// 8 KB per warp), no other thread ever touches a slot, and consecutive lanes own consecutive 16-byte
// pieces, so the read-back is free of bank conflicts.  One commit group per slice; a slot is
// refilled only after the MMAs that consumed it have been issued.
constexpr int kRing = 8;
constexpr int kRingStageBytes = 1024;                      // per warp and slice: 2 pieces x 32 lanes x 16 B
constexpr int kRingWarpBytes = kRing * kRingStageBytes;

__device__ __forceinline__ void ring_issue(unsigned char* warp_ring, int stage, int lane, const __nv_bfloat16* p0,
                                           const __nv_bfloat16* p1) {
    unsigned char* d = warp_ring + stage * kRingStageBytes + lane * 16;
    cp_async16(d, p0);
    cp_async16(d + 512, p1);
}

// acc[n] += A(slice) * B(slice, column tile n); xs points at this thread's 16 bytes of column tile 0.
template <int NT>
__device__ __forceinline__ void ring_consume(const unsigned char* warp_ring, int stage, int lane, const unsigned char* xs,
                                             int x_tile_stride, float (&acc)[NT][4]) {
    const unsigned char* s = warp_ring + stage * kRingStageBytes + lane * 16;
    const uint4 w0 = *reinterpret_cast<const uint4*>(s);
    const uint4 w1 = *reinterpret_cast<const uint4*>(s + 512);
#pragma unroll
    for (int n = 0; n < NT; ++n) {
        const uint4 x = *reinterpret_cast<const uint4*>(xs + (size_t)n * x_tile_stride);
        mma_16816(acc[n], w0.x, w1.x, w0.y, w1.y, x.x, x.y);
        mma_16816(acc[n], w0.z, w1.z, w0.w, w1.w, x.z, x.w);
    }
}

// Activation rows in shared memory are padded by 64 bytes so that the 16-byte B-fragment reads of
// a quarter warp (rows gid, gid+1; four 16-byte pieces each) fall into 32 distinct banks.
__host__ __device__ constexpr int x_row_bytes(int k_elems) { return k_elems * 2 + 64; }

}  // namespace mars
