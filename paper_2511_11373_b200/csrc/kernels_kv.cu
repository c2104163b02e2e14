// Page movers of the paged KV cache: pack a sequence's pages into one contiguous image (device or
// pinned host memory) when a trajectory is parked between rollout segments, unpack such an image
// into freshly reserved pages when it resumes, and copy single pages inside the pool when a group
// member is forked from a shared prompt.
#include "common.cuh"
#include "kernels.h"

namespace mars {

// One unit = the bytes of one page in one layer (n_kv_heads * page_size * head_dim bf16, a multiple
// of 16 bytes).  A block walks units with a grid stride; its threads move 16-byte pieces, four
// loads in flight before the first store.
__global__ void __launch_bounds__(256) kv_page_copy_kernel(PageCopy p) {
    const int units = p.n_pages * p.n_layers;
    const uint32_t pieces = p.page_bytes >> 4;
    for (int u = blockIdx.x; u < units; u += gridDim.x) {
        const int layer = u / p.n_pages, i = u - layer * p.n_pages;
        const int sp = p.src_pages ? p.src_pages[i] : i;
        const int dp = p.dst_pages ? p.dst_pages[i] : i;
        const uint4* __restrict__ s = reinterpret_cast<const uint4*>(p.src + (size_t)layer * p.src_layer_stride +
                                                                    (size_t)sp * p.page_bytes);
        uint4* __restrict__ d = reinterpret_cast<uint4*>(p.dst + (size_t)layer * p.dst_layer_stride + (size_t)dp * p.page_bytes);
        uint32_t c = threadIdx.x;
        for (; c + 3 * blockDim.x < pieces; c += 4 * blockDim.x) {
            const uint4 a0 = s[c], a1 = s[c + blockDim.x], a2 = s[c + 2 * blockDim.x], a3 = s[c + 3 * blockDim.x];
            d[c] = a0; d[c + blockDim.x] = a1; d[c + 2 * blockDim.x] = a2; d[c + 3 * blockDim.x] = a3;
        }
        for (; c < pieces; c += blockDim.x) d[c] = s[c];
    }
}

int launch_kv_page_copy(const PageCopy& p, int sm_count, cudaStream_t st) {
    const int units = p.n_pages * p.n_layers;
    if (units <= 0) return 0;
    const int grid = units < sm_count * 8 ? units : sm_count * 8;
    kv_page_copy_kernel<<<grid, 256, 0, st>>>(p);
    return 1;
}

}  // namespace mars
