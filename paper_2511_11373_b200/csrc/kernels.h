// Launch wrappers of the rollout-step kernels (host side declarations).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "step.h"

namespace mars {

struct KvView {
    __nv_bfloat16* k_pool;
    __nv_bfloat16* v_pool;
    int32_t* block_table;  // [max_seqs][max_pages_per_seq]
    int n_pages, page_size, max_pages_per_seq;
};

struct LayerW {
    const __nv_bfloat16 *attn_norm, *wqkv, *q_norm, *k_norm, *wo, *mlp_norm, *router, *w_gate_up, *w_down;
};

struct DebugTaps {
    float* hidden;            // [L + 1, n_tok, H] or null
    float* router_w;          // [L, n_tok, k] or null
    int32_t* router_idx;      // [L, n_tok, k] or null
    const int32_t* forced_idx;  // [L, n_tok, k] or null
    float* nucleus_mass;      // [n_emit] or null
};

// Launch with programmatic stream serialisation: the kernel's blocks may start while the previous kernel
// of the stream drains (see pdl_wait in common.cuh for the rule the kernels keep).
template <typename... Params, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                  Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Args&&>(args)...);
}

// Each wrapper enqueues its kernel(s) on `st` and returns the number of kernels it launched.
int launch_prep(const Shape& s, const Buffers& b, const StepLayout& lay, const KvView& kv, int n_tok, cudaStream_t st);
int launch_embed(const Shape& s, const Buffers& b, const StepLayout& lay, const __nv_bfloat16* embed,
                 const int32_t* tokens, const __nv_bfloat16* first_gain, float* hidden_tap, int n_tok, cudaStream_t st);
int launch_qkv(const Shape& s, const Buffers& b, const StepLayout& lay, const LayerW& w, const KvView& kv, int layer,
               int n_tok, int sm_count, cudaStream_t st);
// K elements per phase, number of K splits (partials) and phases per CTA of the streaming GEMM.
void gemm_plan(int K, int n_tok, bool many_rows, int* ks, int* ksplit, int* phases);
int launch_oproj(const Shape& s, const Buffers& b, const LayerW& w, int n_tok, int sm_count, cudaStream_t st);
int launch_lm_head(const Shape& s, const Buffers& b, const StepLayout& lay, const __nv_bfloat16* lm_head, int n_emit,
                   int sm_count, cudaStream_t st);

int launch_attention(const Shape& s, const Buffers& b, const StepLayout& lay, const KvView& kv, const CUtensorMap& tm_k,
                     const CUtensorMap& tm_v, int layer, int sm_count, cudaStream_t st);
// Causal attention of a prefill chunk: items are blocks of up to 4 consecutive prompt tokens; writes b.o.
int launch_attention_prefill(const Shape& s, const Buffers& b, const StepLayout& lay, const KvView& kv,
                             const CUtensorMap& tm_k, const CUtensorMap& tm_v, int layer, int sm_count, cudaStream_t st);
// Spans of cached tokens that several decode rows share (same pages): read once per block of up to 4 rows;
// every row gets its partial result in its own slot.
int launch_attention_shared(const Shape& s, const Buffers& b, const StepLayout& lay, const KvView& kv,
                            const CUtensorMap& tm_k, const CUtensorMap& tm_v, int layer, int n_items, int sm_count,
                            cudaStream_t st);

// Causal prefill attention on tcgen05 (head_dim 128, 8 query heads per KV head): items are blocks of up to
// fattn_block_tokens() consecutive prompt tokens; tm_q is the 4-D map (d, head, plane, token) over b.q.
bool fattn_supported(const Shape& s);
int fattn_block_tokens();
int launch_fattn_prefill(const Shape& s, const Buffers& b, const StepLayout& lay, const KvView& kv, const CUtensorMap& tm_q,
                         const CUtensorMap& tm_k, const CUtensorMap& tm_v, int layer, int n_items, int sm_count,
                         cudaStream_t st);
// Shared spans of decode rows on the same kernel: items of fattn_shared_item_words() words, up to
// fattn_shared_rows() rows each; tm_q1 is the query map with one-token boxes.
int fattn_shared_rows();
int fattn_shared_item_words();
int launch_fattn_shared(const Shape& s, const Buffers& b, const StepLayout& lay, const KvView& kv, const CUtensorMap& tm_q1,
                        const CUtensorMap& tm_k, const CUtensorMap& tm_v, int layer, int n_items, int sm_count,
                        cudaStream_t st);
int launch_attn_merge(const Shape& s, const Buffers& b, const StepLayout& lay, int n_tok, cudaStream_t st);

// o_ksplit: number of split-K partials of the output projection that the router kernel adds to the residual.
int launch_router(const Shape& s, const Buffers& b, const LayerW& w, const DebugTaps& dbg, int layer, int n_tok,
                  int group_cap, int o_ksplit, cudaStream_t st);

// Prefill-sized contractions on tcgen05: out[m][n_cols] = A[m][2][K] (hi + lo planes) . B[n_cols][K]^T, and
// the grouped expert pair (gather rows to slot order, gate/up + SwiGLU, down) over the group list.
int launch_resid_norm(const Shape& s, const Buffers& b, const LayerW& w, int n_tok, int o_ksplit, cudaStream_t st);
// n_parts: split-K partials of the gate logits in b.rlogits ([part][n_tok][E]); group_cap <= 0: the streaming
// expert kernels' group size.  Small calls run the token permutation in the selection kernel's last block.
int launch_route_select(const Shape& s, const Buffers& b, const DebugTaps& dbg, int layer, int n_tok, int group_cap, int n_parts,
                        cudaStream_t st);
// The QKV projection with its post-processing in the epilogue of the contraction kernel.  A thread owns one
// token row of a tile and, in it, whole heads (256 / head_dim of them): per-head RMS norm (optional),
// rotary embedding at the token's position, then queries as (hi, lo) bf16 pairs into q_out
// [token][2][nq * D] and keys / values rounded to bf16 into the token's page slot -- the fp32
// projection never goes to memory.
struct QkvEpilogue {
    const int32_t* tok_pos;     // [m_rows]
    const int32_t* tok_seq;     // [m_rows]
    const int32_t* block_table; // [seqs][max_pages_per_seq]
    const float2* rope;         // [m_rows][D / 2] (cos, sin)
    const __nv_bfloat16 *q_gain, *k_gain;
    __nv_bfloat16 *q_out, *k_pool, *v_pool;
    int max_pages_per_seq, n_pages, page_size, layer, nq, nkv, head_dim, qk_norm;
    float eps;
};
// use_lo: 1 accumulates the lo plane of the (hi, lo) activations too; 0 contracts the hi plane only (bf16
// activations: half the tensor work, ~1e-3 relative error per contraction).
int launch_umma_qkv(const CUtensorMap& tm_a, const CUtensorMap& tm_b, int m_rows, int n_cols, int K, const QkvEpilogue& ep,
                    int32_t* err, int use_lo, cudaStream_t st);
int launch_umma_dense(const CUtensorMap& tm_a, const CUtensorMap& tm_b, int m_rows, int n_cols, int K, float* out,
                      int32_t* err, int use_lo, cudaStream_t st);
// Decode-sized projection on tcgen05 with swapped operands: out[split][t][row], t < n_tok <= umma_swap_max_tokens().
int umma_swap_max_tokens();
int umma_swap_splits(int rows, int n_tok, int K);
int launch_umma_swap(const CUtensorMap& tm_w, const CUtensorMap& tm_x, int rows, int n_tok, int K, int splits, float* out,
                     int32_t* err, cudaStream_t st);
int launch_umma_experts(const Shape& s, const Buffers& b, const CUtensorMap& tm_xperm, const CUtensorMap& tm_wgu,
                        const CUtensorMap& tm_act, const CUtensorMap& tm_wdown, int n_tok, int gate_up_lo, int down_lo, cudaStream_t st);
// Scoring pass: out_logprobs[row] = log softmax(lm_head(h[row]) * inv_temp)[targets[row]] (0 where the
// target is negative).  score_ml: [score_vocab_tiles(vocab)][n_rows] scratch, score_tgt: [n_rows] scratch.
int score_vocab_tiles(int vocab);
int launch_umma_score(const CUtensorMap& tm_h, const CUtensorMap& tm_lm, int n_rows, int vocab, int K,
                      const int32_t* targets, float inv_temp, float2* score_ml, float* score_tgt, float* logits_tap,
                      float* out_logprobs, int32_t* err, cudaStream_t st);
// One CTA that waits, with a limit of `limit` polls, for an mbarrier arrival that comes (arrive != 0) or
// never comes (arrive == 0): the give-up path of the bounded waits, run without hanging anything.
int launch_wait_probe(int32_t* err, int arrive, uint32_t limit, cudaStream_t st);
int launch_qkv_post(const Shape& s, const Buffers& b, const StepLayout& lay, const LayerW& w, const KvView& kv, int layer,
                    int n_tok, int ksplit, cudaStream_t st);
int launch_gate_up(const Shape& s, const Buffers& b, const LayerW& w, int n_tok, int sm_count, cudaStream_t st);
int launch_down(const Shape& s, const Buffers& b, const LayerW& w, int n_tok, cudaStream_t st);
int launch_combine(const Shape& s, const Buffers& b, const __nv_bfloat16* next_gain, float* hidden_tap, int n_tok,
                   cudaStream_t st);

int launch_sample(const Shape& s, const Buffers& b, const StepLayout& lay, int n_emit, int sm_count, int32_t* out_tokens,
                  float* out_logprobs, float* nucleus_mass, cudaStream_t st);

// Copies n_pages pages in each of n_layers layers: unit (layer, i) goes from
// src + layer * src_layer_stride + src_pages[i] * page_bytes to the same expression on the dst side
// (a null page list means page index i itself, i.e. a packed image).  Page lists are device arrays.
struct PageCopy {
    const unsigned char* src;
    unsigned char* dst;
    size_t src_layer_stride, dst_layer_stride;
    const int32_t* src_pages;
    const int32_t* dst_pages;
    int n_pages, n_layers;
    uint32_t page_bytes;
};
int launch_kv_page_copy(const PageCopy& p, int sm_count, cudaStream_t st);

// Opt-in shared-memory attributes etc.; call once per device before the first launch.
cudaError_t init_kernels();

}  // namespace mars
