// Host side of libmars: argument checking, paged-KV bookkeeping, per-step work lists, launch
// sequence.  Every step of the computation runs in the kernels; nothing here touches tensor data.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/mars.h"
#include "kernels.h"

namespace mars {
cudaError_t init_dense_kernels();
cudaError_t init_attn_kernels();
cudaError_t init_moe_kernels();
cudaError_t init_umma_kernels();
cudaError_t init_fattn_kernels();
}  // namespace mars

using namespace mars;

static thread_local int32_t g_last_cuda_error = 0;

#define CUDA_TRY(expr)                                   \
    do {                                                 \
        cudaError_t _e = (expr);                         \
        if (_e != cudaSuccess) {                         \
            g_last_cuda_error = (int32_t)_e;             \
            return MARS_ERR_CUDA;                        \
        }                                                \
    } while (0)

namespace {

constexpr int kSpanTokens = 1024;   // cached tokens per attention work item at decode
constexpr int kStagingSlots = 4;
constexpr int kUmmaMinTokens = 64;  // calls with more token rows take the tensor-core (tcgen05) contraction path
constexpr int kSharedRows = 4;      // decode rows per work item of the shared-prefix attention kernel on mma.sync
constexpr int kSharedItemWords = 36; // capacity per shared item: the tcgen05 kernel's items hold 16 rows
constexpr int kMinSharedTokens = 128;  // shorter common prefixes are read per row as usual

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Caps {
    int n_tok;     // token rows per call
    int n_emit;    // sampled rows per call
    int n_updates; // block-table writes per call
    int n_items;   // attention work items per call
    bool keep_weights = true;   // room for the sampler's softmax weights (not in the fixed-scratch entry)
};

Caps make_caps(const mars_config_t& c, int max_decode, int max_prefill) {
    Caps k;
    k.n_tok = std::max(max_decode, max_prefill);
    k.n_emit = std::max(max_decode, 1);
    k.n_updates = k.n_tok + k.n_emit;
    k.n_items = max_decode * (c.max_pos / kSpanTokens + 2) + max_prefill;
    return k;
}

StepLayout make_layout(const Caps& k) {
    StepLayout l;
    int at = H_WORDS;
    auto take = [&](int words) { int o = at; at += (words + 3) & ~3; return o; };
    l.tok_seq = take(k.n_tok);
    l.tok_pos = take(k.n_tok);
    l.tok_item_off = take(k.n_tok + 1);
    l.emit_rows = take(k.n_emit);
    l.emit_slot = take(k.n_emit);
    l.updates = take(3 * k.n_updates);
    l.items = take(4 * k.n_items);
    l.sh_items = take(kSharedItemWords * (k.n_items / 2 + 1));   // a shared item stands for the spans of at least two rows
    l.total_words = at;
    return l;
}

bool shape_supported(const mars_config_t& c) {
    if (c.n_layers < 1 || c.hidden < 256 || c.hidden > 8192 || c.hidden % 256) return false;
    if (c.head_dim != 64 && c.head_dim != 128) return false;
    if (c.n_kv_heads < 1 || c.n_q_heads % c.n_kv_heads || c.n_q_heads / c.n_kv_heads > 8) return false;
    if ((c.n_q_heads * c.head_dim) % 256) return false;
    if (c.n_experts < 1 || c.n_experts > 1024 || c.top_k < 1 || c.top_k > 32 || c.top_k > c.n_experts) return false;
    if (c.expert_inter < 64 || c.expert_inter % 64) return false;
    // the streaming down kernel keeps up to 16 tokens x (hi, lo) activation rows of expert_inter elements in
    // shared memory (200 KB are requested for it)
    if ((size_t)32 * (2 * (size_t)c.expert_inter + 64) > 200u * 1024u) return false;
    if (c.vocab < 2 || c.max_pos < 1) return false;
    return true;
}

// Carves the workspace; with base == nullptr only sizes are computed.
size_t carve(const mars_config_t& c, const Caps& k, const StepLayout& lay, unsigned char* base, Buffers* b,
             int32_t** io_in, int32_t** io_out, float** io_lp) {
    size_t at = 0;
    auto take = [&](size_t bytes) { size_t o = at; at = align_up(at + bytes, 256); return base ? base + o : nullptr; };
    const size_t n = k.n_tok, H = c.hidden, D = c.head_dim, nq = c.n_q_heads, nkv = c.n_kv_heads, kk = c.top_k;
    Buffers t;
    t.step = (int32_t*)take((size_t)lay.total_words * 4);
    t.err = (int32_t*)take(256);
    t.x = (float*)take(n * H * 4);
    t.h = (__nv_bfloat16*)take(n * 2 * H * 2);
    // split-K partials: up to K/256 of them for decode-sized calls, one otherwise
    const size_t n_sw = std::min<size_t>(n, (size_t)umma_swap_max_tokens());
    const size_t qkv_parts = std::max(n, n_sw * (H / 256)), o_parts = std::max(n, n_sw * (nq * D / 256));
    t.qkv = (float*)take(qkv_parts * (nq + 2 * nkv) * D * 4);
    t.opart = (float*)take(o_parts * H * 4);
    t.q = (__nv_bfloat16*)take(n * 2 * nq * D * 2);
    t.o = (__nv_bfloat16*)take(n * 2 * nq * D * 2);
    t.rope = (float2*)take(n * (D / 2) * 8);
    t.inv_freq = (double*)take((D / 2) * 8);
    t.part_o = (float*)take((size_t)k.n_items * nq * D * 4);
    t.part_ml = (float2*)take((size_t)k.n_items * nq * 8);
    t.rlogits = (float*)take(n > kUmmaMinTokens ? n * c.n_experts * 4 : 0);
    t.route_idx = (int32_t*)take(n * kk * 4);
    t.route_w = (float*)take(n * kk * 4);
    t.expert_off = (int32_t*)take(((size_t)c.n_experts + 1) * 4);
    t.slot_token = (int32_t*)take(n * kk * 4);
    t.slot_of = (int32_t*)take(n * kk * 4);
    t.groups = (int32_t*)take(((size_t)c.n_experts + n * kk / 4 + 1) * 16);
    t.n_groups = (int32_t*)take(256);
    t.perm_cnt = (int32_t*)take((size_t)c.n_experts * 4);
    t.perm_cur = (int32_t*)take((size_t)c.n_experts * 4);
    t.active = (int32_t*)take((size_t)c.n_layers * 4);
    t.act = (__nv_bfloat16*)take(n * kk * 2 * c.expert_inter * 2);
    t.xperm = (__nv_bfloat16*)take(n > kUmmaMinTokens ? n * kk * 2 * H * 2 : 0);
    t.y = (float*)take(n * kk * H * 4);
    t.logits = (float*)take((size_t)k.n_emit * c.vocab * 4);
    t.expw = (float*)take(k.keep_weights ? (size_t)k.n_emit * c.vocab * 4 : 0);
    if (!k.keep_weights) t.expw = nullptr;
    int32_t* a = (int32_t*)take((size_t)k.n_emit * 4);
    int32_t* o = (int32_t*)take((size_t)k.n_emit * 4);
    float* lp = (float*)take((size_t)k.n_emit * 4);
    if (b) *b = t;
    if (io_in) *io_in = a;
    if (io_out) *io_out = o;
    if (io_lp) *io_lp = lp;
    return at;
}

}  // namespace

// bf16 tensor map with the 128-byte swizzle and a 64-element (128-byte) inner box.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static mars_status_t make_tiled_map(CUtensorMap* tm, const void* base, int rank, const cuuint64_t* dims,
                                    const cuuint64_t* strides_bytes, const cuuint32_t* box) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (!fn || qres != cudaDriverEntryPointSuccess) return MARS_ERR_UNSUPPORTED;
    const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    CUresult r = ((EncodeTiledFn)fn)(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims,
                                     strides_bytes, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        g_last_cuda_error = (int32_t)r;
        return MARS_ERR_CUDA;
    }
    return MARS_OK;
}
// queries [token][2][nq][D] as a 4-D tensor (d, head, plane, token): boxes of 64 elements x 8 heads x 16 tokens
static mars_status_t make_query_map(CUtensorMap* tm, const void* q, uint64_t tokens, uint64_t nq, uint64_t D,
                                    uint32_t box_tokens = 16) {
    const cuuint64_t dims[4] = {D, nq, 2, tokens}, strides[3] = {D * 2, nq * D * 2, 2 * nq * D * 2};
    const cuuint32_t box[4] = {64u, 8u, 1u, box_tokens};
    return make_tiled_map(tm, q, 4, dims, strides, box);
}
// weights [rows][K]: boxes of 64 rows x 64 elements
static mars_status_t make_weight_map(CUtensorMap* tm, const void* w, uint64_t rows, uint64_t K) {
    const cuuint64_t dims[2] = {K, rows}, strides[1] = {K * 2};
    const cuuint32_t box[2] = {64u, 64u};
    return make_tiled_map(tm, w, 2, dims, strides, box);
}
// activations [rows][2][K] (hi plane, lo plane): boxes of 128 rows of one plane x 64 elements
static mars_status_t make_pair_map(CUtensorMap* tm, const void* x, uint64_t rows, uint64_t K, uint32_t box_rows = 128) {
    const cuuint64_t dims[3] = {K, 2, rows}, strides[2] = {K * 2, K * 4};
    const cuuint32_t box[3] = {64u, 1u, box_rows};
    return make_tiled_map(tm, x, 3, dims, strides, box);
}

struct mars_model {
    mars_config_t cfg;
    Shape shape;
    Caps caps;
    StepLayout lay;
    Buffers buf;
    std::vector<LayerW> layers;
    // tensor maps of the prefill (tcgen05) path: weights per layer, activation buffers
    std::vector<CUtensorMap> tm_wqkv, tm_wo, tm_wgu, tm_wdown, tm_router;
    CUtensorMap tm_h, tm_o, tm_xperm, tm_act;
    CUtensorMap tm_h64, tm_o64, tm_lm;      // decode-sized (64 token rows per box) and the lm_head
    CUtensorMap tm_q;                       // queries for the tcgen05 prefill attention: (d, head, plane, token)
    CUtensorMap tm_q1;                      // the same tensor with one-token boxes (shared spans of decode rows)
    int lo_planes;                          // bit per contraction class of large calls: 1 = (hi, lo) activations, 0 = hi only
    bool fattn_ready, fattn_shared_ready;
    bool umma_ready;
    const __nv_bfloat16 *embed, *final_norm, *lm_head;
    int32_t *io_in, *io_out;
    float* io_lp;
    int device, sm_count;
    int max_decode, max_prefill;
    int32_t* staging[kStagingSlots];
    cudaEvent_t staged[kStagingSlots];
    int next_slot;
    cudaStream_t last_stream;
    mars_step_info_t info;
    // per-kernel-class timing (mars_profile_enable)
    bool profiling;
    std::vector<cudaEvent_t> ev_pool;          // all events ever created
    size_t ev_used;                            // events handed out since the last read
    std::vector<int> ev_class;                 // class of every (start, stop) pair handed out
};

struct SeqState {
    bool used = false;
    int len = 0;
    std::vector<int32_t> pages;
};

struct mars_kv {
    mars_model* model;
    KvView view;
    CUtensorMap tm_k, tm_v;
    int max_seqs;
    std::vector<SeqState> seqs;
    std::vector<int32_t> free_list;   // stack of free page ids
    std::vector<int32_t> refs;        // number of sequence slots that list the page (0 = free)
    bool share_reads = true;          // decode rows with a common page prefix read it once (mars_kv_share_reads)
    cudaStream_t copy_stream = nullptr;   // private stream of the block-table uploads (see upload_row)
};

extern "C" {

const char* mars_version(void) { return "mars-rollout-b200 0.1"; }
int32_t mars_last_cuda_error(void) { return g_last_cuda_error; }

const char* mars_status_string(mars_status_t s) {
    switch (s) {
        case MARS_OK: return "ok";
        case MARS_ERR_INVALID_ARG: return "invalid argument";
        case MARS_ERR_UNSUPPORTED: return "unsupported shape";
        case MARS_ERR_CUDA: return "CUDA runtime error";
        case MARS_ERR_KV_FULL: return "KV cache full";
        case MARS_ERR_TIMEOUT: return "bounded device wait gave up";
        case MARS_ERR_BAD_HANDLE: return "bad handle or sequence slot";
        case MARS_ERR_BAD_TOKEN: return "token id out of range";
        case MARS_ERR_TOO_LARGE: return "request exceeds the built-in scratch array (MARS_STATIC_SCRATCH_BYTES)";
        default: return "unknown status";
    }
}

size_t mars_workspace_bytes(const mars_config_t* cfg, int32_t max_decode_seqs, int32_t max_prefill_tokens) {
    if (!cfg || max_decode_seqs < 0 || max_prefill_tokens < 0 || max_decode_seqs + max_prefill_tokens < 1) return 0;
    if (!shape_supported(*cfg)) return 0;
    const Caps k = make_caps(*cfg, max_decode_seqs, max_prefill_tokens);
    const StepLayout lay = make_layout(k);
    return carve(*cfg, k, lay, nullptr, nullptr, nullptr, nullptr, nullptr);
}

mars_status_t mars_model_load(const mars_config_t* cfg, const mars_weights_t* w, void* workspace, size_t workspace_bytes,
                              int32_t max_decode_seqs, int32_t max_prefill_tokens, mars_model_t** out) {
    if (!cfg || !w || !workspace || !out || !w->layers || !w->embed || !w->final_norm || !w->lm_head)
        return MARS_ERR_INVALID_ARG;
    if (max_decode_seqs < 0 || max_prefill_tokens < 0 || max_decode_seqs + max_prefill_tokens < 1)
        return MARS_ERR_INVALID_ARG;
    if (!shape_supported(*cfg)) return MARS_ERR_UNSUPPORTED;
    if ((uintptr_t)workspace % 256) return MARS_ERR_INVALID_ARG;
    for (int l = 0; l < cfg->n_layers; ++l) {
        const mars_layer_t& s = w->layers[l];
        if (!s.attn_norm || !s.wqkv || !s.wo || !s.mlp_norm || !s.router || !s.w_gate_up || !s.w_down)
            return MARS_ERR_INVALID_ARG;
        if (cfg->qk_norm && (!s.q_norm || !s.k_norm)) return MARS_ERR_INVALID_ARG;
    }
    const Caps k = make_caps(*cfg, max_decode_seqs, max_prefill_tokens);
    const StepLayout lay = make_layout(k);
    if (workspace_bytes < carve(*cfg, k, lay, nullptr, nullptr, nullptr, nullptr, nullptr)) return MARS_ERR_INVALID_ARG;

    int dev = 0, major = 0, sms = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    if (major != 10) return MARS_ERR_UNSUPPORTED;
    CUDA_TRY(init_dense_kernels());
    CUDA_TRY(init_attn_kernels());
    CUDA_TRY(init_moe_kernels());
    CUDA_TRY(init_umma_kernels());
    CUDA_TRY(init_fattn_kernels());

    mars_model* m = new (std::nothrow) mars_model();
    if (!m) return MARS_ERR_INVALID_ARG;
    m->cfg = *cfg;
    m->shape = Shape{cfg->n_layers, cfg->hidden, cfg->n_q_heads, cfg->n_kv_heads, cfg->head_dim, cfg->n_experts,
                     cfg->top_k, cfg->expert_inter, cfg->vocab, cfg->qk_norm, cfg->rms_eps};
    m->caps = k;
    m->lay = lay;
    carve(*cfg, k, lay, (unsigned char*)workspace, &m->buf, &m->io_in, &m->io_out, &m->io_lp);
    m->layers.resize(cfg->n_layers);
    for (int l = 0; l < cfg->n_layers; ++l) {
        const mars_layer_t& s = w->layers[l];
        m->layers[l] = LayerW{(const __nv_bfloat16*)s.attn_norm, (const __nv_bfloat16*)s.wqkv,
                              (const __nv_bfloat16*)s.q_norm, (const __nv_bfloat16*)s.k_norm,
                              (const __nv_bfloat16*)s.wo, (const __nv_bfloat16*)s.mlp_norm,
                              (const __nv_bfloat16*)s.router, (const __nv_bfloat16*)s.w_gate_up,
                              (const __nv_bfloat16*)s.w_down};
    }
    m->embed = (const __nv_bfloat16*)w->embed;
    m->final_norm = (const __nv_bfloat16*)w->final_norm;
    m->lm_head = (const __nv_bfloat16*)w->lm_head;
    m->device = dev;
    m->sm_count = sms;
    m->max_decode = max_decode_seqs;
    m->max_prefill = max_prefill_tokens;
    m->next_slot = 0;
    m->last_stream = nullptr;
    m->profiling = false;
    m->lo_planes = MARS_LO_DEFAULT;
    m->ev_used = 0;
    std::memset(&m->info, 0, sizeof(m->info));
    for (int i = 0; i < kStagingSlots; ++i) { m->staging[i] = nullptr; m->staged[i] = nullptr; }
    auto fail = [&](cudaError_t e) {
        g_last_cuda_error = (int32_t)e;
        mars_model_free(m);
        return MARS_ERR_CUDA;
    };
    for (int i = 0; i < kStagingSlots; ++i) {
        cudaError_t e = cudaHostAlloc((void**)&m->staging[i], (size_t)lay.total_words * 4, cudaHostAllocDefault);
        if (e != cudaSuccess) return fail(e);
        e = cudaEventCreateWithFlags(&m->staged[i], cudaEventDisableTiming);
        if (e != cudaSuccess) return fail(e);
    }
    // rotary frequencies theta^(-2i/D) in fp64, status word cleared
    std::vector<double> inv((size_t)cfg->head_dim / 2);
    for (int i = 0; i < cfg->head_dim / 2; ++i)
        inv[i] = std::pow((double)cfg->rope_theta, -2.0 * (double)i / (double)cfg->head_dim);
    cudaError_t e = cudaMemcpy(m->buf.inv_freq, inv.data(), inv.size() * 8, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) return fail(e);
    e = cudaMemset(m->buf.err, 0, 256);
    if (e != cudaSuccess) return fail(e);
    e = cudaMemset(m->buf.active, 0, (size_t)cfg->n_layers * 4);
    if (e != cudaSuccess) return fail(e);
    e = cudaMemset(m->buf.perm_cnt, 0, (size_t)cfg->n_experts * 4);
    if (e != cudaSuccess) return fail(e);
    e = cudaMemset(m->buf.n_groups, 0, 256);      // [1]: arrival counter of the router blocks, zero between kernels
    if (e != cudaSuccess) return fail(e);
    // tensor maps of the prefill path (calls with more than kUmmaMinTokens token rows)
    m->umma_ready = false;
    {
        const uint64_t H = cfg->hidden, QD = (uint64_t)cfg->n_q_heads * cfg->head_dim, I = cfg->expert_inter;
        const uint64_t E = cfg->n_experts, n = k.n_tok, slots = (uint64_t)k.n_tok * cfg->top_k;
        const bool big = k.n_tok > kUmmaMinTokens;
        m->tm_wqkv.resize(cfg->n_layers); m->tm_wo.resize(cfg->n_layers);
        m->tm_wgu.resize(cfg->n_layers); m->tm_wdown.resize(cfg->n_layers); m->tm_router.resize(cfg->n_layers);
        mars_status_t rc = make_weight_map(&m->tm_lm, m->lm_head, (uint64_t)cfg->vocab, H);
        if (rc == MARS_OK) rc = make_pair_map(&m->tm_h64, m->buf.h, n, H, 64);
        if (rc == MARS_OK) rc = make_pair_map(&m->tm_h, m->buf.h, n, H);   // 128-row boxes (scoring pass, prefill)
        if (rc == MARS_OK) rc = make_pair_map(&m->tm_o64, m->buf.o, n, QD, 64);
        for (int l = 0; l < cfg->n_layers && rc == MARS_OK; ++l) {
            const LayerW& q = m->layers[l];
            rc = make_weight_map(&m->tm_wqkv[l], q.wqkv, (uint64_t)(cfg->n_q_heads + 2 * cfg->n_kv_heads) * cfg->head_dim, H);
            if (rc == MARS_OK) rc = make_weight_map(&m->tm_wo[l], q.wo, H, QD);
            if (!big) continue;
            if (rc == MARS_OK) rc = make_weight_map(&m->tm_router[l], q.router, E, H);
            if (rc == MARS_OK) rc = make_weight_map(&m->tm_wgu[l], q.w_gate_up, E * 2 * I, H);
            if (rc == MARS_OK) rc = make_weight_map(&m->tm_wdown[l], q.w_down, E * H, I);
        }
        if (big) {
            if (rc == MARS_OK) rc = make_pair_map(&m->tm_o, m->buf.o, n, QD);
            if (rc == MARS_OK) rc = make_pair_map(&m->tm_xperm, m->buf.xperm, slots, H);
            if (rc == MARS_OK) rc = make_pair_map(&m->tm_act, m->buf.act, slots, I);
        }
        m->fattn_ready = false;
        m->fattn_shared_ready = false;
        if (rc == MARS_OK && fattn_supported(m->shape)) {
            rc = make_query_map(&m->tm_q1, m->buf.q, n, (uint64_t)cfg->n_q_heads, (uint64_t)cfg->head_dim, 1);
            m->fattn_shared_ready = rc == MARS_OK;
        }
        if (rc == MARS_OK && big && fattn_supported(m->shape)) {
            rc = make_query_map(&m->tm_q, m->buf.q, n, (uint64_t)cfg->n_q_heads, (uint64_t)cfg->head_dim);
            m->fattn_ready = rc == MARS_OK;
        }
        if (rc != MARS_OK) {
            mars_model_free(m);
            return rc;
        }
        m->umma_ready = big;
    }
    *out = m;
    return MARS_OK;
}

mars_status_t mars_model_free(mars_model_t* m) {
    if (!m) return MARS_ERR_BAD_HANDLE;
    for (cudaEvent_t e : m->ev_pool) cudaEventDestroy(e);
    for (int i = 0; i < kStagingSlots; ++i) {
        if (m->staged[i]) cudaEventDestroy(m->staged[i]);
        if (m->staging[i]) cudaFreeHost(m->staging[i]);
    }
    delete m;
    return MARS_OK;
}

// ------------------------------------------------------------------------------- paged KV cache

size_t mars_kv_meta_bytes(int32_t max_seqs, int32_t max_pages_per_seq) {
    if (max_seqs < 1 || max_pages_per_seq < 1) return 0;
    return align_up((size_t)max_seqs * max_pages_per_seq * 4, 256);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static mars_status_t make_pool_map(CUtensorMap* tm, void* pool, uint64_t rows, int D, int box_rows) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (!fn || qres != cudaDriverEntryPointSuccess) return MARS_ERR_UNSUPPORTED;
    const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)D * 2};
    const cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1u, 1u};
    CUresult r = ((EncodeTiledFn)fn)(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, pool, dims, strides, box, estr,
                                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        g_last_cuda_error = (int32_t)r;
        return MARS_ERR_CUDA;
    }
    return MARS_OK;
}

mars_status_t mars_kv_alloc(mars_model_t* m, void* k_pool, void* v_pool, size_t pool_bytes_each, int32_t page_size,
                            int32_t max_seqs, int32_t max_pages_per_seq, void* meta, size_t meta_bytes, mars_kv_t** out) {
    if (!m) return MARS_ERR_BAD_HANDLE;
    if (!k_pool || !v_pool || !meta || !out || max_seqs < 1 || max_pages_per_seq < 1) return MARS_ERR_INVALID_ARG;
    if (page_size != 16 && page_size != 32 && page_size != 64 && page_size != 128) return MARS_ERR_INVALID_ARG;
    if ((uintptr_t)k_pool % 256 || (uintptr_t)v_pool % 256 || (uintptr_t)meta % 256) return MARS_ERR_INVALID_ARG;
    if (meta_bytes < mars_kv_meta_bytes(max_seqs, max_pages_per_seq)) return MARS_ERR_INVALID_ARG;
    const mars_config_t& c = m->cfg;
    const size_t page_bytes = (size_t)c.n_kv_heads * page_size * c.head_dim * 2;
    const size_t n_pages = pool_bytes_each / page_bytes / c.n_layers;
    if (n_pages < 1 || n_pages > 0x3fffffff) return MARS_ERR_INVALID_ARG;
    const uint64_t rows = (uint64_t)c.n_layers * n_pages * c.n_kv_heads * page_size;
    if (rows > 0x7fffffffull) return MARS_ERR_UNSUPPORTED;
    mars_kv* kv = new (std::nothrow) mars_kv();
    if (!kv) return MARS_ERR_INVALID_ARG;
    kv->model = m;
    kv->view = KvView{(__nv_bfloat16*)k_pool, (__nv_bfloat16*)v_pool, (int32_t*)meta, (int)n_pages, page_size,
                      max_pages_per_seq};
    kv->max_seqs = max_seqs;
    const int box_rows = std::min(page_size, 64);
    mars_status_t st = make_pool_map(&kv->tm_k, k_pool, rows, c.head_dim, box_rows);
    if (st == MARS_OK) st = make_pool_map(&kv->tm_v, v_pool, rows, c.head_dim, box_rows);
    if (st != MARS_OK) { delete kv; return st; }
    cudaError_t e = cudaStreamCreateWithFlags(&kv->copy_stream, cudaStreamNonBlocking);
    if (e != cudaSuccess) { g_last_cuda_error = (int32_t)e; delete kv; return MARS_ERR_CUDA; }
    e = cudaMemsetAsync(meta, 0, mars_kv_meta_bytes(max_seqs, max_pages_per_seq), kv->copy_stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(kv->copy_stream);
    if (e != cudaSuccess) { g_last_cuda_error = (int32_t)e; cudaStreamDestroy(kv->copy_stream); delete kv; return MARS_ERR_CUDA; }
    kv->seqs.resize(max_seqs);
    kv->refs.assign(n_pages, 0);
    kv->free_list.resize(n_pages);
    for (size_t i = 0; i < n_pages; ++i) kv->free_list[i] = (int32_t)(n_pages - 1 - i);   // page 0 is handed out first
    *out = kv;
    return MARS_OK;
}

mars_status_t mars_kv_free(mars_kv_t* kv) {
    if (!kv) return MARS_ERR_BAD_HANDLE;
    if (kv->copy_stream) cudaStreamDestroy(kv->copy_stream);
    delete kv;
    return MARS_OK;
}

int32_t mars_kv_num_pages(const mars_kv_t* kv) { return kv ? kv->view.n_pages : -1; }
int32_t mars_kv_free_pages(const mars_kv_t* kv) { return kv ? (int32_t)kv->free_list.size() : -1; }

// Writes entries [first, first + count) of a slot's block-table row.  The copy runs on the cache's own
// stream and has finished when this returns, so kernels launched afterwards on ANY stream (blocking or
// not) see the row; a synchronous copy on the default stream would only be ordered against blocking
// streams.  The entries written are new to the device (pages appended to a slot, or a slot that was
// empty), so steps still in flight on the caller's stream never read them.
static mars_status_t upload_row(mars_kv* kv, int seq, int first, int count) {
    if (count <= 0) return MARS_OK;
    CUDA_TRY(cudaMemcpyAsync(kv->view.block_table + (size_t)seq * kv->view.max_pages_per_seq + first,
                             kv->seqs[seq].pages.data() + first, (size_t)count * 4, cudaMemcpyHostToDevice,
                             kv->copy_stream));
    CUDA_TRY(cudaStreamSynchronize(kv->copy_stream));
    return MARS_OK;
}

// The page that receives position `len` must belong to this slot alone (pages shared by
// mars_kv_seq_fork hold only positions below the fork point and are never written again).
static bool next_write_is_private(const mars_kv* kv, const SeqState& s, int len) {
    const size_t idx = (size_t)(len / kv->view.page_size);
    return idx >= s.pages.size() || kv->refs[s.pages[idx]] == 1;
}

mars_status_t mars_kv_seq_reserve(mars_kv_t* kv, int32_t seq, int32_t n_tokens_total) {
    if (!kv || seq < 0 || seq >= kv->max_seqs) return MARS_ERR_BAD_HANDLE;
    if (n_tokens_total < 0 || n_tokens_total > kv->model->cfg.max_pos) return MARS_ERR_INVALID_ARG;
    SeqState& s = kv->seqs[seq];
    const int ps = kv->view.page_size;
    const int need = (n_tokens_total + ps - 1) / ps;
    const int have = (int)s.pages.size();
    if (need > kv->view.max_pages_per_seq) return MARS_ERR_KV_FULL;
    if (need - have > (int)kv->free_list.size()) return MARS_ERR_KV_FULL;
    for (int i = have; i < need; ++i) {
        const int32_t p = kv->free_list.back();
        kv->free_list.pop_back();
        kv->refs[p] = 1;
        s.pages.push_back(p);
    }
    s.used = true;
    return upload_row(kv, seq, have, need - have);
}

mars_status_t mars_kv_seq_adopt(mars_kv_t* kv, int32_t seq, const int32_t* pages, int32_t n_pages, int32_t ctx_len) {
    if (!kv || seq < 0 || seq >= kv->max_seqs) return MARS_ERR_BAD_HANDLE;
    if (!pages || n_pages < 0 || ctx_len < 0) return MARS_ERR_INVALID_ARG;
    if (n_pages > kv->view.max_pages_per_seq || (int64_t)ctx_len > (int64_t)n_pages * kv->view.page_size)
        return MARS_ERR_INVALID_ARG;
    SeqState& s = kv->seqs[seq];
    if (s.used) return MARS_ERR_BAD_HANDLE;
    std::vector<int32_t> sorted(pages, pages + n_pages);
    std::sort(sorted.begin(), sorted.end());
    for (int i = 0; i < n_pages; ++i) {
        if (sorted[i] < 0 || sorted[i] >= kv->view.n_pages) return MARS_ERR_INVALID_ARG;
        if (kv->refs[sorted[i]] || (i > 0 && sorted[i] == sorted[i - 1])) return MARS_ERR_BAD_HANDLE;
    }
    for (int i = 0; i < n_pages; ++i) kv->refs[pages[i]] = 1;
    kv->free_list.erase(std::remove_if(kv->free_list.begin(), kv->free_list.end(),
                                       [&](int32_t p) { return std::binary_search(sorted.begin(), sorted.end(), p); }),
                        kv->free_list.end());
    s.pages.assign(pages, pages + n_pages);
    s.len = ctx_len;
    s.used = true;
    return upload_row(kv, seq, 0, n_pages);
}

mars_status_t mars_kv_seq_set_len(mars_kv_t* kv, int32_t seq, int32_t ctx_len) {
    if (!kv || seq < 0 || seq >= kv->max_seqs || !kv->seqs[seq].used) return MARS_ERR_BAD_HANDLE;
    if (ctx_len < 0 || (int64_t)ctx_len > (int64_t)kv->seqs[seq].pages.size() * kv->view.page_size)
        return MARS_ERR_INVALID_ARG;
    if (!next_write_is_private(kv, kv->seqs[seq], ctx_len)) return MARS_ERR_INVALID_ARG;   // would append into a shared page
    kv->seqs[seq].len = ctx_len;
    return MARS_OK;
}

mars_status_t mars_kv_seq_release(mars_kv_t* kv, int32_t seq) {
    if (!kv || seq < 0 || seq >= kv->max_seqs || !kv->seqs[seq].used) return MARS_ERR_BAD_HANDLE;
    SeqState& s = kv->seqs[seq];
    for (auto it = s.pages.rbegin(); it != s.pages.rend(); ++it)
        if (--kv->refs[*it] == 0) kv->free_list.push_back(*it);   // shared pages stay until their last holder goes
    s = SeqState();
    return MARS_OK;
}

int32_t mars_kv_seq_len(const mars_kv_t* kv, int32_t seq) {
    if (!kv || seq < 0 || seq >= kv->max_seqs || !kv->seqs[seq].used) return -1;
    return kv->seqs[seq].len;
}

mars_status_t mars_kv_block_table(const mars_kv_t* kv, int32_t seq, int32_t* pages_out, int32_t cap, int32_t* n) {
    if (!kv || seq < 0 || seq >= kv->max_seqs || !kv->seqs[seq].used) return MARS_ERR_BAD_HANDLE;
    if (!n || cap < 0 || (cap > 0 && !pages_out)) return MARS_ERR_INVALID_ARG;
    const auto& p = kv->seqs[seq].pages;
    *n = (int32_t)p.size();
    for (int i = 0; i < std::min<int>(cap, (int)p.size()); ++i) pages_out[i] = p[i];
    return MARS_OK;
}

// ---- parking, resuming and forking a sequence (segment rollouts, grouped agent rollouts)

static size_t layer_page_bytes(const mars_kv* kv) {
    const mars_config_t& c = kv->model->cfg;
    return (size_t)c.n_kv_heads * kv->view.page_size * c.head_dim * 2;
}

size_t mars_kv_seq_image_bytes(const mars_kv_t* kv, int32_t n_tokens) {
    if (!kv || n_tokens < 0) return 0;
    const int ps = kv->view.page_size;
    return 2 * (size_t)kv->model->cfg.n_layers * (size_t)((n_tokens + ps - 1) / ps) * layer_page_bytes(kv);
}

// A kernel will read or write `p`: it must be device memory or page-locked host memory.
static mars_status_t kernel_visible(const void* p, unsigned char** dev_ptr) {
    cudaPointerAttributes attr;
    CUDA_TRY(cudaPointerGetAttributes(&attr, p));
    if (attr.type == cudaMemoryTypeUnregistered || !attr.devicePointer) return MARS_ERR_INVALID_ARG;
    *dev_ptr = (unsigned char*)attr.devicePointer;
    return MARS_OK;
}

// Packed image: [K | V][layer][page index in the sequence][n_kv_heads][page_size][head_dim].
static mars_status_t move_image(mars_kv* kv, int seq, unsigned char* image, int n_pages, bool to_image, cudaStream_t st) {
    const mars_config_t& c = kv->model->cfg;
    const size_t pb = layer_page_bytes(kv);
    const int32_t* row = kv->view.block_table + (size_t)seq * kv->view.max_pages_per_seq;
    for (int which = 0; which < 2; ++which) {
        unsigned char* pool = (unsigned char*)(which ? kv->view.v_pool : kv->view.k_pool);
        unsigned char* img = image + (size_t)which * c.n_layers * n_pages * pb;
        PageCopy pc;
        pc.n_pages = n_pages; pc.n_layers = c.n_layers; pc.page_bytes = (uint32_t)pb;
        if (to_image) {
            pc.src = pool; pc.src_layer_stride = (size_t)kv->view.n_pages * pb; pc.src_pages = row;
            pc.dst = img;  pc.dst_layer_stride = (size_t)n_pages * pb;          pc.dst_pages = nullptr;
        } else {
            pc.src = img;  pc.src_layer_stride = (size_t)n_pages * pb;          pc.src_pages = nullptr;
            pc.dst = pool; pc.dst_layer_stride = (size_t)kv->view.n_pages * pb; pc.dst_pages = row;
        }
        launch_kv_page_copy(pc, kv->model->sm_count, st);
    }
    CUDA_TRY(cudaGetLastError());
    kv->model->last_stream = st;
    return MARS_OK;
}

mars_status_t mars_kv_seq_export(mars_kv_t* kv, int32_t seq, void* image, size_t image_bytes, void* cuda_stream) {
    if (!kv || seq < 0 || seq >= kv->max_seqs || !kv->seqs[seq].used) return MARS_ERR_BAD_HANDLE;
    const SeqState& s = kv->seqs[seq];
    const size_t need = mars_kv_seq_image_bytes(kv, s.len);
    if (!image || image_bytes < need || (uintptr_t)image % 16) return MARS_ERR_INVALID_ARG;
    if (need == 0) return MARS_OK;
    unsigned char* img = nullptr;
    const mars_status_t rc = kernel_visible(image, &img);
    if (rc != MARS_OK) return rc;
    const int ps = kv->view.page_size;
    return move_image(kv, seq, img, (s.len + ps - 1) / ps, true, (cudaStream_t)cuda_stream);
}

mars_status_t mars_kv_seq_import(mars_kv_t* kv, int32_t seq, const void* image, size_t image_bytes, int32_t n_tokens,
                                 void* cuda_stream) {
    if (!kv || seq < 0 || seq >= kv->max_seqs || kv->seqs[seq].used) return MARS_ERR_BAD_HANDLE;
    if (n_tokens < 0 || n_tokens > kv->model->cfg.max_pos) return MARS_ERR_INVALID_ARG;
    const size_t need = mars_kv_seq_image_bytes(kv, n_tokens);
    if (!image || image_bytes < need || (uintptr_t)image % 16) return MARS_ERR_INVALID_ARG;
    unsigned char* img = nullptr;
    if (need) {
        const mars_status_t rc = kernel_visible(image, &img);
        if (rc != MARS_OK) return rc;
    }
    mars_status_t rc = mars_kv_seq_reserve(kv, seq, n_tokens);
    if (rc != MARS_OK) return rc;
    const int ps = kv->view.page_size;
    if (need) rc = move_image(kv, seq, img, (n_tokens + ps - 1) / ps, false, (cudaStream_t)cuda_stream);
    if (rc != MARS_OK) {
        mars_kv_seq_release(kv, seq);
        return rc;
    }
    kv->seqs[seq].len = n_tokens;
    return MARS_OK;
}

mars_status_t mars_kv_seq_fork(mars_kv_t* kv, int32_t src, int32_t dst, void* cuda_stream) {
    if (!kv || src < 0 || src >= kv->max_seqs || dst < 0 || dst >= kv->max_seqs || src == dst) return MARS_ERR_BAD_HANDLE;
    if (!kv->seqs[src].used || kv->seqs[dst].used) return MARS_ERR_BAD_HANDLE;
    const SeqState& a = kv->seqs[src];
    SeqState& b = kv->seqs[dst];
    const int ps = kv->view.page_size;
    const int full = a.len / ps;
    const bool tail = a.len % ps != 0;
    if (tail && kv->free_list.empty()) return MARS_ERR_KV_FULL;
    b.pages.assign(a.pages.begin(), a.pages.begin() + full);
    for (int32_t p : b.pages) ++kv->refs[p];
    if (tail) {   // the page both would append to is copied, not shared
        const int32_t p = kv->free_list.back();
        kv->free_list.pop_back();
        kv->refs[p] = 1;
        b.pages.push_back(p);
    }
    b.len = a.len;
    b.used = true;
    mars_status_t rc = upload_row(kv, dst, 0, (int)b.pages.size());
    if (rc == MARS_OK && tail) {
        const size_t pb = layer_page_bytes(kv);
        for (int which = 0; which < 2 && rc == MARS_OK; ++which) {
            unsigned char* pool = (unsigned char*)(which ? kv->view.v_pool : kv->view.k_pool);
            PageCopy pc;
            pc.src = pool; pc.dst = pool;
            pc.src_layer_stride = pc.dst_layer_stride = (size_t)kv->view.n_pages * pb;
            pc.src_pages = kv->view.block_table + (size_t)src * kv->view.max_pages_per_seq + full;
            pc.dst_pages = kv->view.block_table + (size_t)dst * kv->view.max_pages_per_seq + full;
            pc.n_pages = 1; pc.n_layers = kv->model->cfg.n_layers; pc.page_bytes = (uint32_t)pb;
            launch_kv_page_copy(pc, kv->model->sm_count, (cudaStream_t)cuda_stream);
        }
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) { g_last_cuda_error = (int32_t)e; rc = MARS_ERR_CUDA; }
        kv->model->last_stream = (cudaStream_t)cuda_stream;
    }
    if (rc != MARS_OK) mars_kv_seq_release(kv, dst);
    return rc;
}

mars_status_t mars_kv_share_reads(mars_kv_t* kv, int32_t enable) {
    if (!kv) return MARS_ERR_BAD_HANDLE;
    kv->share_reads = enable != 0;
    return MARS_OK;
}

int32_t mars_kv_page_refs(const mars_kv_t* kv, int32_t page) {
    if (!kv || page < 0 || page >= kv->view.n_pages) return -1;
    return kv->refs[page];
}

// ------------------------------------------------------------------------------------- the step

namespace {

struct StepPlan {
    std::vector<int32_t> tok_seq, tok_pos, emit_rows, emit_slot, updates;
    const int32_t* tokens_dev;
    int span;   // cached tokens per attention item (decode)
    bool prefill = false;   // the call has prompt rows (blocks of consecutive tokens for the causal kernel)
    int n_decode = 0;       // rows [0, n_decode) are decode rows (one new token attending over its cache in
                            // spans); rows after them are prompt rows.  Set by the entry points.
    const int32_t* score_targets = nullptr;   // scoring pass: device [n_tok] target token per row (< 0: none)
    float score_temperature = 1.f;
};

mars_status_t run_step(mars_model* m, mars_kv* kv, cudaStream_t st, const StepPlan& plan, const mars_sampling_t& smp,
                       int32_t* out_tokens, float* out_logprobs, const mars_debug_t* dbg) {
    const int n_tok = (int)plan.tok_seq.size();
    const int n_emit = (int)plan.emit_rows.size();
    const StepLayout& lay = m->lay;

    // Decode rows whose sequences list the same pages from position 0 on (forked members of a rollout
    // group): the common prefix, in whole pages strictly below every member's new position, is read
    // once per block of kSharedRows rows by the shared-prefix kernel; the rest of each row as usual.
    const int n_dec = plan.n_decode;
    const int ps = kv->view.page_size;
    struct SharedGroup { std::vector<int> rows; int tokens; };
    std::vector<SharedGroup> shared;
    std::vector<int> row_shared((size_t)n_dec, 0);   // tokens of the row that the shared kernel covers
    if (kv->share_reads && n_dec > 1) {
        std::vector<std::pair<int32_t, int>> first;   // (first page, index in `shared`), few entries
        for (int t = 0; t < n_dec; ++t) {
            const SeqState& q = kv->seqs[plan.tok_seq[t]];
            if (q.pages.empty() || kv->refs[q.pages[0]] < 2) continue;
            size_t gi = 0;
            while (gi < first.size() && first[gi].first != q.pages[0]) ++gi;
            if (gi == first.size()) {
                first.emplace_back(q.pages[0], (int)shared.size());
                shared.push_back(SharedGroup{{}, 0});
            }
            shared[first[gi].second].rows.push_back(t);
        }
        for (SharedGroup& g : shared) {
            if (g.rows.size() < 2) continue;
            const std::vector<int32_t>& p0 = kv->seqs[plan.tok_seq[g.rows[0]]].pages;
            size_t common = p0.size();
            int min_pos = plan.tok_pos[g.rows[0]];
            for (size_t i = 1; i < g.rows.size(); ++i) {
                const std::vector<int32_t>& pi = kv->seqs[plan.tok_seq[g.rows[i]]].pages;
                size_t c = 0;
                while (c < common && c < pi.size() && pi[c] == p0[c]) ++c;
                common = c;
                min_pos = std::min(min_pos, plan.tok_pos[g.rows[i]]);
            }
            const int tokens = (int)std::min<int64_t>((int64_t)common * ps, (int64_t)(min_pos / ps) * ps);
            if (tokens < kMinSharedTokens) continue;
            g.tokens = tokens;
            for (int r : g.rows) row_shared[r] = tokens;
        }
    }

    // attention work items: spans of `span` cached tokens per token row (widened until they fit)
    int span = plan.span;
    int64_t n_items = 0;
    // consecutive prompt tokens per item of the causal prefill kernel: 16 (x 8 heads = 128 tensor-core rows)
    // where the tcgen05 kernel applies, else 4 (one per warp of the mma.sync kernel)
    const bool fattn = m->fattn_ready && n_tok > n_dec;
    const int kPrefillBlock = fattn ? fattn_block_tokens() : 4;
    int64_t pf_items = 0;
    for (int t = n_dec; t < n_tok;) {
        int e = t + 1;
        while (e < n_tok && e - t < kPrefillBlock && plan.tok_seq[e] == plan.tok_seq[t]) ++e;
        t = e;
        ++pf_items;
    }
    if (pf_items > m->caps.n_items) return MARS_ERR_INVALID_ARG;
    // rows per shared item and words per item: 16 rows on the tcgen05 kernel, 4 on the mma.sync kernel
    const bool fa_shared = m->fattn_shared_ready;
    const int sh_rows = fa_shared ? fattn_shared_rows() : kSharedRows;
    const int sh_words = fa_shared ? fattn_shared_item_words() : 12;
    int64_t dec_items = 0, dec_slots = 0, sh_items = 0;
    for (;;) {
        dec_items = dec_slots = sh_items = 0;
        for (int t = 0; t < n_dec; ++t) {
            const int64_t own = ((int64_t)plan.tok_pos[t] + 1 - row_shared[t] + span - 1) / span;
            dec_items += own;
            dec_slots += own + (row_shared[t] + span - 1) / span;
        }
        for (const SharedGroup& g : shared)
            sh_items += (int64_t)((g.tokens + span - 1) / span) * (((int64_t)g.rows.size() + sh_rows - 1) / sh_rows);
        if (dec_slots + pf_items <= m->caps.n_items && sh_items <= m->caps.n_items / 2 + 1) break;
        if (span > (1 << 28)) return MARS_ERR_INVALID_ARG;
        span *= 2;
    }
    n_items = dec_items + pf_items + sh_items;

    const int slot = m->next_slot;
    m->next_slot = (slot + 1) % kStagingSlots;
    CUDA_TRY(cudaEventSynchronize(m->staged[slot]));
    int32_t* blk = m->staging[slot];
    std::memset(blk, 0, H_WORDS * 4);
    blk[H_NTOK] = n_tok;
    blk[H_NITEMS] = (int32_t)dec_items;
    blk[H_PF_FIRST] = (int32_t)dec_items;
    blk[H_PF_ITEMS] = (int32_t)pf_items;
    blk[H_NUPDATES] = (int32_t)(plan.updates.size() / 3);
    blk[H_NEMIT] = n_emit;
    blk[H_GREEDY] = smp.greedy ? 1 : 0;
    std::memcpy(&blk[H_TEMPERATURE], &smp.temperature, 4);
    std::memcpy(&blk[H_TOP_P], &smp.top_p, 4);
    blk[H_SEED_LO] = (int32_t)(uint32_t)smp.seed;
    blk[H_SEED_HI] = (int32_t)(uint32_t)(smp.seed >> 32);
    blk[H_STEP_LO] = (int32_t)(uint32_t)smp.step;
    blk[H_STEP_HI] = (int32_t)(uint32_t)(smp.step >> 32);
    std::memcpy(blk + lay.tok_seq, plan.tok_seq.data(), (size_t)n_tok * 4);
    std::memcpy(blk + lay.tok_pos, plan.tok_pos.data(), (size_t)n_tok * 4);
    if (n_emit) {
        std::memcpy(blk + lay.emit_rows, plan.emit_rows.data(), (size_t)n_emit * 4);
        std::memcpy(blk + lay.emit_slot, plan.emit_slot.data(), (size_t)n_emit * 4);
    }
    if (!plan.updates.empty()) std::memcpy(blk + lay.updates, plan.updates.data(), plan.updates.size() * 4);
    blk[H_SH_ITEMS] = (int32_t)sh_items;
    int64_t kv_tokens = 0, kv_streamed = 0;
    {
        int32_t* items = blk + lay.items;
        int32_t* off = blk + lay.tok_item_off;
        // partial slots of a decode row: its shared spans first, then its own spans
        int slot_at = 0;
        for (int t = 0; t < n_dec; ++t) {
            off[t] = slot_at;
            const int len = plan.tok_pos[t] + 1;
            slot_at += (row_shared[t] + span - 1) / span + (len - row_shared[t] + span - 1) / span;
        }
        int at = 0;
        for (int t = 0; t < n_dec; ++t) {
            const int len = plan.tok_pos[t] + 1;
            kv_tokens += len;
            int slot_i = off[t] + (row_shared[t] + span - 1) / span;
            for (int s0 = row_shared[t]; s0 < len; s0 += span) {
                items[4 * at + 0] = t;
                items[4 * at + 1] = s0;
                items[4 * at + 2] = std::min(span, len - s0);
                items[4 * at + 3] = slot_i++;
                kv_streamed += items[4 * at + 2];
                ++at;
            }
        }
        int32_t* sh = blk + lay.sh_items;
        int sh_at = 0;
        for (const SharedGroup& g : shared) {
            for (int s0 = 0; s0 < g.tokens; s0 += span) {
                for (size_t r0 = 0; r0 < g.rows.size(); r0 += (size_t)sh_rows) {
                    const int nr = (int)std::min<size_t>((size_t)sh_rows, g.rows.size() - r0);
                    int32_t* it = sh + sh_words * sh_at++;
                    it[0] = s0; it[1] = std::min(span, g.tokens - s0); it[2] = nr; it[3] = 0;
                    for (int i = 0; i < sh_rows; ++i) {
                        const int row = g.rows[r0 + (size_t)std::min(i, nr - 1)];
                        it[4 + i] = row;
                        it[4 + sh_rows + i] = off[row] + s0 / span;
                    }
                    kv_streamed += it[1];
                }
            }
        }
        // blocks of consecutive tokens of one request: (first row, 0, keys visible to the last one, count)
        for (int t = n_dec; t < n_tok;) {
            int e = t + 1;
            while (e < n_tok && e - t < kPrefillBlock && plan.tok_seq[e] == plan.tok_seq[t]) ++e;
            items[4 * at + 0] = t;
            items[4 * at + 1] = 0;
            items[4 * at + 2] = plan.tok_pos[e - 1] + 1;
            items[4 * at + 3] = e - t;
            for (int q = t; q < e; ++q) { off[q] = slot_at; kv_tokens += plan.tok_pos[q] + 1; }
            kv_streamed += plan.tok_pos[e - 1] + 1;
            ++at;
            t = e;
        }
        off[n_tok] = slot_at;
    }
    // one copy uploads the whole block up to the last item
    const size_t used_words = (size_t)lay.items + 4 * (size_t)(dec_items + pf_items);
    CUDA_TRY(cudaMemcpyAsync(m->buf.step, blk, used_words * 4, cudaMemcpyHostToDevice, st));
    if (sh_items)
        CUDA_TRY(cudaMemcpyAsync(m->buf.step + lay.sh_items, blk + lay.sh_items, (size_t)sh_items * sh_words * 4,
                                 cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaEventRecord(m->staged[slot], st));

    const Shape& s = m->shape;
    const Buffers& b = m->buf;
    DebugTaps taps{nullptr, nullptr, nullptr, nullptr, nullptr};
    if (dbg) taps = DebugTaps{dbg->hidden, dbg->router_w, dbg->router_idx, dbg->forced_idx, dbg->nucleus_mass};
    const size_t hid_stride = (size_t)n_tok * s.H;

    int launches = 0;
    cudaError_t ev_err = cudaSuccess;
    // runs one launch wrapper, bracketed by an event pair when profiling is on
    auto run = [&](int cls, auto&& fn) {
        cudaEvent_t e0 = nullptr, e1 = nullptr;
        if (m->profiling && ev_err == cudaSuccess) {
            while (m->ev_pool.size() < m->ev_used + 2 && ev_err == cudaSuccess) {
                cudaEvent_t e;
                ev_err = cudaEventCreate(&e);
                if (ev_err == cudaSuccess) m->ev_pool.push_back(e);
            }
            if (ev_err == cudaSuccess) {
                e0 = m->ev_pool[m->ev_used];
                e1 = m->ev_pool[m->ev_used + 1];
                m->ev_used += 2;
                m->ev_class.push_back(cls);
                ev_err = cudaEventRecord(e0, st);
            }
        }
        launches += fn();
        if (e1 && ev_err == cudaSuccess) ev_err = cudaEventRecord(e1, st);
    };
    run(MARS_K_OTHER, [&] { return launch_prep(s, b, lay, kv->view, n_tok, st); });
    run(MARS_K_OTHER, [&] {
        return launch_embed(s, b, lay, m->embed, plan.tokens_dev, m->layers[0].attn_norm, taps.hidden, n_tok, st);
    });
    // Three regimes by token rows: up to 64 and up to 256 rows are weight streams (swap-AB projections with
    // 64 / 128 / 256 token columns, split-K partials, streaming expert kernels); beyond that the
    // projections and the experts are dense contractions on 128 x 256 tensor-core tiles.
    const bool umma = m->umma_ready && n_tok > umma_swap_max_tokens();
    const int qkv_split = umma_swap_splits((s.nq + 2 * s.nkv) * s.D, n_tok, s.H);
    const int o_split = umma_swap_splits(s.H, n_tok, s.nq * s.D);
    for (int l = 0; l < s.L; ++l) {
        const LayerW& w = m->layers[l];
        if (umma) {   // prefill-sized call: dense contractions on tcgen05 / TMEM
            const int qkv_rows = (s.nq + 2 * s.nkv) * s.D;
            run(MARS_K_QKV, [&] {   // per-head norm, RoPE and the cache append happen in the contraction's epilogue
                const QkvEpilogue ep{b.step + lay.tok_pos, b.step + lay.tok_seq, kv->view.block_table, b.rope, w.q_norm, w.k_norm,
                                     b.q, kv->view.k_pool, kv->view.v_pool, kv->view.max_pages_per_seq, kv->view.n_pages,
                                     kv->view.page_size, l, s.nq, s.nkv, s.D, s.qk_norm, s.eps};
                return launch_umma_qkv(m->tm_h, m->tm_wqkv[l], n_tok, qkv_rows, s.H, ep, b.err, (m->lo_planes >> 0) & 1, st);
            });
        } else {      // decode-sized call: weights stream once through tcgen05 with the operands swapped
            run(MARS_K_QKV, [&] {
                const int ksplit = qkv_split;
                int n = launch_umma_swap(m->tm_wqkv[l], m->tm_h64, (s.nq + 2 * s.nkv) * s.D, n_tok, s.H, ksplit, b.qkv, b.err, st);
                return n + launch_qkv_post(s, b, lay, w, kv->view, l, n_tok, ksplit, st);
            });
        }
        if (n_dec > 0) {      // decode rows: spans of cached tokens, then the merge of each row's spans
            if (sh_items)
                run(MARS_K_ATTN, [&] {
                    if (fa_shared)
                        return launch_fattn_shared(s, b, lay, kv->view, m->tm_q1, kv->tm_k, kv->tm_v, l, (int)sh_items,
                                                   m->sm_count, st);
                    return launch_attention_shared(s, b, lay, kv->view, kv->tm_k, kv->tm_v, l, (int)sh_items, m->sm_count, st);
                });
            run(MARS_K_ATTN, [&] { return launch_attention(s, b, lay, kv->view, kv->tm_k, kv->tm_v, l, m->sm_count, st); });
            run(MARS_K_ATTN_MERGE, [&] { return launch_attn_merge(s, b, lay, n_dec, st); });
        }
        if (n_dec < n_tok) {  // prompt rows: causal kernel over blocks of tokens; writes the merged output itself
            run(MARS_K_ATTN, [&] {
                if (fattn)
                    return launch_fattn_prefill(s, b, lay, kv->view, m->tm_q, kv->tm_k, kv->tm_v, l, (int)pf_items,
                                                m->sm_count, st);
                return launch_attention_prefill(s, b, lay, kv->view, kv->tm_k, kv->tm_v, l, m->sm_count, st);
            });
        }
        if (umma) {
            run(MARS_K_OPROJ, [&] {
                return launch_umma_dense(m->tm_o, m->tm_wo[l], n_tok, s.H, s.nq * s.D, b.opart, b.err, (m->lo_planes >> 1) & 1, st);
            });
            run(MARS_K_ROUTER, [&] {
                int n = launch_resid_norm(s, b, w, n_tok, 1, st);
                n += launch_umma_dense(m->tm_h, m->tm_router[l], n_tok, s.E, s.H, b.rlogits, b.err, (m->lo_planes >> 2) & 1, st);
                return n + launch_route_select(s, b, taps, l, n_tok, 128, 1, st);
            });
            run(MARS_K_GATE_UP, [&] {
                return launch_umma_experts(s, b, m->tm_xperm, m->tm_wgu[l], m->tm_act, m->tm_wdown[l], n_tok, (m->lo_planes >> 3) & 1,
                                           (m->lo_planes >> 4) & 1, st);
            });
        } else {
            run(MARS_K_OPROJ, [&] {
                return launch_umma_swap(m->tm_wo[l], m->tm_o64, s.H, n_tok, s.nq * s.D, o_split, b.opart, b.err, st);
            });
            run(MARS_K_ROUTER, [&] { return launch_router(s, b, w, taps, l, n_tok, 0, o_split, st); });
            run(MARS_K_GATE_UP, [&] { return launch_gate_up(s, b, w, n_tok, m->sm_count, st); });
            run(MARS_K_DOWN, [&] { return launch_down(s, b, w, n_tok, st); });
        }
        if (dbg && dbg->expert_off)      // the permutation's integer outputs, for tests
            CUDA_TRY(cudaMemcpyAsync(dbg->expert_off + (size_t)l * (s.E + 1), b.expert_off, ((size_t)s.E + 1) * 4,
                                     cudaMemcpyDeviceToDevice, st));
        if (dbg && dbg->slot_token)
            CUDA_TRY(cudaMemcpyAsync(dbg->slot_token + (size_t)l * n_tok * s.k, b.slot_token, (size_t)n_tok * s.k * 4,
                                     cudaMemcpyDeviceToDevice, st));
        const __nv_bfloat16* next_gain = l + 1 < s.L ? m->layers[l + 1].attn_norm : m->final_norm;
        float* tap = taps.hidden ? taps.hidden + (size_t)(l + 1) * hid_stride : nullptr;
        run(MARS_K_COMBINE, [&] { return launch_combine(s, b, next_gain, tap, n_tok, st); });
    }
    if (n_emit) {
        run(MARS_K_LM_HEAD, [&] {
            // decode: the emitting rows are the token rows in order, so the tensor maps over b.h apply
            // (more token columns would make the swapped kernel re-read the activations once per 128 vocabulary rows)
            if (!plan.prefill && n_emit <= kUmmaMinTokens)
                return launch_umma_swap(m->tm_lm, m->tm_h64, s.V, n_emit, s.H, 1, b.logits, b.err, st);
            if (!plan.prefill && m->umma_ready)
                return launch_umma_dense(m->tm_h, m->tm_lm, n_emit, s.V, s.H, b.logits, b.err, 1, st);
            return launch_lm_head(s, b, lay, m->lm_head, n_emit, m->sm_count, st);
        });
        if (dbg && dbg->logits)
            CUDA_TRY(cudaMemcpyAsync(dbg->logits, b.logits, (size_t)n_emit * s.V * 4, cudaMemcpyDeviceToDevice, st));
        run(MARS_K_SAMPLE, [&] {
            return launch_sample(s, b, lay, n_emit, m->sm_count, out_tokens, out_logprobs, taps.nucleus_mass, st);
        });
    }
    if (plan.score_targets) {
        // the last combine left rms(x) * final_norm of EVERY row in b.h; the expert outputs in b.y are dead
        float2* ml = reinterpret_cast<float2*>(b.y);
        float* zt = b.y + 2 * (size_t)score_vocab_tiles(s.V) * n_tok;
        run(MARS_K_LM_HEAD, [&] {
            return launch_umma_score(m->tm_h, m->tm_lm, n_tok, s.V, s.H, plan.score_targets, 1.f / plan.score_temperature,
                                     ml, zt, dbg ? dbg->logits : nullptr, out_logprobs, b.err, st);
        });
    }
    CUDA_TRY(ev_err);
    CUDA_TRY(cudaGetLastError());
    m->last_stream = st;
    m->info.kernel_launches = launches;
    m->info.attn_items = n_items;
    m->info.kv_tokens_read = kv_tokens;
    m->info.kv_tokens_streamed = kv_streamed;
    return MARS_OK;
}

}  // namespace

mars_status_t mars_decode_step(mars_model_t* m, mars_kv_t* kv, void* cuda_stream, int32_t n_seqs, const int32_t* seq_ids,
                               const int32_t* in_tokens, const mars_sampling_t* sampling, int32_t* out_tokens,
                               float* out_logprobs, const mars_debug_t* debug) {
    if (!m || !kv || kv->model != m) return MARS_ERR_BAD_HANDLE;
    if (!seq_ids || !in_tokens || !sampling || !out_tokens || !out_logprobs) return MARS_ERR_INVALID_ARG;
    if (n_seqs < 1 || n_seqs > m->max_decode) return MARS_ERR_INVALID_ARG;
    if (!sampling->greedy && (!(sampling->temperature > 0.f) || !(sampling->top_p > 0.f) || sampling->top_p > 1.f))
        return MARS_ERR_INVALID_ARG;
    const int ps = kv->view.page_size;
    StepPlan plan;
    plan.tokens_dev = in_tokens;
    plan.span = kSpanTokens;
    plan.n_decode = n_seqs;
    std::vector<uint8_t> seen(kv->max_seqs, 0);
    int new_pages = 0;
    for (int i = 0; i < n_seqs; ++i) {
        const int sq = seq_ids[i];
        if (sq < 0 || sq >= kv->max_seqs || !kv->seqs[sq].used || seen[sq]) return MARS_ERR_BAD_HANDLE;
        seen[sq] = 1;
        const SeqState& s = kv->seqs[sq];
        if (s.len + 1 > m->cfg.max_pos) return MARS_ERR_INVALID_ARG;
        if (!next_write_is_private(kv, s, s.len)) return MARS_ERR_BAD_HANDLE;
        if (s.len / ps >= (int)s.pages.size()) {
            if ((int)s.pages.size() + 1 > kv->view.max_pages_per_seq) return MARS_ERR_KV_FULL;
            ++new_pages;
        }
    }
    if (new_pages > (int)kv->free_list.size()) return MARS_ERR_KV_FULL;
    // nothing can fail on the host from here on except CUDA calls
    std::vector<std::pair<int, int32_t>> taken;
    for (int i = 0; i < n_seqs; ++i) {
        const int sq = seq_ids[i];
        SeqState& s = kv->seqs[sq];
        if (s.len / ps >= (int)s.pages.size()) {
            const int32_t p = kv->free_list.back();
            kv->free_list.pop_back();
            kv->refs[p] = 1;
            plan.updates.push_back(sq);
            plan.updates.push_back((int32_t)s.pages.size());
            plan.updates.push_back(p);
            s.pages.push_back(p);
            taken.emplace_back(sq, p);
        }
        plan.tok_seq.push_back(sq);
        plan.tok_pos.push_back(s.len);
        plan.emit_rows.push_back(i);
        plan.emit_slot.push_back(sq);
    }
    mars_status_t r = run_step(m, kv, (cudaStream_t)cuda_stream, plan, *sampling, out_tokens, out_logprobs, debug);
    if (r != MARS_OK) {
        for (auto it = taken.rbegin(); it != taken.rend(); ++it) {   // undo the page grabs
            kv->seqs[it->first].pages.pop_back();
            kv->refs[it->second] = 0;
            kv->free_list.push_back(it->second);
        }
        return r;
    }
    for (int i = 0; i < n_seqs; ++i) kv->seqs[seq_ids[i]].len += 1;
    return MARS_OK;
}

// Chunks of prompt tokens appended to their sequences, optionally together with decode rows (one new
// token per listed sequence) that travel through the same pass.  With score_targets == null this is
// the prefill / mixed call (sampling from the decode rows and from the last position of the chunks
// that ask for it), otherwise the scoring pass (a log-prob per row, chunks only).
static mars_status_t feed_chunks(mars_model_t* m, mars_kv_t* kv, void* cuda_stream, int32_t n_dec, const int32_t* dec_ids,
                                 const int32_t* dec_tokens, int32_t n_reqs, const int32_t* seq_ids,
                                 const int32_t* chunk_lens, const int32_t* tokens, const int32_t* emit_last,
                                 const mars_sampling_t* sampling, int32_t* out_tokens, float* out_logprobs,
                                 const mars_debug_t* debug, const int32_t* score_targets, float score_temperature) {
    if (!m || !kv || kv->model != m) return MARS_ERR_BAD_HANDLE;
    if (!seq_ids || !chunk_lens || !tokens || !sampling || n_reqs < 1 || n_dec < 0) return MARS_ERR_INVALID_ARG;
    if (n_dec > 0 && (!dec_ids || !dec_tokens)) return MARS_ERR_INVALID_ARG;
    if (!sampling->greedy && (!(sampling->temperature > 0.f) || !(sampling->top_p > 0.f) || sampling->top_p > 1.f))
        return MARS_ERR_INVALID_ARG;
    const int ps = kv->view.page_size;
    int64_t total = 0, new_pages = 0;
    int n_emit = n_dec;
    std::vector<uint8_t> seen(kv->max_seqs, 0);
    for (int i = 0; i < n_dec; ++i) {
        const int sq = dec_ids[i];
        if (sq < 0 || sq >= kv->max_seqs || !kv->seqs[sq].used || seen[sq]) return MARS_ERR_BAD_HANDLE;
        seen[sq] = 1;
        const SeqState& s = kv->seqs[sq];
        if (s.len + 1 > m->cfg.max_pos) return MARS_ERR_INVALID_ARG;
        if (!next_write_is_private(kv, s, s.len)) return MARS_ERR_BAD_HANDLE;
        if (s.len / ps >= (int)s.pages.size()) {
            if ((int)s.pages.size() + 1 > kv->view.max_pages_per_seq) return MARS_ERR_KV_FULL;
            ++new_pages;
        }
    }
    for (int r = 0; r < n_reqs; ++r) {
        const int sq = seq_ids[r];
        if (sq < 0 || sq >= kv->max_seqs || !kv->seqs[sq].used || seen[sq]) return MARS_ERR_BAD_HANDLE;
        seen[sq] = 1;
        if (chunk_lens[r] < 1) return MARS_ERR_INVALID_ARG;
        const SeqState& s = kv->seqs[sq];
        const int64_t end = (int64_t)s.len + chunk_lens[r];
        if (end > m->cfg.max_pos) return MARS_ERR_INVALID_ARG;
        if (!next_write_is_private(kv, s, s.len)) return MARS_ERR_BAD_HANDLE;
        const int64_t need = (end + ps - 1) / ps;
        if (need > kv->view.max_pages_per_seq) return MARS_ERR_KV_FULL;
        new_pages += std::max<int64_t>(0, need - (int64_t)s.pages.size());
        total += chunk_lens[r];
        if (emit_last && emit_last[r]) ++n_emit;
    }
    if (n_dec == 0 && total > m->max_prefill) return MARS_ERR_INVALID_ARG;
    if (n_dec + total > m->caps.n_tok) return MARS_ERR_INVALID_ARG;
    if (n_emit > m->caps.n_emit) return MARS_ERR_INVALID_ARG;
    if (n_emit && (!out_tokens || !out_logprobs)) return MARS_ERR_INVALID_ARG;
    if (new_pages > (int64_t)kv->free_list.size()) return MARS_ERR_KV_FULL;

    StepPlan plan;
    plan.tokens_dev = tokens;
    plan.span = kSpanTokens;
    plan.prefill = true;
    plan.n_decode = n_dec;
    plan.score_targets = score_targets;
    plan.score_temperature = score_temperature;
    std::vector<std::pair<int, int32_t>> taken;
    auto take_page = [&](int sq) {
        SeqState& s = kv->seqs[sq];
        const int32_t p = kv->free_list.back();
        kv->free_list.pop_back();
        kv->refs[p] = 1;
        plan.updates.push_back(sq);
        plan.updates.push_back((int32_t)s.pages.size());
        plan.updates.push_back(p);
        s.pages.push_back(p);
        taken.emplace_back(sq, p);
    };
    for (int i = 0; i < n_dec; ++i) {
        const int sq = dec_ids[i];
        SeqState& s = kv->seqs[sq];
        if (s.len / ps >= (int)s.pages.size()) take_page(sq);
        plan.tok_seq.push_back(sq);
        plan.tok_pos.push_back(s.len);
        plan.emit_rows.push_back(i);
        plan.emit_slot.push_back(sq);
    }
    int row = n_dec;
    for (int r = 0; r < n_reqs; ++r) {
        const int sq = seq_ids[r];
        SeqState& s = kv->seqs[sq];
        const int need = (s.len + chunk_lens[r] + ps - 1) / ps;
        while ((int)s.pages.size() < need) take_page(sq);
        for (int i = 0; i < chunk_lens[r]; ++i) {
            plan.tok_seq.push_back(sq);
            plan.tok_pos.push_back(s.len + i);
        }
        row += chunk_lens[r];
        if (emit_last && emit_last[r]) {
            plan.emit_rows.push_back(row - 1);
            plan.emit_slot.push_back(sq);
        }
    }
    auto undo = [&] {
        for (auto it = taken.rbegin(); it != taken.rend(); ++it) {
            kv->seqs[it->first].pages.pop_back();
            kv->refs[it->second] = 0;
            kv->free_list.push_back(it->second);
        }
    };
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (n_dec > 0) {
        // one token array for the embedding: decode tokens, then the chunks.  The routing-index buffer is
        // free until the first layer's router runs, which is after the embedding has read the tokens.
        int32_t* cat = m->buf.route_idx;
        cudaError_t e = cudaMemcpyAsync(cat, dec_tokens, (size_t)n_dec * 4, cudaMemcpyDeviceToDevice, stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(cat + n_dec, tokens, (size_t)total * 4, cudaMemcpyDeviceToDevice, stream);
        if (e != cudaSuccess) {
            g_last_cuda_error = (int32_t)e;
            undo();
            return MARS_ERR_CUDA;
        }
        plan.tokens_dev = cat;
    }
    mars_status_t st = run_step(m, kv, stream, plan, *sampling, out_tokens, out_logprobs, debug);
    if (st != MARS_OK) {
        undo();
        return st;
    }
    for (int i = 0; i < n_dec; ++i) kv->seqs[dec_ids[i]].len += 1;
    for (int r = 0; r < n_reqs; ++r) kv->seqs[seq_ids[r]].len += chunk_lens[r];
    return MARS_OK;
}

mars_status_t mars_prefill_chunk(mars_model_t* m, mars_kv_t* kv, void* cuda_stream, int32_t n_reqs,
                                 const int32_t* seq_ids, const int32_t* chunk_lens, const int32_t* tokens,
                                 const int32_t* emit_last, const mars_sampling_t* sampling, int32_t* out_tokens,
                                 float* out_logprobs, const mars_debug_t* debug) {
    return feed_chunks(m, kv, cuda_stream, 0, nullptr, nullptr, n_reqs, seq_ids, chunk_lens, tokens, emit_last, sampling,
                       out_tokens, out_logprobs, debug, nullptr, 1.f);
}

mars_status_t mars_mixed_step(mars_model_t* m, mars_kv_t* kv, void* cuda_stream, int32_t n_seqs, const int32_t* seq_ids,
                              const int32_t* in_tokens, int32_t n_reqs, const int32_t* req_ids, const int32_t* chunk_lens,
                              const int32_t* chunk_tokens, const int32_t* emit_last, const mars_sampling_t* sampling,
                              int32_t* out_tokens, float* out_logprobs, const mars_debug_t* debug) {
    if (n_seqs < 1) return MARS_ERR_INVALID_ARG;
    return feed_chunks(m, kv, cuda_stream, n_seqs, seq_ids, in_tokens, n_reqs, req_ids, chunk_lens, chunk_tokens, emit_last,
                       sampling, out_tokens, out_logprobs, debug, nullptr, 1.f);
}

mars_status_t mars_score_chunk(mars_model_t* m, mars_kv_t* kv, void* cuda_stream, int32_t n_reqs, const int32_t* seq_ids,
                               const int32_t* chunk_lens, const int32_t* tokens, const int32_t* targets,
                               float temperature, float* out_logprobs, const mars_debug_t* debug) {
    if (!m) return MARS_ERR_BAD_HANDLE;
    if (!targets || !out_logprobs || !(temperature > 0.f)) return MARS_ERR_INVALID_ARG;
    // the per-tile softmax statistics borrow the expert-output buffer: [tiles][rows] pairs + [rows]
    if ((size_t)score_vocab_tiles(m->cfg.vocab) * 8 + 4 > (size_t)m->cfg.top_k * m->cfg.hidden * 4) return MARS_ERR_UNSUPPORTED;
    mars_sampling_t none;
    std::memset(&none, 0, sizeof(none));
    none.greedy = 1; none.temperature = 1.f; none.top_p = 1.f;
    return feed_chunks(m, kv, cuda_stream, 0, nullptr, nullptr, n_reqs, seq_ids, chunk_lens, tokens, nullptr, &none, nullptr,
                       out_logprobs, debug, targets, temperature);
}

mars_status_t mars_decode_step_host(mars_model_t* m, mars_kv_t* kv, void* cuda_stream, int32_t n_seqs,
                                    const int32_t* seq_ids, const int32_t* in_tokens_host,
                                    const mars_sampling_t* sampling, int32_t* out_tokens_host, float* out_logprobs_host) {
    if (!m || !kv) return MARS_ERR_BAD_HANDLE;
    if (!in_tokens_host || !out_tokens_host || !out_logprobs_host || n_seqs < 1 || n_seqs > m->max_decode)
        return MARS_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    CUDA_TRY(cudaMemcpyAsync(m->io_in, in_tokens_host, (size_t)n_seqs * 4, cudaMemcpyHostToDevice, st));
    mars_status_t r = mars_decode_step(m, kv, cuda_stream, n_seqs, seq_ids, m->io_in, sampling, m->io_out, m->io_lp,
                                       nullptr);
    if (r != MARS_OK) return r;
    CUDA_TRY(cudaMemcpyAsync(out_tokens_host, m->io_out, (size_t)n_seqs * 4, cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaMemcpyAsync(out_logprobs_host, m->io_lp, (size_t)n_seqs * 4, cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    return MARS_OK;
}

// ------------------------------------------------------------- allocation-free decode step
// Scratch for mars_decode_step_static.  In host code the name below is only a handle for the
// runtime; the device address is obtained once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[MARS_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
unsigned char* g_static_ptr[kMaxDevices] = {nullptr};

// Device address of the built-in array for the current device (looked up on first use).
mars_status_t static_scratch(unsigned char** out) {
    int dev = 0, major = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return MARS_ERR_UNSUPPORTED;
    if (!g_static_ptr[dev]) {
        CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
        if (major != 10) return MARS_ERR_UNSUPPORTED;
        CUDA_TRY(init_dense_kernels());
        CUDA_TRY(init_attn_kernels());
        CUDA_TRY(init_moe_kernels());
        unsigned char* p = nullptr;
        CUDA_TRY(cudaGetSymbolAddress((void**)&p, g_static_scratch));
        if (!p) return MARS_ERR_CUDA;
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return MARS_OK;
}
}  // namespace

mars_status_t mars_decode_step_static(const mars_config_t* cfg, const mars_weights_t* w, void* k_pool, void* v_pool,
                                      size_t pool_bytes_each, int32_t page_size, const int32_t* block_table,
                                      int32_t max_pages_per_seq, const int32_t* ctx_lens, void* cuda_stream,
                                      int32_t n_seqs, const int32_t* in_tokens, const mars_sampling_t* sampling,
                                      int32_t* out_tokens, float* out_logprobs) {
    if (!cfg || !w || !w->layers || !w->embed || !w->final_norm || !w->lm_head || !k_pool || !v_pool || !block_table ||
        !ctx_lens || !in_tokens || !sampling || !out_tokens || !out_logprobs)
        return MARS_ERR_INVALID_ARG;
    if (n_seqs < 1 || max_pages_per_seq < 1) return MARS_ERR_INVALID_ARG;
    if (page_size != 16 && page_size != 32 && page_size != 64 && page_size != 128) return MARS_ERR_INVALID_ARG;
    if ((uintptr_t)k_pool % 256 || (uintptr_t)v_pool % 256) return MARS_ERR_INVALID_ARG;
    if (!sampling->greedy && (!(sampling->temperature > 0.f) || !(sampling->top_p > 0.f) || sampling->top_p > 1.f))
        return MARS_ERR_INVALID_ARG;
    if (!shape_supported(*cfg)) return MARS_ERR_UNSUPPORTED;
    {   // The call reads ctx_lens on the host and uploads its step block from host memory that dies when it
        // returns: a captured copy of it would replay stale lengths from freed memory.  Refuse a capturing stream
        // before anything is enqueued.
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        CUDA_TRY(cudaStreamIsCapturing((cudaStream_t)cuda_stream, &cap));
        if (cap != cudaStreamCaptureStatusNone) return MARS_ERR_UNSUPPORTED;
    }
    for (int l = 0; l < cfg->n_layers; ++l) {
        const mars_layer_t& s = w->layers[l];
        if (!s.attn_norm || !s.wqkv || !s.wo || !s.mlp_norm || !s.router || !s.w_gate_up || !s.w_down)
            return MARS_ERR_INVALID_ARG;
        if (cfg->qk_norm && (!s.q_norm || !s.k_norm)) return MARS_ERR_INVALID_ARG;
    }
    for (int b = 0; b < n_seqs; ++b) {
        if (ctx_lens[b] < 0 || ctx_lens[b] + 1 > cfg->max_pos) return MARS_ERR_INVALID_ARG;
        if (ctx_lens[b] / page_size >= max_pages_per_seq) return MARS_ERR_INVALID_ARG;
    }
    const size_t page_bytes = (size_t)cfg->n_kv_heads * page_size * cfg->head_dim * 2;
    const size_t n_pages = pool_bytes_each / page_bytes / cfg->n_layers;
    if (n_pages < 1 || n_pages > 0x3fffffff) return MARS_ERR_INVALID_ARG;
    const uint64_t rows = (uint64_t)cfg->n_layers * n_pages * cfg->n_kv_heads * page_size;
    if (rows > 0x7fffffffull) return MARS_ERR_UNSUPPORTED;

    // everything the step needs must fit the built-in array
    Caps caps = make_caps(*cfg, n_seqs, 0);
    caps.keep_weights = false;             // the sampler recomputes its weights: the fixed scratch has no room to keep them
    const StepLayout lay = make_layout(caps);
    const size_t need = carve(*cfg, caps, lay, nullptr, nullptr, nullptr, nullptr, nullptr);
    if (need > (size_t)MARS_STATIC_SCRATCH_BYTES) return MARS_ERR_TOO_LARGE;

    unsigned char* base = nullptr;
    mars_status_t rc = static_scratch(&base);
    if (rc != MARS_OK) return rc;
    int dev = 0, sms = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    Buffers buf;
    carve(*cfg, caps, lay, base, &buf, nullptr, nullptr, nullptr);
    cudaStream_t st = (cudaStream_t)cuda_stream;

    CUtensorMap tm_k, tm_v;
    const int box_rows = std::min(page_size, 64);
    rc = make_pool_map(&tm_k, k_pool, rows, cfg->head_dim, box_rows);
    if (rc == MARS_OK) rc = make_pool_map(&tm_v, v_pool, rows, cfg->head_dim, box_rows);
    if (rc != MARS_OK) return rc;

    // step block (host heap, copied from pageable memory: the runtime stages it before returning)
    int64_t n_items = 0;
    for (int b = 0; b < n_seqs; ++b) n_items += (ctx_lens[b] + 1 + kSpanTokens - 1) / kSpanTokens;
    if (n_items > caps.n_items) return MARS_ERR_TOO_LARGE;
    std::vector<int32_t> blk((size_t)lay.items + 4 * (size_t)n_items, 0);
    blk[H_NTOK] = n_seqs;
    blk[H_NITEMS] = (int32_t)n_items;
    blk[H_NUPDATES] = 0;
    blk[H_NEMIT] = n_seqs;
    blk[H_GREEDY] = sampling->greedy ? 1 : 0;
    std::memcpy(&blk[H_TEMPERATURE], &sampling->temperature, 4);
    std::memcpy(&blk[H_TOP_P], &sampling->top_p, 4);
    blk[H_SEED_LO] = (int32_t)(uint32_t)sampling->seed;
    blk[H_SEED_HI] = (int32_t)(uint32_t)(sampling->seed >> 32);
    blk[H_STEP_LO] = (int32_t)(uint32_t)sampling->step;
    blk[H_STEP_HI] = (int32_t)(uint32_t)(sampling->step >> 32);
    int at = 0;
    for (int b = 0; b < n_seqs; ++b) {
        blk[lay.tok_seq + b] = b;
        blk[lay.tok_pos + b] = ctx_lens[b];
        blk[lay.emit_rows + b] = b;
        blk[lay.emit_slot + b] = b;
        blk[lay.tok_item_off + b] = at;
        const int len = ctx_lens[b] + 1;
        for (int s0 = 0; s0 < len; s0 += kSpanTokens) {
            blk[lay.items + 4 * at + 0] = b;
            blk[lay.items + 4 * at + 1] = s0;
            blk[lay.items + 4 * at + 2] = std::min(kSpanTokens, len - s0);
            blk[lay.items + 4 * at + 3] = at;      // partial slot = item index (nothing is shared here)
            ++at;
        }
    }
    blk[lay.tok_item_off + n_seqs] = at;
    std::vector<double> inv((size_t)cfg->head_dim / 2);
    for (int i = 0; i < cfg->head_dim / 2; ++i)
        inv[i] = std::pow((double)cfg->rope_theta, -2.0 * (double)i / (double)cfg->head_dim);

    // the array keeps the previous call's contents: clear what the kernels only OR into or count in
    CUDA_TRY(cudaMemsetAsync(buf.err, 0, 256, st));
    CUDA_TRY(cudaMemsetAsync(buf.active, 0, (size_t)cfg->n_layers * 4, st));
    CUDA_TRY(cudaMemsetAsync(buf.perm_cnt, 0, (size_t)cfg->n_experts * 4, st));   // its offset moves with the shape
    CUDA_TRY(cudaMemsetAsync(buf.n_groups, 0, 256, st));                         // the router blocks' arrival counter
    CUDA_TRY(cudaMemcpyAsync(buf.step, blk.data(), blk.size() * 4, cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaMemcpyAsync(buf.inv_freq, inv.data(), inv.size() * 8, cudaMemcpyHostToDevice, st));

    const Shape s{cfg->n_layers, cfg->hidden, cfg->n_q_heads, cfg->n_kv_heads, cfg->head_dim, cfg->n_experts,
                  cfg->top_k, cfg->expert_inter, cfg->vocab, cfg->qk_norm, cfg->rms_eps};
    const KvView view{(__nv_bfloat16*)k_pool, (__nv_bfloat16*)v_pool, const_cast<int32_t*>(block_table), (int)n_pages,
                      page_size, max_pages_per_seq};
    const DebugTaps taps{nullptr, nullptr, nullptr, nullptr, nullptr};
    auto layer_w = [&](int l) {
        const mars_layer_t& q = w->layers[l];
        return LayerW{(const __nv_bfloat16*)q.attn_norm, (const __nv_bfloat16*)q.wqkv, (const __nv_bfloat16*)q.q_norm,
                      (const __nv_bfloat16*)q.k_norm, (const __nv_bfloat16*)q.wo, (const __nv_bfloat16*)q.mlp_norm,
                      (const __nv_bfloat16*)q.router, (const __nv_bfloat16*)q.w_gate_up, (const __nv_bfloat16*)q.w_down};
    };
    launch_prep(s, buf, lay, view, n_seqs, st);
    launch_embed(s, buf, lay, (const __nv_bfloat16*)w->embed, in_tokens, (const __nv_bfloat16*)w->layers[0].attn_norm,
                 nullptr, n_seqs, st);
    for (int l = 0; l < s.L; ++l) {
        const LayerW lw = layer_w(l);
        launch_qkv(s, buf, lay, lw, view, l, n_seqs, sms, st);
        launch_attention(s, buf, lay, view, tm_k, tm_v, l, sms, st);
        launch_attn_merge(s, buf, lay, n_seqs, st);
        launch_oproj(s, buf, lw, n_seqs, sms, st);
        {
            int ks, o_ksplit, phases;      // as launch_oproj plans it
            gemm_plan(s.nq * s.D, n_seqs, false, &ks, &o_ksplit, &phases);
            launch_router(s, buf, lw, taps, l, n_seqs, 0, o_ksplit, st);
        }
        launch_gate_up(s, buf, lw, n_seqs, sms, st);
        launch_down(s, buf, lw, n_seqs, st);
        const __nv_bfloat16* next_gain =
            l + 1 < s.L ? (const __nv_bfloat16*)w->layers[l + 1].attn_norm : (const __nv_bfloat16*)w->final_norm;
        launch_combine(s, buf, next_gain, nullptr, n_seqs, st);
    }
    launch_lm_head(s, buf, lay, (const __nv_bfloat16*)w->lm_head, n_seqs, sms, st);
    launch_sample(s, buf, lay, n_seqs, 0, out_tokens, out_logprobs, nullptr, st);      // one block per row
    CUDA_TRY(cudaGetLastError());
    return MARS_OK;
}

mars_status_t mars_poll_status(mars_model_t* m) {
    if (!m) return MARS_ERR_BAD_HANDLE;
    CUDA_TRY(cudaStreamSynchronize(m->last_stream));
    int32_t word = 0;
    CUDA_TRY(cudaMemcpy(&word, m->buf.err, 4, cudaMemcpyDeviceToHost));
    if (word) CUDA_TRY(cudaMemset(m->buf.err, 0, 4));
    if (word & kErrTimeout) return MARS_ERR_TIMEOUT;
    if (word & kErrBadToken) return MARS_ERR_BAD_TOKEN;
    return MARS_OK;
}

mars_status_t mars_debug_bounded_wait(mars_model_t* m, void* cuda_stream, int32_t arrive) {
    if (!m) return MARS_ERR_BAD_HANDLE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    launch_wait_probe(m->buf.err, arrive ? 1 : 0, 4096u, st);
    CUDA_TRY(cudaGetLastError());
    m->last_stream = st;
    return MARS_OK;
}

mars_status_t mars_set_prefill_lo_planes(mars_model_t* m, int32_t mask) {
    if (!m) return MARS_ERR_BAD_HANDLE;
    if (mask < 0 || mask > MARS_LO_ALL) return MARS_ERR_INVALID_ARG;
    m->lo_planes = mask;
    return MARS_OK;
}

mars_status_t mars_profile_enable(mars_model_t* m, int32_t enable) {
    if (!m) return MARS_ERR_BAD_HANDLE;
    m->profiling = enable != 0;
    return MARS_OK;
}

mars_status_t mars_profile_read(mars_model_t* m, double* ms_per_class, int64_t* launches_per_class) {
    if (!m) return MARS_ERR_BAD_HANDLE;
    if (!ms_per_class || !launches_per_class) return MARS_ERR_INVALID_ARG;
    CUDA_TRY(cudaStreamSynchronize(m->last_stream));
    for (size_t i = 0; i < m->ev_class.size(); ++i) {
        float ms = 0.f;
        CUDA_TRY(cudaEventElapsedTime(&ms, m->ev_pool[2 * i], m->ev_pool[2 * i + 1]));
        ms_per_class[m->ev_class[i]] += (double)ms;
        launches_per_class[m->ev_class[i]] += 1;
    }
    m->ev_class.clear();
    m->ev_used = 0;
    return MARS_OK;
}

mars_status_t mars_last_step_info(const mars_model_t* m, mars_step_info_t* out) {
    if (!m) return MARS_ERR_BAD_HANDLE;
    if (!out) return MARS_ERR_INVALID_ARG;
    *out = m->info;
    return MARS_OK;
}

const int32_t* mars_active_experts_device(const mars_model_t* m) { return m ? m->buf.active : nullptr; }

}  // extern "C"
