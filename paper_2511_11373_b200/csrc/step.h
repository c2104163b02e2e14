// Host/device description of one step: the model shape, the workspace carve-up and the per-step
// metadata block that the host builds in pinned memory and uploads with a single copy.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace mars {

// Bits of the device status word (read and cleared by mars_poll_status).
constexpr int kErrBadToken = 1;
constexpr int kErrTimeout = 2;

// Header words of the step block (int32 each).
enum StepHdr {
    H_NTOK = 0,       // token rows in this call
    H_NITEMS = 1,     // attention work items of the decode kernel (spans of cached tokens), items [0, H_NITEMS)
    H_NUPDATES = 2,   // block-table entries to write before the step
    H_NEMIT = 3,      // rows that sample a token
    H_GREEDY = 4,
    H_TEMPERATURE = 5,  // float bits
    H_TOP_P = 6,        // float bits
    H_SEED_LO = 7, H_SEED_HI = 8, H_STEP_LO = 9, H_STEP_HI = 10,
    H_PF_FIRST = 11,  // first work item of the causal (prompt) attention kernel; decode spans come before it
    H_PF_ITEMS = 12,  // number of such items
    H_SH_ITEMS = 13,  // work items of the shared-prefix kernel (a span of cached tokens read once for up to 4 rows)
    H_WORDS = 16
};

// Offsets (in int32 words) of the arrays inside the step block.
struct StepLayout {
    int tok_seq;       // [n_tok] sequence slot (block-table row) of every token row
    int tok_pos;       // [n_tok] position of the token in its sequence
    int tok_item_off;  // [n_tok + 1] first partial slot (span result) of every token row
    int emit_rows;     // [n_emit] token row whose hidden state is sampled
    int emit_slot;     // [n_emit] sequence slot of that row (random-number counter)
    int updates;       // [n_updates][3] (slot, page index, page id)
    int items;         // [n_items][4] decode spans: (token row, first cached token, number of tokens, partial slot);
                       // prompt blocks after them: (first row, 0, keys visible to the last row, rows)
    int sh_items;      // [n_sh][12] (first cached token, tokens, rows <= 4, 0, token row x 4, partial slot x 4)
    int total_words;
};

struct Shape {
    int L, H, nq, nkv, D, E, k, I, V, qk_norm;
    float eps;
};

// Everything the kernels need to find their buffers.  All pointers are device pointers into the
// caller's workspace unless noted.
struct Buffers {
    int32_t* step;          // the uploaded step block
    int32_t* err;           // status word
    float* x;               // [n_tok, H] residual stream (fp32)
    __nv_bfloat16* h;       // [n_tok, 2, H] normalised input of the next projection, (hi, lo) rows
    float* qkv;             // [ksplit, n_tok, (nq + 2 nkv) D] raw projection (split-K partials)
    float* opart;           // [ksplit, n_tok, H] output-projection partials, added to x by the router kernel
    __nv_bfloat16* q;       // [n_tok, 2, nq D] rotated queries, (hi, lo) rows
    __nv_bfloat16* o;       // [n_tok, 2, nq D] attention output, (hi, lo) rows
    float2* rope;           // [n_tok, D/2] (cos, sin) of pos * theta_i
    double* inv_freq;       // [D/2] theta^(-2i/D)
    float* part_o;          // [slots, nq, D] unnormalised partial outputs, one slot per (token row, span)
    float2* part_ml;        // [slots, nq] (running max in log2 units, sum)
    float* rlogits;         // [n_tok, E] gate logits (prefill path: computed by one contraction for all rows)
    int32_t* route_idx;     // [n_tok, k]
    float* route_w;         // [n_tok, k]
    int32_t* expert_off;    // [E + 1]
    int32_t* slot_token;    // [n_tok k] token row served by every expert slot
    int32_t* slot_of;       // [n_tok k] slot of (token, j)
    int32_t* groups;        // [n_groups][4] (expert, first slot, tokens, 0): the expert kernels' work list
    int32_t* n_groups;
    int32_t* perm_cnt;      // [E] tokens per expert, counted by many blocks (large calls); zero between uses
    int32_t* perm_cur;      // [E] next free slot of every expert while the slots are handed out (large calls)
    int32_t* active;        // [L] distinct experts per layer
    __nv_bfloat16* act;     // [n_tok k, 2, I] SwiGLU activations, (hi, lo) rows
    __nv_bfloat16* xperm;   // [n_tok k, 2, H] activations gathered into expert-slot order (prefill path only)
    float* y;               // [n_tok k, H]
    float* logits;          // [n_emit, V]
    float* expw;            // [n_emit, V] softmax weights exp((l - max) / T) kept between the sampler's passes, or null
};

}  // namespace mars
