// Prompt processing (Eq. 3 of the paper: KV <- Prefill(x_1:T)) as dense contractions on the 5th-generation tensor cores.
// Host-side interface between the C ABI (edgefm.cu) and the kernels of prefill.cu.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"
#include "../../include/edgefm.h"

namespace edgefm {

constexpr int PF_HEAD_GRID_MAX = 1024;   // CTAs of the output-layer kernels (candidate slots: PF_HEAD_GRID_MAX x PF_VERIFY_MAX)
constexpr int PF_VERIFY_MAX = 8;         // tokens of a block verified through the dense path
#ifndef PF_CHUNK_MAX_VALUE
#define PF_CHUNK_MAX_VALUE 4096
#endif
constexpr int PF_CHUNK_MAX = PF_CHUNK_MAX_VALUE;   // tokens per pass over the layers (longer prompts take several passes); 4096 instead of
                                                  // 2048 took a 32768-token prompt of the 1.5B shape from 393 to 351 ms   // tokens per pass over the layers (longer prompts take several passes)

// Work buffers of one pass, owned by the context, allocated at the first prefill call.
struct PrefillBuffers {
    int chunk = 0;               // rows the buffers hold
    float *resid = nullptr;      // residual stream fp32 [chunk][H]
    float *part = nullptr;       // K-split partial sums of the O / down contraction, fp32 [8][chunk][H]
    // activations as two bf16 planes each (hi = bf16(x), lo = bf16(x - hi)):
    uint16_t *xn = nullptr;      // normalised activations [2][chunk][H]
    uint16_t *q = nullptr;       // rotated queries [2][chunk][nq d]
    uint16_t *attn = nullptr;    // attention output [2][chunk][nq d]
    uint16_t *act = nullptr;     // SwiGLU output [2][chunk][F]
    float *kv_stage = nullptr;   // compressed cache only: fp32 k and v rows of the pass [2][nkv][chunk][d], before compression
    float2 *rope = nullptr;      // (cos, sin) of the chunk's positions, [chunk][d/2]
    int *tokens = nullptr;       // device copy of the chunk's token ids
    int *error = nullptr;        // device word: non-zero when a bounded wait of a GEMM ran out
    float *att_o = nullptr;      // attention of a lone query tile shared out among CTAs: partial rows fp32 [8][128][nq d]
    float *att_ml = nullptr;     // ... and their (reference maximum, row sum) [8][128][nq][2]
    float *logits = nullptr;     // verified blocks: logits of the block's rows when the caller wants none, fp32 [8][vocab]
    int logits_rows = 0;
    float *head_val = nullptr;   // output layer: the CTAs' greedy candidates
    int *head_idx = nullptr;
    unsigned *head_ticket = nullptr;
    uint32_t wait_limit = 1u << 24;   // polls per wait (far beyond any legitimate wait of a tile)
    uint32_t extra_arrivals = 0;      // tests only: 1 makes the first wait of every contraction run out
};

struct PrefillModel {
    edgefm_shape shape;
    const edgefm_layer_weights *layers;   // host array
    const void *embed;
    uint16_t *k_cache, *v_cache;          // bf16 [L][nkv][max_context][d], or one signed byte per element (k_scale != nullptr)
    float *k_scale, *v_scale;             // compressed cache: [L][nkv][max_context], else nullptr
    int max_context;
    StepState *state;
    int num_sms;
};

// Tile shape and K split a contraction of [M x K] x [K x N] gets on num_sms SMs (host logic, no device needed).
// epilogue: 0 = QKV, 1 = added to the residual stream (O, down), 2 = gate/up.  *wide: 256-column tiles; *splits: K units per tile.
void prefill_plan_contraction(int epilogue, int M, int N, int K, int num_sms, int *wide, int *splits);

// Bytes the work buffers of a pass over `chunk` tokens take.
size_t prefill_buffer_bytes(const edgefm_shape &sh, int chunk);
// Allocate / free.  Returns a CUDA error.
cudaError_t prefill_alloc(PrefillBuffers *b, const edgefm_shape &sh, int chunk, bool kv8);
void prefill_free(PrefillBuffers *b);

// Enqueue the layers for `n` tokens (host ids) whose cache rows go to slots [slot0, slot0 + n) at rotary positions
// position .. position + n - 1.  Every layer's K and V rows are written.  whole_last_layer = false: the last layer's attention
// and MLP are skipped (their result would only feed an output layer nobody reads); true: they run, and the residual stream
// behind the last layer is left in PrefillBuffers::resid for prefill_head.  Sets the device state to cache length slot0 + n.
// Returns nullptr or a message.
const char *prefill_run(const PrefillModel &m, PrefillBuffers *b, const int32_t *tokens, int n, int slot0, int position, bool whole_last_layer,
                        cudaStream_t stream, int *launches);

// The output layer for row `row` of the residual stream of the last pass: final norm, logits over `rows` rows of `lm` (ids:
// their token ids when the vocabulary is pruned, else nullptr), greedy token; leaves the device state as a decode step of
// `token` at `pos` would.  logits_out / next_token_out: device pointers or nullptr.
const char *prefill_head(const PrefillModel &m, PrefillBuffers *b, int row, const void *final_norm, const void *lm, const int *ids, int rows,
                         float *logits_out, int *next_token_out, int token, int pos, cudaStream_t stream);

// Block verification through the dense path (Sec. 3.11): after prefill_run(..., n tokens, whole_last_layer = true), the logits of
// all n rows ([n][rows], or nullptr), the greedy acceptance on the device and the state update (cache length slot0 + accepted).
const char *prefill_verify_head(const PrefillModel &m, PrefillBuffers *b, int n, const void *final_norm, const void *lm, const int *ids, int rows,
                                float *logits_out, int *n_accepted_out, int *next_token_out, int slot0, int pos, cudaStream_t stream);

}  // namespace edgefm
