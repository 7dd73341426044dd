// C ABI of the batch-1 decode step (see include/edgefm.h) and the assembly of the step as a CUDA graph.
#include "../../include/edgefm.h"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"
#include "megakernel_types.cuh"
#include "step_plan.h"
#include "prefill.h"
// the persistent kernel is built twice: 11 consumer warps per CTA (short contexts, here) and 7 (long contexts,
// in the megakernel_long_*.cu translation units), plus the warp that prefetches into L2
#define MK_NS mk_short
#define MK_NW_VALUE MK_NW_SHORT
#include "megakernel.cuh"
#undef MK_NS
#undef MK_NW_VALUE

namespace edgefm {

// ---- small kernels -------------------------------------------------------------------------------

// Strided copy of n caller-provided KV positions into cache slots [slot0, slot0 + n); also sets the device state
// (cache length slot0 + n).
__global__ void __launch_bounds__(256) prefill_copy_kernel(const uint16_t *k, const uint16_t *v, uint16_t *kc, uint16_t *vc,
                                                           int L, int nkv, int n, int d, int max_context, long long s_layer,
                                                           long long s_head, long long s_pos, int vec_ok, StepState *st, int slot0) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        st->cur_len = slot0 + n;
        st->next_position = slot0 + n;
        st->status = 0;
    }
    const long long total = static_cast<long long>(L) * nkv * n * d;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    if (vec_ok) {  // 16-byte pieces: d % 8 == 0, all strides % 8 == 0, bases 16-byte aligned
        const int dp = d >> 3;
        for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total >> 3; i += stride) {
            const int j = static_cast<int>(i % dp);
            long long r = i / dp;
            const int t = static_cast<int>(r % n); r /= n;
            const int g = static_cast<int>(r % nkv);
            const int l = static_cast<int>(r / nkv);
            const long long src = l * s_layer + g * s_head + t * s_pos + j * 8;
            const long long dst = ((static_cast<long long>(l) * nkv + g) * max_context + slot0 + t) * d + j * 8;
            *reinterpret_cast<uint4 *>(kc + dst) = *reinterpret_cast<const uint4 *>(k + src);
            *reinterpret_cast<uint4 *>(vc + dst) = *reinterpret_cast<const uint4 *>(v + src);
        }
    } else {
        for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total; i += stride) {
            const int j = static_cast<int>(i % d);
            long long r = i / d;
            const int t = static_cast<int>(r % n); r /= n;
            const int g = static_cast<int>(r % nkv);
            const int l = static_cast<int>(r / nkv);
            const long long src = l * s_layer + g * s_head + t * s_pos + j;
            const long long dst = ((static_cast<long long>(l) * nkv + g) * max_context + slot0 + t) * d + j;
            kc[dst] = k[src];
            vc[dst] = v[src];
        }
    }
}

// The same for the compressed cache (Sec. 3.9): one warp per given row; the row's largest magnitude fixes its scale,
// scale = amax / 127, code = clamp(rint(x * (127 / amax))) in fp32.
__global__ void __launch_bounds__(256) prefill_quantize_kernel(const uint16_t *k, const uint16_t *v, signed char *kc, signed char *vc,
                                                               float *ks, float *vs, int L, int nkv, int n, int d, int max_context,
                                                               long long s_layer, long long s_head, long long s_pos, StepState *st,
                                                               int slot0) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        st->cur_len = slot0 + n;
        st->next_position = slot0 + n;
        st->status = 0;
    }
    const int warps = (gridDim.x * blockDim.x) >> 5, lane = threadIdx.x & 31;
    const long long rows = static_cast<long long>(L) * nkv * n * 2;          // K rows, then V rows
    for (long long r = (blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x) >> 5; r < rows; r += warps) {
        const bool is_v = r >= rows / 2;
        long long rr = is_v ? r - rows / 2 : r;
        const int t = static_cast<int>(rr % n); rr /= n;
        const int g = static_cast<int>(rr % nkv);
        const int l = static_cast<int>(rr / nkv);
        const uint16_t *src = (is_v ? v : k) + l * s_layer + g * s_head + t * s_pos;
        const long long row = (static_cast<long long>(l) * nkv + g) * max_context + slot0 + t;
        float x[4];                                                          // d <= 128: at most 4 values per lane
        float amax = 0.f;
        for (int e = 0; e < 4; ++e) {
            const int j = lane + 32 * e;
            x[e] = j < d ? bf16_bits_to_f32(src[j]) : 0.f;
            amax = fmaxf(amax, fabsf(x[e]));
        }
        amax = warp_max(amax);
        const float inv = amax > 0.f ? __fdiv_rn(127.0f, amax) : 0.f;
        signed char *dst = (is_v ? vc : kc) + row * d;
        for (int e = 0; e < 4; ++e) {
            const int j = lane + 32 * e;
            if (j < d) dst[j] = static_cast<signed char>(static_cast<int>(fminf(fmaxf(rintf(__fmul_rn(x[e], inv)), -127.f), 127.f)));
        }
        if (lane == 0) (is_v ? vs : ks)[row] = amax > 0.f ? __fdiv_rn(amax, 127.0f) : 0.f;
    }
}

// Vocabulary pruning: row r of the compact lm_head is row ids[r] of the full one.  One warp per row, 16-byte pieces.
__global__ void __launch_bounds__(256) gather_rows_kernel(const uint16_t *src, const int *ids, uint16_t *dst, int n, int H) {
    const int warps = (gridDim.x * blockDim.x) >> 5;
    const int lane = threadIdx.x & 31;
    const int k16 = H >> 3;
    for (int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < n; r += warps) {
        const uint4 *s4 = reinterpret_cast<const uint4 *>(src + static_cast<size_t>(ids[r]) * H);
        uint4 *d4 = reinterpret_cast<uint4 *>(dst + static_cast<size_t>(r) * H);
        for (int c = lane; c < k16; c += 32) d4[c] = s4[c];
    }
}

// long_ctx = false: the variant without the grouped (one CTA per GQA group) attention code, for contexts that
// never need it.
MegaKernel mega_kernel_block2(int head_dim);   // megakernel_block2.cu
MegaKernel mega_kernel_block4(int head_dim);   // megakernel_block4.cu

template <int D>
MegaKernel mega_kernel_g(int G, bool long_ctx, bool kv8 = false, int block_tokens = 1) {
    if (block_tokens == 2) return mega_kernel_block2(D);
    if (block_tokens == 4) return mega_kernel_block4(D);
    if (kv8) {
        if (D == 64) return G <= 4 ? mega_kernel_q8_d64_lo(G) : mega_kernel_q8_d64_hi(G);
        return G <= 4 ? mega_kernel_q8_d128_lo(G) : mega_kernel_q8_d128_hi(G);
    }
    if (!long_ctx) return mk_short::decode_megakernel<D, 1, false>;   // G is only used by the grouped attention
    if (D == 64) return G <= 4 ? mega_kernel_long_d64_lo(G) : mega_kernel_long_d64_hi(G);
    return G <= 4 ? mega_kernel_long_d128_lo(G) : mega_kernel_long_d128_hi(G);
}

// ---- launch plan of the persistent step kernel (shared by edgefm_create and edgefm_decode_step_static) ----------------
struct StepPlan {
    MegaKernel kernel = nullptr;
    bool long_ctx = false;
    int nw = 0;            // consumer warps per CTA of the chosen kernel build
    int grid = 0;          // CTAs (one per SM)
    int max_chunks = 0;    // row stride of the attention partial buffers
    int n_ops = 0;         // 4 per layer + lm_head
    size_t xbuf = 0, ops_bytes = 0, tab_bytes = 0, sched_bytes = 0;   // shared memory: activation / attention scratch, operators, schedule table, tile lists
    int slots = 0, slot_bytes = 0, slot_rows = 0;   // ring of one consumer warp
    size_t dyn_smem = 0;
    int block_tokens = 1;  // tokens a call may carry (the M of the chosen kernel build)
};

// Kernel variant and shared-memory split for a model shape.  Returns null, or why the shape does not fit.
// sched_reserve: bytes to set aside for the CTA's tile lists.
inline const char *plan_step(const edgefm_shape &sh, int max_context, int num_sms, int smem_optin, size_t sched_reserve, StepPlan *pl, cudaError_t *cuda_err,
                             bool kv8 = false, int block_tokens = 1) {
    const int H = sh.hidden, d = sh.head_dim, nq = sh.n_q_heads, nkv = sh.n_kv_heads, G = nq / nkv;
    *cuda_err = cudaSuccess;
    // (the compressed cache is attended by the grouped attention of the long-context build only)
    pl->long_ctx = kv8 || max_context > 8192 || static_cast<long long>(nq) * MK_ATT_SPLIT_MAXC * 2 > MK_PARTIAL_FLOATS;
    if (block_tokens > 1 && pl->long_ctx) return "blocks of several tokens need the plain cache and max_context <= 8192";
    pl->block_tokens = block_tokens;
    pl->kernel = d == 64 ? mega_kernel_g<64>(G, pl->long_ctx, kv8, block_tokens) : mega_kernel_g<128>(G, pl->long_ctx, kv8, block_tokens);
    pl->nw = pl->long_ctx ? MK_NW_LONG : MK_NW_SHORT;
    pl->grid = num_sms;
    pl->max_chunks = pl->grid / nkv > 0 ? pl->grid / nkv : 1;
    pl->n_ops = 4 * sh.n_layers + 1;
    const int NW = pl->nw, ATT_MW = NW;   // every warp has an entry in the attention merge area
    int max_k = H;                       // vectors staged in shared memory: the residual stream and the attention output
    if (nq * d > max_k) max_k = nq * d;   // (the down projection reads the MLP activations from global memory)
    max_k = (max_k + MK_TILE_COLS - 1) / MK_TILE_COLS * MK_TILE_COLS;   // whole 256-column pieces (zero-padded)
    // attention scratch: queries, probabilities, warp merge area, chunk statistics
    // (the short-context build always runs attention with one query head per CTA)
    const int AG = pl->long_ctx ? G : 1;
    const size_t att_bytes = (static_cast<size_t>(AG) * d + NW * (AG * MK_ATT_TILE > 32 / MK_ATT_LPP_SPLIT ? AG * MK_ATT_TILE : 32 / MK_ATT_LPP_SPLIT) +
                              2 * ATT_MW * AG + static_cast<size_t>(ATT_MW) * AG * d + 2 * static_cast<size_t>(AG) * pl->max_chunks) * 4;
    size_t xbuf = block_tokens * mk_splits(block_tokens) * (static_cast<size_t>(max_k) * 2 + MK_XS_PAD);   // the staged activations: three bf16 arrays per token
    if (att_bytes > xbuf) xbuf = att_bytes;
    pl->xbuf = (xbuf + 1023) / 1024 * 1024;
    cudaFuncAttributes fa{};
    *cuda_err = cudaFuncGetAttributes(&fa, pl->kernel);
    if (*cuda_err != cudaSuccess) return "cudaFuncGetAttributes";
    const size_t static_smem = fa.sharedSizeBytes + (1024 - fa.sharedSizeBytes % 1024) % 1024;   // the kernel's static shared memory (mbarriers, tables, scratch) + the padding in
                                                            // front of the 1 KB-aligned dynamic part
    pl->ops_bytes = static_cast<size_t>(pl->n_ops) * sizeof(MkOp);
    const size_t tab = static_cast<size_t>(cta_tab_ints_for(NW)) * sizeof(int);
    pl->tab_bytes = (tab + 15) / 16 * 16;
    const size_t head = (pl->ops_bytes + pl->tab_bytes + sched_reserve + 1023) / 1024 * 1024;   // the rings start on a 1 KB boundary
    pl->sched_bytes = head - pl->ops_bytes - pl->tab_bytes;
    const size_t tail = pl->xbuf + static_cast<size_t>(NW) * mk_wbuf_bytes(block_tokens);   // behind the rings: the activation vector and the warps' small buffers
    if (head + tail + static_smem + static_cast<size_t>(NW) * 2 * 2048 > static_cast<size_t>(smem_optin))
        return "model shape does not fit the shared-memory plan";
    const size_t per_warp = (smem_optin - static_smem - head - tail) / NW;
    // two slots per warp at least; a slot holds up to 16 rows x 256 columns (8 KB) and is a whole number of KB (an even number of rows)
    size_t slot = per_warp / 2 / 1024 * 1024;
    if (slot > static_cast<size_t>(MK_TILE_ROWS) * MK_TILE_COLS * 2) slot = static_cast<size_t>(MK_TILE_ROWS) * MK_TILE_COLS * 2;
    if (slot < 2048) return "model shape does not fit the shared-memory plan";
    pl->slot_bytes = static_cast<int>(slot);
    pl->slot_rows = pl->slot_bytes / (MK_TILE_COLS * 2);
    pl->slots = static_cast<int>(per_warp / slot);
    if (pl->slots > MK_MAX_SLOTS) pl->slots = MK_MAX_SLOTS;
    pl->dyn_smem = head + static_cast<size_t>(NW) * pl->slots * slot + tail;
    return nullptr;
}

// Raise the kernel's dynamic shared-memory limit to the most any plan can ask for (a function attribute, not an
// allocation).  Always the same value, so contexts and static calls of different shapes never lower it for one another.
inline cudaError_t allow_max_dynamic_smem(MegaKernel kern, int smem_optin) {
    cudaFuncAttributes fa{};
    cudaError_t e = cudaFuncGetAttributes(&fa, kern);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin - static_cast<int>(fa.sharedSizeBytes));
}

// Shapes of the five streaming operators (0..3 of a layer, 4 = output layer over `lm_rows` rows).
inline void op_shapes(const edgefm_shape &sh, int lm_rows, OpShape os[5]) {
    const int H = sh.hidden, d = sh.head_dim, nq = sh.n_q_heads, nkv = sh.n_kv_heads, F = sh.ffn;
    const int R = (nq + 2 * nkv) * d;
    os[0] = {PH_QKV, R / 2, H, R, d / 2};
    os[1] = {PH_RESID, H, nq * d, H, 0};
    os[2] = {PH_SWIGLU, F, H, 2 * F, 0};
    os[3] = {PH_RESID, H, F, H, 0};
    os[4] = {PH_LMHEAD, lm_rows, H, lm_rows, 0};
}

// The operators of the step in execution order, wired to the work buffers.
inline void fill_ops(const edgefm_shape &sh, const edgefm_layer_weights *layers, const void *final_norm, const void *lm_head, float *x, float *attn, float *q,
                     float *act, MkOp *out, const uint16_t **weights_out, int block_tokens = 1) {
    // distance between the vectors of consecutive tokens of a block (see MkParams::block_tokens)
    const int sx = sh.hidden, sq = sh.n_q_heads * sh.head_dim, sa = mk_splits(block_tokens) * ((sh.ffn + MK_TILE_COLS - 1) / MK_TILE_COLS * MK_TILE_COLS);
    OpShape os[5];
    op_shapes(sh, sh.vocab, os);
    int n = 0;
    auto mk = [&](const OpShape &o, const void *W, const void *bias, const void *norm, const float *x_src, float *dst, int layer, int flags, int xs_ = 0,
                  int os_ = 0) {
        MkOp op{};
        op.x_tok_stride = xs_; op.out_tok_stride = os_;
        weights_out[n] = static_cast<const uint16_t *>(W);
        op.bias = static_cast<const uint16_t *>(bias); op.norm_w = static_cast<const uint16_t *>(norm); op.x_src = x_src; op.out = dst;
        op.K = o.K; op.kind = o.kind; op.units_total = o.units; op.layer_flags = layer << 8 | flags | (o.K % 64 ? PHF_RAGGED : 0);
        out[n++] = op;
    };
    for (int l = 0; l < sh.n_layers; ++l) {
        const edgefm_layer_weights &w = layers[l];
        mk(os[0], w.wqkv, sh.qkv_bias ? w.bqkv : nullptr, w.input_norm, l == 0 ? nullptr : x, q, l, 0, sx, sq);
        mk(os[1], w.wo, nullptr, nullptr, attn, x, l, 0, sq, sx);
        mk(os[2], w.w_gate_up, nullptr, w.post_norm, x, act, l, PHF_OUT_SPLIT, sx, sa);  // the MLP activations go to memory in the form the down projection multiplies
        mk(os[3], w.w_down, nullptr, nullptr, act, x, l, PHF_X_GLOBAL, sa, sx);
    }
    mk(os[4], lm_head, nullptr, final_norm, x, nullptr, sh.n_layers, 0, sx, 0);
}

// Tile schedule of the step for the plan's geometry.  Returns null, or why the shape does not fit.
inline const char *plan_schedule(const StepPlan &pl, const edgefm_shape &sh, int lm_rows, StepSchedule *ss) {
    OpShape os[5];
    op_shapes(sh, lm_rows, os);
    for (int o = 0; o < 5; ++o)
        if (const char *why = plan_op(os[o], o, pl.grid, pl.nw, pl.slot_rows, &ss->ops[o])) return why;
    assemble_schedule(ss, pl.grid, pl.nw);
    return nullptr;
}

// Shared-memory plan and tile schedule together: the tile lists live in shared memory, so their size (known only once
// the schedule exists) takes room from the rings, whose slot size shapes the schedule.  A few rounds settle it.
inline const char *plan_step_and_schedule(const edgefm_shape &sh, int max_context, int num_sms, int smem_optin, StepPlan *pl, StepSchedule *ss,
                                          cudaError_t *cuda_err, bool kv8 = false, int block_tokens = 1) {
    size_t reserve = 0;
    for (int attempt = 0; attempt < 6; ++attempt) {
        if (const char *why = plan_step(sh, max_context, num_sms, smem_optin, reserve, pl, cuda_err, kv8, block_tokens)) return why;
        if (const char *why = plan_schedule(*pl, sh, sh.vocab, ss)) return why;
        const size_t need = ss->smem_bytes();
        if (need <= pl->sched_bytes) return nullptr;
        reserve = need + (attempt > 0 ? need / 8 : 0);
    }
    return "model shape does not fit the shared-memory plan";
}

// Tensor maps of all weight matrices: [(4 l + op) * MK_MAX_VARIANTS + variant]; the output layer's come last.
inline const char *encode_maps(const StepSchedule &ss, const edgefm_shape &sh, const edgefm_layer_weights *layers, const void *lm_head, int lm_rows,
                               CUtensorMap *maps) {
    OpShape os[5];
    op_shapes(sh, lm_rows, os);
    auto enc = [&](int opi, int o, const void *W) {
        for (int v = 0; v < MK_MAX_VARIANTS; ++v) {
            CUtensorMap *m = &maps[static_cast<size_t>(opi) * MK_MAX_VARIANTS + v];
            if (v >= ss.ops[o].n_variants) { std::memset(m, 0, sizeof *m); continue; }
            const int pair_rows = os[o].kind == PH_QKV ? os[o].head_half : (os[o].kind == PH_SWIGLU ? os[o].units : 0);
            if (!encode_weight_map(m, W, os[o].rows, os[o].K, ss.ops[o].variant_rows[v], pair_rows, os[o].kind == PH_QKV)) return false;
        }
        return true;
    };
    for (int l = 0; l < sh.n_layers; ++l) {
        const edgefm_layer_weights &w = layers[l];
        if (!enc(4 * l + 0, 0, w.wqkv) || !enc(4 * l + 1, 1, w.wo) || !enc(4 * l + 2, 2, w.w_gate_up) || !enc(4 * l + 3, 3, w.w_down))
            return "cuTensorMapEncodeTiled failed";
    }
    if (!enc(4 * sh.n_layers, 4, lm_head)) return "cuTensorMapEncodeTiled failed";
    return nullptr;
}

// Shape-derived kernel parameters common to both entry points (buffers, cache and schedule pointers are the caller's).
inline void fill_shape_params(MkParams *m, const edgefm_shape &sh, int max_context, const StepPlan &pl, const StepSchedule &ss) {
    m->nph = pl.n_ops; m->n_layers = sh.n_layers; m->H = sh.hidden; m->nq = sh.n_q_heads; m->nkv = sh.n_kv_heads;
    m->d = sh.head_dim; m->F = sh.ffn; m->V = sh.vocab;
    m->half_shift = sh.head_dim == 64 ? 5 : 6;
    m->eps = sh.rms_eps; m->scale = static_cast<float>(1.0 / std::sqrt(static_cast<double>(sh.head_dim)));
    m->max_context = max_context; m->max_chunks = pl.max_chunks; m->block_tokens = pl.block_tokens;
    m->att_chunk_shared = 256; m->att_chunk_split = 64; m->att_split_max_n = 8192;
    m->slots = pl.slots; m->slot_bytes = pl.slot_bytes;
    m->xbuf_bytes = static_cast<int>(pl.xbuf); m->ops_bytes = static_cast<int>(pl.ops_bytes); m->tab_bytes = static_cast<int>(pl.tab_bytes);
    m->sched_bytes = static_cast<int>(pl.sched_bytes);
    m->cta_tab_ints = ss.cta_tab_ints;
    m->barrier_extra = 0;
    m->pf_tiles = MK_PF_TILES;   // measured: 3 .. 8 equal, 16 thrashes L2 (1.5B shape)
    m->map_fence = 1;   // edgefm_set_vocab_subset rewrites the output layer's maps between steps
    m->spin_limit = 1000000000u;   // 1 s
}

}  // namespace edgefm

using namespace edgefm;

// ---- the context -----------------------------------------------------------------------------------

struct edgefm_ctx {
    edgefm_shape shape{};
    int max_context = 0;
    int device = -1;
    int num_sms = 0;
    std::vector<edgefm_layer_weights> layers;
    const void *embed = nullptr, *final_norm = nullptr, *lm_head = nullptr;

    // owned device memory
    uint16_t *k_cache = nullptr, *v_cache = nullptr;  // [L][nkv][max_context][d] (bf16, or one signed byte per element)
    int kv_format = EDGEFM_KV_BF16;
    int block_tokens = 1;        // tokens a call may carry (edgefm_verify_block)
    float *k_scale = nullptr, *v_scale = nullptr;     // compressed cache: [L][nkv][max_context]
    float *kv_stage = nullptr;                        // compressed cache: fp32 k, v rows of the step's token [2][nkv][d]
    float *x = nullptr;          // residual stream [H]
    float *q = nullptr;          // rotated queries [nq*d]
    float *attn = nullptr;       // attention output [nq*d]
    float *act = nullptr;        // SwiGLU output [F]
    double *inv_freq = nullptr;  // [d/2]
    float *part_m = nullptr, *part_l = nullptr, *part_o = nullptr;
    float *lm_part_val = nullptr;
    int *lm_part_idx = nullptr;
    unsigned *tickets = nullptr;  // [nq] attention + [1] lm_head
    StepState *state = nullptr;
    StepRequest *req = nullptr;
    MkOp *d_ops = nullptr;
    const uint16_t **d_op_w = nullptr;   // base of every operator's weight matrix
    unsigned char *d_maps = nullptr;   // CUtensorMap [(4 L + 1) * MK_MAX_VARIANTS]
    uint2 *d_tiles = nullptr;
    int *d_cta_tab = nullptr;
    MkCombine *d_combines = nullptr;
    size_t tiles_cap = 0, combines_cap = 0;
    unsigned *grid_bar = nullptr;
    unsigned long long *prof = nullptr;
    int prof_stride = 0;

    // the persistent step kernel
    StepPlan plan;
    MkParams mk{};
    // vocabulary pruning: the full-vocabulary schedule and maps to return to, the gathered rows of the current subset
    // and their token ids
    StepSchedule sched_full;
    std::vector<CUtensorMap> maps_full_lm;   // MK_MAX_VARIANTS maps of the full output layer
    MkOp lm_op_full{};
    int *vocab_ids = nullptr;       // [vocab]
    uint16_t *sub_lm = nullptr;     // [vocab_subset][hidden] or null
    int vocab_subset = 0;           // 0 = full vocabulary

    cudaStream_t build_stream = nullptr;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    int launches_per_step = 0;
    PrefillBuffers pf;           // work buffers of edgefm_prefill, allocated at its first call
    int prefill_launches = 0;    // kernels the last edgefm_prefill enqueued
    uint32_t pf_wait_limit = 1u << 24, pf_extra_arrivals = 0;   // edgefm_debug_set_prefill_wait

    // host mirrors
    int cur_len = 0;
    bool have_token = false;
    bool len_exact = true;       // false between a verified block (the device decides how far the cache grows) and edgefm_sync_length
    bool req_valid = false;
    StepRequest last_req{};
    std::string err;
};

namespace {

thread_local std::string g_create_error;

edgefm_status fail(edgefm_ctx *ctx, edgefm_status st, const char *fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    if (ctx) ctx->err = buf; else g_create_error = buf;
    return st;
}

#define CUDA_TRY(ctx, call)                                                                                   \
    do {                                                                                                      \
        cudaError_t e_ = (call);                                                                              \
        if (e_ != cudaSuccess)                                                                                \
            return fail(ctx, e_ == cudaErrorMemoryAllocation ? EDGEFM_ERR_OUT_OF_MEMORY : EDGEFM_ERR_CUDA,    \
                        "%s failed: %s", #call, cudaGetErrorString(e_));                                      \
    } while (0)

struct DeviceGuard {
    int prev = -1;
    bool active = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) { cudaSetDevice(dev); active = true; }
    }
    ~DeviceGuard() { if (active) cudaSetDevice(prev); }
};

template <typename T>
cudaError_t dev_alloc(T **p, size_t count) {
    return cudaMalloc(reinterpret_cast<void **>(p), count * sizeof(T) + 256);  // + guard bytes behind every buffer
}

void free_all(edgefm_ctx *c) {
    if (c->exec) cudaGraphExecDestroy(c->exec);
    if (c->graph) cudaGraphDestroy(c->graph);
    if (c->build_stream) cudaStreamDestroy(c->build_stream);
    void *bufs[] = {c->k_cache, c->v_cache, c->x, c->q, c->attn, c->act, c->inv_freq, c->part_m, c->part_l,
                    c->part_o, c->lm_part_val, c->lm_part_idx, c->tickets, c->state, c->req, c->d_ops, c->d_op_w, c->d_maps, c->d_tiles,
                    c->d_cta_tab, c->d_combines, c->grid_bar, c->prof, c->vocab_ids, c->sub_lm, c->k_scale, c->v_scale, c->kv_stage};
    for (void *b : bufs) if (b) cudaFree(b);
    if (c->pf.chunk) prefill_free(&c->pf);
}

edgefm_status ensure_prefill_buffers(edgefm_ctx *ctx);
PrefillModel prefill_model(edgefm_ctx *ctx);

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// One cooperative launch of the step kernel: all CTAs are co-resident, which the grid barriers rely on.
cudaError_t launch_step(MegaKernel kern, const StepPlan &pl, const MkParams &mk, cudaStream_t s) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(pl.grid);
    cfg.blockDim = dim3((pl.nw + 1) * 32);
    cfg.dynamicSmemBytes = pl.dyn_smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, mk);
}

// Record the step once; every decode step replays this graph (one kernel node).
cudaError_t record_graph(edgefm_ctx *c) {
    if (c->exec) { cudaGraphExecDestroy(c->exec); c->exec = nullptr; }
    if (c->graph) { cudaGraphDestroy(c->graph); c->graph = nullptr; }
    cudaError_t e = cudaStreamBeginCapture(c->build_stream, cudaStreamCaptureModeThreadLocal);
    if (e != cudaSuccess) return e;
    const cudaError_t le = launch_step(c->plan.kernel, c->plan, c->mk, c->build_stream);
    e = cudaStreamEndCapture(c->build_stream, &c->graph);
    if (le != cudaSuccess) return le;
    if (e != cudaSuccess) return e;
    c->launches_per_step = 1;
    return cudaGraphInstantiate(&c->exec, c->graph, 0);
}

}  // namespace

extern "C" {

const char *edgefm_version(void) { return "edgefm-b200 0.2 (sm_100a)"; }

const char *edgefm_last_error(const edgefm_ctx *ctx) { return ctx ? ctx->err.c_str() : g_create_error.c_str(); }

edgefm_status edgefm_create(const edgefm_shape *shape, const edgefm_weights *weights, int32_t max_context,
                            edgefm_ctx **out) {
    return edgefm_create_with_options(shape, weights, max_context, nullptr, out);
}

edgefm_status edgefm_create_with_options(const edgefm_shape *shape, const edgefm_weights *weights, int32_t max_context,
                                         const edgefm_options *options, edgefm_ctx **out) {
    if (out) *out = nullptr;
    if (options) {
        if (options->kv_format != EDGEFM_KV_BF16 && options->kv_format != EDGEFM_KV_INT8)
            return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "unknown kv_format %d", options->kv_format);
        for (int r : options->reserved)
            if (r != 0) return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "reserved option fields must be zero");
    }
    const bool kv8 = options && options->kv_format == EDGEFM_KV_INT8;
    if (options && options->block_tokens != 0 && options->block_tokens != 1 && options->block_tokens != 2 && options->block_tokens != 4)
        return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "block_tokens %d is not supported (0, 1, 2 or 4)", options->block_tokens);
    const int M = options && options->block_tokens > 1 ? options->block_tokens : 1;
    if (M > 1 && kv8) return fail(nullptr, EDGEFM_ERR_BAD_SHAPE, "blocks of several tokens need the plain bf16 cache");
    if (!shape || !weights || !out) return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "null argument");
    if (max_context < 1) return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "max_context must be >= 1");
    const edgefm_shape &sh = *shape;
    if (sh.n_layers < 1 || sh.hidden < 8 || sh.n_q_heads < 1 || sh.n_kv_heads < 1 || sh.ffn < 8 || sh.vocab < 1)
        return fail(nullptr, EDGEFM_ERR_BAD_SHAPE, "non-positive dimension");
    if (sh.hidden % 8 || sh.ffn % 8) return fail(nullptr, EDGEFM_ERR_BAD_SHAPE, "hidden and ffn must be multiples of 8");
    if (sh.head_dim != 64 && sh.head_dim != 128) return fail(nullptr, EDGEFM_ERR_BAD_SHAPE, "head_dim must be 64 or 128");
    if (sh.n_q_heads % sh.n_kv_heads) return fail(nullptr, EDGEFM_ERR_BAD_SHAPE, "n_q_heads must be a multiple of n_kv_heads");
    const int G = sh.n_q_heads / sh.n_kv_heads;
    if (G > 8) return fail(nullptr, EDGEFM_ERR_BAD_SHAPE, "group size n_q/n_kv must be <= 8");
    if (!(sh.rms_eps >= 0.f) || !(sh.rope_theta > 0.f)) return fail(nullptr, EDGEFM_ERR_BAD_SHAPE, "bad rms_eps / rope_theta");
    if (static_cast<long long>(sh.vocab) * sh.hidden > (1LL << 40)) return fail(nullptr, EDGEFM_ERR_BAD_SHAPE, "model too large");
    if (!weights->embed || !weights->final_norm || !weights->lm_head || !weights->layers)
        return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "null weight pointer");
    if (!aligned16(weights->embed) || !aligned16(weights->lm_head) || !aligned16(weights->final_norm))
        return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "weight pointers must be 16-byte aligned");
    for (int l = 0; l < sh.n_layers; ++l) {
        const edgefm_layer_weights &w = weights->layers[l];
        if (!w.input_norm || !w.wqkv || !w.wo || !w.post_norm || !w.w_gate_up || !w.w_down || (sh.qkv_bias && !w.bqkv))
            return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "null weight pointer in layer %d", l);
        if (!aligned16(w.input_norm) || !aligned16(w.wqkv) || !aligned16(w.wo) || !aligned16(w.post_norm) ||
            !aligned16(w.w_gate_up) || !aligned16(w.w_down))
            return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "weight pointers must be 16-byte aligned (layer %d)", l);
    }

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return fail(nullptr, EDGEFM_ERR_CUDA, "no CUDA device available (this library has no CPU path)");
    }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
        cudaGetLastError();
        return fail(nullptr, EDGEFM_ERR_CUDA, "cudaGetDeviceProperties failed");
    }
    if (prop.major < 10) return fail(nullptr, EDGEFM_ERR_CUDA, "device sm_%d%d is not supported (built for sm_100a)", prop.major, prop.minor);

    edgefm_ctx *c = new (std::nothrow) edgefm_ctx();
    if (!c) return fail(nullptr, EDGEFM_ERR_OUT_OF_MEMORY, "host allocation failed");
    c->shape = sh;
    c->kv_format = kv8 ? EDGEFM_KV_INT8 : EDGEFM_KV_BF16;
    c->block_tokens = M;
    c->max_context = max_context;
    c->device = dev;
    c->num_sms = prop.multiProcessorCount;
    c->layers.assign(weights->layers, weights->layers + sh.n_layers);
    c->embed = weights->embed; c->final_norm = weights->final_norm; c->lm_head = weights->lm_head;

    auto bail = [&](edgefm_status st, const char *what, cudaError_t e) {
        g_create_error = std::string(what) + ": " + cudaGetErrorString(e);
        cudaGetLastError();
        free_all(c);
        delete c;
        return st;
    };
#define CREATE_TRY(call)                                                                                            \
    do {                                                                                                            \
        cudaError_t e_ = (call);                                                                                    \
        if (e_ != cudaSuccess) return bail(e_ == cudaErrorMemoryAllocation ? EDGEFM_ERR_OUT_OF_MEMORY : EDGEFM_ERR_CUDA, #call, e_); \
    } while (0)

    const int H = sh.hidden, d = sh.head_dim, nq = sh.n_q_heads, nkv = sh.n_kv_heads, F = sh.ffn;

    StepPlan &pl = c->plan;
    int smem_optin = 0, coop = 0;
    CREATE_TRY(cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    CREATE_TRY(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
    if (!coop) return bail(EDGEFM_ERR_CUDA, "device lacks cooperative launch", cudaErrorNotSupported);
    {
        cudaError_t ce = cudaSuccess;
        if (const char *why = plan_step_and_schedule(sh, max_context, c->num_sms, smem_optin, &pl, &c->sched_full, &ce, kv8, M))
            return bail(ce != cudaSuccess ? EDGEFM_ERR_CUDA : EDGEFM_ERR_BAD_SHAPE, why, ce != cudaSuccess ? ce : cudaErrorInvalidValue);
    }
    const StepSchedule &ss = c->sched_full;

    const size_t kv_elems = static_cast<size_t>(sh.n_layers) * nkv * max_context * d;
    const size_t kv_bytes = kv8 ? kv_elems : kv_elems * 2;
    CREATE_TRY(dev_alloc(&c->k_cache, (kv_bytes + 1) / 2));
    CREATE_TRY(dev_alloc(&c->v_cache, (kv_bytes + 1) / 2));
    if (kv8) {
        const size_t kv_rows = static_cast<size_t>(sh.n_layers) * nkv * max_context;
        CREATE_TRY(dev_alloc(&c->k_scale, kv_rows));
        CREATE_TRY(dev_alloc(&c->v_scale, kv_rows));
        CREATE_TRY(dev_alloc(&c->kv_stage, static_cast<size_t>(2) * nkv * d));
        CREATE_TRY(cudaMemset(c->k_scale, 0, kv_rows * sizeof(float)));
        CREATE_TRY(cudaMemset(c->v_scale, 0, kv_rows * sizeof(float)));
        CREATE_TRY(cudaMemset(c->kv_stage, 0, static_cast<size_t>(2) * nkv * d * sizeof(float)));
    }
    // (work buffers hold one vector per token of a block)
    CREATE_TRY(dev_alloc(&c->x, static_cast<size_t>(M) * H));
    CREATE_TRY(dev_alloc(&c->q, static_cast<size_t>(M) * nq * d));
    CREATE_TRY(dev_alloc(&c->attn, static_cast<size_t>(M) * nq * d));
    CREATE_TRY(dev_alloc(&c->act, static_cast<size_t>(M) * mk_splits(M) * ((F + MK_TILE_COLS - 1) / MK_TILE_COLS * MK_TILE_COLS) / 2));   // three bf16 arrays of F rounded
                                                                                         // up to whole column pieces (the pieces of every value)
    CREATE_TRY(dev_alloc(&c->inv_freq, d / 2));
    CREATE_TRY(dev_alloc(&c->part_m, static_cast<size_t>(M) * nq * pl.max_chunks));
    CREATE_TRY(dev_alloc(&c->part_l, static_cast<size_t>(M) * nq * pl.max_chunks));
    CREATE_TRY(dev_alloc(&c->part_o, static_cast<size_t>(M) * nq * pl.max_chunks * d));
    CREATE_TRY(dev_alloc(&c->lm_part_val, static_cast<size_t>(M) * pl.grid));
    CREATE_TRY(dev_alloc(&c->lm_part_idx, static_cast<size_t>(M) * pl.grid));
    CREATE_TRY(dev_alloc(&c->tickets, nq + nkv + 2 + nq + 2 * nkv));   // tickets, then the per-head counters of the QKV projection
    CREATE_TRY(dev_alloc(&c->state, 1));
    CREATE_TRY(dev_alloc(&c->req, 1));
    CREATE_TRY(cudaMemset(c->k_cache, 0, kv_bytes));
    CREATE_TRY(cudaMemset(c->v_cache, 0, kv_bytes));
    CREATE_TRY(cudaMemset(c->tickets, 0, (nq + nkv + 2 + nq + 2 * nkv) * sizeof(unsigned)));
    CREATE_TRY(cudaMemset(c->state, 0, sizeof(StepState)));
    {
        StepRequest r{-1, -1, nullptr, nullptr};
        CREATE_TRY(cudaMemcpy(c->req, &r, sizeof r, cudaMemcpyHostToDevice));
        std::vector<double> inv(d / 2);
        for (int i = 0; i < d / 2; ++i) inv[i] = std::pow(static_cast<double>(sh.rope_theta), -2.0 * i / d);
        CREATE_TRY(cudaMemcpy(c->inv_freq, inv.data(), inv.size() * sizeof(double), cudaMemcpyHostToDevice));
    }

    // the operators of the step wired to the work buffers, the tile schedule and the tensor maps of the weights
    {
        std::vector<MkOp> ops(static_cast<size_t>(pl.n_ops));
        std::vector<const uint16_t *> op_w(static_cast<size_t>(pl.n_ops));
        fill_ops(sh, c->layers.data(), c->final_norm, c->lm_head, c->x, c->attn, c->q, c->act, ops.data(), op_w.data(), M);
        c->lm_op_full = ops.back();
        std::vector<CUtensorMap> maps(static_cast<size_t>(pl.n_ops) * MK_MAX_VARIANTS);
        if (const char *why = encode_maps(ss, sh, c->layers.data(), c->lm_head, sh.vocab, maps.data()))
            return bail(EDGEFM_ERR_CUDA, why, cudaErrorUnknown);
        c->maps_full_lm.assign(maps.end() - MK_MAX_VARIANTS, maps.end());
        c->tiles_cap = ss.tiles.size();
        c->combines_cap = static_cast<size_t>(pl.grid) * 5 * (2 * pl.nw + 4);
        if (ss.combines.size() > c->combines_cap) c->combines_cap = ss.combines.size();
        CREATE_TRY(dev_alloc(&c->d_ops, ops.size()));
        CREATE_TRY(dev_alloc(&c->d_op_w, op_w.size()));
        CREATE_TRY(cudaMemcpy(c->d_op_w, op_w.data(), op_w.size() * sizeof(op_w[0]), cudaMemcpyHostToDevice));
        CREATE_TRY(cudaMalloc(reinterpret_cast<void **>(&c->d_maps), maps.size() * sizeof(CUtensorMap)));
        CREATE_TRY(dev_alloc(&c->d_tiles, c->tiles_cap));
        CREATE_TRY(dev_alloc(&c->d_cta_tab, ss.cta_tab.size()));
        CREATE_TRY(dev_alloc(&c->d_combines, c->combines_cap));
        CREATE_TRY(cudaMemcpy(c->d_ops, ops.data(), ops.size() * sizeof(MkOp), cudaMemcpyHostToDevice));
        CREATE_TRY(cudaMemcpy(c->d_maps, maps.data(), maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice));
        CREATE_TRY(cudaMemcpy(c->d_tiles, ss.tiles.data(), ss.tiles.size() * sizeof(uint2), cudaMemcpyHostToDevice));
        CREATE_TRY(cudaMemcpy(c->d_cta_tab, ss.cta_tab.data(), ss.cta_tab.size() * sizeof(int), cudaMemcpyHostToDevice));
        if (!ss.combines.empty())
            CREATE_TRY(cudaMemcpy(c->d_combines, ss.combines.data(), ss.combines.size() * sizeof(MkCombine), cudaMemcpyHostToDevice));
    }
    CREATE_TRY(allow_max_dynamic_smem(pl.kernel, smem_optin));
    int per_sm = 0;
    CREATE_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, pl.kernel, (pl.nw + 1) * 32, pl.dyn_smem));
    if (per_sm < 1) return bail(EDGEFM_ERR_CUDA, "persistent kernel does not fit one CTA per SM", cudaErrorInvalidValue);
    CREATE_TRY(dev_alloc(&c->grid_bar, 1));
    CREATE_TRY(cudaMemset(c->grid_bar, 0, sizeof(unsigned)));
    CREATE_TRY(dev_alloc(&c->vocab_ids, static_cast<size_t>(sh.vocab)));
    CREATE_TRY(cudaMemset(c->vocab_ids, 0, static_cast<size_t>(sh.vocab) * sizeof(int)));
    MkParams &m = c->mk;
    fill_shape_params(&m, sh, max_context, pl, ss);
    m.ops = c->d_ops; m.op_weights = c->d_op_w; m.maps = c->d_maps; m.tiles = c->d_tiles; m.cta_tab = c->d_cta_tab; m.combines = c->d_combines;
    m.vocab_ids = c->vocab_ids;
    m.k_cache = c->k_cache; m.v_cache = c->v_cache; m.embed = (const uint16_t *)c->embed;
    m.kv8 = kv8 ? 1 : 0; m.k_scale = c->k_scale; m.v_scale = c->v_scale; m.kv_stage = c->kv_stage;
    m.inv_freq = c->inv_freq; m.x = c->x; m.q = c->q; m.attn = c->attn; m.part_m = c->part_m; m.part_l = c->part_l;
    m.part_o = c->part_o; m.tickets = c->tickets; m.barrier = c->grid_bar;
    m.head_ready = c->tickets + nq + nkv + 2; m.head_flags = pl.long_ctx ? 0 : MK_HEAD_FLAGS;
    m.lm_part_val = c->lm_part_val; m.lm_part_idx = c->lm_part_idx; m.state = c->state; m.req = c->req;
    const char *pe_ = getenv("EDGEFM_PROFILE");
    if (pe_ && pe_[0] == '1') {
        c->prof_stride = 3 + 14 * sh.n_layers;
        const size_t n_prof = static_cast<size_t>(pl.grid) * c->prof_stride + MK_NW_MAX * 16 * 4 + 8;   // + the optional per-warp trace
        CREATE_TRY(dev_alloc(&c->prof, n_prof));
        CREATE_TRY(cudaMemset(c->prof, 0, n_prof * 8));
        m.prof = c->prof; m.prof_stride = c->prof_stride;
    }

    CREATE_TRY(cudaStreamCreateWithFlags(&c->build_stream, cudaStreamNonBlocking));
    CREATE_TRY(record_graph(c));
    CREATE_TRY(cudaDeviceSynchronize());
#undef CREATE_TRY
    g_create_error.clear();
    *out = c;
    return EDGEFM_OK;
}

namespace {
// Common part of edgefm_prefill_kv (slot0 = 0) and edgefm_append_kv.
edgefm_status copy_kv_in(edgefm_ctx *ctx, const void *k, const void *v, int32_t slot0, int32_t n_positions, int64_t stride_layer,
                         int64_t stride_head, int64_t stride_pos, void *stream) {
    if (n_positions < 0) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "n_positions < 0");
    if (static_cast<int64_t>(slot0) + n_positions > ctx->max_context)
        return fail(ctx, EDGEFM_ERR_CONTEXT_FULL, "%d positions from slot %d exceed max_context %d", n_positions, slot0, ctx->max_context);
    if (n_positions > 0 && (!k || !v)) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "null k or v");
    if (n_positions > 0 && (stride_layer < 0 || stride_head < 0 || stride_pos < ctx->shape.head_dim))
        return fail(ctx, EDGEFM_ERR_INVALID_ARG, "bad strides");
    DeviceGuard guard(ctx->device);
    const edgefm_shape &sh = ctx->shape;
    if (ctx->kv_format == EDGEFM_KV_INT8) {
        long long blocks = (static_cast<long long>(sh.n_layers) * sh.n_kv_heads * n_positions * 2 + 7) / 8;   // 8 warps (rows) per block
        if (blocks < 1) blocks = 1;
        if (blocks > ctx->num_sms * 16) blocks = ctx->num_sms * 16;
        prefill_quantize_kernel<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(
            static_cast<const uint16_t *>(k), static_cast<const uint16_t *>(v), reinterpret_cast<signed char *>(ctx->k_cache),
            reinterpret_cast<signed char *>(ctx->v_cache), ctx->k_scale, ctx->v_scale, sh.n_layers, sh.n_kv_heads, n_positions, sh.head_dim,
            ctx->max_context, stride_layer, stride_head, stride_pos, ctx->state, slot0);
        CUDA_TRY(ctx, cudaGetLastError());
        ctx->cur_len = slot0 + n_positions;
        ctx->len_exact = true;
        ctx->err.clear();
        return EDGEFM_OK;
    }
    const int vec_ok = n_positions > 0 && aligned16(k) && aligned16(v) && stride_layer % 8 == 0 && stride_head % 8 == 0 &&
                       stride_pos % 8 == 0;
    const long long total = static_cast<long long>(sh.n_layers) * sh.n_kv_heads * n_positions * sh.head_dim;
    long long blocks = (total / (vec_ok ? 8 : 1) + 255) / 256;
    if (blocks < 1) blocks = 1;
    if (blocks > ctx->num_sms * 16) blocks = ctx->num_sms * 16;
    prefill_copy_kernel<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint16_t *>(k), static_cast<const uint16_t *>(v), ctx->k_cache, ctx->v_cache, sh.n_layers,
        sh.n_kv_heads, n_positions, sh.head_dim, ctx->max_context, stride_layer, stride_head, stride_pos, vec_ok, ctx->state, slot0);
    CUDA_TRY(ctx, cudaGetLastError());
    ctx->cur_len = slot0 + n_positions;
    ctx->len_exact = true;
    ctx->err.clear();
    return EDGEFM_OK;
}
}  // namespace

edgefm_status edgefm_prefill_kv(edgefm_ctx *ctx, const void *k, const void *v, int32_t n_positions, int64_t stride_layer,
                                int64_t stride_head, int64_t stride_pos, void *stream) {
    if (!ctx) return EDGEFM_ERR_INVALID_ARG;
    return copy_kv_in(ctx, k, v, 0, n_positions, stride_layer, stride_head, stride_pos, stream);
}

edgefm_status edgefm_append_kv(edgefm_ctx *ctx, const void *k, const void *v, int32_t start, int32_t n_positions, int64_t stride_layer,
                               int64_t stride_head, int64_t stride_pos, void *stream) {
    if (!ctx) return EDGEFM_ERR_INVALID_ARG;
    if (start < 0 || start > ctx->cur_len)
        return fail(ctx, EDGEFM_ERR_INVALID_ARG, "start %d outside [0, %d]: the cache may not have holes", start, ctx->cur_len);
    return copy_kv_in(ctx, k, v, start, n_positions, stride_layer, stride_head, stride_pos, stream);
}

edgefm_status edgefm_decode_step(edgefm_ctx *ctx, int32_t token_id, int32_t position, void *stream, float *logits_out,
                                 int32_t *next_token_out) {
    if (!ctx) return EDGEFM_ERR_INVALID_ARG;
    if (token_id < -1 || token_id >= ctx->shape.vocab) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "token_id %d out of range", token_id);
    if (position < -1) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "position %d out of range", position);
    if (token_id == -1 && !ctx->have_token)
        return fail(ctx, EDGEFM_ERR_INVALID_ARG, "token_id -1 needs a previous step on this context");
    if (ctx->cur_len >= ctx->max_context)
        return fail(ctx, EDGEFM_ERR_CONTEXT_FULL, "KV cache is full (%d slots)", ctx->max_context);
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    StepRequest r{token_id, position, logits_out, next_token_out};
    if (!ctx->req_valid || std::memcmp(&r, &ctx->last_req, sizeof r) != 0) {
        // small pageable copy: the runtime stages the bytes before returning, so `r` may live on the stack
        CUDA_TRY(ctx, cudaMemcpyAsync(ctx->req, &r, sizeof r, cudaMemcpyHostToDevice, s));
        ctx->last_req = r;
        ctx->req_valid = true;
    }
    CUDA_TRY(ctx, cudaGraphLaunch(ctx->exec, s));
    ctx->cur_len += 1;
    ctx->have_token = true;
    ctx->err.clear();
    return EDGEFM_OK;
}

edgefm_status edgefm_verify_block(edgefm_ctx *ctx, const int32_t *tokens, int32_t m, int32_t position, void *stream, float *logits_out,
                                  int32_t *n_accepted_out, int32_t *next_token_out) {
    if (!ctx) return EDGEFM_ERR_INVALID_ARG;
    if (!tokens) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "null tokens");
    const bool dense = m > ctx->block_tokens;   // longer blocks go through the dense path (the prefill kernels)
    if (m < 1 || m > std::max(ctx->block_tokens, PF_VERIFY_MAX))
        return fail(ctx, EDGEFM_ERR_INVALID_ARG, "m = %d: blocks of 1 .. %d tokens", m, std::max(ctx->block_tokens, PF_VERIFY_MAX));
    if (dense && (tokens[0] < 0 || position < 0))
        return fail(ctx, EDGEFM_ERR_INVALID_ARG, "a block of %d tokens on this context (block_tokens = %d) takes the dense path, which needs tokens[0] and position given", m, ctx->block_tokens);
    if (dense && !ctx->len_exact)
        return fail(ctx, EDGEFM_ERR_INVALID_ARG, "the dense path places the block behind the host's cache length: call edgefm_sync_length after the previous block first");
    if (tokens[0] < -1 || tokens[0] >= ctx->shape.vocab) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "tokens[0] = %d out of range", tokens[0]);
    for (int t = 1; t < m; ++t)
        if (tokens[t] < 0 || tokens[t] >= ctx->shape.vocab) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "tokens[%d] = %d out of range", t, tokens[t]);
    if (position < -1) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "position %d out of range", position);
    if (tokens[0] == -1 && !ctx->have_token) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "tokens[0] = -1 needs a previous step on this context");
    if (ctx->cur_len + m > ctx->max_context)
        return fail(ctx, EDGEFM_ERR_CONTEXT_FULL, "%d tokens do not fit behind %d of %d cache slots", m, ctx->cur_len, ctx->max_context);
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (dense) {
        if (const edgefm_status st = ensure_prefill_buffers(ctx)) return st;
        PrefillModel pm = prefill_model(ctx);
        int launches = 0;
        const int slot0 = ctx->cur_len;
        if (const char *e = prefill_run(pm, &ctx->pf, tokens, m, slot0, position, true, s, &launches)) {
            cudaGetLastError();
            return fail(ctx, EDGEFM_ERR_CUDA, "%s", e);
        }
        const bool sub = ctx->vocab_subset > 0;
        if (const char *e = prefill_verify_head(pm, &ctx->pf, m, ctx->final_norm, sub ? static_cast<const void *>(ctx->sub_lm) : ctx->lm_head,
                                                sub ? ctx->vocab_ids : nullptr, sub ? ctx->vocab_subset : ctx->shape.vocab, logits_out, n_accepted_out,
                                                next_token_out, slot0, position, s)) {
            cudaGetLastError();
            return fail(ctx, EDGEFM_ERR_CUDA, "%s", e);
        }
        ctx->prefill_launches = launches + 1;
        ctx->cur_len += m;     // an upper bound until edgefm_sync_length
        ctx->len_exact = false;
        ctx->have_token = true;
        ctx->err.clear();
        return EDGEFM_OK;
    }
    StepRequest r{tokens[0], position, logits_out, next_token_out};
    r.m = m;
    for (int t = 1; t < m && t <= 3; ++t) r.draft[t - 1] = tokens[t];
    r.n_accepted_out = n_accepted_out;
    if (!ctx->req_valid || std::memcmp(&r, &ctx->last_req, sizeof r) != 0) {
        CUDA_TRY(ctx, cudaMemcpyAsync(ctx->req, &r, sizeof r, cudaMemcpyHostToDevice, s));
        ctx->last_req = r;
        ctx->req_valid = true;
    }
    CUDA_TRY(ctx, cudaGraphLaunch(ctx->exec, s));
    ctx->cur_len += m;     // an upper bound until edgefm_sync_length: the device decides how many tokens are accepted
    if (m > 1) ctx->len_exact = false;
    ctx->have_token = true;
    ctx->err.clear();
    return EDGEFM_OK;
}

edgefm_status edgefm_prefill_tokens(edgefm_ctx *ctx, const int32_t *tokens, int32_t n, int32_t position, void *stream) {
    if (!ctx) return EDGEFM_ERR_INVALID_ARG;
    if (n < 0 || (n > 0 && !tokens)) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "bad token list");
    if (position < 0) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "position %d out of range", position);
    for (int i = 0; i < n; ++i)
        if (tokens[i] < 0 || tokens[i] >= ctx->shape.vocab) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "tokens[%d] = %d out of range", i, tokens[i]);
    if (ctx->cur_len + n > ctx->max_context)
        return fail(ctx, EDGEFM_ERR_CONTEXT_FULL, "%d tokens do not fit behind %d of %d cache slots", n, ctx->cur_len, ctx->max_context);
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int M = ctx->block_tokens;
    for (int i = 0; i < n; i += M) {   // the step kernel, as many given tokens per call as the context's build carries
        const int m = n - i < M ? n - i : M;
        StepRequest r{tokens[i], position + i, nullptr, nullptr};
        r.m = m;
        for (int t = 1; t < m; ++t) r.draft[t - 1] = tokens[i + t];
        r.flags = 1;
        CUDA_TRY(ctx, cudaMemcpyAsync(ctx->req, &r, sizeof r, cudaMemcpyHostToDevice, s));
        ctx->last_req = r;
        ctx->req_valid = true;
        CUDA_TRY(ctx, cudaGraphLaunch(ctx->exec, s));
        ctx->cur_len += m;
        ctx->have_token = true;
    }
    ctx->err.clear();
    return EDGEFM_OK;
}

}  // extern "C" (helpers of the dense path follow)

namespace {

// Work buffers of the dense path (prefill, long verified blocks): allocated at the first use, kept.
edgefm_status ensure_prefill_buffers(edgefm_ctx *ctx) {
    if (ctx->pf.chunk == 0) {
        const int chunk = std::min(PF_CHUNK_MAX, ctx->max_context);
        if (prefill_alloc(&ctx->pf, ctx->shape, chunk, ctx->kv_format == EDGEFM_KV_INT8) != cudaSuccess) {
            cudaGetLastError();
            prefill_free(&ctx->pf);
            return fail(ctx, EDGEFM_ERR_OUT_OF_MEMORY, "work buffers of the dense path (%zu bytes)", prefill_buffer_bytes(ctx->shape, chunk));
        }
    }
    ctx->pf.wait_limit = ctx->pf_wait_limit;
    ctx->pf.extra_arrivals = ctx->pf_extra_arrivals;
    return EDGEFM_OK;
}

PrefillModel prefill_model(edgefm_ctx *ctx) {
    return PrefillModel{ctx->shape, ctx->layers.data(), ctx->embed, ctx->k_cache, ctx->v_cache,
                        ctx->kv_format == EDGEFM_KV_INT8 ? ctx->k_scale : nullptr, ctx->kv_format == EDGEFM_KV_INT8 ? ctx->v_scale : nullptr,
                        ctx->max_context, ctx->state, ctx->num_sms};
}

}  // namespace

extern "C" {

edgefm_status edgefm_prefill(edgefm_ctx *ctx, const int32_t *tokens, int32_t n, int32_t position, void *stream, float *logits_out,
                             int32_t *next_token_out) {
    if (!ctx) return EDGEFM_ERR_INVALID_ARG;
    if (n < 1 || !tokens) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "bad token list");
    if (position < 0) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "position %d out of range", position);
    for (int i = 0; i < n; ++i)
        if (tokens[i] < 0 || tokens[i] >= ctx->shape.vocab) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "tokens[%d] = %d out of range", i, tokens[i]);
    if (ctx->cur_len + n > ctx->max_context)
        return fail(ctx, EDGEFM_ERR_CONTEXT_FULL, "%d tokens do not fit behind %d of %d cache slots", n, ctx->cur_len, ctx->max_context);
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // Prompts of at least 8 tokens go through the dense path whole, and the output layer runs for the last row alone (one pass
    // over its matrix); shorter ones leave their last token to a decode step (which streams all weights again: 1.1 ms at the
    // 1.5B shape, against one more layer for a handful of rows).
    if (!ctx->len_exact)
        return fail(ctx, EDGEFM_ERR_INVALID_ARG, "the prompt is placed behind the host's cache length: call edgefm_sync_length after a verified block first");
    const bool dense_all = n >= 8;
    const int n_dense = dense_all ? n : n - 1;
    if (n_dense > 0)
        if (const edgefm_status st = ensure_prefill_buffers(ctx)) return st;
    PrefillModel pm = prefill_model(ctx);
    ctx->prefill_launches = 0;
    for (int i = 0; i < n_dense;) {
        const int c = std::min(ctx->pf.chunk, n_dense - i);
        int launches = 0;
        if (const char *e = prefill_run(pm, &ctx->pf, tokens + i, c, ctx->cur_len, position + i, dense_all && i + c == n_dense, s, &launches)) {
            cudaGetLastError();
            return fail(ctx, EDGEFM_ERR_CUDA, "%s", e);
        }
        ctx->prefill_launches += launches;
        ctx->cur_len += c;
        i += c;
        if (dense_all && i == n_dense) {   // the output layer for the prompt's last token, and the state a decode step would leave
            const bool sub = ctx->vocab_subset > 0;
            if (const char *e = prefill_head(pm, &ctx->pf, c - 1, ctx->final_norm, sub ? static_cast<const void *>(ctx->sub_lm) : ctx->lm_head,
                                             sub ? ctx->vocab_ids : nullptr, sub ? ctx->vocab_subset : ctx->shape.vocab, logits_out, next_token_out,
                                             tokens[n - 1], position + n - 1, s)) {
                cudaGetLastError();
                return fail(ctx, EDGEFM_ERR_CUDA, "%s", e);
            }
            ctx->prefill_launches += 1;
            ctx->have_token = true;
            ctx->err.clear();
            return EDGEFM_OK;
        }
    }
    const edgefm_status st = edgefm_decode_step(ctx, tokens[n - 1], position + n - 1, stream, logits_out, next_token_out);
    if (st == EDGEFM_OK) ctx->prefill_launches += ctx->launches_per_step;
    return st;
}

edgefm_status edgefm_sync_length(edgefm_ctx *ctx, void *stream, int32_t *cur_len_host) {
    if (!ctx || !cur_len_host) return EDGEFM_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    CUDA_TRY(ctx, cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    StepState st{};
    CUDA_TRY(ctx, cudaMemcpy(&st, ctx->state, sizeof st, cudaMemcpyDeviceToHost));
    ctx->cur_len = st.cur_len;
    ctx->len_exact = true;
    *cur_len_host = st.cur_len;
    return EDGEFM_OK;
}

edgefm_status edgefm_destroy(edgefm_ctx *ctx) {
    if (!ctx) return EDGEFM_OK;
    DeviceGuard guard(ctx->device);
    cudaError_t e = cudaDeviceSynchronize();
    free_all(ctx);
    delete ctx;
    return e == cudaSuccess ? EDGEFM_OK : EDGEFM_ERR_CUDA;
}

edgefm_status edgefm_get_length(const edgefm_ctx *ctx, int32_t *cur_len_host) {
    if (!ctx || !cur_len_host) return EDGEFM_ERR_INVALID_ARG;
    *cur_len_host = ctx->cur_len;
    return EDGEFM_OK;
}

edgefm_status edgefm_set_vocab_subset(edgefm_ctx *ctx, const int32_t *token_ids, int32_t n, void *stream) {
    if (!ctx) return EDGEFM_ERR_INVALID_ARG;
    if (n < 0 || n > ctx->shape.vocab) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "subset size %d outside [0, %d]", n, ctx->shape.vocab);
    if (n > 0 && !token_ids) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "null token_ids");
    for (int i = 0; i < n; ++i) {
        if (token_ids[i] < 0 || token_ids[i] >= ctx->shape.vocab)
            return fail(ctx, EDGEFM_ERR_INVALID_ARG, "token_ids[%d] = %d out of range", i, token_ids[i]);
        if (i > 0 && token_ids[i] <= token_ids[i - 1])
            return fail(ctx, EDGEFM_ERR_INVALID_ARG, "token_ids must be strictly ascending (entry %d)", i);
    }
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int H = ctx->shape.hidden;
    const StepPlan &pl = ctx->plan;
    // the schedule of the step with the output layer cut down to n rows (the other operators keep their lists), its
    // tensor maps over the gathered rows, and the operator descriptor
    StepSchedule sub;
    const StepSchedule *ss = &ctx->sched_full;
    std::vector<CUtensorMap> lm_maps = ctx->maps_full_lm;
    MkOp op = ctx->lm_op_full;
    uint16_t *fresh = nullptr;
    if (n > 0) {
        for (int o = 0; o < 4; ++o) sub.ops[o] = ctx->sched_full.ops[o];
        OpShape os[5];
        op_shapes(ctx->shape, n, os);
        if (const char *why = plan_op(os[4], 4, pl.grid, pl.nw, pl.slot_rows, &sub.ops[4]))
            return fail(ctx, EDGEFM_ERR_BAD_SHAPE, "a subset of %d rows does not fit the tile plan of this context: %s", n, why);
        assemble_schedule(&sub, pl.grid, pl.nw);
        if (sub.tiles.size() > ctx->tiles_cap || sub.combines.size() > ctx->combines_cap ||
            sub.smem_bytes() > static_cast<size_t>(ctx->mk.sched_bytes))
            return fail(ctx, EDGEFM_ERR_BAD_SHAPE, "a subset of %d rows does not fit the tile plan of this context", n);
        ss = &sub;
        CUDA_TRY(ctx, cudaMalloc(&fresh, static_cast<size_t>(n) * H * sizeof(uint16_t)));
        for (int v = 0; v < MK_MAX_VARIANTS; ++v) {
            std::memset(&lm_maps[v], 0, sizeof(CUtensorMap));
            if (v < sub.ops[4].n_variants && !encode_weight_map(&lm_maps[v], fresh, n, H, sub.ops[4].variant_rows[v])) {
                cudaFree(fresh);
                return fail(ctx, EDGEFM_ERR_CUDA, "cuTensorMapEncodeTiled failed");
            }
        }
        op.units_total = n;
        op.layer_flags = (op.layer_flags & ~0xff) | PHF_REMAP;
    }
    // steps already enqueued on the stream still read the previous subset
    cudaError_t e = cudaStreamSynchronize(s);
    if (e == cudaSuccess && n > 0) {
        e = cudaMemcpyAsync(ctx->vocab_ids, token_ids, static_cast<size_t>(n) * sizeof(int32_t), cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess) {
            int blocks = (n + 7) / 8;
            if (blocks > ctx->num_sms * 8) blocks = ctx->num_sms * 8;
            gather_rows_kernel<<<blocks, 256, 0, s>>>(static_cast<const uint16_t *>(ctx->lm_head), ctx->vocab_ids, fresh, n, H);
            e = cudaGetLastError();
        }
    }
    const size_t lm_index = static_cast<size_t>(ctx->mk.nph - 1);
    const uint16_t *lm_w = n > 0 ? fresh : static_cast<const uint16_t *>(ctx->lm_head);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->d_ops + lm_index, &op, sizeof op, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->d_op_w + lm_index, &lm_w, sizeof lm_w, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(ctx->d_maps + lm_index * MK_MAX_VARIANTS * sizeof(CUtensorMap), lm_maps.data(), MK_MAX_VARIANTS * sizeof(CUtensorMap),
                            cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->d_tiles, ss->tiles.data(), ss->tiles.size() * sizeof(uint2), cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->d_cta_tab, ss->cta_tab.data(), ss->cta_tab.size() * sizeof(int), cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess && !ss->combines.empty())
        e = cudaMemcpyAsync(ctx->d_combines, ss->combines.data(), ss->combines.size() * sizeof(MkCombine), cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);   // the host buffers are read before the call returns
    if (e != cudaSuccess) {
        if (fresh) cudaFree(fresh);
        return fail(ctx, EDGEFM_ERR_CUDA, "set_vocab_subset: %s", cudaGetErrorString(e));
    }
    if (ctx->sub_lm) cudaFree(ctx->sub_lm);
    ctx->sub_lm = fresh;
    ctx->vocab_subset = n;
    ctx->err.clear();
    return EDGEFM_OK;
}

edgefm_status edgefm_get_launches_per_step(const edgefm_ctx *ctx, int32_t *n) {
    if (!ctx || !n) return EDGEFM_ERR_INVALID_ARG;
    *n = ctx->launches_per_step;
    return EDGEFM_OK;
}

edgefm_status edgefm_debug_profile(edgefm_ctx *ctx, uint64_t *out_host, int64_t capacity, int32_t *n_ctas, int32_t *stride) {
    if (!ctx || !n_ctas || !stride) return EDGEFM_ERR_INVALID_ARG;
    *n_ctas = ctx->prof ? ctx->plan.grid : 0;
    *stride = ctx->prof_stride;
    if (!ctx->prof || !out_host) return EDGEFM_OK;
    int64_t n = static_cast<int64_t>(ctx->plan.grid) * ctx->prof_stride;
    if (capacity < n) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "profile buffer too small");
    if (capacity >= n + MK_NW_MAX * 16 * 4 + 8) n += MK_NW_MAX * 16 * 4 + 8;   // optional per-warp trace behind the table
    DeviceGuard guard(ctx->device);
    CUDA_TRY(ctx, cudaDeviceSynchronize());
    CUDA_TRY(ctx, cudaMemcpy(out_host, ctx->prof, static_cast<size_t>(n) * 8, cudaMemcpyDeviceToHost));
    return EDGEFM_OK;
}

edgefm_status edgefm_debug_plan(const edgefm_ctx *ctx, int32_t *out8) {
    if (!ctx || !out8) return EDGEFM_ERR_INVALID_ARG;
    const StepPlan &pl = ctx->plan;
    out8[0] = pl.grid; out8[1] = pl.nw; out8[2] = pl.slots; out8[3] = pl.slot_bytes; out8[4] = static_cast<int32_t>(pl.dyn_smem);
    out8[5] = ctx->sched_full.max_cta_tiles; out8[6] = static_cast<int32_t>(pl.sched_bytes); out8[7] = pl.long_ctx ? 1 : 0;
    return EDGEFM_OK;
}

edgefm_status edgefm_debug_set_wait_limit(edgefm_ctx *ctx, uint32_t limit_ns, int32_t extra_barrier_arrivals) {
    if (!ctx) return EDGEFM_ERR_INVALID_ARG;
    if (limit_ns < 1000u || extra_barrier_arrivals < 0 || extra_barrier_arrivals > 1)
        return fail(ctx, EDGEFM_ERR_INVALID_ARG, "limit_ns must be >= 1000 and extra_barrier_arrivals 0 or 1");
    DeviceGuard guard(ctx->device);
    CUDA_TRY(ctx, cudaDeviceSynchronize());
    ctx->mk.spin_limit = limit_ns;
    ctx->mk.barrier_extra = extra_barrier_arrivals;
    CUDA_TRY(ctx, record_graph(ctx));
    ctx->err.clear();
    return EDGEFM_OK;
}

edgefm_status edgefm_debug_set_prefill_wait(edgefm_ctx *ctx, uint32_t polls, int32_t extra_arrivals) {
    if (!ctx) return EDGEFM_ERR_INVALID_ARG;
    if (polls < 1024u || extra_arrivals < 0 || extra_arrivals > 1)
        return fail(ctx, EDGEFM_ERR_INVALID_ARG, "polls must be >= 1024 and extra_arrivals 0 or 1");
    ctx->pf_wait_limit = polls;
    ctx->pf_extra_arrivals = static_cast<uint32_t>(extra_arrivals);
    ctx->err.clear();
    return EDGEFM_OK;
}

edgefm_status edgefm_debug_prefill_plan(int32_t epilogue, int32_t M, int32_t N, int32_t K, int32_t num_sms, int32_t *out2) {
    if (!out2 || epilogue < 0 || epilogue > 2 || M < 1 || N < 1 || K < 1 || num_sms < 1) return EDGEFM_ERR_INVALID_ARG;
    int wide = 0, splits = 0;
    prefill_plan_contraction(epilogue, M, N, K, num_sms, &wide, &splits);
    out2[0] = wide;
    out2[1] = splits;
    return EDGEFM_OK;
}

edgefm_status edgefm_export_kv(edgefm_ctx *ctx, void *k_out, void *v_out, void *stream) {
    if (!ctx) return EDGEFM_ERR_INVALID_ARG;
    if (!k_out || !v_out) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "null output");
    if (ctx->kv_format != EDGEFM_KV_BF16) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "this context has a compressed cache: use edgefm_export_kv_int8");
    DeviceGuard guard(ctx->device);
    const edgefm_shape &sh = ctx->shape;
    const size_t bytes = static_cast<size_t>(sh.n_layers) * sh.n_kv_heads * ctx->max_context * sh.head_dim * 2;
    CUDA_TRY(ctx, cudaMemcpyAsync(k_out, ctx->k_cache, bytes, cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream)));
    CUDA_TRY(ctx, cudaMemcpyAsync(v_out, ctx->v_cache, bytes, cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream)));
    return EDGEFM_OK;
}

edgefm_status edgefm_export_kv_int8(edgefm_ctx *ctx, void *k_codes_out, void *v_codes_out, float *k_scales_out, float *v_scales_out,
                                    void *stream) {
    if (!ctx) return EDGEFM_ERR_INVALID_ARG;
    if (!k_codes_out || !v_codes_out || !k_scales_out || !v_scales_out) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "null output");
    if (ctx->kv_format != EDGEFM_KV_INT8) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "this context has the plain bf16 cache: use edgefm_export_kv");
    DeviceGuard guard(ctx->device);
    const edgefm_shape &sh = ctx->shape;
    const size_t rows = static_cast<size_t>(sh.n_layers) * sh.n_kv_heads * ctx->max_context;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CUDA_TRY(ctx, cudaMemcpyAsync(k_codes_out, ctx->k_cache, rows * sh.head_dim, cudaMemcpyDeviceToDevice, s));
    CUDA_TRY(ctx, cudaMemcpyAsync(v_codes_out, ctx->v_cache, rows * sh.head_dim, cudaMemcpyDeviceToDevice, s));
    CUDA_TRY(ctx, cudaMemcpyAsync(k_scales_out, ctx->k_scale, rows * sizeof(float), cudaMemcpyDeviceToDevice, s));
    CUDA_TRY(ctx, cudaMemcpyAsync(v_scales_out, ctx->v_scale, rows * sizeof(float), cudaMemcpyDeviceToDevice, s));
    return EDGEFM_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------------------
// edgefm_decode_step_static -- one decode step that allocates nothing.
//
// Some callers must not allocate device memory at all: a step issued from inside another framework's
// allocation-free region (a phase in which that framework has frozen its memory plan), from a process whose
// device memory is handed out entirely by a pool it does not own, or from a latency-critical thread where the
// implicit device synchronisation of cudaMalloc / cudaFree is not acceptable.  For them the work buffers of the
// persistent step kernel (residual stream, queries, attention partials, MLP activations, operator table, tile
// schedule, tensor maps, counters, device state: everything edgefm_create would allocate except the KV cache)
// live in a fixed array that is part of the loaded library image.  The caller owns the KV cache and the cache
// length and passes them in, so the call keeps no context.
//
// The array is EDGEFM_STATIC_SCRATCH_BYTES (4 MiB) on every GPU that loads the library, until exit.
namespace {

constexpr size_t EDGEFM_STATIC_SCRATCH_BYTES = 4u << 20;
static __device__ __align__(256) unsigned char g_static_scratch[EDGEFM_STATIC_SCRATCH_BYTES];

// In host code `g_static_scratch` is only a host-side stand-in for the symbol, not a device address.
// The device address is looked up once per device, with that device current.
constexpr int kMaxDevices = 64;
unsigned char *g_scratch_dev_ptr[kMaxDevices] = {};
StepState *g_static_state[kMaxDevices] = {};   // where the last static call on the device put its state word

struct ScratchCarver {
    unsigned char *base;
    size_t off = 0;
    template <typename T>
    T *take(size_t count) {
        T *p = reinterpret_cast<T *>(base + off);
        off = (off + count * sizeof(T) + 255) / 256 * 256;
        return p;
    }
};

}  // namespace

extern "C" edgefm_status edgefm_decode_step_static(const edgefm_shape *shape, const edgefm_weights *weights, void *k_cache,
                                                   void *v_cache, int32_t max_context, int32_t cur_len, int32_t token_id,
                                                   int32_t position, void *stream, float *logits_out,
                                                   int32_t *next_token_out) {
    if (!shape || !weights || !weights->layers || !k_cache || !v_cache)
        return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "null argument");
    const edgefm_shape &sh = *shape;
    constexpr int kMaxLayers = 96;
    if (sh.n_layers < 1 || sh.n_layers > kMaxLayers || sh.hidden < 8 || sh.hidden % 8 || sh.ffn < 8 || sh.ffn % 8 ||
        (sh.head_dim != 64 && sh.head_dim != 128) || sh.n_q_heads < 1 || sh.n_kv_heads < 1 || sh.n_q_heads % sh.n_kv_heads ||
        sh.n_q_heads / sh.n_kv_heads > 8 || sh.vocab < 1 || !(sh.rms_eps >= 0.f) || !(sh.rope_theta > 0.f))
        return fail(nullptr, EDGEFM_ERR_BAD_SHAPE, "unsupported model shape (same limits as edgefm_create; at most %d layers)", kMaxLayers);
    if (max_context < 1 || cur_len < 0 || cur_len >= max_context)
        return fail(nullptr, cur_len >= max_context ? EDGEFM_ERR_CONTEXT_FULL : EDGEFM_ERR_INVALID_ARG, "cur_len %d / max_context %d", cur_len, max_context);
    if (token_id < 0 || token_id >= sh.vocab || position < 0) return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "token or position out of range");
    if (!weights->embed || !weights->final_norm || !weights->lm_head) return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "null weight pointer");
    for (int l = 0; l < sh.n_layers; ++l) {
        const edgefm_layer_weights &w = weights->layers[l];
        if (!w.input_norm || !w.wqkv || !w.wo || !w.post_norm || !w.w_gate_up || !w.w_down || (sh.qkv_bias && !w.bqkv))
            return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "null weight pointer in layer %d", l);
        if (!aligned16(w.wqkv) || !aligned16(w.wo) || !aligned16(w.w_gate_up) || !aligned16(w.w_down) || !aligned16(w.input_norm) ||
            !aligned16(w.post_norm))
            return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "weight pointers must be 16-byte aligned (layer %d)", l);
    }
    if (!aligned16(weights->embed) || !aligned16(weights->lm_head) || !aligned16(weights->final_norm) || !aligned16(k_cache) || !aligned16(v_cache))
        return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "pointers must be 16-byte aligned");

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return fail(nullptr, EDGEFM_ERR_CUDA, "no usable CUDA device (this library has no CPU path)");
    }
    // The small copies below read host buffers of this call; recorded into a capture they would be replayed from memory
    // that is gone by then.  A capturing stream is therefore refused before anything is enqueued.
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    {
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(s, &cap) != cudaSuccess) {
            cudaGetLastError();
            return fail(nullptr, EDGEFM_ERR_CUDA, "cudaStreamIsCapturing failed");
        }
        if (cap != cudaStreamCaptureStatusNone)
            return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "edgefm_decode_step_static must not be called on a stream that is being captured");
    }
    const int H = sh.hidden, d = sh.head_dim, nq = sh.n_q_heads, nkv = sh.n_kv_heads, F = sh.ffn;
    int num_sms = 0, smem_optin = 0, coop = 0;
    CUDA_TRY(nullptr, cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev));
    CUDA_TRY(nullptr, cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    CUDA_TRY(nullptr, cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
    if (!coop) return fail(nullptr, EDGEFM_ERR_CUDA, "device lacks cooperative launch");

    // ---- set-up, once per device: the device address of the scratch array (never the host-side symbol) ----
    if (!g_scratch_dev_ptr[dev]) {
        unsigned char *ptr = nullptr;
        CUDA_TRY(nullptr, cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_static_scratch));
        if (!ptr) return fail(nullptr, EDGEFM_ERR_CUDA, "cudaGetSymbolAddress returned a null scratch address");
        g_scratch_dev_ptr[dev] = ptr;
    }
    // ---- the same plan edgefm_create makes, in host memory -------------------------------------------------
    StepPlan pl;
    StepSchedule ss;
    {
        cudaError_t ce = cudaSuccess;
        if (const char *why = plan_step_and_schedule(sh, max_context, num_sms, smem_optin, &pl, &ss, &ce))
            return fail(nullptr, ce != cudaSuccess ? EDGEFM_ERR_CUDA : EDGEFM_ERR_BAD_SHAPE, "%s", why);
    }
    const int grid = pl.grid, max_chunks = pl.max_chunks, n_ops = pl.n_ops;

    // carve the scratch array; reject shapes that need more than it holds
    ScratchCarver sc{g_scratch_dev_ptr[dev]};
    unsigned char *d_maps = sc.take<unsigned char>(static_cast<size_t>(n_ops) * MK_MAX_VARIANTS * sizeof(CUtensorMap));
    MkOp *d_ops = sc.take<MkOp>(n_ops);
    const uint16_t **d_op_w = sc.take<const uint16_t *>(n_ops);
    uint2 *d_tiles = sc.take<uint2>(ss.tiles.size());
    int *d_cta_tab = sc.take<int>(ss.cta_tab.size());
    MkCombine *d_combines = sc.take<MkCombine>(ss.combines.size() + 1);
    float *x = sc.take<float>(H);
    float *q = sc.take<float>(static_cast<size_t>(nq) * d);
    float *attn = sc.take<float>(static_cast<size_t>(nq) * d);
    float *act = sc.take<float>(static_cast<size_t>(MK_X_SPLITS) * ((F + MK_TILE_COLS - 1) / MK_TILE_COLS * MK_TILE_COLS) / 2);
    double *inv_freq = sc.take<double>(d / 2);
    float *part_m = sc.take<float>(static_cast<size_t>(nq) * max_chunks);
    float *part_l = sc.take<float>(static_cast<size_t>(nq) * max_chunks);
    float *part_o = sc.take<float>(static_cast<size_t>(nq) * max_chunks * d);
    float *lm_val = sc.take<float>(grid);
    int *lm_idx = sc.take<int>(grid);
    unsigned *counters = sc.take<unsigned>(static_cast<size_t>(nq) + nkv + 2 + 64 + nq + 2 * nkv);   // tickets, the grid barrier counter, the per-head counters
    StepState *state = sc.take<StepState>(1);
    StepRequest *req = sc.take<StepRequest>(1);
    if (sc.off > EDGEFM_STATIC_SCRATCH_BYTES)
        return fail(nullptr, EDGEFM_ERR_BAD_SHAPE, "this shape needs %zu bytes of work buffers; the static scratch holds %zu", sc.off,
                    EDGEFM_STATIC_SCRATCH_BYTES);
    unsigned *tickets = counters;
    unsigned *grid_bar = counters + nq + nkv + 2 + 32;

    std::vector<MkOp> ops(static_cast<size_t>(n_ops));
    std::vector<const uint16_t *> op_w(static_cast<size_t>(n_ops));
    fill_ops(sh, weights->layers, weights->final_norm, weights->lm_head, x, attn, q, act, ops.data(), op_w.data());
    std::vector<CUtensorMap> maps(static_cast<size_t>(n_ops) * MK_MAX_VARIANTS);
    if (const char *why = encode_maps(ss, sh, weights->layers, weights->lm_head, sh.vocab, maps.data()))
        return fail(nullptr, EDGEFM_ERR_CUDA, "%s", why);
    CUDA_TRY(nullptr, allow_max_dynamic_smem(pl.kernel, smem_optin));

    MkParams m{};
    fill_shape_params(&m, sh, max_context, pl, ss);
    m.ops = d_ops; m.op_weights = d_op_w; m.maps = d_maps; m.tiles = d_tiles; m.cta_tab = d_cta_tab; m.combines = d_combines;
    m.k_cache = static_cast<uint16_t *>(k_cache); m.v_cache = static_cast<uint16_t *>(v_cache);
    m.embed = (const uint16_t *)weights->embed; m.inv_freq = inv_freq; m.x = x; m.q = q; m.attn = attn;
    m.part_m = part_m; m.part_l = part_l; m.part_o = part_o;
    m.head_ready = counters + nq + nkv + 2 + 64; m.head_flags = pl.long_ctx ? 0 : MK_HEAD_FLAGS;
    m.tickets = tickets; m.barrier = grid_bar; m.lm_part_val = lm_val; m.lm_part_idx = lm_idx; m.state = state; m.req = req;
    m.prof = nullptr; m.prof_stride = 0;
    m.map_fence = 2;   // every call rewrites all tensor maps in the shared scratch

    // ---- stream-ordered set-up of the shared scratch: it still holds the previous call's contents ----------
    double inv[64];
    for (int i = 0; i < d / 2; ++i) inv[i] = std::pow(static_cast<double>(sh.rope_theta), -2.0 * i / d);
    StepState st{};
    st.cur_len = cur_len; st.next_position = position;
    StepRequest rq{token_id, position, logits_out, next_token_out};
    // counters (attention tickets, lm_head ticket, grid barrier) must start at zero
    CUDA_TRY(nullptr, cudaMemsetAsync(counters, 0, (static_cast<size_t>(nq) + nkv + 2 + 64 + nq + 2 * nkv) * sizeof(unsigned), s));
    // pageable copies: the runtime stages the bytes before returning, so the sources may be freed after the call
    CUDA_TRY(nullptr, cudaMemcpyAsync(d_ops, ops.data(), ops.size() * sizeof(MkOp), cudaMemcpyHostToDevice, s));
    CUDA_TRY(nullptr, cudaMemcpyAsync(d_op_w, op_w.data(), op_w.size() * sizeof(op_w[0]), cudaMemcpyHostToDevice, s));
    CUDA_TRY(nullptr, cudaMemcpyAsync(d_maps, maps.data(), maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice, s));
    CUDA_TRY(nullptr, cudaMemcpyAsync(d_tiles, ss.tiles.data(), ss.tiles.size() * sizeof(uint2), cudaMemcpyHostToDevice, s));
    CUDA_TRY(nullptr, cudaMemcpyAsync(d_cta_tab, ss.cta_tab.data(), ss.cta_tab.size() * sizeof(int), cudaMemcpyHostToDevice, s));
    if (!ss.combines.empty())
        CUDA_TRY(nullptr, cudaMemcpyAsync(d_combines, ss.combines.data(), ss.combines.size() * sizeof(MkCombine), cudaMemcpyHostToDevice, s));
    CUDA_TRY(nullptr, cudaMemcpyAsync(inv_freq, inv, static_cast<size_t>(d / 2) * sizeof(double), cudaMemcpyHostToDevice, s));
    CUDA_TRY(nullptr, cudaMemcpyAsync(state, &st, sizeof st, cudaMemcpyHostToDevice, s));
    CUDA_TRY(nullptr, cudaMemcpyAsync(req, &rq, sizeof rq, cudaMemcpyHostToDevice, s));
    CUDA_TRY(nullptr, launch_step(pl.kernel, pl, m, s));
    g_static_state[dev] = state;
    g_create_error.clear();
    return EDGEFM_OK;
}

extern "C" edgefm_status edgefm_sync_status(edgefm_ctx *ctx, void *stream) {
    // ctx == NULL: the status word the last edgefm_decode_step_static on the current device left in the static scratch
    int dev = -1;
    StepState *where = nullptr;
    if (ctx) {
        where = ctx->state;
    } else {
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices || !g_static_state[dev]) {
            cudaGetLastError();
            return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "no static step has run on the current device");
        }
        where = g_static_state[dev];
    }
    DeviceGuard guard(ctx ? ctx->device : dev);
    CUDA_TRY(ctx, cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    StepState st;
    CUDA_TRY(ctx, cudaMemcpy(&st, where, sizeof st, cudaMemcpyDeviceToHost));
    if (ctx && ctx->pf.chunk) {
        int pe = 0;
        CUDA_TRY(ctx, cudaMemcpy(&pe, ctx->pf.error, sizeof pe, cudaMemcpyDeviceToHost));
        if (pe != 0) return fail(ctx, EDGEFM_ERR_TIMEOUT, "a bounded wait of a prefill contraction expired; the context must be destroyed");
    }
    if (st.status != 0)
        return fail(ctx, EDGEFM_ERR_TIMEOUT, "device status %d (6 = a bounded wait expired, 100+ = self-check code) operands %d %d; "
                    "the context must be destroyed", st.status, st.pad[0], st.pad[1]);
    return EDGEFM_OK;
}

// Host-only diagnostics: the tile schedule of one operator, in the form the kernel reads, for checking the planner
// without a GPU.  tiles_out receives the tiles CTA by CTA, warp by warp (tiles_per_warp [n_ctas * n_warps] counts them);
// combines_out four words per entry (combines_per_cta [n_ctas]); variant_rows [4] the box heights of the tensor maps.
extern "C" edgefm_status edgefm_debug_plan_operator(int32_t kind, int32_t units, int32_t K, int32_t head_half, int32_t op_index, int32_t n_ctas,
                                                    int32_t n_warps, int32_t slot_rows, uint64_t *tiles_out, int64_t tiles_cap,
                                                    int32_t *tiles_per_warp, uint32_t *combines_out, int64_t combines_cap,
                                                    int32_t *combines_per_cta, int32_t *variant_rows, int64_t *n_tiles, int64_t *n_combines) {
    if (!tiles_per_warp || !combines_per_cta || !variant_rows || !n_tiles || !n_combines || n_ctas < 1 || n_warps < 1)
        return fail(nullptr, EDGEFM_ERR_INVALID_ARG, "bad argument");
    OpShape os{kind, units, K, op_paired(kind) ? 2 * units : units, head_half};
    OpSchedule S;
    if (const char *why = plan_op(os, op_index, n_ctas, n_warps, slot_rows, &S)) return fail(nullptr, EDGEFM_ERR_BAD_SHAPE, "%s", why);
    int64_t nt = 0, nc = 0;
    for (int c = 0; c < n_ctas; ++c) {
        for (int w = 0; w < n_warps; ++w) {
            tiles_per_warp[c * n_warps + w] = static_cast<int32_t>(S.tiles[c][w].size());
            for (const uint2 &d : S.tiles[c][w]) {
                if (tiles_out && nt < tiles_cap) tiles_out[nt] = static_cast<uint64_t>(d.x) | static_cast<uint64_t>(d.y) << 32;
                ++nt;
            }
        }
        combines_per_cta[c] = static_cast<int32_t>(S.combines[c].size());
        for (const MkCombine &e : S.combines[c]) {
            if (combines_out && nc < combines_cap) { combines_out[4 * nc] = e.x; combines_out[4 * nc + 1] = e.y; combines_out[4 * nc + 2] = e.z; combines_out[4 * nc + 3] = e.w; }
            ++nc;
        }
    }
    for (int v = 0; v < MK_MAX_VARIANTS; ++v) variant_rows[v] = v < S.n_variants ? S.variant_rows[v] : 0;
    *n_tiles = nt; *n_combines = nc;
    return EDGEFM_OK;
}
