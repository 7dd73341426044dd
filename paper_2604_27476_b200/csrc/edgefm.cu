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

#include "attention.cuh"
#include "common.cuh"
#include "gemv.cuh"
#include "megakernel_types.cuh"
// the persistent kernel is built twice: 12 warps per CTA (short contexts, here) and 8 warps per CTA (long contexts,
// in the megakernel_long_*.cu translation units)
#define MK_NS mk_short
#define MK_NW_VALUE MK_NW_SHORT
#include "megakernel.cuh"
#undef MK_NS
#undef MK_NW_VALUE

namespace edgefm {

// ---- small kernels -------------------------------------------------------------------------------

// First node of the step graph: resolve the request into (token, position), gather the embedding
// row into the fp32 residual stream and build the cos/sin table of the rotary position.  The
// angle is evaluated in fp64 (position up to ~33k times the fastest frequency needs more than
// fp32's 24 bits to stay accurate), rounded to fp32 once.
__global__ void __launch_bounds__(256) step_begin_kernel(const StepRequest *req, StepState *st, const uint16_t *embed,
                                                         const double *inv_freq, float *x, float *rope_cs, int H,
                                                         int half_d) {
    pdl_launch_dependents();
    pdl_wait();
    const int rt = req->token, rp = req->position;
    const int token = rt >= 0 ? rt : st->next_token;
    const int pos = rp >= 0 ? rp : st->next_position;
    __syncthreads();  // every thread has read the previous state before it is overwritten
    if (threadIdx.x == 0) { st->token = token; st->position = pos; }
    const uint16_t *row = embed + static_cast<size_t>(token) * H;
    for (int i = threadIdx.x; i < H; i += blockDim.x) x[i] = bf16_bits_to_f32(row[i]);
    for (int i = threadIdx.x; i < half_d; i += blockDim.x) {
        double s, c;
        sincos(static_cast<double>(pos) * inv_freq[i], &s, &c);
        rope_cs[i] = static_cast<float>(c);
        rope_cs[half_d + i] = static_cast<float>(s);
    }
}

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

// ---- launch helpers ------------------------------------------------------------------------------

template <typename Kern, typename... Args>
cudaError_t launch(Kern kern, dim3 grid, dim3 block, size_t smem, cudaStream_t s, bool pdl, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

using GemvKernel = void (*)(const GemvArgs);
using AttnKernel = void (*)(const AttnArgs);

struct GemvPlan {
    GemvKernel kern = nullptr;
    int threads = 0, tile_rows = 0, wk = 0;
    int grid = 0;
    size_t smem = 0;
};

struct AttnPlan {
    AttnKernel kern = nullptr;
    int threads = 0;
    size_t smem = 0;
    int max_chunks = 0, min_chunk = 0;
};

template <int PRO, int EPI, int RW, int WR, int WK, int U>
GemvPlan make_gemv_plan(int units, int K, int num_sms, cudaError_t *err) {
    GemvPlan p;
    p.kern = gemv_kernel<PRO, EPI, RW, WR, WK, U>;
    p.threads = WR * WK * 32;
    p.tile_rows = RW * WR;
    p.wk = WK;
    p.smem = (static_cast<size_t>(K) + (WK + 1) * RW * WR) * sizeof(float);
    *err = cudaFuncSetAttribute(p.kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(p.smem));
    if (*err != cudaSuccess) return p;
    int per_sm = 0;
    *err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, p.kern, p.threads, p.smem);
    if (*err != cudaSuccess) return p;
    if (per_sm < 1) per_sm = 1;
    const int paired = (EPI == EPI_QKV || EPI == EPI_SWIGLU) ? 2 : 1;
    const int per_tile = p.tile_rows / paired;
    const int ntiles = (units + per_tile - 1) / per_tile;
    const int cap = num_sms * per_sm;
    p.grid = ntiles < cap ? ntiles : cap;
    if (p.grid < 1) p.grid = 1;
    return p;
}

template <int D, int G, int LPP, int NW>
AttnPlan make_attn_plan_t(cudaError_t *err) {
    AttnPlan p;
    p.kern = attn_kernel<D, G, LPP, NW>;
    p.threads = NW * 32;
    p.smem = AttnSmem<D, G, LPP, NW>::TOTAL;
    *err = cudaFuncSetAttribute(p.kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(p.smem));
    return p;
}

template <int D, int LPP, int NW>
AttnPlan make_attn_plan_g(int G, cudaError_t *err) {
    switch (G) {
        case 1: return make_attn_plan_t<D, 1, LPP, NW>(err);
        case 2: return make_attn_plan_t<D, 2, LPP, NW>(err);
        case 3: return make_attn_plan_t<D, 3, LPP, NW>(err);
        case 4: return make_attn_plan_t<D, 4, LPP, NW>(err);
        case 5: return make_attn_plan_t<D, 5, LPP, NW>(err);
        case 6: return make_attn_plan_t<D, 6, LPP, NW>(err);
        case 7: return make_attn_plan_t<D, 7, LPP, NW>(err);
        case 8: return make_attn_plan_t<D, 8, LPP, NW>(err);
    }
    *err = cudaErrorInvalidValue;
    return AttnPlan();
}

// long_ctx = false: the variant without the grouped (one CTA per GQA group) attention code, for contexts that
// never need it.
template <int D>
MegaKernel mega_kernel_g(int G, bool long_ctx) {
    if (!long_ctx) return mk_short::decode_megakernel<D, 1, false>;   // G is only used by the grouped attention
    if (D == 64) return G <= 4 ? mega_kernel_long_d64_lo(G) : mega_kernel_long_d64_hi(G);
    return G <= 4 ? mega_kernel_long_d128_lo(G) : mega_kernel_long_d128_hi(G);
}
// Tile geometry of one weight-streaming operator.
//  * long operators (many rows per CTA): whole rows, as many per tile (rw rows or row pairs) as fit the
//    slot budget while every warp keeps about two tiles;
//  * short operators, and rows longer than a slot: one row (pair) per item, cut into `ksplit` K slices
//    (a power of two dividing the row) that go to different warps, so that all warps of a CTA share the
//    latency of the operator; their partial sums meet in shared memory.
inline void choose_tile(int K, bool paired, int pair_align, int units, int ncta, int nw, int budget_bytes, int *rw, int *ksplit, int *split) {
    const int kc = K / 8;
    const int mult = paired ? 2 : 1;
    const long long row_bytes = static_cast<long long>(K) * 2 * mult;
    const double per_cta = static_cast<double>(units) / ncta;
    *rw = 1; *ksplit = 1; *split = 0;
    if (row_bytes <= budget_bytes && per_cta >= 2.0 * nw) {
        int r = paired ? 4 : 8;
        while (r > 1 && (row_bytes * r > budget_bytes || (paired && pair_align % r != 0) || per_cta / r < 2.0 * nw)) r >>= 1;
        *rw = r;
        return;
    }
    int s = 1;
    auto can_double = [&](int min_kcs) { return kc % (2 * s) == 0 && kc / (2 * s) >= min_kcs && 2 * s <= 16; };
    while (row_bytes / s > budget_bytes && kc % (2 * s) == 0) s *= 2;           // must fit a slot
    // at least one tile per warp, as long as a tile keeps 3 KB: below that the fixed cost of a tile (wait, copy issue,
    // reduction) outweighs the idle warps (measured on the O projection of the 1.5B shape: 10 whole-row tiles on 12 warps
    // beat 21 half-row tiles)
    while (per_cta * s < nw && can_double(64) && row_bytes / (2 * s) >= 3072) s *= 2;
    while (per_cta * s < 2.0 * nw && can_double(256)) s *= 2;                // two per warp while slices stay long
    *ksplit = s;
    *split = s > 1 ? 1 : 0;
}


// Bytes of one tile of an operator.
inline int phase_tile_bytes(const MkPhase &ph) {
    const bool paired = ph.kind == PH_QKV || ph.kind == PH_SWIGLU;
    return ph.rw * (paired ? 2 : 1) * ph.kcs * 16;
}

// ---- launch plan of the persistent step kernel (shared by edgefm_create and edgefm_decode_step_static) ----------------
struct StepPlan {
    MegaKernel kernel = nullptr;
    bool long_ctx = false;
    int nw = 0;            // warps per CTA of the chosen kernel build
    int grid = 0;          // CTAs (one per SM)
    int max_chunks = 0;    // row stride of the attention partial buffers
    int n_phases = 0;      // 4 per layer + lm_head
    int budget = 0;        // upper bound of one weight tile, bytes
    size_t xbuf = 0, sched = 0, avail = 0;   // shared memory: activation / attention scratch, schedule, what is left for the rings
    int ring_bytes = 0, slot_bytes = 0;      // filled by plan_phases
    size_t dyn_smem = 0;
};

// Kernel variant and shared-memory split for a model shape.  Returns null, or why the shape does not fit.
inline const char *plan_step(const edgefm_shape &sh, int max_context, int num_sms, int smem_optin, StepPlan *pl, cudaError_t *cuda_err) {
    const int H = sh.hidden, d = sh.head_dim, nq = sh.n_q_heads, nkv = sh.n_kv_heads, F = sh.ffn, G = nq / nkv;
    *cuda_err = cudaSuccess;
    pl->long_ctx = max_context > 8192 || static_cast<long long>(nq) * MK_ATT_SPLIT_MAXC * 2 > MK_PARTIAL_FLOATS;
    pl->kernel = d == 64 ? mega_kernel_g<64>(G, pl->long_ctx) : mega_kernel_g<128>(G, pl->long_ctx);
    pl->nw = pl->long_ctx ? MK_NW_LONG : MK_NW_SHORT;
    pl->grid = num_sms;
    pl->max_chunks = pl->grid / nkv > 0 ? pl->grid / nkv : 1;
    pl->n_phases = 4 * sh.n_layers + 1;
    const int NW = pl->nw, ATT_MW = (NW + 1) / 2;
    int max_k = H;
    if (nq * d > max_k) max_k = nq * d;
    if (F > max_k) max_k = F;
    // attention scratch: queries, probabilities, warp merge area, chunk statistics
    const size_t att_bytes = (static_cast<size_t>(G) * d + NW * (G * MK_ATT_TILE > 32 / MK_ATT_LPP_SPLIT ? G * MK_ATT_TILE : 32 / MK_ATT_LPP_SPLIT) +
                              2 * ATT_MW * G + static_cast<size_t>(ATT_MW) * G * d + 2 * static_cast<size_t>(G) * pl->max_chunks) * 4;
    size_t xbuf = static_cast<size_t>(max_k) * 4;
    if (att_bytes > xbuf) xbuf = att_bytes;
    pl->xbuf = (xbuf + 255) / 256 * 256;
    cudaFuncAttributes fa{};
    *cuda_err = cudaFuncGetAttributes(&fa, pl->kernel);
    if (*cuda_err != cudaSuccess) return "cudaFuncGetAttributes";
    const size_t static_smem = fa.sharedSizeBytes + 1024;   // the kernel's static shared memory (mbarriers, tables, scratch) + margin
    pl->sched = (static_cast<size_t>(pl->n_phases) * (sizeof(MkPhase) + sizeof(int2)) + 127) / 128 * 128;
    if (pl->xbuf + pl->sched + static_smem + static_cast<size_t>(NW) * 1024 > static_cast<size_t>(smem_optin))
        return "model shape does not fit the shared-memory plan";
    pl->avail = smem_optin - static_smem - pl->xbuf - pl->sched;
    pl->budget = 8192;
    if (const char *tb = getenv("EDGEFM_TILE_BYTES")) { const int v = atoi(tb); if (v >= 1024 && v <= 65536) pl->budget = v; }
    const int fit1 = static_cast<int>(pl->avail / NW / 128 * 128);   // a tile must fit a warp's ring
    if (pl->budget > fit1) pl->budget = fit1;
    return nullptr;
}

// Descriptor of one weight-streaming operator (tile shape chosen for its aspect ratio).  False: it does not fit the plan.
inline bool plan_phase(const StepPlan &pl, int head_dim, int kind, const void *W, int K, int units, const void *bias, const void *norm,
                       const float *x_src, float *out, int layer, MkPhase *ph_out) {
    MkPhase ph{};
    const bool paired = kind == PH_QKV || kind == PH_SWIGLU;
    choose_tile(K, paired, kind == PH_QKV ? head_dim / 2 : 4, units, pl.grid, pl.nw, pl.budget, &ph.rw, &ph.ksplit, &ph.split);
    ph.s_shift = 0;
    while ((1 << ph.s_shift) < ph.ksplit) ++ph.s_shift;
    ph.W = static_cast<const uint16_t *>(W); ph.bias = static_cast<const uint16_t *>(bias); ph.norm_w = static_cast<const uint16_t *>(norm);
    ph.x_src = x_src; ph.out = out; ph.K = K; ph.kind = kind; ph.kcs = K / 8 / ph.ksplit;
    ph.units_total = units; ph.items_total = (units + ph.rw - 1) / ph.rw; ph.layer = layer;
    *ph_out = ph;
    if (phase_tile_bytes(ph) > pl.budget) return false;
    if (ph.split) {   // partial sums of one CTA's share must fit the shared-memory scratch
        const long long per_cta = (ph.items_total + pl.grid - 1) / pl.grid + 1;
        if (per_cta * ph.ksplit * (paired ? 2 : 1) > MK_PARTIAL_FLOATS) return false;
    }
    return true;
}

// All operators of the step, in execution order, wired to the work buffers; then the ring geometry.
// Returns null, or why the shape does not fit.
inline const char *plan_phases(StepPlan *pl, const edgefm_shape &sh, const edgefm_layer_weights *layers, const void *final_norm,
                               const void *lm_head, float *x, float *q, float *attn, float *act, MkPhase *out) {
    const int H = sh.hidden, d = sh.head_dim, nq = sh.n_q_heads, nkv = sh.n_kv_heads, F = sh.ffn;
    const int R = (nq + 2 * nkv) * d;
    bool fits = true;
    int n = 0;
    for (int l = 0; l < sh.n_layers; ++l) {
        const edgefm_layer_weights &w = layers[l];
        fits &= plan_phase(*pl, d, PH_QKV, w.wqkv, H, R / 2, sh.qkv_bias ? w.bqkv : nullptr, w.input_norm, l == 0 ? nullptr : x, q, l, &out[n++]);
        fits &= plan_phase(*pl, d, PH_RESID, w.wo, nq * d, H, nullptr, nullptr, attn, x, l, &out[n++]);
        out[n - 1].flags |= PHF_X_BULK;      // the attention phase stores its output in the staged layout
        fits &= plan_phase(*pl, d, PH_SWIGLU, w.w_gate_up, H, F, nullptr, w.post_norm, x, act, l, &out[n++]);
        out[n - 1].flags |= PHF_OUT_SPLIT;   // the MLP activations go to memory in the layout the down projection stages
        fits &= plan_phase(*pl, d, PH_RESID, w.w_down, F, H, nullptr, nullptr, act, x, l, &out[n++]);
        out[n - 1].flags |= PHF_X_BULK;
    }
    fits &= plan_phase(*pl, d, PH_LMHEAD, lm_head, H, sh.vocab, nullptr, final_norm, x, nullptr, sh.n_layers, &out[n++]);
    if (!fits) return "model shape does not fit the tile plan";
    int max_tile = 0;
    for (int i = 0; i < n; ++i) max_tile = std::max(max_tile, phase_tile_bytes(out[i]));
    pl->slot_bytes = (max_tile + 127) / 128 * 128;
    pl->ring_bytes = static_cast<int>(pl->avail / pl->nw / 128 * 128);
    if (pl->slot_bytes > pl->ring_bytes || pl->ring_bytes > (0xffff << 4)) return "weight rows do not fit the shared-memory ring";
    pl->dyn_smem = pl->xbuf + pl->sched + static_cast<size_t>(pl->ring_bytes) * pl->nw;
    return nullptr;
}

// Shape-derived kernel parameters common to both entry points (buffers, cache and schedule pointers are the caller's).
inline void fill_shape_params(MkParams *m, const edgefm_shape &sh, int max_context, const StepPlan &pl) {
    m->nph = pl.n_phases; m->n_layers = sh.n_layers; m->H = sh.hidden; m->nq = sh.n_q_heads; m->nkv = sh.n_kv_heads;
    m->d = sh.head_dim; m->F = sh.ffn; m->V = sh.vocab;
    m->half_shift = sh.head_dim == 64 ? 5 : 6;
    m->eps = sh.rms_eps; m->scale = static_cast<float>(1.0 / std::sqrt(static_cast<double>(sh.head_dim)));
    m->max_context = max_context; m->max_chunks = pl.max_chunks;
    m->att_chunk_shared = 256; m->att_chunk_split = 64; m->att_split_max_n = 8192;
    m->ring_bytes = pl.ring_bytes; m->slot_bytes = pl.slot_bytes; m->xbuf_bytes = static_cast<int>(pl.xbuf);
    m->sched_bytes = static_cast<int>(pl.sched);
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
    bool use_pdl = true;
    std::vector<edgefm_layer_weights> layers;
    const void *embed = nullptr, *final_norm = nullptr, *lm_head = nullptr;

    // owned device memory
    uint16_t *k_cache = nullptr, *v_cache = nullptr;  // [L][nkv][max_context][d]
    float *x = nullptr;          // residual stream [H]
    float *q = nullptr;          // rotated queries [nq*d]
    float *attn = nullptr;       // attention output [nq*d]
    float *act = nullptr;        // SwiGLU output [F]
    float *rope_cs = nullptr;    // [d]
    double *inv_freq = nullptr;  // [d/2]
    float *part_m = nullptr, *part_l = nullptr, *part_o = nullptr;
    float *lm_part_val = nullptr;
    int *lm_part_idx = nullptr;
    unsigned *tickets = nullptr;  // [nkv] attention + [1] lm_head
    StepState *state = nullptr;
    StepRequest *req = nullptr;

    GemvPlan p_qkv, p_o, p_gu, p_down, p_lm;
    AttnPlan p_attn;

    // persistent-kernel path
    bool use_mega = true;
    MegaKernel mega = nullptr;
    MkPhase *d_phases = nullptr;
    unsigned *grid_bar = nullptr;
    unsigned long long *prof = nullptr;
    int prof_stride = 0;
    MkParams mk{};
    size_t mega_smem = 0;
    int mega_threads = 0;
    int mega_grid = 0;
    // vocabulary pruning: the full-vocabulary lm_head descriptor, the tile budget it was planned with, the
    // gathered rows of the current subset and their token ids
    MkPhase lm_phase_full{};
    int tile_budget = 0;
    int *vocab_ids = nullptr;       // [vocab]
    uint16_t *sub_lm = nullptr;     // [vocab_subset][hidden] or null
    int vocab_subset = 0;           // 0 = full vocabulary

    cudaStream_t build_stream = nullptr;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    int launches_per_step = 0;

    // host mirrors
    int cur_len = 0;
    bool have_token = false;
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
    void *bufs[] = {c->k_cache, c->v_cache, c->x, c->q, c->attn, c->act, c->rope_cs, c->inv_freq, c->part_m, c->part_l,
                    c->part_o, c->lm_part_val, c->lm_part_idx, c->tickets, c->state, c->req, c->d_phases, c->grid_bar, c->prof,
                    c->vocab_ids, c->sub_lm};
    for (void *b : bufs) if (b) cudaFree(b);
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Enqueue the kernels of one decode step (used once, under stream capture).
cudaError_t enqueue_step(edgefm_ctx *c, cudaStream_t s, int *n_launches) {
    const edgefm_shape &sh = c->shape;
    const int H = sh.hidden, d = sh.head_dim, nq = sh.n_q_heads, nkv = sh.n_kv_heads, F = sh.ffn;
    const int R = (nq + 2 * nkv) * d;
    const bool pdl = c->use_pdl;
    int n = 0;
    cudaError_t e;
    if (c->use_mega) {
        // one cooperative launch: all CTAs are co-resident, which the grid barriers rely on
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(c->mega_grid);
        cfg.blockDim = dim3(c->mega_threads);
        cfg.dynamicSmemBytes = c->mega_smem;
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, c->mega, c->mk);
        if (e != cudaSuccess) return e;
        *n_launches = 1;
        return cudaSuccess;
    }
    // The first node follows the previous graph launch by ordinary stream order.
    e = launch(step_begin_kernel, dim3(1), dim3(256), 0, s, false, (const StepRequest *)c->req, c->state,
               (const uint16_t *)c->embed, (const double *)c->inv_freq, c->x, c->rope_cs, H, d / 2);
    if (e != cudaSuccess) return e;
    ++n;
    const size_t kv_layer = static_cast<size_t>(nkv) * c->max_context * d;
    for (int l = 0; l < sh.n_layers; ++l) {
        const edgefm_layer_weights &w = c->layers[l];
        GemvArgs a{};
        a.W = (const uint16_t *)w.wqkv; a.rows = R; a.K = H; a.x_in = c->x; a.norm_w = (const uint16_t *)w.input_norm;
        a.eps = sh.rms_eps; a.bias = sh.qkv_bias ? (const uint16_t *)w.bqkv : nullptr; a.out = c->q;
        a.k_cache = c->k_cache + l * kv_layer; a.v_cache = c->v_cache + l * kv_layer; a.max_context = c->max_context;
        a.nq = nq; a.nkv = nkv; a.d = d; a.rope_cs = c->rope_cs; a.state = c->state;
        e = launch(c->p_qkv.kern, dim3(c->p_qkv.grid), dim3(c->p_qkv.threads), c->p_qkv.smem, s, pdl, a);
        if (e != cudaSuccess) return e;
        ++n;

        AttnArgs t{};
        t.q = c->q; t.k_cache = a.k_cache; t.v_cache = a.v_cache; t.out = c->attn; t.part_m = c->part_m;
        t.part_l = c->part_l; t.part_o = c->part_o; t.tickets = c->tickets; t.state = c->state;
        t.max_context = c->max_context; t.max_chunks = c->p_attn.max_chunks; t.min_chunk = c->p_attn.min_chunk;
        t.scale = static_cast<float>(1.0 / std::sqrt(static_cast<double>(d)));
        e = launch(c->p_attn.kern, dim3(c->p_attn.max_chunks, nkv), dim3(c->p_attn.threads), c->p_attn.smem, s, pdl, t);
        if (e != cudaSuccess) return e;
        ++n;

        GemvArgs o{};
        o.W = (const uint16_t *)w.wo; o.rows = H; o.K = nq * d; o.x_in = c->attn; o.out = c->x;
        e = launch(c->p_o.kern, dim3(c->p_o.grid), dim3(c->p_o.threads), c->p_o.smem, s, pdl, o);
        if (e != cudaSuccess) return e;
        ++n;

        GemvArgs gu{};
        gu.W = (const uint16_t *)w.w_gate_up; gu.rows = 2 * F; gu.K = H; gu.x_in = c->x;
        gu.norm_w = (const uint16_t *)w.post_norm; gu.eps = sh.rms_eps; gu.out = c->act; gu.F = F;
        e = launch(c->p_gu.kern, dim3(c->p_gu.grid), dim3(c->p_gu.threads), c->p_gu.smem, s, pdl, gu);
        if (e != cudaSuccess) return e;
        ++n;

        GemvArgs dn{};
        dn.W = (const uint16_t *)w.w_down; dn.rows = H; dn.K = F; dn.x_in = c->act; dn.out = c->x;
        e = launch(c->p_down.kern, dim3(c->p_down.grid), dim3(c->p_down.threads), c->p_down.smem, s, pdl, dn);
        if (e != cudaSuccess) return e;
        ++n;
    }
    GemvArgs lm{};
    lm.W = (const uint16_t *)c->lm_head; lm.rows = sh.vocab; lm.K = H; lm.x_in = c->x;
    lm.norm_w = (const uint16_t *)c->final_norm; lm.eps = sh.rms_eps; lm.state = c->state; lm.req = c->req;
    lm.part_val = c->lm_part_val; lm.part_idx = c->lm_part_idx; lm.ticket = c->tickets + nkv;
    e = launch(c->p_lm.kern, dim3(c->p_lm.grid), dim3(c->p_lm.threads), c->p_lm.smem, s, pdl, lm);
    if (e != cudaSuccess) return e;
    ++n;
    *n_launches = n;
    return cudaSuccess;
}

}  // namespace

extern "C" {

const char *edgefm_version(void) { return "edgefm-b200 0.1 (sm_100a)"; }

const char *edgefm_last_error(const edgefm_ctx *ctx) { return ctx ? ctx->err.c_str() : g_create_error.c_str(); }

edgefm_status edgefm_create(const edgefm_shape *shape, const edgefm_weights *weights, int32_t max_context,
                            edgefm_ctx **out) {
    if (out) *out = nullptr;
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
    c->max_context = max_context;
    c->device = dev;
    c->num_sms = prop.multiProcessorCount;
    const char *env = getenv("EDGEFM_PDL");
    c->use_pdl = !(env && env[0] == '0');
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
    const int R = (nq + 2 * nkv) * d;
    cudaError_t pe = cudaSuccess;

    // kernel variants per operator (tile rows x split-K chosen for the operator's aspect ratio)
    c->p_qkv = make_gemv_plan<PRO_RMSNORM, EPI_QKV, 2, 8, 1, 4>(R / 2, H, c->num_sms, &pe);
    CREATE_TRY(pe);
    c->p_o = make_gemv_plan<PRO_PLAIN, EPI_RESIDUAL, 1, 8, 1, 6>(H, nq * d, c->num_sms, &pe);
    CREATE_TRY(pe);
    c->p_gu = make_gemv_plan<PRO_RMSNORM, EPI_SWIGLU, 2, 8, 1, 4>(F, H, c->num_sms, &pe);
    CREATE_TRY(pe);
    c->p_down = make_gemv_plan<PRO_PLAIN, EPI_RESIDUAL, 4, 1, 8, 2>(H, F, c->num_sms, &pe);
    CREATE_TRY(pe);
    c->p_lm = make_gemv_plan<PRO_RMSNORM, EPI_LMHEAD, 2, 8, 1, 4>(sh.vocab, H, c->num_sms, &pe);
    CREATE_TRY(pe);
    if (d == 64) c->p_attn = make_attn_plan_g<64, 2, 4>(G, &pe); else c->p_attn = make_attn_plan_g<128, 2, 4>(G, &pe);
    CREATE_TRY(pe);
    c->p_attn.min_chunk = 64;
    {
        int per_head = (2 * c->num_sms + nkv - 1) / nkv;
        const int need = (max_context + c->p_attn.min_chunk - 1) / c->p_attn.min_chunk;
        if (per_head > need) per_head = need;
        if (per_head < 1) per_head = 1;
        c->p_attn.max_chunks = per_head;
    }

    {
        const char *impl = getenv("EDGEFM_IMPL");
        c->use_mega = !(impl && std::strcmp(impl, "kernels") == 0);
    }
    StepPlan pl;
    if (c->use_mega) {
        int smem_optin = 0, coop = 0;
        CREATE_TRY(cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
        CREATE_TRY(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
        if (!coop) return bail(EDGEFM_ERR_CUDA, "device lacks cooperative launch", cudaErrorNotSupported);
        cudaError_t ce = cudaSuccess;
        if (const char *why = plan_step(sh, max_context, c->num_sms, smem_optin, &pl, &ce))
            return bail(EDGEFM_ERR_CUDA, why, ce != cudaSuccess ? ce : cudaErrorInvalidValue);
        c->mega = pl.kernel;
        c->mega_threads = pl.nw * 32;
        c->mega_grid = pl.grid;
        c->tile_budget = pl.budget;
        c->p_attn.max_chunks = pl.max_chunks;  // sizes the partial buffers below
        c->p_lm.grid = pl.grid;
    }

    const size_t kv_elems = static_cast<size_t>(sh.n_layers) * nkv * max_context * d;
    CREATE_TRY(dev_alloc(&c->k_cache, kv_elems));
    CREATE_TRY(dev_alloc(&c->v_cache, kv_elems));
    CREATE_TRY(dev_alloc(&c->x, H));
    CREATE_TRY(dev_alloc(&c->q, nq * d));
    CREATE_TRY(dev_alloc(&c->attn, nq * d));
    CREATE_TRY(dev_alloc(&c->act, F));
    CREATE_TRY(dev_alloc(&c->rope_cs, d));
    CREATE_TRY(dev_alloc(&c->inv_freq, d / 2));
    CREATE_TRY(dev_alloc(&c->part_m, static_cast<size_t>(nq) * c->p_attn.max_chunks));
    CREATE_TRY(dev_alloc(&c->part_l, static_cast<size_t>(nq) * c->p_attn.max_chunks));
    CREATE_TRY(dev_alloc(&c->part_o, static_cast<size_t>(nq) * c->p_attn.max_chunks * d));
    CREATE_TRY(dev_alloc(&c->lm_part_val, c->p_lm.grid));
    CREATE_TRY(dev_alloc(&c->lm_part_idx, c->p_lm.grid));
    CREATE_TRY(dev_alloc(&c->tickets, nq + nkv + 2));
    CREATE_TRY(dev_alloc(&c->state, 1));
    CREATE_TRY(dev_alloc(&c->req, 1));
    CREATE_TRY(cudaMemset(c->k_cache, 0, kv_elems * 2));
    CREATE_TRY(cudaMemset(c->v_cache, 0, kv_elems * 2));
    CREATE_TRY(cudaMemset(c->tickets, 0, (nq + nkv + 2) * sizeof(unsigned)));
    CREATE_TRY(cudaMemset(c->state, 0, sizeof(StepState)));
    {
        StepRequest r{-1, -1, nullptr, nullptr};
        CREATE_TRY(cudaMemcpy(c->req, &r, sizeof r, cudaMemcpyHostToDevice));
        std::vector<double> inv(d / 2);
        for (int i = 0; i < d / 2; ++i) inv[i] = std::pow(static_cast<double>(sh.rope_theta), -2.0 * i / d);
        CREATE_TRY(cudaMemcpy(c->inv_freq, inv.data(), inv.size() * sizeof(double), cudaMemcpyHostToDevice));
    }

    if (c->use_mega) {
        // the operators of the step wired to the work buffers, then the shared-memory rings
        std::vector<MkPhase> phases(static_cast<size_t>(pl.n_phases));
        if (const char *why = plan_phases(&pl, sh, c->layers.data(), c->final_norm, c->lm_head, c->x, c->q, c->attn, c->act, phases.data()))
            return bail(EDGEFM_ERR_CUDA, why, cudaErrorInvalidValue);
        c->mega_smem = pl.dyn_smem;
        CREATE_TRY(cudaFuncSetAttribute(c->mega, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(c->mega_smem)));
        int per_sm = 0;
        CREATE_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, c->mega, c->mega_threads, c->mega_smem));
        if (per_sm < 1) return bail(EDGEFM_ERR_CUDA, "persistent kernel does not fit one CTA per SM", cudaErrorInvalidValue);
        CREATE_TRY(dev_alloc(&c->d_phases, phases.size()));
        CREATE_TRY(dev_alloc(&c->grid_bar, 1));
        CREATE_TRY(cudaMemset(c->grid_bar, 0, sizeof(unsigned)));
        CREATE_TRY(cudaMemcpy(c->d_phases, phases.data(), phases.size() * sizeof(MkPhase), cudaMemcpyHostToDevice));
        c->lm_phase_full = phases.back();
        CREATE_TRY(dev_alloc(&c->vocab_ids, static_cast<size_t>(sh.vocab)));
        CREATE_TRY(cudaMemset(c->vocab_ids, 0, static_cast<size_t>(sh.vocab) * sizeof(int)));
        MkParams &m = c->mk;
        fill_shape_params(&m, sh, max_context, pl);
        m.phases = c->d_phases; m.vocab_ids = c->vocab_ids;
        m.k_cache = c->k_cache; m.v_cache = c->v_cache; m.embed = (const uint16_t *)c->embed;
        m.inv_freq = c->inv_freq; m.x = c->x; m.q = c->q; m.attn = c->attn; m.part_m = c->part_m; m.part_l = c->part_l;
        m.part_o = c->part_o; m.tickets = c->tickets; m.barrier = c->grid_bar;
        if (max_context > 8192) {   // only the long-context kernel variant has both attention modes
            if (const char *ac = getenv("EDGEFM_ATT_SPLIT_MAX")) { const int v = atoi(ac); if (v >= 0) m.att_split_max_n = v; }
        }
        if (const char *ac = getenv("EDGEFM_ATT_CHUNK")) { const int v = atoi(ac); if (v >= 8) { m.att_chunk_shared = v; m.att_chunk_split = v; } }
        m.lm_part_val = c->lm_part_val; m.lm_part_idx = c->lm_part_idx; m.state = c->state; m.req = c->req;
        const char *pe_ = getenv("EDGEFM_PROFILE");
        if (pe_ && pe_[0] == '1') {
            c->prof_stride = 3 + 14 * sh.n_layers;
            CREATE_TRY(dev_alloc(&c->prof, static_cast<size_t>(c->mega_grid + 1) * c->prof_stride + MK_NW_SHORT * 16));
            CREATE_TRY(cudaMemset(c->prof, 0, (static_cast<size_t>(c->mega_grid + 1) * c->prof_stride + MK_NW_SHORT * 16) * 8));
            m.prof = c->prof; m.prof_stride = c->prof_stride;
        }
    }

    // record the step once; every decode step replays this graph
    CREATE_TRY(cudaStreamCreateWithFlags(&c->build_stream, cudaStreamNonBlocking));
    CREATE_TRY(cudaStreamBeginCapture(c->build_stream, cudaStreamCaptureModeThreadLocal));
    cudaError_t le = enqueue_step(c, c->build_stream, &c->launches_per_step);
    cudaError_t ce = cudaStreamEndCapture(c->build_stream, &c->graph);
    if (le != cudaSuccess) return bail(EDGEFM_ERR_CUDA, "kernel launch during graph capture", le);
    CREATE_TRY(ce);
    CREATE_TRY(cudaGraphInstantiate(&c->exec, c->graph, 0));
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
    if (!ctx->use_mega) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "vocabulary pruning needs the persistent-kernel path");
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
    MkPhase ph = ctx->lm_phase_full;
    uint16_t *fresh = nullptr;
    if (n > 0) {
        // plan the operator for n rows with the tile budget of the context; it has to fit what the step kernel was
        // launched with (largest tile, partial-sum scratch)
        StepPlan pl;
        pl.grid = ctx->mega_grid; pl.nw = ctx->mega_threads / 32; pl.budget = ctx->tile_budget;
        const MkPhase &full = ctx->lm_phase_full;
        const bool fits = plan_phase(pl, ctx->shape.head_dim, PH_LMHEAD, nullptr, H, n, nullptr, full.norm_w, full.x_src, nullptr, full.layer, &ph);
        ph.flags = PHF_REMAP;
        if (!fits || phase_tile_bytes(ph) > ctx->mk.slot_bytes)
            return fail(ctx, EDGEFM_ERR_BAD_SHAPE, "a subset of %d rows does not fit the tile plan of this context", n);
        CUDA_TRY(ctx, cudaMalloc(&fresh, static_cast<size_t>(n) * H * sizeof(uint16_t)));
        ph.W = fresh;
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
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(ctx->d_phases + (ctx->mk.nph - 1), &ph, sizeof ph, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);   // token_ids and ph are read before the call returns
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
    *n_ctas = ctx->prof ? ctx->mega_grid : 0;
    *stride = ctx->prof_stride;
    if (!ctx->prof || !out_host) return EDGEFM_OK;
    int64_t n = static_cast<int64_t>(ctx->mega_grid) * ctx->prof_stride;
    if (capacity >= n + MK_NW_SHORT * 16) n += MK_NW_SHORT * 16;   // optional per-warp trace behind the table
    if (capacity < n) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "profile buffer too small");
    DeviceGuard guard(ctx->device);
    CUDA_TRY(ctx, cudaDeviceSynchronize());
    CUDA_TRY(ctx, cudaMemcpy(out_host, ctx->prof, static_cast<size_t>(n) * 8, cudaMemcpyDeviceToHost));
    return EDGEFM_OK;
}

edgefm_status edgefm_sync_status(edgefm_ctx *ctx, void *stream) {
    if (!ctx) return EDGEFM_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    CUDA_TRY(ctx, cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    StepState st;
    CUDA_TRY(ctx, cudaMemcpy(&st, ctx->state, sizeof st, cudaMemcpyDeviceToHost));
    if (st.status != 0)
        return fail(ctx, EDGEFM_ERR_TIMEOUT, "device status %d (6 = a bounded wait expired, 100+ = self-check code) operands %d %d; "
                    "the context must be destroyed", st.status, st.pad[0], st.pad[1]);
    return EDGEFM_OK;
}

edgefm_status edgefm_export_kv(edgefm_ctx *ctx, void *k_out, void *v_out, void *stream) {
    if (!ctx) return EDGEFM_ERR_INVALID_ARG;
    if (!k_out || !v_out) return fail(ctx, EDGEFM_ERR_INVALID_ARG, "null output");
    DeviceGuard guard(ctx->device);
    const edgefm_shape &sh = ctx->shape;
    const size_t bytes = static_cast<size_t>(sh.n_layers) * sh.n_kv_heads * ctx->max_context * sh.head_dim * 2;
    CUDA_TRY(ctx, cudaMemcpyAsync(k_out, ctx->k_cache, bytes, cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream)));
    CUDA_TRY(ctx, cudaMemcpyAsync(v_out, ctx->v_cache, bytes, cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream)));
    return EDGEFM_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------------------
// edgefm_decode_step_static -- one decode step that allocates nothing.
//
// Some callers must not allocate device memory at all: a step issued from inside another framework's
// allocation-free region (for example while that framework is replaying or recording its own work with a
// fixed memory plan), from a process whose device memory is handed out entirely by a pool it does not own,
// or from a latency-critical thread where the implicit device synchronisation of cudaMalloc / cudaFree is
// not acceptable.  For them the work buffers of the persistent step kernel (residual stream, queries,
// attention partials, MLP activations, schedule, counters, device state: everything edgefm_create would
// allocate except the KV cache) live in a fixed array that is part of the loaded library image.  The
// caller owns the KV cache and the cache length and passes them in, so the call keeps no context.
//
// The array is EDGEFM_STATIC_SCRATCH_BYTES (2 MiB) on every GPU that loads the library, until exit.
namespace {

constexpr size_t EDGEFM_STATIC_SCRATCH_BYTES = 2u << 20;
static __device__ __align__(256) unsigned char g_static_scratch[EDGEFM_STATIC_SCRATCH_BYTES];

// In host code `g_static_scratch` is only a host-side stand-in for the symbol, not a device address.
// The device address is looked up once per device, with that device current.
constexpr int kMaxDevices = 64;
unsigned char *g_scratch_dev_ptr[kMaxDevices] = {};

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
    // ---- the same plan edgefm_create makes, on the stack ----------------------------------------------------
    StepPlan pl;
    {
        cudaError_t ce = cudaSuccess;
        if (const char *why = plan_step(sh, max_context, num_sms, smem_optin, &pl, &ce))
            return fail(nullptr, ce != cudaSuccess ? EDGEFM_ERR_CUDA : EDGEFM_ERR_BAD_SHAPE, "%s", why);
    }
    MegaKernel kern = pl.kernel;
    const int NW = pl.nw, grid = pl.grid, max_chunks = pl.max_chunks, n_phases = pl.n_phases;

    // carve the scratch array; reject shapes that need more than it holds
    ScratchCarver sc{g_scratch_dev_ptr[dev]};
    MkPhase *d_phases = sc.take<MkPhase>(n_phases);
    float *x = sc.take<float>(H);
    float *q = sc.take<float>(static_cast<size_t>(nq) * d);
    float *attn = sc.take<float>(static_cast<size_t>(nq) * d);
    float *act = sc.take<float>(F);
    double *inv_freq = sc.take<double>(d / 2);
    float *part_m = sc.take<float>(static_cast<size_t>(nq) * max_chunks);
    float *part_l = sc.take<float>(static_cast<size_t>(nq) * max_chunks);
    float *part_o = sc.take<float>(static_cast<size_t>(nq) * max_chunks * d);
    float *lm_val = sc.take<float>(grid);
    int *lm_idx = sc.take<int>(grid);
    unsigned *counters = sc.take<unsigned>(static_cast<size_t>(nq) + nkv + 2 + 64);   // tickets, then the grid barrier counter
    StepState *state = sc.take<StepState>(1);
    StepRequest *req = sc.take<StepRequest>(1);
    if (sc.off > EDGEFM_STATIC_SCRATCH_BYTES)
        return fail(nullptr, EDGEFM_ERR_BAD_SHAPE, "this shape needs %zu bytes of work buffers; the static scratch holds %zu", sc.off,
                    EDGEFM_STATIC_SCRATCH_BYTES);
    unsigned *tickets = counters;
    unsigned *grid_bar = counters + nq + nkv + 2 + 32;

    MkPhase phases[4 * kMaxLayers + 1];
    if (const char *why = plan_phases(&pl, sh, weights->layers, weights->final_norm, weights->lm_head, x, q, attn, act, phases))
        return fail(nullptr, EDGEFM_ERR_BAD_SHAPE, "%s", why);
    const int n_ph = n_phases;
    const size_t dyn_smem = pl.dyn_smem;
    // raise the kernel's dynamic shared-memory limit (a function attribute, not an allocation); repeated on every
    // call because edgefm_create sets the same attribute for its own contexts
    CUDA_TRY(nullptr, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(dyn_smem)));

    MkParams m{};
    fill_shape_params(&m, sh, max_context, pl);
    m.phases = d_phases;
    m.k_cache = static_cast<uint16_t *>(k_cache); m.v_cache = static_cast<uint16_t *>(v_cache);
    m.embed = (const uint16_t *)weights->embed; m.inv_freq = inv_freq; m.x = x; m.q = q; m.attn = attn;
    m.part_m = part_m; m.part_l = part_l; m.part_o = part_o;
    m.tickets = tickets; m.barrier = grid_bar; m.lm_part_val = lm_val; m.lm_part_idx = lm_idx; m.state = state; m.req = req;
    m.prof = nullptr; m.prof_stride = 0;

    // ---- stream-ordered set-up of the shared scratch: it still holds the previous call's contents ----------
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    double inv[64];
    for (int i = 0; i < d / 2; ++i) inv[i] = std::pow(static_cast<double>(sh.rope_theta), -2.0 * i / d);
    StepState st{};
    st.cur_len = cur_len; st.next_position = position;
    StepRequest rq{token_id, position, logits_out, next_token_out};
    // counters (attention tickets, lm_head ticket, grid barrier) must start at zero
    CUDA_TRY(nullptr, cudaMemsetAsync(counters, 0, (static_cast<size_t>(nq) + nkv + 2 + 64) * sizeof(unsigned), s));
    // small pageable copies: the runtime stages the bytes before returning, so stack sources are fine
    CUDA_TRY(nullptr, cudaMemcpyAsync(d_phases, phases, static_cast<size_t>(n_ph) * sizeof(MkPhase), cudaMemcpyHostToDevice, s));
    CUDA_TRY(nullptr, cudaMemcpyAsync(inv_freq, inv, static_cast<size_t>(d / 2) * sizeof(double), cudaMemcpyHostToDevice, s));
    CUDA_TRY(nullptr, cudaMemcpyAsync(state, &st, sizeof st, cudaMemcpyHostToDevice, s));
    CUDA_TRY(nullptr, cudaMemcpyAsync(req, &rq, sizeof rq, cudaMemcpyHostToDevice, s));

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(NW * 32);
    cfg.dynamicSmemBytes = dyn_smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    CUDA_TRY(nullptr, cudaLaunchKernelEx(&cfg, kern, m));
    g_create_error.clear();
    return EDGEFM_OK;
}
