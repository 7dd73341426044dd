// Types and constants of the persistent decode kernel that do not depend on the number of warps per CTA.
#pragma once
#include "common.cuh"

namespace edgefm {

constexpr int MK_ATT_LPP = 2;                    // lanes per cached position in the score phase (one CTA per GQA group)
constexpr int MK_ATT_LPP_SPLIT = 2;              // ... when every query head has its own CTAs (16 positions per warp iteration)
constexpr int MK_ATT_TILE = 32 / MK_ATT_LPP;     // positions per warp iteration (grouped mode)
#ifndef MK_ATT_SPLIT_MAXC_VALUE
#define MK_ATT_SPLIT_MAXC_VALUE 12
#endif
constexpr int MK_ATT_SPLIT_MAXC = MK_ATT_SPLIT_MAXC_VALUE;   // chunks per head when every query head has its own CTAs
constexpr int MK_PARTIAL_SLOTS = 48;             // shared-memory scratch: partial row sums, 16 floats per slot
constexpr int MK_PARTIAL_FLOATS = MK_PARTIAL_SLOTS * 16;   // (also the chunk statistics of the attention merge)
constexpr int MK_TILE_COLS = 256;                // columns of a weight tile: four blocks of 64 columns (128-byte rows, the swizzle span)
constexpr int MK_TILE_ROWS = 16;                 // rows of a tile: the M of one m16n8k16 tensor-core instruction (largest tile: 8 KB)
constexpr int MK_X_SPLITS = 3;                   // (the most; see mk_splits)
// bf16 pieces an fp32 activation is staged as.  Three (24 mantissa bits) while the tokens of a call fit the eight B columns
// that way (1 or 2 tokens); the build for blocks of up to four tokens keeps two pieces per token (16 mantissa bits, twice the
// precision of the bf16 weights it multiplies).
__host__ __device__ constexpr int mk_splits(int block_tokens) { return block_tokens > 2 ? 2 : 3; }
                   // an fp32 activation is staged as the sum of three bf16 pieces (24 mantissa bits)
constexpr int MK_XS_PAD = 64;                    // bytes between the three staged arrays beyond the row length (bank spread)
// A consumer warp's buffer for one tile's worth of a vector read from global memory: 3 arrays of 512 bytes per token of the
// call.  The single-token build spreads them over the banks (pad); a block build has no room for that (its shared memory
// decides the size of the ring slots) and packs them.
__host__ __device__ constexpr int mk_wbuf_array_bytes(int block_tokens) { return MK_TILE_COLS * 2 + (block_tokens > 1 ? 0 : MK_XS_PAD); }
__host__ __device__ constexpr int mk_wbuf_bytes(int block_tokens) { return block_tokens * mk_splits(block_tokens) * mk_wbuf_array_bytes(block_tokens); }
constexpr int MK_MAX_VARIANTS = 4;               // tensor maps (box heights) per weight matrix
constexpr int MK_MAX_SLOTS = 4;                  // ring slots per consumer warp
constexpr int MK_WARP_TAB = 8;                   // ints per warp in the per-CTA table
// Consumer warps per CTA of the two builds of the kernel (one more warp prefetches into L2): the short-context build favours
// instruction streams, the long-context build (grouped attention keeps G heads of accumulators per warp) registers.
#ifndef MK_HEAD_FLAGS
#define MK_HEAD_FLAGS 1   // short build: per-head completion counters instead of the grid barrier between QKV and attention
#endif
#ifndef MK_PF_TILES
#define MK_PF_TILES 4   // tiles per consumer warp the helper warp asks L2 for ahead of the ring
#endif
#ifndef MK_PF_TILES_LM
#define MK_PF_TILES_LM 8   // the same within the output layer
#endif
#ifndef MK_NW_SHORT_VALUE
#define MK_NW_SHORT_VALUE 11
#endif
#ifndef MK_NW_LONG_VALUE
#define MK_NW_LONG_VALUE 7
#endif
constexpr int MK_NW_SHORT = MK_NW_SHORT_VALUE;
constexpr int MK_NW_LONG = MK_NW_LONG_VALUE;
constexpr int MK_NW_MAX = MK_NW_SHORT > MK_NW_LONG ? MK_NW_SHORT : MK_NW_LONG;

enum { PH_QKV = 0, PH_RESID = 1, PH_SWIGLU = 2, PH_LMHEAD = 3 };

// MkOp::flags
enum : int {
    PHF_REMAP = 1,      // PH_LMHEAD: rows are a vocabulary subset; row r stands for token MkParams::vocab_ids[r]
    PHF_OUT_SPLIT = 2,  // PH_SWIGLU: the output vector is stored the way the next operator reads it: three bf16 arrays
                        // [3][F rounded up to 256] (the pieces of every value) in tensor-core fragment order (mk_xs_index)
    PHF_X_GLOBAL = 4,   // the input vector has that form already: the consumer warps read their B fragments straight from
                        // global memory (L2), a tile ahead; nothing is staged in shared memory
    PHF_RAGGED = 8,     // K is not a multiple of 64: the tile's four 64-column blocks are fetched by one copy each
};

// Position of column c in a staged activation array.  The columns of every group of 32 are reordered so that the two 32-bit
// B-fragment registers of two consecutive k-steps of mma.m16n8k16 are one 16-byte piece per lane quad index q:
// [q][k-step parity][k half][2 values].
__host__ __device__ inline int mk_xs_index(int c) {
    const int kk = c & 15;
    return (c & ~31) + ((kk & 7) >> 1) * 8 + ((c >> 4) & 1) * 4 + (kk >> 3) * 2 + (kk & 1);
}

// One weight-streaming operator of the step (its weights are reached through tensor maps, see MkParams::maps).
struct alignas(16) MkOp {
    const uint16_t *bias;    // PH_QKV: bf16 [rows] or null
    const uint16_t *norm_w;  // RMSNorm weight of the prologue (bf16 [K]) or null = plain copy of x_src
    const float *x_src;      // fp32 [K] input vector in global memory; null = embedding row of the token
    float *out;              // PH_QKV: q fp32; PH_RESID: x (+=); PH_SWIGLU: act; PH_LMHEAD: unused
    int K;                   // columns (multiple of 8)
    int kind;
    int units_total;         // rows (PH_RESID, PH_LMHEAD), pairs (PH_QKV: rows/2, PH_SWIGLU: F)
    int layer_flags;         // layer << 8 | PHF_* bits
    int x_tok_stride;        // a block of several tokens: elements (of x_src's type; PHF_X_GLOBAL: bf16) between the tokens' input vectors
    int out_tok_stride;      // ... and between their output vectors (floats; PHF_OUT_SPLIT: bf16)
    int pad_[2];
    __host__ __device__ int layer() const { return layer_flags >> 8; }
    __host__ __device__ int flags() const { return layer_flags & 0xff; }
};
static_assert(sizeof(MkOp) % 16 == 0, "descriptor is copied in 16-byte pieces");

// ---- the tile schedule ------------------------------------------------------------------------------------------
// A tile is a box of m rows x 256 columns of one weight matrix (for PH_QKV / PH_SWIGLU: m "low" rows and their m
// partner rows), fetched by one TMA tensor copy into a ring slot of the consumer warp that owns it, where it lies as
// [4 column blocks][partner][m][128 bytes] with the 128-byte swizzle (conflict-free ldmatrix reads).
// The host lays out, for every CTA and every consumer warp, the list of tiles of one layer (operators in order) and of
// the output layer; the lists are the same for every layer.  8 bytes per tile:
//   x: unit_base [0,20) | column piece [20,28) | tensor-map variant [28,30) | FIRST 30 | FLUSH 31
//   y: m [0,5) | first valid unit v0 [5,9) | DIRECT 9 | partial slot [10,20) | operator in layer (4 = output layer) [20,23) |
//      RAGGED 23 (K is not a multiple of 64: the tile is fetched as four copies, see PHF_RAGGED)
// FIRST: the warp's accumulators start at zero with this tile.  FLUSH: after this tile the 16 row sums are reduced
// across the lanes; DIRECT: the warp has seen all columns of these rows and finishes them itself; otherwise the sums
// go to partial slot `slot` and the units are finished after the operator by summing their slots in order.
constexpr uint32_t MKT_FIRST = 1u << 30, MKT_FLUSH = 1u << 31, MKT_DIRECT = 1u << 9, MKT_RAGGED = 1u << 23;
__host__ __device__ inline uint2 mk_tile_desc(uint32_t unit_base, uint32_t kcol, uint32_t variant, bool first, bool flush, uint32_t m,
                                              uint32_t v0, bool direct, uint32_t slot, uint32_t op, bool ragged = false) {
    uint2 d;
    d.x = (unit_base & 0xfffffu) | (kcol & 0xffu) << 20 | (variant & 3u) << 28 | (first ? MKT_FIRST : 0u) | (flush ? MKT_FLUSH : 0u);
    d.y = (m & 31u) | (v0 & 15u) << 5 | (direct ? MKT_DIRECT : 0u) | (slot & 1023u) << 10 | (op & 7u) << 20 | (ragged ? MKT_RAGGED : 0u);
    return d;
}
// Units whose row sums were left in partial slots: unit_base, m | v0 << 8, first slot, number of slots.
using MkCombine = uint4;

struct MkParams {
    const MkOp *ops;         // [nph]
    int nph;                 // 4 * n_layers + 1
    int n_layers, H, nq, nkv, d, F, V;
    int half_shift;          // log2(d / 2)
    float eps, scale;
    int max_context;
    uint16_t *k_cache, *v_cache;   // [L][nkv][max_context][d] bf16; compressed cache (kv8): the same shape in signed bytes
    int kv8;                       // 1: compressed cache (8-bit codes + one fp32 scale per cached row)
    float *k_scale, *v_scale;      // kv8: [L][nkv][max_context]
    float *kv_stage;               // kv8: the fp32 k (after RoPE) and v rows of the step's token, [2][nkv][d], reused by every layer
    const uint16_t *embed;
    const double *inv_freq;        // [d/2]
    float *x, *q, *attn;
    float *part_m, *part_l, *part_o;
    int max_chunks;                // row stride of the attention partial buffers (>= any chunk count)
    int block_tokens;              // tokens a call may carry (1, or the M of the block build); buffers below hold that many vectors:
                                   // x [M][H], q / attn [M][nq d], part_m / part_l [M][nq][max_chunks], part_o [M][nq][max_chunks][d],
                                   // lm_part_val / lm_part_idx [M][gridDim.x]
    int att_chunk_shared;          // smallest chunk (positions) when one CTA serves a whole GQA group
    int att_chunk_split;           // smallest chunk when every query head has its own CTAs
    int att_split_max_n;           // contexts up to this length use one-head-per-CTA attention
    unsigned *tickets;             // [nq] attention, [nq] = lm_head
    unsigned *barrier;             // grid barrier counter (0 between launches)
    unsigned *head_ready;          // [nq + 2 nkv] finished units per head of the QKV projection, all layers of the step (0 between launches)
    int head_flags;                // 1: no grid barrier between the QKV projection and attention; attention waits on head_ready (short build)
    float *lm_part_val;
    int *lm_part_idx;
    const int *vocab_ids;          // [V] token id of every row of a pruned lm_head (used when the last operator has PHF_REMAP)
    StepState *state;
    const StepRequest *req;
    // weight streaming
    const uint16_t *const *op_weights;   // [nph] base of every operator's matrix (the L2 prefetch uses plain addresses)
    const unsigned char *maps;     // CUtensorMap [(4 * n_layers + 1) * MK_MAX_VARIANTS], 128 bytes each, index (4 l + op) * 4 + variant
    const uint2 *tiles;            // all tile lists, one contiguous block per CTA (copied to shared memory when the kernel starts)
    const int *cta_tab;            // [gridDim.x][cta_tab_ints]: per consumer warp {layer list offset in the CTA's block, tiles per
                                   // operator x4, output-layer list offset, output-layer tiles, tiles per layer}, then per operator (5) {combine
                                   // offset in the CTA's block, combine count}, then {first tile of the CTA's block, tiles in the block, first combine
                                   // entry of the CTA's block, entries in the block}
    const MkCombine *combines;
    int cta_tab_ints;
    int slots;                     // ring slots per consumer warp
    int slot_bytes;                // bytes of one slot (a multiple of 1024)
    int xbuf_bytes, ops_bytes, tab_bytes, sched_bytes;   // shared-memory areas: operators, table, tile lists, [rings], activation vector
    int pf_tiles;                  // tiles per consumer warp the L2 prefetch runs ahead of the ring
    int map_fence;                 // tensor maps the host may have rewritten since the last launch: 0 none, 1 the output layer's, 2 all
    int barrier_extra;             // test hook: arrivals the grid barrier expects beyond the CTAs present (0 in production)
    unsigned spin_limit;           // upper bound of every device-side wait, nanoseconds
    unsigned long long *prof;      // optional timestamps [gridDim.x][prof_stride] (diagnostics), or null
    int prof_stride;
};

using MegaKernel = void (*)(const MkParams);
// long-context kernel variants, defined in megakernel_long_d*_*.cu
MegaKernel mega_kernel_long_d64_lo(int G);
MegaKernel mega_kernel_long_d64_hi(int G);
MegaKernel mega_kernel_long_d128_lo(int G);
MegaKernel mega_kernel_long_d128_hi(int G);
// ... and their variants for the compressed cache, defined in megakernel_q8_d*_*.cu
MegaKernel mega_kernel_q8_d64_lo(int G);
MegaKernel mega_kernel_q8_d64_hi(int G);
MegaKernel mega_kernel_q8_d128_lo(int G);
MegaKernel mega_kernel_q8_d128_hi(int G);

}  // namespace edgefm
