// Types and constants of the persistent decode kernel that do not depend on the number of warps per CTA.
#pragma once
#include "common.cuh"

namespace edgefm {

constexpr int MK_MAXF = 4;                       // tiles in flight per warp (one mbarrier each)
constexpr int MK_BAR_POLLERS = 1;                // warps whose lane 0 polls the grid barrier counter
constexpr int MK_ATT_LPP = 2;                    // lanes per cached position in the score phase (one CTA per GQA group)
constexpr int MK_ATT_LPP_SPLIT = 2;              // ... when every query head has its own CTAs (16 positions per warp iteration)
constexpr int MK_ATT_TILE = 32 / MK_ATT_LPP;     // positions per warp iteration (grouped mode)
constexpr int MK_ATT_SPLIT_MAXC = 12;            // chunks per head when every query head has its own CTAs
constexpr int MK_PARTIAL_FLOATS = 2048;          // shared-memory scratch: split-K partial sums / chunk statistics
// Warps per CTA of the two builds of the kernel: the short-context build favours instruction streams, the
// long-context build (grouped attention keeps G heads of accumulators per warp) favours registers.
#ifndef MK_NW_SHORT_VALUE
#define MK_NW_SHORT_VALUE 12
#endif
#ifndef MK_NW_LONG_VALUE
#define MK_NW_LONG_VALUE 8
#endif
constexpr int MK_NW_SHORT = MK_NW_SHORT_VALUE;
constexpr int MK_NW_LONG = MK_NW_LONG_VALUE;

enum { PH_QKV = 0, PH_RESID = 1, PH_SWIGLU = 2, PH_LMHEAD = 3 };

// One weight-streaming operator of the step.
// MkPhase::flags
enum : int {
    PHF_REMAP = 1,      // PH_LMHEAD: rows are a vocabulary subset; row r stands for token MkParams::vocab_ids[r]
    PHF_OUT_SPLIT = 2,  // PH_SWIGLU: the output vector is stored as [even 16-byte pieces | odd 16-byte pieces]
    PHF_X_BULK = 4,     // the input vector has that layout already and needs no transform: staged by two bulk copies
};

struct alignas(16) MkPhase {
    const uint16_t *W;       // bf16 [rows][K]
    const uint16_t *bias;    // PH_QKV: bf16 [rows] or null
    const uint16_t *norm_w;  // RMSNorm weight of the prologue (bf16 [K]) or null = plain copy of x_src
    const float *x_src;      // fp32 [K] input vector in global memory; null = embedding row of the token
    float *out;              // PH_QKV: q fp32; PH_RESID: x (+=); PH_SWIGLU: act; PH_LMHEAD: unused
    int K;                   // columns (multiple of 8)
    int kind;
    int rw;                  // units per work item (rows, or row pairs for PH_QKV / PH_SWIGLU); 1 when split
    int ksplit;              // K slices per item (tiles per item)
    int kcs;                 // 16-byte pieces per row slice = K / 8 / ksplit
    int units_total;         // rows (PH_RESID, PH_LMHEAD), pairs (PH_QKV: rows/2, PH_SWIGLU: F)
    int items_total;         // ceil(units_total / rw)
    int layer;
    int s_shift;             // log2(ksplit); ksplit is a power of two
    int split;               // 1: the tiles of an item go to different warps, partial sums meet in shared memory
    int flags;               // PHF_* bits
};
static_assert(sizeof(MkPhase) % 16 == 0, "descriptor is copied in 16-byte pieces");

struct MkParams {
    const MkPhase *phases;   // [nph]
    int nph;                 // 4 * n_layers + 1
    int n_layers, H, nq, nkv, d, F, V;
    int half_shift;          // log2(d / 2)
    float eps, scale;
    int max_context;
    uint16_t *k_cache, *v_cache;   // [L][nkv][max_context][d]
    const uint16_t *embed;
    const double *inv_freq;        // [d/2]
    float *x, *q, *attn;
    float *part_m, *part_l, *part_o;
    int max_chunks;                // row stride of the attention partial buffers (>= any chunk count)
    int att_chunk_shared;          // smallest chunk (positions) when one CTA serves a whole GQA group
    int att_chunk_split;           // smallest chunk when every query head has its own CTAs
    int att_split_max_n;           // contexts up to this length use one-head-per-CTA attention
    unsigned *tickets;             // [nq] attention, [nq] = lm_head
    unsigned *barrier;             // grid barrier counter (0 between launches)
    float *lm_part_val;
    int *lm_part_idx;
    const int *vocab_ids;          // [V] token id of every row of a pruned lm_head (used when the last operator has PHF_REMAP)
    StepState *state;
    const StepRequest *req;
    int ring_bytes;                // shared-memory ring of one warp
    int slot_bytes;                // largest tile (checked against ring_bytes on the host)
    int xbuf_bytes, sched_bytes;
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

}  // namespace edgefm
