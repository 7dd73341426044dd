// Host side of the persistent step kernel: the static tile schedule of the weight stream and its tensor maps.
//
// Every weight matrix is row-major bf16 [rows][K].  A CTA owns a contiguous range of the "units" of every operator (a
// unit is an output row; for the QKV and gate/up operators a pair of rows whose sums meet in one epilogue: the rotate-half
// RoPE partners i, i + d/2 of a head, or gate row i and up row F + i).  The range is cut into blocks of up to 16 rows (8
// pairs), every block into tiles of 256 columns, and the tiles, in (block, column) order, into one contiguous run per
// consumer warp.  A warp therefore sees consecutive column pieces of the same rows: it keeps their 16 sums in
// registers and reduces them once per run; runs that cover all columns of a block finish the rows in the warp, the
// others leave partial sums in shared-memory slots that are added in slot order after the operator (deterministic).
#pragma once
#include <cuda.h>   // CUtensorMap and its enums only: the encoder is looked up at run time, nothing links against the driver library
#include <algorithm>
#include <cstring>
#include <vector>

#include "megakernel_types.cuh"

namespace edgefm {

struct OpShape {
    int kind = 0;        // PH_*
    int units = 0;       // rows, or row pairs
    int K = 0;           // columns
    int rows = 0;        // rows of the matrix (tensor-map extent)
    int head_half = 0;   // PH_QKV: d / 2 (a block may not cross a head)
};

struct OpSchedule {
    int n_variants = 0;
    int variant_rows[MK_MAX_VARIANTS] = {0, 0, 0, 0};            // box heights of the operator's tensor maps
    std::vector<std::vector<std::vector<uint2>>> tiles;          // [cta][warp] tile list
    std::vector<std::vector<MkCombine>> combines;                // [cta]
    int max_slots = 0;                                           // partial slots the busiest CTA uses
};

inline bool op_paired(int kind) { return kind == PH_QKV || kind == PH_SWIGLU; }

// Schedule of one operator for `ncta` CTAs of `nw` consumer warps; slot_rows = rows a ring slot holds.
// op_index: 0..3 inside a layer, 4 = output layer.  Returns null, or why the operator does not fit.
inline const char *plan_op(const OpShape &os, int op_index, int ncta, int nw, int slot_rows, OpSchedule *out) {
    const bool paired = op_paired(os.kind);
    int B = paired ? std::min(8, slot_rows / 2) : std::min(MK_TILE_ROWS, slot_rows);   // units per block
    if (B < 1) return "ring slots too small for a tile";
    const int nkb = (os.K + MK_TILE_COLS - 1) / MK_TILE_COLS;
    if (nkb > 255) return "rows too long for the tile schedule";
    if (os.units >= (1 << 20)) return "too many rows for the tile schedule";
    OpSchedule &S = *out;
    S = OpSchedule();
    S.tiles.assign(ncta, std::vector<std::vector<uint2>>(nw));
    S.combines.assign(ncta, {});
    auto variant_of = [&](int rows, bool may_add) -> int {
        for (int v = 0; v < S.n_variants; ++v) if (S.variant_rows[v] == rows) return v;
        if (!may_add || S.n_variants == MK_MAX_VARIANTS) return -1;
        S.variant_rows[S.n_variants] = rows;
        return S.n_variants++;
    };
    // unit ranges of the CTAs.  QKV: in granules that divide a head's pairs, the granule that gives the smallest
    // largest share (so that blocks never cross a head and at most four box heights occur).
    int granule = 1;
    if (os.kind == PH_QKV) {
        long long best = -1;
        for (int g : {8, 4, 2}) {
            if (g > B || os.head_half % g) continue;
            const long long ng = os.units / g;
            const long long worst = ((ng + ncta - 1) / ncta) * g;
            if (best < 0 || worst < best) { best = worst; granule = g; }
        }
        if (best < 0) granule = 1;
        if (os.units % granule) return "QKV rows do not split into blocks";
        B = B / granule * granule;   // blocks of whole granules: at most four different heights (granule, 2 granules, ...)
    }
    struct Block { int u0, m, v0, variant; };
    for (int c = 0; c < ncta; ++c) {
        const long long ng = os.units / granule;
        const int u0 = static_cast<int>(ng * c / ncta) * granule, u1 = static_cast<int>(ng * (c + 1) / ncta) * granule;
        std::vector<Block> blocks;
        int u = u0;
        while (u < u1) {
            int m = std::min(B, u1 - u);
            if (os.kind == PH_QKV) m = std::min(m, os.head_half - u % os.head_half);   // stay inside the head
            int v = variant_of(m, true), v0 = 0, ub = u;
            if (v < 0) {
                // no tensor map of this height left: take a full block that ends where this one ends; its first units
                // repeat units that are already covered and are skipped in the epilogue
                if (os.kind == PH_QKV || u + m - B < u0) return "too many tile heights for one operator";
                v = variant_of(B, false);
                if (v < 0) return "too many tile heights for one operator";
                ub = u + m - B; v0 = B - m; m = B;
            }
            blocks.push_back({ub, m, v0, v});
            u = ub + m;
        }
        // tiles in (block, column) order, one contiguous run per warp
        const int T = static_cast<int>(blocks.size()) * nkb;
        int next_slot = 0;
        std::vector<int> first_slot(blocks.size(), -1), n_slots(blocks.size(), 0);
        for (int w = 0; w < nw; ++w) {
            const int t0 = static_cast<int>(static_cast<long long>(T) * w / nw), t1 = static_cast<int>(static_cast<long long>(T) * (w + 1) / nw);
            int t = t0;
            while (t < t1) {
                const int b = t / nkb, k0 = t % nkb;
                const int k1 = std::min(nkb, k0 + (t1 - t));        // columns [k0, k1) of block b
                const bool direct = k0 == 0 && k1 == nkb;
                int slot = 0;
                if (!direct) {
                    slot = next_slot++;
                    if (first_slot[b] < 0) first_slot[b] = slot;
                    ++n_slots[b];
                }
                for (int k = k0; k < k1; ++k)
                    S.tiles[c][w].push_back(mk_tile_desc(blocks[b].u0, k, blocks[b].variant, k == k0, k == k1 - 1, blocks[b].m, blocks[b].v0,
                                                         direct, slot, op_index, os.K % 64 != 0));
                t += k1 - k0;
            }
        }
        for (size_t b = 0; b < blocks.size(); ++b)
            if (n_slots[b] > 0)
                S.combines[c].push_back(make_uint4(static_cast<unsigned>(blocks[b].u0), static_cast<unsigned>(blocks[b].m | blocks[b].v0 << 8),
                                                   static_cast<unsigned>(first_slot[b]), static_cast<unsigned>(n_slots[b])));
        S.max_slots = std::max(S.max_slots, next_slot);
    }
    if (S.max_slots > MK_PARTIAL_SLOTS) return "too many partial sums per CTA";
    return nullptr;
}

// The step's schedule in the form the kernel reads.
struct StepSchedule {
    OpSchedule ops[5];
    std::vector<uint2> tiles;        // per CTA one block: the warps' layer lists (operators 0..3), then their output-layer lists
    std::vector<int> cta_tab;        // [ncta][cta_tab_ints]
    std::vector<MkCombine> combines;
    int cta_tab_ints = 0;
    int max_cta_tiles = 0;           // largest block (sizes the shared-memory copy)
    int max_cta_combines = 0;
    // bytes of shared memory the largest CTA block needs: tiles (8 bytes each, padded to 16), then combine entries (16 bytes each)
    size_t smem_bytes() const { return (static_cast<size_t>(max_cta_tiles) * 8 + 15) / 16 * 16 + static_cast<size_t>(max_cta_combines) * 16; }
};

inline int cta_tab_ints_for(int nw) { return (nw * MK_WARP_TAB + 14 + 3) / 4 * 4; }

inline void assemble_schedule(StepSchedule *ss, int ncta, int nw) {
    ss->cta_tab_ints = cta_tab_ints_for(nw);
    ss->cta_tab.assign(static_cast<size_t>(ncta) * ss->cta_tab_ints, 0);
    ss->tiles.clear();
    ss->combines.clear();
    ss->max_cta_tiles = 0;
    ss->max_cta_combines = 0;
    for (int c = 0; c < ncta; ++c) {
        int *ctab = &ss->cta_tab[static_cast<size_t>(c) * ss->cta_tab_ints];
        const size_t base = ss->tiles.size();
        for (int w = 0; w < nw; ++w) {
            int *tab = ctab + w * MK_WARP_TAB;
            tab[0] = static_cast<int>(ss->tiles.size() - base);
            for (int o = 0; o < 4; ++o) {
                const auto &l = ss->ops[o].tiles[c][w];
                tab[1 + o] = static_cast<int>(l.size());
                tab[7] += static_cast<int>(l.size());          // tiles per layer
                ss->tiles.insert(ss->tiles.end(), l.begin(), l.end());
            }
        }
        for (int w = 0; w < nw; ++w) {
            int *tab = ctab + w * MK_WARP_TAB;
            const auto &l = ss->ops[4].tiles[c][w];
            tab[5] = static_cast<int>(ss->tiles.size() - base);
            tab[6] = static_cast<int>(l.size());
            ss->tiles.insert(ss->tiles.end(), l.begin(), l.end());
        }
        const size_t cbase = ss->combines.size();
        for (int o = 0; o < 5; ++o) {
            int *ct = ctab + nw * MK_WARP_TAB + 2 * o;
            const auto &l = ss->ops[o].combines[c];
            ct[0] = static_cast<int>(ss->combines.size() - cbase);     // inside the CTA's block
            ct[1] = static_cast<int>(l.size());
            ss->combines.insert(ss->combines.end(), l.begin(), l.end());
        }
        ctab[nw * MK_WARP_TAB + 10] = static_cast<int>(base);
        ctab[nw * MK_WARP_TAB + 11] = static_cast<int>(ss->tiles.size() - base);
        ctab[nw * MK_WARP_TAB + 12] = static_cast<int>(cbase);
        ctab[nw * MK_WARP_TAB + 13] = static_cast<int>(ss->combines.size() - cbase);
        ss->max_cta_combines = std::max(ss->max_cta_combines, static_cast<int>(ss->combines.size() - cbase));
        ss->max_cta_tiles = std::max(ss->max_cta_tiles, static_cast<int>(ss->tiles.size() - base));
    }
}

// ---- tensor maps ---------------------------------------------------------------------------------------------------
using TensorMapEncodeFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                       const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                       CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline TensorMapEncodeFn tensor_map_encoder() {
    static TensorMapEncodeFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            p = nullptr;
        }
        return reinterpret_cast<TensorMapEncodeFn>(p);
    }();
    return fn;
}

// Tensor map of a row-major bf16 [rows][K] matrix on THIS GPU.  A box is box_rows rows x 256 columns, delivered to shared
// memory as four blocks of 64 columns ([block][rows][128 bytes], 128-byte swizzle); columns and rows outside the matrix read as
// zero.  The 64-column blocks of a row are the LAST dimension of the map (stride 128 bytes), so the column coordinate is
// always 0 and the block coordinate is 4 * (column piece).  (No multicast is ever used with these maps.)
//   pair_rows == 0                : (0, row, block);
//   pair_rows  > 0, !grouped      : view [2][pair_rows][K] (gate rows, up rows): (0, row, 0, block), a box = box_rows low rows
//                                   and their partners;
//   pair_rows  > 0, grouped       : view [rows / (2 pair_rows)][2][pair_rows][K] (heads of the QKV matrix, rotate-half partners):
//                                   (0, row in half, 0, head, block).
// K not a multiple of 64: the block dimension is left out (its last block would reach into the next row); the map's first
// dimension is then the K columns, a box is ONE 64-column block, and the caller copies the four blocks of a tile one by one.
inline bool encode_weight_map(CUtensorMap *m, const void *base, int rows, int K, int box_rows, int pair_rows = 0, bool grouped = false) {
    TensorMapEncodeFn enc = tensor_map_encoder();
    if (!enc) return false;
    const cuuint64_t row_bytes = static_cast<cuuint64_t>(K) * 2;
    const bool ragged = K % 64 != 0;
    // dimensions, innermost first: 64 columns (or all K columns when K has a ragged last block), rows [, partner, head],
    // and last the 64-column blocks of a row (128 bytes apart), so that a box lands block by block
    cuuint64_t dims[5] = {static_cast<cuuint64_t>(ragged ? K : 64), static_cast<cuuint64_t>(rows), 1, 1, 1};
    cuuint64_t strides[4] = {row_bytes, 0, 0, 0};
    cuuint32_t box[5] = {64, static_cast<cuuint32_t>(box_rows), 1, 1, 1};
    const cuuint32_t es[5] = {1, 1, 1, 1, 1};
    cuuint32_t rank = 2;
    if (pair_rows > 0) {
        dims[1] = static_cast<cuuint64_t>(pair_rows); dims[2] = 2;
        strides[1] = row_bytes * pair_rows;
        box[2] = 2;
        rank = 3;
        if (grouped) {
            dims[3] = static_cast<cuuint64_t>(rows / (2 * pair_rows));
            strides[2] = row_bytes * pair_rows * 2;
            rank = 4;
        }
    }
    if (!ragged) {
        dims[rank] = static_cast<cuuint64_t>(K / 64);
        strides[rank - 1] = 128;
        box[rank] = MK_TILE_COLS / 64;
        ++rank;
    }
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void *>(base), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace edgefm
