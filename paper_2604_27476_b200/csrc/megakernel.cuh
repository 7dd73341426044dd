// The whole decode step as ONE persistent cooperative kernel (one CTA per SM).
//
// Why: at batch 1 a layer of a 1.5B-parameter decoder is ~94 MB of weights, i.e. ~14 us of HBM time,
// split over five operators that depend on one another.  Separate kernels drain and refill the memory
// pipeline at every boundary.  Here the weight stream is decoupled from the dependency chain:
//
//   * The step's weight traffic is a static schedule (QKV, O, gate/up, down of every layer, then
//     lm_head).  Every CTA owns a fixed share of each operator's rows, and every warp of the CTA a fixed
//     sequence of tiles (a few rows, or one K slice of a long row) across the WHOLE step.
//   * Each warp keeps a private byte ring in shared memory filled with its next tiles (up to MK_MAXF in
//     flight, variable size, allocated first-in first-out) by bulk async copies (TMA: cp.async.bulk +
//     mbarrier complete_tx).  When it has consumed a tile it immediately fetches as many further tiles
//     as now fit -- regardless of operator boundaries -- so the short operators of a layer are already
//     on chip when their turn comes, and HBM keeps streaming while the arithmetic waits at a grid
//     barrier, stages an activation vector or runs attention.
//     Ring space and mbarriers are armed and drained by the same warp, in program order, so the one-bit
//     mbarrier phase parity cannot alias and no "empty" barrier is needed (a proxy fence orders the
//     warp's reads before the next asynchronous write).
//   * A tile is multiplied with the activation vector staged in shared memory; the fused epilogues
//     (bias + RoPE + KV append, residual add, SwiGLU, logits + argmax) run in the warp that owns the rows.
//   * Between dependent operators all CTAs meet at a grid barrier (monotonic counter in global memory,
//     release/acquire, bounded spin).  Attention (split-KV, exact log-sum-exp merge) runs between two
//     barriers.
//
// Every wait is bounded: on expiry the CTA records EDGEFM_ERR_TIMEOUT in the device state, stops
// issuing copies, waits (bounded) for the copies it has in flight and returns.
// This file is the body of the kernel.  It is included once per build (MK_NS = namespace, MK_NW_VALUE = warps per
// CTA); everything that does not depend on the number of warps lives in megakernel_types.cuh.
#include "megakernel_types.cuh"

namespace edgefm {
namespace MK_NS {

constexpr int MK_NW = MK_NW_VALUE;               // warps per CTA (each streams and consumes its own tiles)
constexpr int MK_NT = MK_NW * 32;
constexpr int MK_ATT_MW = (MK_NW + 1) / 2;       // warps whose partials fit the merge area at once

// Optional fine-grained trace of one operator in CTA 0 (compile with -DEDGEFM_TRACE_PHASE=<operator index>):
// lane 0 of every warp appends %globaltimer stamps behind the regular profile table.
#ifndef MK_TRACE
#ifdef EDGEFM_TRACE_PHASE
#define MK_TRACE(p, ph, warp, lane, slot)                                                                          \
    do {                                                                                                           \
        if ((p).prof && (ph) == EDGEFM_TRACE_PHASE && blockIdx.x == 0 && (lane) == 0 && (slot) < 16)               \
            (p).prof[static_cast<size_t>(gridDim.x) * (p).prof_stride + (warp) * 16 + (slot)] = global_ns();        \
    } while (0)
#else
#define MK_TRACE(p, ph, warp, lane, slot) do {} while (0)
#endif
#endif  // MK_TRACE

// 1: one-head-per-CTA attention leaves the merge of its chunks to the O projection's prologue (every CTA merges);
// 0: the last CTA of every head merges (atomic ticket) and the O projection stages the finished vector
#ifndef MK_SPLIT_DEFER
#define MK_SPLIT_DEFER 1
#endif

// ---- mbarrier / bulk copy primitives -----------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void *p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(unsigned long long *b, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long *b, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long *b, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(b)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait (limit in nanoseconds); false = gave up (or another thread of the CTA already did).
__device__ __forceinline__ bool mbar_wait(unsigned long long *b, unsigned parity, volatile int *abort_flag, unsigned limit_ns) {
    if (mbar_try_wait(b, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (unsigned it = 1;; ++it) {
        if (mbar_try_wait(b, parity)) return true;
        if ((it & 31u) == 0u) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > limit_ns) break;
        }
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void bulk_copy_g2s(void *dst, const void *src, unsigned bytes, unsigned long long *bar,
                                              unsigned long long policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void bulk_copy_g2s_plain(void *dst, const void *src, unsigned bytes, unsigned long long *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void cta_sync() { __syncthreads(); }

__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned *p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Diagnostics: thread 0 of every CTA records %globaltimer at fixed points of the step.
__device__ __forceinline__ void prof_stamp(const MkParams &p, int tid, int &idx) {
    if (p.prof && tid == 0) {
        if (idx < p.prof_stride) p.prof[static_cast<size_t>(blockIdx.x) * p.prof_stride + idx] = global_ns();
        ++idx;
    }
}

// Self-check: record the first violated bound (status 100 + code, two operands) instead of touching memory.
__device__ __forceinline__ bool diag_fail(const MkParams &p, volatile int *abort_flag, int code, long long a, long long b) {
    if (atomicCAS(&p.state->status, 0, 100 + code) == 0) {
        p.state->pad[0] = static_cast<int>(a);
        p.state->pad[1] = static_cast<int>(b);
    }
    *abort_flag = 1;
    return false;
}

// All threads of all CTAs meet here.  Returns false when the wait expired (step aborted).
// While the CTA waits, every warp tops up its weight ring (the fetches short operators skipped).
template <typename Refill>
__device__ __forceinline__ bool grid_barrier(const MkParams &p, unsigned target, volatile int *abort_flag, volatile int *s_released,
                                             int tid, int &prof_idx, Refill &&refill_fn) {
    cta_sync();
    prof_stamp(p, tid, prof_idx);   // this CTA's share of the operator is done
    if (tid == 0 && !*abort_flag) {
        *s_released = 0;
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.barrier) : "memory");
    }
    refill_fn();
    // lane 0 of the first MK_BAR_POLLERS warps polls the counter; their polls interleave in time, which shortens the
    // delay between the last arrival and its detection; whoever sees it first releases the others
    if ((tid & 31) == 0 && (tid >> 5) < MK_BAR_POLLERS && !*abort_flag) {
        unsigned it = 0;
        unsigned long long t0 = 0;
        while (ld_acquire_gpu(p.barrier) < target) {
            if (*s_released) break;
            if ((++it & 63u) == 0u) {
                const unsigned long long now = global_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > p.spin_limit) { *abort_flag = 1; p.state->status = 6; break; }
            }
        }
        *s_released = 1;
    }
    cta_sync();
    prof_stamp(p, tid, prof_idx);   // released by the slowest CTA
    return !*abort_flag;
}

// Work items [it0, it1) of CTA `cta` in a phase with `total` items.
__device__ __forceinline__ void item_range(int total, int cta, int ncta, int &it0, int &it1) {
    it0 = static_cast<int>((static_cast<long long>(total) * cta) / ncta);
    it1 = static_cast<int>((static_cast<long long>(total) * (cta + 1)) / ncta);
}

// First row of block `blk` (0 = low/plain, 1 = partner rows) of item `it`, and the number of valid units.
__device__ __forceinline__ int item_rows(const MkPhase &P, const MkParams &p, int it, int blk, int &cnt) {
    const int u0 = it * P.rw;
    cnt = min(P.rw, P.units_total - u0);
    if (P.kind == PH_QKV) {
        const int half = p.d >> 1;
        const int head = u0 >> p.half_shift, i0 = u0 & (half - 1);
        return head * p.d + i0 + blk * half;
    }
    if (P.kind == PH_SWIGLU) return u0 + blk * p.F;
    return u0;
}

// ---- a warp's position in its tile sequence over the whole step ----------------------------------------
// Tile j of a CTA's share of an operator is slice (j & (ksplit-1)) of item (j >> s_shift); warp w owns the
// tiles j = w, w + NW, ...  The CTA's item range of every operator is tabulated once per launch (s_rng).
// The cursor keeps the constants of its operator in registers so that issuing a tile costs no shared-memory
// round trips.
struct TileCursor {
    int ph;        // operator index (nph = past the end)
    int j;         // tile index inside this CTA's share of the operator
    int it0;       // first item of this CTA in operator ph
    int n_tiles;   // tiles of this CTA in operator ph
    // cached from s_ph[ph]
    const uint16_t *W;
    int K, rw, s_shift, smask, units_total, kind;
    unsigned seg_bytes;      // bytes of one row slice
    unsigned alloc_bytes;    // ring bytes of one tile
    unsigned partner_elems;  // elements between the two blocks of a paired tile (0: single block)
};
__device__ __forceinline__ void cursor_enter_phase(TileCursor &c, const MkParams &p, const MkPhase *s_ph, const int2 *s_rng, int warp) {
    while (c.ph < p.nph) {  // skip operators in which this warp owns no tile
        const MkPhase &P = s_ph[c.ph];
        const int2 r = s_rng[c.ph];
        c.it0 = r.x;
        c.n_tiles = (r.y - r.x) << P.s_shift;
        if (warp < c.n_tiles) {
            c.j = warp;
            c.W = P.W; c.K = P.K; c.rw = P.rw; c.s_shift = P.s_shift; c.smask = P.ksplit - 1; c.units_total = P.units_total;
            c.kind = P.kind;
            c.seg_bytes = static_cast<unsigned>(P.kcs) * 16u;
            const bool paired = P.kind == PH_QKV || P.kind == PH_SWIGLU;
            c.alloc_bytes = (paired ? 2u : 1u) * P.rw * c.seg_bytes;
            c.partner_elems = !paired ? 0u : static_cast<unsigned>(P.kind == PH_QKV ? (p.d >> 1) : p.F) * static_cast<unsigned>(P.K);
            return;
        }
        ++c.ph;
    }
}
__device__ __forceinline__ void cursor_advance(TileCursor &c, const MkParams &p, const MkPhase *s_ph, const int2 *s_rng, int warp) {
    c.j += MK_NW;
    if (c.j < c.n_tiles) return;
    ++c.ph;
    cursor_enter_phase(c, p, s_ph, s_rng, warp);
}

// Fetch the tile under cursor `c` into ring space.  Called by a whole warp after __syncwarp(); lane 0 issues.
__device__ __forceinline__ bool issue_tile(const MkParams &p, const TileCursor &c, unsigned char *dst, unsigned long long *bar,
                                           unsigned long long policy, volatile int *abort_flag, int lane) {
    const int it = c.it0 + (c.j >> c.s_shift);
    const int sl = c.j & c.smask;
    const int u0 = it * c.rw;
    const int cnt = min(c.rw, c.units_total - u0);
    int row_lo = u0;
    if (c.kind == PH_QKV) {
        const int half = p.d >> 1;
        row_lo = (u0 >> p.half_shift) * p.d + (u0 & (half - 1));
    }
    const unsigned bytes = static_cast<unsigned>(cnt) * c.seg_bytes;   // one contiguous run per block
    // bounds: at least one row, inside the matrix (16-byte rule holds by construction: K % 8 == 0, slices of
    // kcs 16-byte pieces, 16-byte aligned bases and ring offsets, all checked on the host)
    if (cnt < 1 || (sl + 1) * static_cast<int>(c.seg_bytes >> 1) > c.K) return diag_fail(p, abort_flag, 1, c.ph, it);
    if (lane == 0) {
        const uint16_t *src = c.W + static_cast<size_t>(row_lo) * c.K + static_cast<size_t>(sl) * (c.seg_bytes >> 1);
        if (c.partner_elems) {
            mbar_arrive_expect_tx(bar, bytes * 2u);
            bulk_copy_g2s(dst, src, bytes, bar, policy);
            bulk_copy_g2s(dst + static_cast<size_t>(c.rw) * c.seg_bytes, src + c.partner_elems, bytes, bar, policy);
        } else {
            mbar_arrive_expect_tx(bar, bytes);
            bulk_copy_g2s(dst, src, bytes, bar, policy);
        }
    }
    return true;
}

// Per-warp streaming state.
struct WarpStream {
    TileCursor pf;            // next tile to fetch into shared memory
    unsigned consumed;        // tiles consumed so far by this warp
    unsigned issued;          // tiles fetched so far (issued - consumed <= MK_MAXF)
    unsigned char *ring;      // this warp's byte ring
    int head, tail;           // ring offsets: [head, tail) (cyclically) holds the tiles in flight
    bool wrapped;             // tail has wrapped around the ring end and head has not yet
    unsigned long long fifo;  // ring offset / 16 of tile k in the 16-bit field k % MK_MAXF
    unsigned long long *bars; // [MK_MAXF]
    unsigned long long policy;
};
static_assert(MK_MAXF == 4, "fifo packs four 16-bit offsets into one register");
__device__ __forceinline__ int fifo_get(const WarpStream &ws, unsigned k) {
    return static_cast<int>((ws.fifo >> ((k & 3u) * 16u)) & 0xffffull) << 4;
}
__device__ __forceinline__ void fifo_set(WarpStream &ws, unsigned k, int off) {
    const unsigned sh = (k & 3u) * 16u;
    ws.fifo = (ws.fifo & ~(0xffffull << sh)) | (static_cast<unsigned long long>(off >> 4) << sh);
}

// Fetch as many of this warp's next tiles as fit its ring (first-in first-out space, at most MK_MAXF in
// flight).  Whole warp, after __syncwarp() when ring space has just been read.
__device__ __forceinline__ bool refill(const MkParams &p, const MkPhase *s_ph, const int2 *s_rng, WarpStream &ws,
                                       volatile int *abort_flag, int warp, int lane) {
    bool fenced = false;
    while (ws.issued - ws.consumed < MK_MAXF && ws.pf.ph < p.nph) {
        const int sz = static_cast<int>(ws.pf.alloc_bytes);
        if (ws.issued == ws.consumed) { ws.head = 0; ws.tail = 0; ws.wrapped = false; }   // empty: restart at the base
        int off;
        if (!ws.wrapped) {                   // in flight: [head, tail); free: [tail, R) and [0, head)
            if (ws.tail + sz <= p.ring_bytes) off = ws.tail;
            else if (sz <= ws.head) { off = 0; ws.wrapped = true; }   // wrap (the bytes behind tail stay unused this round)
            else break;
        } else {                              // in flight: [head, R) and [0, tail); free: [tail, head)
            if (ws.tail + sz <= ws.head) off = ws.tail;
            else break;
        }
        if (!fenced) {
            // ring space was read through the generic proxy by this warp: order those reads before async writes
            if (lane == 0) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            fenced = true;
        }
        if (!issue_tile(p, ws.pf, ws.ring + off, &ws.bars[ws.issued & (MK_MAXF - 1)], ws.policy, abort_flag, lane)) return false;
        fifo_set(ws, ws.issued, off);
        ws.tail = off + sz;
        ++ws.issued;
        cursor_advance(ws.pf, p, s_ph, s_rng, warp);
    }
    return true;
}

struct ItemCtx {
    float rscale;          // deferred RMSNorm factor (1 for plain prologues)
    int slot_row;          // cache slot written by this step
    const float *rope;     // smem cos[d/2], sin[d/2]
    float best_v;          // PH_LMHEAD running argmax of this lane
    int best_i;
    float *logits_out;
};

// ---- fused epilogue of one output unit (a row, or a row pair) ------------------------------------------------
// pre: the value the epilogue adds (old residual / the two biases) was fetched ahead into pre_lo, pre_hi.
__device__ __forceinline__ void apply_epilogue(const MkParams &p, const MkPhase &P, ItemCtx &cx, int u, float lo, float hi,
                                               bool pre = false, float pre_lo = 0.f, float pre_hi = 0.f) {
    if (P.kind == PH_RESID) {
        P.out[u] = (pre ? pre_lo : __ldcg(P.out + u)) + lo;
    } else if (P.kind == PH_LMHEAD) {
        if (cx.logits_out) cx.logits_out[u] = lo;
        if (arg_better(lo, u, cx.best_v, cx.best_i)) { cx.best_v = lo; cx.best_i = u; }
    } else if (P.kind == PH_SWIGLU) {
        const float a = lo / (1.f + expf(-lo)) * hi;
        if (P.flags & PHF_OUT_SPLIT) {   // the layout the next operator's prologue copies straight into shared memory
            const int i4 = u >> 2;
            P.out[(i4 & 1) * (P.units_total >> 1) + ((i4 >> 1) << 2) + (u & 3)] = a;
        } else {
            P.out[u] = a;
        }
    } else {  // PH_QKV: bias, rotate-half RoPE of q and k, q to the work buffer, k and v to the cache row of this step
        const int half = p.d >> 1;
        const int head = u >> p.half_shift, i = u & (half - 1);
        const int row_lo = head * p.d + i, row_hi = row_lo + half;
        if (P.bias) {
            lo += pre ? pre_lo : bf16_bits_to_f32(P.bias[row_lo]);
            hi += pre ? pre_hi : bf16_bits_to_f32(P.bias[row_hi]);
        }
        const size_t layer_off = static_cast<size_t>(P.layer) * p.nkv * p.max_context * p.d;
        if (head < p.nq + p.nkv) {
            const float c = cx.rope[i], sn = cx.rope[half + i];
            const float rlo = lo * c - hi * sn, rhi = hi * c + lo * sn;
            if (head < p.nq) {
                P.out[row_lo] = rlo;
                P.out[row_hi] = rhi;
            } else {
                uint16_t *dst = p.k_cache + layer_off + (static_cast<size_t>(head - p.nq) * p.max_context + cx.slot_row) * p.d;
                dst[i] = f32_to_bf16_bits(rlo);
                dst[i + half] = f32_to_bf16_bits(rhi);
            }
        } else {
            uint16_t *dst = p.v_cache + layer_off + (static_cast<size_t>(head - p.nq - p.nkv) * p.max_context + cx.slot_row) * p.d;
            dst[i] = f32_to_bf16_bits(lo);
            dst[i + half] = f32_to_bf16_bits(hi);
        }
    }
}

// ---- one tile (NR row slices of kcs 16-byte pieces) by one warp: wait, multiply, re-arm the slot ------------
template <int NR>
__device__ __forceinline__ bool consume_tile(const MkParams &p, const MkPhase *s_ph, const int2 *s_rng, int kcs, int slice, bool do_refill,
                                             WarpStream &ws, const float4 *xsA, const float4 *xsB, volatile int *abort_flag,
                                             float (&out)[NR], int warp, int lane) {
    float acc[NR], acc2[NR];   // two chains per row halve the dependent-FMA latency
#pragma unroll
    for (int r = 0; r < NR; ++r) { acc[r] = 0.f; acc2[r] = 0.f; }
    if (ws.consumed == ws.issued) {   // not fetched yet (short operator whose tiles exceed the ring): fetch on demand
        __syncwarp();
        if (!refill(p, s_ph, s_rng, ws, abort_flag, warp, lane)) return false;
        if (ws.consumed == ws.issued) return diag_fail(p, abort_flag, 2, kcs, NR);
    }
    const unsigned q = ws.consumed & (MK_MAXF - 1);
    const unsigned par = (ws.consumed / MK_MAXF) & 1u;
    if (!mbar_wait(&ws.bars[q], par, abort_flag, p.spin_limit)) return false;
    const uint4 *t = reinterpret_cast<const uint4 *>(ws.ring + fifo_get(ws, ws.consumed));
    const float4 *a = xsA + slice * kcs, *b = xsB + slice * kcs;
    auto fma_chunk = [&](const uint4 &w, const float4 &x0, const float4 &x1, int r) {
        acc[r] = fmaf(bf16lo(w.x), x0.x, acc[r]);  acc2[r] = fmaf(bf16hi(w.x), x0.y, acc2[r]);
        acc[r] = fmaf(bf16lo(w.y), x0.z, acc[r]);  acc2[r] = fmaf(bf16hi(w.y), x0.w, acc2[r]);
        acc[r] = fmaf(bf16lo(w.z), x1.x, acc[r]);  acc2[r] = fmaf(bf16hi(w.z), x1.y, acc2[r]);
        acc[r] = fmaf(bf16lo(w.w), x1.z, acc[r]);  acc2[r] = fmaf(bf16hi(w.w), x1.w, acc2[r]);
    };
    constexpr int UN = NR >= 8 ? 1 : (NR == 4 ? 2 : 3);   // lane-chunks whose loads are issued together
    int c = lane;
    for (; c + 32 * (UN - 1) < kcs; c += 32 * UN) {
        float4 x0[UN], x1[UN];
        uint4 w[UN][NR];
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            x0[u] = a[c + 32 * u]; x1[u] = b[c + 32 * u];
#pragma unroll
            for (int r = 0; r < NR; ++r) w[u][r] = t[r * kcs + c + 32 * u];
        }
#pragma unroll
        for (int u = 0; u < UN; ++u)
#pragma unroll
            for (int r = 0; r < NR; ++r) fma_chunk(w[u][r], x0[u], x1[u], r);
    }
    for (; c < kcs; c += 32) {
        const float4 x0 = a[c], x1 = b[c];
#pragma unroll
        for (int r = 0; r < NR; ++r) fma_chunk(t[r * kcs + c], x0, x1, r);
    }
    ++ws.consumed;
    {   // free the tile's bytes: head moves to the next tile in flight (back to the ring start once it passes the wrap)
        const int nh = ws.consumed < ws.issued ? fifo_get(ws, ws.consumed) : ws.tail;
        if (nh < ws.head) ws.wrapped = false;
        ws.head = nh;
    }
    __syncwarp();
    if (do_refill && !refill(p, s_ph, s_rng, ws, abort_flag, warp, lane)) return false;
#pragma unroll
    for (int r = 0; r < NR; ++r) out[r] = warp_sum(acc[r] + acc2[r]);
    return true;
}

// Tiles of this warp in one operator.  Whole items (ksplit == 1): the warp that owns the rows finishes
// them (lane r = unit r).  Split items: the partial sum of every tile goes to shared memory.
template <int NR>
__device__ __forceinline__ bool consume_tiles(const MkParams &p, const MkPhase *s_ph, const int2 *s_rng, const MkPhase &P, int it0,
                                              int n_tiles, WarpStream &ws, const float4 *xsA, const float4 *xsB,
                                              volatile int *abort_flag, ItemCtx &cx, float *s_partial, int warp, int lane,
                                              int ph_index) {
    int trace_slot = 1;
    // operator constants in registers (the asm memory clobbers would otherwise force shared-memory reloads)
    const int kcs = P.kcs, smask = P.ksplit - 1, rw = P.rw, kind = P.kind, units_total = P.units_total;
    const bool split = P.split != 0;
    if (NR * kcs * 16 > p.slot_bytes || P.ksplit * kcs * 32 > p.xbuf_bytes) return diag_fail(p, abort_flag, 2, kcs, NR);
    // short operators leave the ring alone (it is topped up while the CTA waits at the grid barrier), so that
    // nothing but the arithmetic sits on their critical path; streaming operators refill after every tile
    const bool do_refill = n_tiles > 2 * MK_NW;
    for (int j = warp; j < n_tiles; j += MK_NW) {
        float y[NR];
        MK_TRACE(p, ph_index, warp, lane, trace_slot); ++trace_slot;
        if (!consume_tile<NR>(p, s_ph, s_rng, kcs, j & smask, do_refill, ws, xsA, xsB, abort_flag, y, warp, lane)) return false;
        MK_TRACE(p, ph_index, warp, lane, trace_slot); ++trace_slot;
        // every lane holds all sums of the tile; lane r takes those of unit r, so that the units finish side by side in one
        // pass over one copy of the epilogue code
        const bool paired = kind == PH_QKV || kind == PH_SWIGLU;
        constexpr int NU = NR >= 2 ? NR / 2 : 1;
        float lo = y[0], hi = NR >= 2 ? y[NU] : 0.f;
#pragma unroll
        for (int r = 1; r < NR; ++r) {
            if (lane == r) {
                lo = y[r];
                if (r < NU) hi = y[r + NU];
            }
        }
        if (split) {
            if (lane < NR) s_partial[j * NR + lane] = lo;
        } else {
            const int u = (it0 + j) * rw + lane;
            const int cnt = paired ? NU : NR;
            if ((NR >= 2 || !paired) && lane < cnt && u < units_total) apply_epilogue(p, P, cx, u, lo * cx.rscale, hi * cx.rscale);
        }
    }
    return true;
}

// Attention chunking shared by the attention phase and by the consumer of its partial results.
__device__ __forceinline__ void att_chunking(const MkParams &p, int n, int hg, int min_chunk, int tile, int ncta, int &nch, int &chunk_len) {
    const int groups = p.nq / hg;
    nch = (n + min_chunk - 1) / min_chunk;
    nch = min(nch, min(ncta / groups, p.max_chunks));
    if (hg == 1) nch = min(nch, MK_ATT_SPLIT_MAXC);
    nch = max(nch, 1);
    chunk_len = (n + nch - 1) / nch;
    chunk_len = (chunk_len + tile - 1) / tile * tile;
    nch = (n + chunk_len - 1) / chunk_len;
}

// One weight-streaming operator: prologue (stage the activation vector, RMSNorm folded in: x*w is staged
// and the scalar rsqrt(mean x^2 + eps) is applied to the dot products), then this warp's tiles.
// merge_attn > 0: the input is the attention output, still split into merge_attn chunk partials per head
// (m, l, unnormalised o); the exact log-sum-exp merge is done here, in chunk order, by every CTA.
__device__ __forceinline__ bool gemv_phase(const MkParams &p, const MkPhase *s_ph, const int2 *s_rng, int ph, WarpStream &ws, float4 *xsA,
                                           float4 *xsB, volatile int *abort_flag, float *s_part, float *s_partial, ItemCtx &cx, int token,
                                           int merge_attn, int tid, int &prof_idx, unsigned long long *x_bar, unsigned &x_parity) {
    const MkPhase &P = s_ph[ph];
    const int lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x;
    const int n4 = P.K >> 2;
    float ss = 0.f;
    if (merge_attn > 0) {
        const int nch = merge_attn;
        const int d4 = p.d >> 2;
        float *sm_m = s_partial;                 // [nq][nch] chunk maxima
        float *sm_l = s_partial + p.nq * nch;    // [nq][nch] chunk denominators
        float4 ob[MK_ATT_SPLIT_MAXC];
        auto load_partials = [&](int o4) {
            const int h = o4 / d4, j4 = o4 - h * d4;
            const float4 *po = reinterpret_cast<const float4 *>(p.part_o + static_cast<size_t>(h) * p.max_chunks * p.d) + j4;
#pragma unroll
            for (int c = 0; c < MK_ATT_SPLIT_MAXC; ++c)
                if (c < nch) ob[c] = __ldcg(po + static_cast<size_t>(c) * d4);
        };
        if (tid < n4) load_partials(tid);        // issued before the statistics are waited for
        for (int i = tid; i < p.nq * nch; i += MK_NT) {
            const int h = i / nch, c = i - h * nch;
            sm_m[i] = __ldcg(p.part_m + h * p.max_chunks + c);
            sm_l[i] = __ldcg(p.part_l + h * p.max_chunks + c);
        }
        cta_sync();
        for (int o4 = tid; o4 < n4; o4 += MK_NT) {
            if (o4 != tid) load_partials(o4);
            const int h = o4 / d4;
            const float *hm = sm_m + h * nch, *hl = sm_l + h * nch;
            float mm = -INFINITY;
            for (int c = 0; c < nch; ++c) mm = fmaxf(mm, hm[c]);
            float ll = 0.f;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int c = 0; c < MK_ATT_SPLIT_MAXC; ++c) {
                if (c < nch) {
                    const float e = __expf(hm[c] - mm);
                    ll = fmaf(hl[c], e, ll);
                    acc.x = fmaf(ob[c].x, e, acc.x); acc.y = fmaf(ob[c].y, e, acc.y);
                    acc.z = fmaf(ob[c].z, e, acc.z); acc.w = fmaf(ob[c].w, e, acc.w);
                }
            }
            const float inv = 1.f / ll;
            acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
            if (o4 & 1) xsB[o4 >> 1] = acc; else xsA[o4 >> 1] = acc;
        }
    } else if (P.flags & PHF_X_BULK) {
        // the vector is already in the split layout and needs no transform: two bulk copies, every thread waits for them
        // (the CTA-wide sync of the grid barrier ordered all earlier reads of the buffer before this point)
        if (tid == 0) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            const unsigned half_bytes = static_cast<unsigned>(P.K) * 2u;
            mbar_arrive_expect_tx(x_bar, 2u * half_bytes);
            bulk_copy_g2s_plain(xsA, P.x_src, half_bytes, x_bar);
            bulk_copy_g2s_plain(xsB, P.x_src + (P.K >> 1), half_bytes, x_bar);
        }
        const bool arrived = mbar_wait(x_bar, x_parity, abort_flag, p.spin_limit);
        x_parity ^= 1u;
        if (!arrived && tid == 0) p.state->status = 6;
    } else {
        constexpr int PU = 4;  // loads in flight per thread
        for (int base = tid; base < n4; base += MK_NT * PU) {
            float4 v[PU];
            uint2 w[PU];
#pragma unroll
            for (int u = 0; u < PU; ++u) {
                const int i4 = base + u * MK_NT;
                if (i4 < n4) {
                    if (P.x_src) {
                        v[u] = __ldcg(reinterpret_cast<const float4 *>(P.x_src) + i4);
                    } else {  // first operator of the step: the embedding row is the residual stream
                        const uint2 e = *reinterpret_cast<const uint2 *>(p.embed + static_cast<size_t>(token) * p.H + i4 * 4);
                        v[u] = make_float4(bf16lo(e.x), bf16hi(e.x), bf16lo(e.y), bf16hi(e.y));
                    }
                    if (P.norm_w) w[u] = *reinterpret_cast<const uint2 *>(P.norm_w + i4 * 4);
                }
            }
#pragma unroll
            for (int u = 0; u < PU; ++u) {
                const int i4 = base + u * MK_NT;
                if (i4 < n4) {
                    float4 t = v[u];
                    if (!P.x_src && cta == 0) reinterpret_cast<float4 *>(p.x)[i4] = t;
                    if (P.norm_w) {
                        ss = fmaf(t.x, t.x, ss); ss = fmaf(t.y, t.y, ss); ss = fmaf(t.z, t.z, ss); ss = fmaf(t.w, t.w, ss);
                        t.x *= bf16lo(w[u].x); t.y *= bf16hi(w[u].x); t.z *= bf16lo(w[u].y); t.w *= bf16hi(w[u].y);
                    }
                    if (i4 & 1) xsB[i4 >> 1] = t; else xsA[i4 >> 1] = t;
                }
            }
        }
    }
    if (P.norm_w) {
        ss = warp_sum(ss);
        if (lane == 0) s_part[warp] = ss;
    }
    cta_sync();
    prof_stamp(p, tid, prof_idx);   // activation vector staged
    cx.rscale = 1.f;
    if (P.norm_w) {
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < MK_NW; ++w) tot += s_part[w];
        cx.rscale = rsqrtf(tot / static_cast<float>(P.K) + p.eps);
    }
    MK_TRACE(p, ph, warp, lane, 0);
    const int2 rng = s_rng[ph];
    const int n_items = rng.y - rng.x;
    const int n_tiles = n_items << P.s_shift;
    const bool paired = P.kind == PH_QKV || P.kind == PH_SWIGLU;
    // split operators: thread u finishes unit u after the tiles; fetch what its epilogue adds (old residual
    // value, bias) now, so that the load latency overlaps the arithmetic
    float pre_lo = 0.f, pre_hi = 0.f;
    if (P.split && tid < n_items) {
        const int u = rng.x + tid;
        if (P.kind == PH_RESID) {
            pre_lo = __ldcg(P.out + u);
        } else if (P.kind == PH_QKV && P.bias) {
            const int half = p.d >> 1;
            const int row_lo = (u >> p.half_shift) * p.d + (u & (half - 1));
            pre_lo = bf16_bits_to_f32(P.bias[row_lo]);
            pre_hi = bf16_bits_to_f32(P.bias[row_lo + half]);
        }
    }
    const int nr = paired ? 2 * P.rw : P.rw;
    bool ok;
    switch (nr) {
        case 1: ok = consume_tiles<1>(p, s_ph, s_rng, P, rng.x, n_tiles, ws, xsA, xsB, abort_flag, cx, s_partial, warp, lane, ph); break;
        case 2: ok = consume_tiles<2>(p, s_ph, s_rng, P, rng.x, n_tiles, ws, xsA, xsB, abort_flag, cx, s_partial, warp, lane, ph); break;
        case 4: ok = consume_tiles<4>(p, s_ph, s_rng, P, rng.x, n_tiles, ws, xsA, xsB, abort_flag, cx, s_partial, warp, lane, ph); break;
        default: ok = consume_tiles<8>(p, s_ph, s_rng, P, rng.x, n_tiles, ws, xsA, xsB, abort_flag, cx, s_partial, warp, lane, ph); break;
    }
    MK_TRACE(p, ph, warp, lane, 12);
    if (P.split) {
        // partial sums of the K slices meet here; thread u finishes unit u of this CTA (rw == 1), slices in order
        cta_sync();
        MK_TRACE(p, ph, warp, lane, 13);
        if (!*abort_flag) {
            for (int u = tid; u < n_items; u += MK_NT) {
                float lo = 0.f, hi = 0.f;
                for (int sl = 0; sl < P.ksplit; ++sl) {
                    const int j = (u << P.s_shift) + sl;
                    if (paired) { lo += s_partial[2 * j]; hi += s_partial[2 * j + 1]; } else { lo += s_partial[j]; }
                }
                const bool pre = u == tid;   // operands fetched ahead (first MK_NT units)
                apply_epilogue(p, P, cx, rng.x + u, lo * cx.rscale, hi * cx.rscale, pre, pre_lo, pre_hi);
            }
        }
        MK_TRACE(p, ph, warp, lane, 14);
    }
    return ok;
}

// The attention output vector (n4 16-byte pieces) is stored as [even pieces | odd pieces], the layout of the shared-memory
// activation buffers, so that the O projection stages it with two bulk copies.
__device__ __forceinline__ int split_piece(int i4, int n4) { return (i4 & 1) * (n4 >> 1) + (i4 >> 1); }

// ---- attention -----------------------------------------------------------------------------------------------
// A CTA serves HG query heads of one GQA group over one chunk of the cached positions: HG = G (the whole
// group shares every K/V row read: least traffic, for long contexts) or HG = 1 (every query head has
// its own CTAs: G times more parallelism for short, latency-bound contexts; K/V re-reads hit L2).
// Scores: MK_ATT_LPP lanes per position, each lane reads interleaved 16-byte pieces of the K row from
// global memory; P V: every lane owns d/32 dims.  Shared memory (the idle activation buffer): q,
// probabilities, warp merge area, chunk statistics.  The CTA that arrives last for its head group
// (atomic ticket, no waiting) merges the chunks exactly:  m = max m_c, l = sum l_c e^{m_c - m},
// o = sum o_c e^{m_c - m} / l, in index order.
template <int D, int HG, int LPP>
__device__ __forceinline__ void attention_phase(const MkParams &p, int layer, int n, int min_chunk, bool defer_merge,
                                                unsigned char *xbuf, int tid, int *s_flag) {
    constexpr int TILE = 32 / LPP;   // positions per warp iteration
    constexpr int DV = D / 32, CPR = D / 8, CPL = CPR / LPP;
    constexpr int MW = MK_ATT_MW;
    const int lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x, ncta = gridDim.x;
    const int G = p.nq / p.nkv;
    const int groups = p.nq / HG;                       // head groups served by separate CTAs
    int nch, chunk_len;
    att_chunking(p, n, HG, min_chunk, TILE, ncta, nch, chunk_len);
    if (cta >= nch * groups) return;
    const int grp = cta / nch, c = cta - grp * nch;
    const int qh0 = grp * HG;                            // first query head of this CTA
    const int g = qh0 / G;                               // its kv head
    const int t0 = c * chunk_len, t1 = min(n, t0 + chunk_len);

    float *qs = reinterpret_cast<float *>(xbuf);               // [HG][D]
    float *ps = qs + HG * D;                                    // [NW][HG][TILE]
    float *mg_m = ps + MK_NW * HG * TILE;                       // [MW][HG]
    float *mg_l = mg_m + MW * HG;                               // [MW][HG]
    float *mg_o = mg_l + MW * HG;                               // [MW][HG][D]
    float *cm = mg_o + MW * HG * D;                             // [HG][max_chunks] chunk maxima
    float *cl = cm + HG * p.max_chunks;                         // [HG][max_chunks] chunk denominators

    for (int i = tid; i < HG * D; i += MK_NT) qs[i] = __ldcg(p.q + static_cast<size_t>(qh0) * D + i) * p.scale;
    cta_sync();

    const size_t head_off = (static_cast<size_t>(layer) * p.nkv + g) * p.max_context * D;
    const uint16_t *kg = p.k_cache + head_off;
    const uint16_t *vg = p.v_cache + head_off;
    float *pw = ps + warp * (HG * TILE);
    const int pi = lane / LPP, part = lane % LPP;

    float m[HG], l[HG], o[HG][DV];
#pragma unroll
    for (int h = 0; h < HG; ++h) {
        m[h] = -INFINITY; l[h] = 0.f;
#pragma unroll
        for (int e = 0; e < DV; ++e) o[h][e] = 0.f;
    }

    for (int tt = t0 + warp * TILE; tt < t1; tt += MK_NW * TILE) {
        const bool pvalid = tt + pi < t1;
        uint4 kk[CPL];
#pragma unroll
        for (int j = 0; j < CPL; ++j)
            kk[j] = pvalid ? __ldcg(reinterpret_cast<const uint4 *>(kg + static_cast<size_t>(tt + pi) * D) + j * LPP + part)
                           : make_uint4(0, 0, 0, 0);
        // V rows of the tile, raw bf16 pairs (converted when used to keep the register footprint small)
        uint32_t vraw[TILE][DV / 2];
#pragma unroll
        for (int x = 0; x < TILE; ++x) {
            const int t = tt + x;
            const uint16_t *vp = vg + static_cast<size_t>(t) * D + lane * DV;
            if constexpr (DV == 4) {
                const uint2 w = t < t1 ? __ldcg(reinterpret_cast<const uint2 *>(vp)) : make_uint2(0u, 0u);
                vraw[x][0] = w.x; vraw[x][1] = w.y;
            } else {
                vraw[x][0] = t < t1 ? __ldcg(reinterpret_cast<const unsigned *>(vp)) : 0u;
            }
        }
        float s[HG];
#pragma unroll
        for (int h = 0; h < HG; ++h) s[h] = 0.f;
#pragma unroll
        for (int j = 0; j < CPL; ++j) {
            const int cc = j * LPP + part;
#pragma unroll
            for (int h = 0; h < HG; ++h) {
                const float4 q0 = *reinterpret_cast<const float4 *>(qs + h * D + cc * 8);
                const float4 q1 = *reinterpret_cast<const float4 *>(qs + h * D + cc * 8 + 4);
                s[h] = dot8(kk[j], q0, q1, s[h]);
            }
        }
#pragma unroll
        for (int h = 0; h < HG; ++h) {
#pragma unroll
            for (int x = 1; x < LPP; x <<= 1) s[h] += __shfl_xor_sync(0xffffffffu, s[h], x);
            if (!pvalid) s[h] = -INFINITY;
            const float mn = fmaxf(m[h], warp_max(s[h]));
            const float corr = __expf(m[h] - mn);
            const float pr = pvalid ? __expf(s[h] - mn) : 0.f;
            l[h] = l[h] * corr + (part == 0 ? pr : 0.f);
#pragma unroll
            for (int e = 0; e < DV; ++e) o[h][e] *= corr;
            m[h] = mn;
            if (part == 0) pw[h * TILE + pi] = pr;
        }
        __syncwarp();
#pragma unroll
        for (int tb = 0; tb < TILE; tb += 4) {
            float v[4][DV];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
#pragma unroll
                for (int e = 0; e < DV; e += 2) {
                    v[x][e] = bf16lo(vraw[tb + x][e / 2]);
                    v[x][e + 1] = bf16hi(vraw[tb + x][e / 2]);
                }
            }
#pragma unroll
            for (int h = 0; h < HG; ++h) {
                const float4 p4 = *reinterpret_cast<const float4 *>(pw + h * TILE + tb);
#pragma unroll
                for (int e = 0; e < DV; ++e) {
                    o[h][e] = fmaf(p4.x, v[0][e], o[h][e]);
                    o[h][e] = fmaf(p4.y, v[1][e], o[h][e]);
                    o[h][e] = fmaf(p4.z, v[2][e], o[h][e]);
                    o[h][e] = fmaf(p4.w, v[3][e], o[h][e]);
                }
            }
        }
        __syncwarp();
    }

    // merge the warps of the CTA in two passes through a merge area of MW entries (idle warps carry
    // m = -inf and weigh 0): upper warps publish, lower warps fold them in, then publish themselves.
    float lt[HG];
#pragma unroll
    for (int h = 0; h < HG; ++h) lt[h] = warp_sum(l[h]);
    if (warp >= MW) {
        const int u = warp - MW;
#pragma unroll
        for (int h = 0; h < HG; ++h) {
            if (lane == 0) { mg_m[u * HG + h] = m[h]; mg_l[u * HG + h] = lt[h]; }
#pragma unroll
            for (int e = 0; e < DV; ++e) mg_o[(u * HG + h) * D + lane * DV + e] = o[h][e];
        }
    }
    cta_sync();
    if (warp < MK_NW - MW) {
#pragma unroll
        for (int h = 0; h < HG; ++h) {
            const float m2 = mg_m[warp * HG + h], l2 = mg_l[warp * HG + h];
            const float mn = fmaxf(m[h], m2);
            const float e1 = m[h] == mn ? 1.f : __expf(m[h] - mn);
            const float e2 = m2 == mn ? 1.f : __expf(m2 - mn);
            lt[h] = lt[h] * e1 + l2 * e2;
#pragma unroll
            for (int e = 0; e < DV; ++e) o[h][e] = o[h][e] * e1 + mg_o[(warp * HG + h) * D + lane * DV + e] * e2;
            m[h] = mn;
        }
    }
    cta_sync();
    if (warp < MW) {
#pragma unroll
        for (int h = 0; h < HG; ++h) {
            if (lane == 0) { mg_m[warp * HG + h] = m[h]; mg_l[warp * HG + h] = lt[h]; }
#pragma unroll
            for (int e = 0; e < DV; ++e) mg_o[(warp * HG + h) * D + lane * DV + e] = o[h][e];
        }
    }
    cta_sync();
    for (int i = tid; i < HG * D; i += MK_NT) {
        const int h = i / D, j = i - h * D;
        float mm = -INFINITY;
#pragma unroll
        for (int w = 0; w < MW; ++w) mm = fmaxf(mm, mg_m[w * HG + h]);
        float ll = 0.f, oo = 0.f;
#pragma unroll
        for (int w = 0; w < MW; ++w) {
            const float e = __expf(mg_m[w * HG + h] - mm);
            ll = fmaf(mg_l[w * HG + h], e, ll);
            oo = fmaf(mg_o[(w * HG + h) * D + j], e, oo);
        }
        const int qh = qh0 + h;
        if (nch == 1 && !defer_merge) {  // nothing to merge across CTAs
            p.attn[split_piece((qh * D + j) >> 2, (p.nq * D) >> 2) * 4 + (j & 3)] = oo / ll;
        } else {
            p.part_o[(static_cast<size_t>(qh) * p.max_chunks + c) * D + j] = oo;
            if (j == 0) { p.part_m[qh * p.max_chunks + c] = mm; p.part_l[qh * p.max_chunks + c] = ll; }
        }
    }
    if (nch == 1 || defer_merge) return;   // deferred: the next operator's prologue merges the chunks
    __threadfence();
    cta_sync();
    if (tid == 0) *s_flag = (atomicAdd(p.tickets + grp, 1u) == static_cast<unsigned>(nch - 1)) ? 1 : 0;
    cta_sync();
    if (!*s_flag) return;

    // Last CTA of this head group: merge the chunks.  All loads of a batch (chunk statistics and up to
    // CB partial vectors per thread) are issued before any is used.
    __threadfence();
    constexpr int CB = 8;
    const bool has_out = tid < HG * D / 4;       // output (h, j4) of this thread, if any
    const int oh = has_out ? tid / (D / 4) : 0, oj4 = has_out ? tid - oh * (D / 4) : 0;
    const float4 *po = reinterpret_cast<const float4 *>(p.part_o + static_cast<size_t>(qh0 + oh) * p.max_chunks * D) + oj4;
    float4 ob[CB];
#pragma unroll
    for (int u = 0; u < CB; ++u)
        ob[u] = (has_out && u < nch) ? __ldcg(po + static_cast<size_t>(u) * (D / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
    for (int i = tid; i < HG * nch; i += MK_NT) {
        const int h = i / nch, cc = i - h * nch;
        cm[h * p.max_chunks + cc] = __ldcg(p.part_m + (qh0 + h) * p.max_chunks + cc);
        cl[h * p.max_chunks + cc] = __ldcg(p.part_l + (qh0 + h) * p.max_chunks + cc);
    }
    cta_sync();
    if (has_out) {
        const float *hm = cm + oh * p.max_chunks, *hl = cl + oh * p.max_chunks;
        float mm = -INFINITY;
        for (int cc = 0; cc < nch; ++cc) mm = fmaxf(mm, hm[cc]);
        float ll = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int c0 = 0; c0 < nch; c0 += CB) {
            if (c0 > 0) {
#pragma unroll
                for (int u = 0; u < CB; ++u)
                    ob[u] = (c0 + u < nch) ? __ldcg(po + static_cast<size_t>(c0 + u) * (D / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < CB; ++u) {
                if (c0 + u < nch) {
                    const float e = __expf(hm[c0 + u] - mm);
                    ll = fmaf(hl[c0 + u], e, ll);
                    acc.x = fmaf(ob[u].x, e, acc.x); acc.y = fmaf(ob[u].y, e, acc.y);
                    acc.z = fmaf(ob[u].z, e, acc.z); acc.w = fmaf(ob[u].w, e, acc.w);
                }
            }
        }
        const float inv = 1.f / ll;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
        reinterpret_cast<float4 *>(p.attn)[split_piece((qh0 + oh) * (D / 4) + oj4, (p.nq * D) >> 2)] = acc;
    }
    if (tid == 0) p.tickets[grp] = 0u;
}

// ---- the kernel -----------------------------------------------------------------------------------------------
// LONG = false: contexts that always run attention with one query head per CTA group (max_context <=
// att_split_max_n); the grouped variant is then not compiled in, which keeps the register footprint of the
// streaming state small.
template <int D, int G, bool LONG>
__global__ void __launch_bounds__(MK_NT, 1) decode_megakernel(const MkParams p) {
    extern __shared__ __align__(128) unsigned char mk_smem[];
    unsigned char *smem = mk_smem;
    float4 *xsA = reinterpret_cast<float4 *>(smem);
    float4 *xsB = reinterpret_cast<float4 *>(smem + p.xbuf_bytes / 2);
    MkPhase *s_ph = reinterpret_cast<MkPhase *>(smem + p.xbuf_bytes);          // the step's schedule
    int2 *s_rng = reinterpret_cast<int2 *>(s_ph + p.nph);                      // this CTA's item range per operator
    unsigned char *ring = smem + p.xbuf_bytes + p.sched_bytes;
    __shared__ __align__(8) unsigned long long full_bar[MK_NW * MK_MAXF];
    __shared__ __align__(8) unsigned long long x_bar;   // completion of bulk-copied activation vectors
    __shared__ float s_rope[128];
    __shared__ float s_part[MK_NW];
    __shared__ float s_partial[MK_PARTIAL_FLOATS];
    __shared__ float s_bv[MK_NW];
    __shared__ int s_bi[MK_NW];
    __shared__ int s_flag;
    __shared__ int s_abort;
    __shared__ int s_released;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x, ncta = gridDim.x;
    if (tid == 0) {
        for (int i = 0; i < MK_NW * MK_MAXF; ++i) mbar_init(&full_bar[i], 1);
        mbar_init(&x_bar, 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    {
        const int n16 = p.nph * static_cast<int>(sizeof(MkPhase) / 16);
        const uint4 *src = reinterpret_cast<const uint4 *>(p.phases);
        uint4 *dst = reinterpret_cast<uint4 *>(s_ph);
        for (int i = tid; i < n16; i += MK_NT) dst[i] = src[i];
        for (int i = tid; i < p.nph; i += MK_NT) {
            int it0, it1;
            item_range(p.phases[i].items_total, cta, ncta, it0, it1);
            s_rng[i] = make_int2(it0, it1);
        }
    }
    __syncthreads();
    volatile int *abort_flag = &s_abort;

    // The small per-layer vectors (norm weights, biases) are read on the critical path right after a grid barrier;
    // ask L2 for all of them now (they stay: the weight stream is evict-first).
    for (int i = cta * MK_NT + tid; i < p.nph * 64; i += ncta * MK_NT) {
        const MkPhase &P = s_ph[i >> 6];
        const int line = i & 63;   // 128-byte line of the vector
        if (P.norm_w && line * 64 < P.K) asm volatile("prefetch.global.L2 [%0];" ::"l"(P.norm_w + line * 64));
        if (P.bias && P.kind == PH_QKV && line * 64 < 2 * P.units_total) asm volatile("prefetch.global.L2 [%0];" ::"l"(P.bias + line * 64));
    }

    // ---- start this warp's weight stream: fill its ring, then run the L2 prefetch ahead ---------------
    WarpStream ws;
    ws.consumed = 0; ws.issued = 0; ws.head = 0; ws.tail = 0; ws.wrapped = false; ws.fifo = 0;
    ws.ring = ring + static_cast<size_t>(warp) * p.ring_bytes;
    ws.bars = &full_bar[warp * MK_MAXF];
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(ws.policy));
    ws.pf.ph = 0;
    cursor_enter_phase(ws.pf, p, s_ph, s_rng, warp);
    bool ok = refill(p, s_ph, s_rng, ws, abort_flag, warp, lane);
    const int rt = p.req->token, rp = p.req->position;
    const int token = rt >= 0 ? rt : p.state->next_token;
    const int pos = rp >= 0 ? rp : p.state->next_position;
    const int slot_row = p.state->cur_len;
    const int half = p.d >> 1;
    if (token < 0 || token >= p.V || slot_row < 0 || slot_row >= p.max_context || pos < 0) {
        if (tid == 0) diag_fail(p, abort_flag, 3, token, slot_row);   // corrupt request/state: compute nothing
        ok = false;
    }
    if (ok && tid < half) {  // rotary table of this step's position; fp64 angle, rounded once
        double sn, cs;
        sincos(static_cast<double>(pos) * p.inv_freq[tid], &sn, &cs);
        s_rope[tid] = static_cast<float>(cs);
        s_rope[half + tid] = static_cast<float>(sn);
    }
    if (ok && cta == 0 && tid == 0) { p.state->token = token; p.state->position = pos; }
    // (s_rope is published by the __syncthreads of the first prologue)

    ItemCtx cx;
    cx.rscale = 1.f; cx.slot_row = slot_row; cx.rope = s_rope; cx.best_v = -INFINITY; cx.best_i = 0x7fffffff;
    cx.logits_out = p.req->logits_out;

    unsigned bar_no = 0;
    unsigned x_parity = 0;
    int prof_idx = 0;
    prof_stamp(p, tid, prof_idx);
    auto top_up = [&]() { __syncwarp(); if (ok && !*abort_flag) refill(p, s_ph, s_rng, ws, abort_flag, warp, lane); };
    const int n_att = slot_row + 1;
    const bool att_split = !LONG || (n_att <= p.att_split_max_n && static_cast<long long>(p.nq) * MK_ATT_SPLIT_MAXC * 2 <= MK_PARTIAL_FLOATS);
    int merge_chunks = 0;   // chunks per head the O-projection prologue has to merge (split mode)
    if (att_split && MK_SPLIT_DEFER) { int cl; att_chunking(p, n_att, 1, p.att_chunk_split, 32 / MK_ATT_LPP_SPLIT, ncta, merge_chunks, cl); }
    // One loop over the operators of the step, with a single inlined copy of the streaming operator and of the grid barrier
    // (the code of a step is executed once per layer: a small instruction footprint matters).  Operator 4l+1 (the O
    // projection) is preceded by the attention of layer l.
    const int n_layer_ops = 4 * p.n_layers;
    for (int ph = 0; ph < p.nph && ok; ++ph) {
        const bool layer_op = ph < n_layer_ops;
        const bool after_attention = layer_op && (ph & 3) == 1;
        if (after_attention) {
            const int l = ph >> 2;
            if constexpr (LONG) {
                if (att_split) attention_phase<D, 1, MK_ATT_LPP_SPLIT>(p, l, n_att, p.att_chunk_split, MK_SPLIT_DEFER != 0, smem, tid, &s_flag);
                else attention_phase<D, G, MK_ATT_LPP>(p, l, n_att, p.att_chunk_shared, false, smem, tid, &s_flag);
            } else {
                attention_phase<D, 1, MK_ATT_LPP_SPLIT>(p, l, n_att, p.att_chunk_split, MK_SPLIT_DEFER != 0, smem, tid, &s_flag);
            }
            ok = grid_barrier(p, ++bar_no * ncta, abort_flag, &s_released, tid, prof_idx, top_up) && ok;
            if (!ok) break;
        }
        ok = gemv_phase(p, s_ph, s_rng, ph, ws, xsA, xsB, abort_flag, s_part, s_partial, cx, token, after_attention ? merge_chunks : 0, tid,
                        prof_idx, &x_bar, x_parity);
        if (layer_op) ok = grid_barrier(p, ++bar_no * ncta, abort_flag, &s_released, tid, prof_idx, top_up) && ok;
    }
    prof_stamp(p, tid, prof_idx);
    if (!ok || *abort_flag) {
        // aborted: wait (bounded) for the copies this warp still has in flight, then leave
        if (tid == 0 && p.state->status == 0) p.state->status = 6;
        for (unsigned k = ws.consumed; k < ws.issued; ++k) {
            const unsigned q = k & (MK_MAXF - 1);
            const unsigned par = (k / MK_MAXF) & 1u;
            const unsigned long long t0 = global_ns();
            while (!mbar_try_wait(&ws.bars[q], par))
                if (global_ns() - t0 > p.spin_limit) break;
        }
        return;
    }

    // ---- greedy sampling: warp -> CTA -> last CTA reduces all partials, then the state advances -------------
    float bv = cx.best_v;
    int bi = cx.best_i;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (arg_better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
    }
    if (lane == 0) { s_bv[warp] = bv; s_bi[warp] = bi; }
    cta_sync();
    if (tid == 0) {
        for (int w = 1; w < MK_NW; ++w)
            if (arg_better(s_bv[w], s_bi[w], bv, bi)) { bv = s_bv[w]; bi = s_bi[w]; }
        p.lm_part_val[cta] = bv;
        p.lm_part_idx[cta] = bi;
        __threadfence();
        s_flag = (atomicAdd(p.tickets + p.nq, 1u) == static_cast<unsigned>(ncta - 1)) ? 1 : 0;
    }
    cta_sync();
    if (!s_flag) return;
    __threadfence();
    if (warp == 0) {
        bv = -INFINITY; bi = 0x7fffffff;
        for (int i = lane; i < ncta; i += 32) {
            const float v = __ldcg(p.lm_part_val + i);
            const int ix = __ldcg(p.lm_part_idx + i);
            if (arg_better(v, ix, bv, bi)) { bv = v; bi = ix; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (arg_better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
        }
        if (lane == 0) {
            if (bi == 0x7fffffff) bi = 0;
            if (s_ph[p.nph - 1].flags & PHF_REMAP) bi = p.vocab_ids[bi];   // pruned vocabulary: row index -> token id
            int *nto = p.req->next_token_out;
            if (nto) *nto = bi;
            p.state->next_token = bi;
            p.state->next_position = pos + 1;
            p.state->cur_len = slot_row + 1;
            p.tickets[p.nq] = 0u;
            *p.barrier = 0u;  // every CTA has passed the last grid barrier
        }
    }
}

}  // namespace MK_NS
}  // namespace edgefm
