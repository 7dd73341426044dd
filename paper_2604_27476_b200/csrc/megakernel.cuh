// The whole decode step as ONE persistent cooperative kernel (one CTA per SM).
//
// Why: at batch 1 a layer of a 1.5B-parameter decoder is ~94 MB of weights, i.e. ~14 us of HBM time,
// split over five operators that depend on one another.  Separate kernels drain and refill the memory
// pipeline at every boundary.  Here the weight stream is decoupled from the dependency chain:
//
//   * a PRODUCER warp per CTA walks the step's static schedule (QKV, O, gate/up, down of every layer,
//     then lm_head) and keeps a ring of shared-memory slots full with bulk async copies (TMA,
//     cp.async.bulk + mbarrier complete_tx) of this CTA's weight tiles.  It never waits for the
//     arithmetic, only for a free slot, so HBM stays busy across operator boundaries and grid barriers;
//   * CONSUMER warps take tiles from the ring (one warp per work item, no intra-tile cross-warp sync),
//     multiply them with the activation vector staged in shared memory, and run the fused epilogues
//     (bias + RoPE + KV append, residual add, SwiGLU, logits + argmax);
//   * between dependent operators the consumers meet at a grid barrier (monotonic counter in global
//     memory, release/acquire, bounded spin).  Attention (split-KV with an exact log-sum-exp merge) runs
//     on the consumer warps between two barriers while the producer prefetches the next operators.
//
// Every wait is bounded: on expiry the CTA records EDGEFM_ERR_TIMEOUT in the device state, stops
// issuing copies, waits (bounded) for the copies it has in flight and returns.
#pragma once
#include "common.cuh"

namespace edgefm {

constexpr int MK_NWC = 15;                       // consumer warps per CTA
constexpr int MK_NTC = MK_NWC * 32;              // consumer threads
constexpr int MK_THREADS = MK_NTC + 32;          // + one producer warp
constexpr int MK_MAX_SLOTS = 32;
constexpr int MK_ATT_LPP = 4;                    // lanes per cached position in the score phase
constexpr int MK_ATT_TILE = 32 / MK_ATT_LPP;     // positions per warp iteration
constexpr int MK_ATT_MW = (MK_NWC + 1) / 2;      // warps whose partials fit the merge area at once

static_assert(2 * MK_NWC <= MK_MAX_SLOTS && MK_MAX_SLOTS <= 32, "one producer lane per ring slot");

enum { PH_QKV = 0, PH_RESID = 1, PH_SWIGLU = 2, PH_LMHEAD = 3 };

// One weight-streaming operator of the step.
struct alignas(16) MkPhase {
    const uint16_t *W;       // bf16 [rows][K]
    const uint16_t *bias;    // PH_QKV: bf16 [rows] or null
    const uint16_t *norm_w;  // RMSNorm weight of the prologue (bf16 [K]) or null = plain copy of x_src
    const float *x_src;      // fp32 [K] input vector in global memory; null = embedding row of the token
    float *out;              // PH_QKV: q fp32; PH_RESID: x (+=); PH_SWIGLU: act; PH_LMHEAD: unused
    int K;                   // columns (multiple of 8)
    int kind;
    int rw;                  // units per work item (rows, or row pairs for PH_QKV / PH_SWIGLU)
    int ksplit;              // K slices per item (tiles per item)
    int kcs;                 // 16-byte pieces per row slice = K / 8 / ksplit
    int units_total;         // rows (PH_RESID, PH_LMHEAD), pairs (PH_QKV: rows/2, PH_SWIGLU: F)
    int items_total;         // ceil(units_total / rw)
    int layer;
    int pad_[3];
};
static_assert(sizeof(MkPhase) % 16 == 0, "descriptor is copied in 16-byte pieces");

struct MkParams {
    const MkPhase *phases;   // [4 * n_layers + 1]
    int n_layers, H, nq, nkv, d, F, V;
    float eps, scale;
    int max_context;
    uint16_t *k_cache, *v_cache;   // [L][nkv][max_context][d]
    const uint16_t *embed;
    const double *inv_freq;        // [d/2]
    float *x, *q, *attn;
    float *part_m, *part_l, *part_o;
    int max_chunks;                // attention chunks per kv head (<= gridDim.x / nkv)
    int att_min_chunk;
    unsigned *tickets;             // [nkv] attention, [nkv] lm_head
    unsigned *barrier;             // grid barrier counter (0 between launches)
    float *lm_part_val;
    int *lm_part_idx;
    StepState *state;
    const StepRequest *req;
    int nslot, slot_bytes, xbuf_bytes, sched_bytes;
    unsigned spin_limit;           // upper bound of every device-side wait, nanoseconds
    unsigned long long *prof;      // optional timestamps [gridDim.x][prof_stride] (diagnostics), or null
    int prof_stride;
};

// ---- mbarrier / bulk copy primitives -----------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void *p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(unsigned long long *b, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long *b) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
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
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(MK_NTC) : "memory"); }

__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned *p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Diagnostics: consumer thread 0 of every CTA records %globaltimer at fixed points of the step.
__device__ __forceinline__ void prof_stamp(const MkParams &p, int tidc, int &idx) {
    if (p.prof && tidc == 0) {
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

// All consumer threads of all CTAs meet here.  Returns false when the wait expired (step aborted).
__device__ __forceinline__ bool grid_barrier(const MkParams &p, unsigned target, volatile int *abort_flag, int tidc, int &prof_idx) {
    consumer_sync();
    prof_stamp(p, tidc, prof_idx);   // this CTA's share of the operator is done
    if (tidc == 0 && !*abort_flag) {
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.barrier) : "memory");
        unsigned it = 0;
        unsigned long long t0 = 0;
        while (ld_acquire_gpu(p.barrier) < target) {
            if ((++it & 63u) == 0u) {
                const unsigned long long now = global_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > p.spin_limit) { *abort_flag = 1; p.state->status = 6; break; }
            }
        }
    }
    consumer_sync();
    prof_stamp(p, tidc, prof_idx);   // released by the slowest CTA
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
        const int head = u0 / half, i0 = u0 - head * half;
        return head * p.d + i0 + blk * half;
    }
    if (P.kind == PH_SWIGLU) return u0 + blk * p.F;
    return u0;
}

// ---- producer: keep the ring full -----------------------------------------------------------------------
// Every consumer warp w has a private sub-ring of `depth` slots (slot = w * depth + q).  Warp w consumes
// its own tiles strictly in order, so a slot is always filled and drained by the same pair of threads
// in alternation: the one-bit mbarrier phase parity can never alias (a warp cannot run a whole ring
// round ahead of a slot it does not own), and a slow warp never blocks the supply of the others.
// Lane (w, q) of the producer warp issues the tiles k = q, q + depth, ... of warp w's tile sequence over
// the whole step; the lanes work independently, so their address arithmetic overlaps.
__device__ __noinline__ void producer_loop(const MkParams &p, const MkPhase *s_ph, unsigned char *ring,
                                           unsigned long long *full_bar, unsigned long long *empty_bar,
                                           volatile int *abort_flag, int lane) {
    if (lane >= p.nslot) return;
    unsigned long long policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    const int cta = blockIdx.x, ncta = gridDim.x;
    const int nph = 4 * p.n_layers + 1;
    const int depth = p.nslot / MK_NWC;
    const int w = lane / depth;          // consumer warp served by this lane
    unsigned char *dst = ring + static_cast<size_t>(lane) * p.slot_bytes;
    unsigned long long *fb = &full_bar[lane], *eb = &empty_bar[lane];
    int ph = 0, it0 = 0, ntiles = 0;
    int local = lane - w * depth;  // index in warp w's tile sequence of the current phase
    unsigned round = 0;            // how often this slot has been filled
    bool ok = true;
    bool fresh = true;             // phase changed: recompute the warp's share
    while (ok) {
        if (fresh) {
            if (ph >= nph) break;
            int it1;
            item_range(s_ph[ph].items_total, cta, ncta, it0, it1);
            const int n_items = it1 - it0;
            const int mine = n_items > w ? (n_items - w + MK_NWC - 1) / MK_NWC : 0;   // items i = w, w + NWC, ...
            ntiles = mine * s_ph[ph].ksplit;
            fresh = false;
        }
        if (local >= ntiles) { local -= ntiles; ++ph; fresh = true; continue; }
        const MkPhase &P = s_ph[ph];
        const int S = P.ksplit;
        const int it = it0 + w + (S == 1 ? local : local / S) * MK_NWC;
        const int sl = S == 1 ? 0 : local % S;
        const int nblk = (P.kind == PH_QKV || P.kind == PH_SWIGLU) ? 2 : 1;
        const unsigned seg_bytes = static_cast<unsigned>(P.kcs) * 16u;
        int cnt;
        const int row_lo = item_rows(P, p, it, 0, cnt);
        {   // bounds of the tile about to be fetched (rows inside the matrix, bytes inside the slot, 16-byte rule)
            const long long rows_total = P.kind == PH_QKV ? 2LL * P.units_total : (P.kind == PH_SWIGLU ? 2LL * p.F : P.units_total);
            const int row_hi_chk = nblk == 2 ? item_rows(P, p, it, 1, cnt) : row_lo;
            const bool bad = cnt < 1 || seg_bytes == 0 || (seg_bytes & 15u) || row_lo < 0 || row_lo + cnt > rows_total ||
                             row_hi_chk + cnt > rows_total || static_cast<long long>(nblk - 1) * P.rw * seg_bytes + static_cast<long long>(cnt) * seg_bytes > p.slot_bytes ||
                             (sl + 1) * P.kcs * 8 > P.K || (reinterpret_cast<unsigned long long>(P.W) & 15ull) || (smem_u32(dst) & 15u);
            if (bad) { ok = diag_fail(p, abort_flag, 1, ph, it); break; }
        }
        if (!mbar_wait(eb, (round & 1u) ^ 1u, abort_flag, p.spin_limit)) { ok = false; break; }
        mbar_arrive_expect_tx(fb, static_cast<unsigned>(cnt * nblk) * seg_bytes);
        for (int b = 0; b < nblk; ++b) {
            const int row0 = b ? item_rows(P, p, it, 1, cnt) : row_lo;
            unsigned char *d = dst + static_cast<size_t>(b * P.rw) * seg_bytes;
            if (S == 1) {  // whole rows are contiguous: one copy per block
                bulk_copy_g2s(d, P.W + static_cast<size_t>(row0) * P.K, static_cast<unsigned>(cnt) * seg_bytes, fb, policy);
            } else {
                for (int r = 0; r < cnt; ++r)
                    bulk_copy_g2s(d + static_cast<size_t>(r) * seg_bytes,
                                  P.W + static_cast<size_t>(row0 + r) * P.K + static_cast<size_t>(sl) * P.kcs * 8, seg_bytes, fb, policy);
            }
        }
        ++round;
        local += depth;
    }
    if (!ok && round > 0) {
        // aborted: wait (bounded) until the last copy this lane issued has landed before the CTA may exit
        if (p.state->status == 0) p.state->status = 6;
        const unsigned long long t0 = global_ns();
        while (!mbar_try_wait(fb, (round - 1u) & 1u))
            if (global_ns() - t0 > p.spin_limit) break;
    }
}

// ---- consumer: one work item (rw rows or row pairs, all K slices) by one warp -----------------------------
struct ItemCtx {
    float rscale;          // deferred RMSNorm factor (1 for plain prologues)
    int slot_row;          // cache slot written by this step
    const float *rope;     // smem cos[d/2], sin[d/2]
    float best_v;          // PH_LMHEAD running argmax of this lane
    int best_i;
    float *logits_out;
    unsigned warp;         // consumer warp index
};

template <int NR>
__device__ __forceinline__ bool consume_item(const MkParams &p, const MkPhase &P, int it, unsigned &tile_no, const float4 *xsA,
                                             const float4 *xsB, const unsigned char *ring, unsigned long long *full_bar,
                                             unsigned long long *empty_bar, volatile int *abort_flag, ItemCtx &cx, int lane) {
    float acc[NR], acc2[NR];   // two chains per row halve the dependent-FMA latency
#pragma unroll
    for (int r = 0; r < NR; ++r) { acc[r] = 0.f; acc2[r] = 0.f; }
    const int kcs = P.kcs;
    for (int s = 0; s < P.ksplit; ++s) {
        const unsigned depth = static_cast<unsigned>(p.nslot) / MK_NWC;       // this warp's private sub-ring
        const unsigned slot = cx.warp * depth + tile_no % depth;
        const unsigned par = (tile_no / depth) & 1u;
        ++tile_no;
        if (NR * kcs * 16 > p.slot_bytes || (s + 1) * kcs * 32 > p.xbuf_bytes) return diag_fail(p, abort_flag, 2, kcs, NR);
        if (!mbar_wait(&full_bar[slot], par, abort_flag, p.spin_limit)) return false;
        const uint4 *t = reinterpret_cast<const uint4 *>(ring + static_cast<size_t>(slot) * p.slot_bytes);
        const float4 *a = xsA + s * kcs, *b = xsB + s * kcs;
#pragma unroll 2
        for (int c = lane; c < kcs; c += 32) {
            const float4 x0 = a[c], x1 = b[c];
#pragma unroll
            for (int r = 0; r < NR; ++r) {
                const uint4 w = t[r * kcs + c];
                acc[r] = fmaf(bf16lo(w.x), x0.x, acc[r]);  acc2[r] = fmaf(bf16hi(w.x), x0.y, acc2[r]);
                acc[r] = fmaf(bf16lo(w.y), x0.z, acc[r]);  acc2[r] = fmaf(bf16hi(w.y), x0.w, acc2[r]);
                acc[r] = fmaf(bf16lo(w.z), x1.x, acc[r]);  acc2[r] = fmaf(bf16hi(w.z), x1.y, acc2[r]);
                acc[r] = fmaf(bf16lo(w.w), x1.z, acc[r]);  acc2[r] = fmaf(bf16hi(w.w), x1.w, acc2[r]);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[slot]);
    }
#pragma unroll
    for (int r = 0; r < NR; ++r) acc[r] = warp_sum(acc[r] + acc2[r]) * cx.rscale;

    // ---- fused epilogue: lane r finishes unit r of the item ---------------------------------------------
    const int u0 = it * P.rw;
    if (P.kind == PH_RESID) {
#pragma unroll
        for (int r = 0; r < NR; ++r)
            if (lane == r && u0 + r < P.units_total) P.out[u0 + r] = __ldcg(P.out + u0 + r) + acc[r];
    } else if (P.kind == PH_LMHEAD) {
#pragma unroll
        for (int r = 0; r < NR; ++r)
            if (lane == r && u0 + r < P.units_total) {
                if (cx.logits_out) cx.logits_out[u0 + r] = acc[r];
                if (arg_better(acc[r], u0 + r, cx.best_v, cx.best_i)) { cx.best_v = acc[r]; cx.best_i = u0 + r; }
            }
    } else if constexpr (NR >= 2) {
        constexpr int RWP = NR / 2;  // pairs in the tile: low rows [0, RWP), partner rows [RWP, NR)
#pragma unroll
        for (int r = 0; r < RWP; ++r) {
            if (lane == r && u0 + r < P.units_total) {
                float lo = acc[r], hi = acc[r + RWP];
                if (P.kind == PH_SWIGLU) {
                    P.out[u0 + r] = lo / (1.f + expf(-lo)) * hi;
                } else {  // PH_QKV
                    const int half = p.d >> 1;
                    const int u = u0 + r;
                    const int head = u / half, i = u - head * half;
                    const int row_lo = head * p.d + i, row_hi = row_lo + half;
                    if (P.bias) { lo += bf16_bits_to_f32(P.bias[row_lo]); hi += bf16_bits_to_f32(P.bias[row_hi]); }
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
        }
    }
    return true;
}

// One weight-streaming operator on the consumer warps: prologue (stage the activation vector, RMSNorm
// folded in: x*w is staged and the scalar rsqrt(mean x^2 + eps) is applied to the dot products), items.
__device__ __forceinline__ bool gemv_phase(const MkParams &p, const MkPhase &P, unsigned &tile_no, float4 *xsA, float4 *xsB,
                                           const unsigned char *ring, unsigned long long *full_bar, unsigned long long *empty_bar,
                                           volatile int *abort_flag, float *s_part, ItemCtx &cx, int token, int tidc, int &prof_idx) {
    const int lane = tidc & 31, warp = tidc >> 5;
    const int cta = blockIdx.x, ncta = gridDim.x;
    const int n4 = P.K >> 2;
    float ss = 0.f;
    constexpr int PU = 4;  // loads in flight per thread
    for (int base = tidc; base < n4; base += MK_NTC * PU) {
        float4 v[PU];
        uint2 w[PU];
#pragma unroll
        for (int u = 0; u < PU; ++u) {
            const int i4 = base + u * MK_NTC;
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
            const int i4 = base + u * MK_NTC;
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
    if (P.norm_w) {
        ss = warp_sum(ss);
        if (lane == 0) s_part[warp] = ss;
    }
    consumer_sync();
    prof_stamp(p, tidc, prof_idx);   // activation vector staged
    cx.rscale = 1.f;
    if (P.norm_w) {
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < MK_NWC; ++w) tot += s_part[w];
        cx.rscale = rsqrtf(tot / static_cast<float>(P.K) + p.eps);
    }
    int it0, it1;
    item_range(P.items_total, cta, ncta, it0, it1);
    const int nr = (P.kind == PH_QKV || P.kind == PH_SWIGLU) ? 2 * P.rw : P.rw;
    bool ok = true;
    for (int i = warp; i < it1 - it0 && ok; i += MK_NWC) {
        switch (nr) {
            case 1: ok = consume_item<1>(p, P, it0 + i, tile_no, xsA, xsB, ring, full_bar, empty_bar, abort_flag, cx, lane); break;
            case 2: ok = consume_item<2>(p, P, it0 + i, tile_no, xsA, xsB, ring, full_bar, empty_bar, abort_flag, cx, lane); break;
            case 4: ok = consume_item<4>(p, P, it0 + i, tile_no, xsA, xsB, ring, full_bar, empty_bar, abort_flag, cx, lane); break;
            default: ok = consume_item<8>(p, P, it0 + i, tile_no, xsA, xsB, ring, full_bar, empty_bar, abort_flag, cx, lane); break;
        }
    }
    return ok;
}

// ---- attention on the consumer warps ------------------------------------------------------------------
// CTA (g, c) = chunk c of kv head g; all G query heads of the group share each K/V row read.
// Scores: MK_ATT_LPP lanes per position, each lane reads interleaved 16-byte pieces of the K row from
// global memory; P V: every lane owns d/32 dims.  Shared memory (the idle activation buffer): q,
// probabilities, warp merge area, chunk statistics.
template <int D, int G>
__device__ __forceinline__ void attention_phase(const MkParams &p, int layer, int n, unsigned char *xbuf, int tidc, int *s_flag) {
    constexpr int TILE = MK_ATT_TILE, LPP = MK_ATT_LPP;
    constexpr int DV = D / 32, CPR = D / 8, CPL = CPR / LPP;
    const int lane = tidc & 31, warp = tidc >> 5;
    const int cta = blockIdx.x;
    int nch = (n + p.att_min_chunk - 1) / p.att_min_chunk;
    nch = min(nch, p.max_chunks);
    int chunk_len = (n + nch - 1) / nch;
    chunk_len = (chunk_len + TILE - 1) / TILE * TILE;
    nch = (n + chunk_len - 1) / chunk_len;
    if (cta >= nch * p.nkv) return;
    const int g = cta / nch, c = cta - g * nch;
    const int t0 = c * chunk_len, t1 = min(n, t0 + chunk_len);

    float *qs = reinterpret_cast<float *>(xbuf);               // [G][D]
    float *ps = qs + G * D;                                     // [NWC][G][TILE]
    constexpr int MW = MK_ATT_MW;
    float *mg_m = ps + MK_NWC * G * TILE;                       // [MW][G]
    float *mg_l = mg_m + MW * G;                                // [MW][G]
    float *mg_o = mg_l + MW * G;                                // [MW][G][D]
    float *cm = mg_o + MW * G * D;                              // [G][max_chunks] chunk maxima
    float *cl = cm + G * p.max_chunks;                          // [G][max_chunks] chunk denominators

    for (int i = tidc; i < G * D; i += MK_NTC) qs[i] = __ldcg(p.q + static_cast<size_t>(g) * G * D + i) * p.scale;
    consumer_sync();

    const size_t head_off = (static_cast<size_t>(layer) * p.nkv + g) * p.max_context * D;
    const uint16_t *kg = p.k_cache + head_off;
    const uint16_t *vg = p.v_cache + head_off;
    float *pw = ps + warp * (G * TILE);
    const int pi = lane / LPP, part = lane % LPP;

    float m[G], l[G], o[G][DV];
#pragma unroll
    for (int h = 0; h < G; ++h) {
        m[h] = -INFINITY; l[h] = 0.f;
#pragma unroll
        for (int e = 0; e < DV; ++e) o[h][e] = 0.f;
    }

    for (int tt = t0 + warp * TILE; tt < t1; tt += MK_NWC * TILE) {
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
        float s[G];
#pragma unroll
        for (int h = 0; h < G; ++h) s[h] = 0.f;
#pragma unroll
        for (int j = 0; j < CPL; ++j) {
            const int cc = j * LPP + part;
#pragma unroll
            for (int h = 0; h < G; ++h) {
                const float4 q0 = *reinterpret_cast<const float4 *>(qs + h * D + cc * 8);
                const float4 q1 = *reinterpret_cast<const float4 *>(qs + h * D + cc * 8 + 4);
                s[h] = dot8(kk[j], q0, q1, s[h]);
            }
        }
#pragma unroll
        for (int h = 0; h < G; ++h) {
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
            for (int h = 0; h < G; ++h) {
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
    float lt[G];
#pragma unroll
    for (int h = 0; h < G; ++h) lt[h] = warp_sum(l[h]);
    if (warp >= MW) {
        const int u = warp - MW;
#pragma unroll
        for (int h = 0; h < G; ++h) {
            if (lane == 0) { mg_m[u * G + h] = m[h]; mg_l[u * G + h] = lt[h]; }
#pragma unroll
            for (int e = 0; e < DV; ++e) mg_o[(u * G + h) * D + lane * DV + e] = o[h][e];
        }
    }
    consumer_sync();
    if (warp < MK_NWC - MW) {
#pragma unroll
        for (int h = 0; h < G; ++h) {
            const float m2 = mg_m[warp * G + h], l2 = mg_l[warp * G + h];
            const float mn = fmaxf(m[h], m2);
            const float e1 = m[h] == mn ? 1.f : __expf(m[h] - mn);
            const float e2 = m2 == mn ? 1.f : __expf(m2 - mn);
            lt[h] = lt[h] * e1 + l2 * e2;
#pragma unroll
            for (int e = 0; e < DV; ++e) o[h][e] = o[h][e] * e1 + mg_o[(warp * G + h) * D + lane * DV + e] * e2;
            m[h] = mn;
        }
    }
    consumer_sync();
    if (warp < MW) {
#pragma unroll
        for (int h = 0; h < G; ++h) {
            if (lane == 0) { mg_m[warp * G + h] = m[h]; mg_l[warp * G + h] = lt[h]; }
#pragma unroll
            for (int e = 0; e < DV; ++e) mg_o[(warp * G + h) * D + lane * DV + e] = o[h][e];
        }
    }
    consumer_sync();
    for (int i = tidc; i < G * D; i += MK_NTC) {
        const int h = i / D, j = i - h * D;
        float mm = -INFINITY;
#pragma unroll
        for (int w = 0; w < MW; ++w) mm = fmaxf(mm, mg_m[w * G + h]);
        float ll = 0.f, oo = 0.f;
#pragma unroll
        for (int w = 0; w < MW; ++w) {
            const float e = __expf(mg_m[w * G + h] - mm);
            ll = fmaf(mg_l[w * G + h], e, ll);
            oo = fmaf(mg_o[(w * G + h) * D + j], e, oo);
        }
        const int qh = g * G + h;
        if (nch == 1) {  // nothing to merge across CTAs
            p.attn[qh * D + j] = oo / ll;
        } else {
            p.part_o[(static_cast<size_t>(qh) * p.max_chunks + c) * D + j] = oo;
            if (j == 0) { p.part_m[qh * p.max_chunks + c] = mm; p.part_l[qh * p.max_chunks + c] = ll; }
        }
    }
    if (nch == 1) return;
    __threadfence();
    consumer_sync();
    if (tidc == 0) *s_flag = (atomicAdd(p.tickets + g, 1u) == static_cast<unsigned>(nch - 1)) ? 1 : 0;
    consumer_sync();
    if (!*s_flag) return;

    // Last CTA of this kv head: exact log-sum-exp merge of the chunks, in index order.  All loads of a
    // batch (chunk statistics and up to CB partial vectors per thread) are issued before any is used.
    __threadfence();
    constexpr int CB = 8;
    const int i0 = tidc;                       // output (h, j4) of this thread, if any
    const bool has_out = i0 < G * D / 4;
    const int oh = has_out ? i0 / (D / 4) : 0, oj4 = has_out ? i0 - oh * (D / 4) : 0;
    const float4 *po = reinterpret_cast<const float4 *>(p.part_o + static_cast<size_t>(g * G + oh) * p.max_chunks * D) + oj4;
    float4 ob[CB];
#pragma unroll
    for (int u = 0; u < CB; ++u)
        ob[u] = (has_out && u < nch) ? __ldcg(po + static_cast<size_t>(u) * (D / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
    for (int i = tidc; i < G * nch; i += MK_NTC) {
        const int h = i / nch, cc = i - h * nch;
        cm[h * p.max_chunks + cc] = __ldcg(p.part_m + (g * G + h) * p.max_chunks + cc);
        cl[h * p.max_chunks + cc] = __ldcg(p.part_l + (g * G + h) * p.max_chunks + cc);
    }
    consumer_sync();
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
        reinterpret_cast<float4 *>(p.attn + (g * G + oh) * D)[oj4] = acc;
    }
    if (tidc == 0) p.tickets[g] = 0u;
}

// ---- the kernel -----------------------------------------------------------------------------------------------
template <int D, int G>
__global__ void __launch_bounds__(MK_THREADS, 1) decode_megakernel(const MkParams p) {
    extern __shared__ __align__(128) unsigned char mk_smem[];
    unsigned char *smem = mk_smem;
    float4 *xsA = reinterpret_cast<float4 *>(smem);
    float4 *xsB = reinterpret_cast<float4 *>(smem + p.xbuf_bytes / 2);
    MkPhase *s_ph = reinterpret_cast<MkPhase *>(smem + p.xbuf_bytes);          // the step's schedule
    unsigned char *ring = smem + p.xbuf_bytes + p.sched_bytes;
    __shared__ __align__(8) unsigned long long full_bar[MK_MAX_SLOTS];
    __shared__ __align__(8) unsigned long long empty_bar[MK_MAX_SLOTS];
    __shared__ float s_rope[128];
    __shared__ float s_part[MK_NWC];
    __shared__ float s_bv[MK_NWC];
    __shared__ int s_bi[MK_NWC];
    __shared__ int s_flag;
    __shared__ int s_abort;

    const int tid = threadIdx.x;
    if (tid == 0) {
        for (int i = 0; i < p.nslot; ++i) { mbar_init(&full_bar[i], 1); mbar_init(&empty_bar[i], 1); }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    {
        const int n16 = (4 * p.n_layers + 1) * static_cast<int>(sizeof(MkPhase) / 16);
        const uint4 *src = reinterpret_cast<const uint4 *>(p.phases);
        uint4 *dst = reinterpret_cast<uint4 *>(s_ph);
        for (int i = tid; i < n16; i += MK_THREADS) dst[i] = src[i];
    }
    __syncthreads();
    volatile int *abort_flag = &s_abort;

    if (tid >= MK_NTC) {  // ---- producer warp ----
        producer_loop(p, s_ph, ring, full_bar, empty_bar, abort_flag, tid - MK_NTC);
        return;
    }

    // ---- consumer warps ----
    const int tidc = tid, lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x, ncta = gridDim.x;
    const int rt = p.req->token, rp = p.req->position;
    const int token = rt >= 0 ? rt : p.state->next_token;
    const int pos = rp >= 0 ? rp : p.state->next_position;
    const int slot_row = p.state->cur_len;
    const int half = p.d >> 1;
    if (tidc < half) {  // rotary table of this step's position; fp64 angle, rounded once
        double sn, cs;
        sincos(static_cast<double>(pos) * p.inv_freq[tidc], &sn, &cs);
        s_rope[tidc] = static_cast<float>(cs);
        s_rope[half + tidc] = static_cast<float>(sn);
    }
    if (token < 0 || token >= p.V || slot_row < 0 || slot_row >= p.max_context || pos < 0) {
        if (tidc == 0) diag_fail(p, abort_flag, 3, token, slot_row);   // corrupt request/state: touch nothing
        return;
    }
    if (cta == 0 && tidc == 0) { p.state->token = token; p.state->position = pos; }
    // (s_rope is published by the consumer_sync of the first prologue)

    ItemCtx cx;
    cx.rscale = 1.f; cx.slot_row = slot_row; cx.rope = s_rope; cx.best_v = -INFINITY; cx.best_i = 0x7fffffff;
    cx.logits_out = p.req->logits_out;
    cx.warp = static_cast<unsigned>(warp);

    unsigned tile_no = 0, bar_no = 0;   // tile_no: tiles this warp has consumed so far
    int prof_idx = 0;
    prof_stamp(p, tidc, prof_idx);
    bool ok = true;
    for (int l = 0; l < p.n_layers && ok; ++l) {
        ok = gemv_phase(p, s_ph[4 * l], tile_no, xsA, xsB, ring, full_bar, empty_bar, abort_flag, s_part, cx, token, tidc, prof_idx);
        ok = grid_barrier(p, ++bar_no * ncta, abort_flag, tidc, prof_idx) && ok;
        if (ok) attention_phase<D, G>(p, l, slot_row + 1, smem, tidc, &s_flag);
        ok = grid_barrier(p, ++bar_no * ncta, abort_flag, tidc, prof_idx) && ok;
        for (int k = 1; k < 4 && ok; ++k) {
            ok = gemv_phase(p, s_ph[4 * l + k], tile_no, xsA, xsB, ring, full_bar, empty_bar, abort_flag, s_part, cx, token, tidc, prof_idx);
            ok = grid_barrier(p, ++bar_no * ncta, abort_flag, tidc, prof_idx) && ok;
        }
    }
    if (ok) ok = gemv_phase(p, s_ph[4 * p.n_layers], tile_no, xsA, xsB, ring, full_bar, empty_bar, abort_flag, s_part, cx, token, tidc, prof_idx);
    prof_stamp(p, tidc, prof_idx);
    if (!ok) {
        if (tidc == 0) p.state->status = 6;
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
    consumer_sync();
    if (tidc == 0) {
        for (int w = 1; w < MK_NWC; ++w)
            if (arg_better(s_bv[w], s_bi[w], bv, bi)) { bv = s_bv[w]; bi = s_bi[w]; }
        p.lm_part_val[cta] = bv;
        p.lm_part_idx[cta] = bi;
        __threadfence();
        s_flag = (atomicAdd(p.tickets + p.nkv, 1u) == static_cast<unsigned>(ncta - 1)) ? 1 : 0;
    }
    consumer_sync();
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
            int *nto = p.req->next_token_out;
            if (nto) *nto = bi;
            p.state->next_token = bi;
            p.state->next_position = pos + 1;
            p.state->cur_len = slot_row + 1;
            p.tickets[p.nkv] = 0u;
            *p.barrier = 0u;  // every CTA has passed the last grid barrier
        }
    }
}

}  // namespace edgefm
