// The whole decode step as ONE persistent cooperative kernel (one CTA per SM).
//
// Why: at batch 1 a layer of a 1.5B-parameter decoder is ~94 MB of weights, i.e. ~14 us of HBM time,
// split over five operators that depend on one another.  Separate kernels drain and refill the memory
// pipeline at every boundary.  Here the weight stream is decoupled from the dependency chain:
//
//   * The step's weight traffic is a static schedule made on the host (QKV, O, gate/up, down of every layer,
//     then lm_head).  Every CTA owns a fixed share of each operator's rows; the share is cut into tiles of up
//     to 16 rows x 256 columns, and every consumer warp owns a fixed list of tiles (the same for every layer).
//   * Every consumer warp keeps a private ring of shared-memory slots filled with its next tiles by TMA tensor copies
//     (cp.async.bulk.tensor, 128-byte swizzle, mbarrier complete_tx): when it has multiplied a tile, its lane 0 at once fetches
//     the tile that comes S places later in its sequence into the freed slot -- regardless of operator boundaries,
//     the weights do not depend on the computation.  So the short operators of a layer are on chip when their turn
//     comes and HBM keeps streaming while the arithmetic waits at a grid barrier, stages an activation vector or
//     runs attention.  One more warp of the CTA computes nothing: it runs ahead of the rings and pulls the tiles
//     that come next into L2 (prefetch.global.L2), because the rings alone hold too little to keep HBM busy through
//     the stalls and a refill from L2 returns much sooner than one from HBM.
//   * A consumer warp waits for its next tile, multiplies it with the 256 activations of the tile's columns and releases
//     the slot.  The multiplication is 16 x (ldmatrix + mma.m16n8k16): the fp32 activations are staged as three bf16
//     pieces (columns 0..2 of the B operand), the products are exact and accumulate in fp32.  Consecutive tiles of a warp
//     cover the same rows; only at the end of a run of tiles are the row sums taken out of the accumulator fragments
//     (three shuffles).  The fused epilogues (bias + RoPE + KV append,
//     residual add, SwiGLU, logits + argmax) run in the warp when it has seen all columns of its rows, else the
//     sums meet in shared memory after the operator, in a fixed order.
//   * Between dependent operators all CTAs meet at a grid barrier (monotonic counter in global memory,
//     release/acquire, bounded spin).  Attention (split-KV, exact log-sum-exp merge) runs between two
//     barriers.
//
// Every wait is bounded: on expiry the CTA records EDGEFM_ERR_TIMEOUT in the device state, stops
// issuing copies, waits (bounded) for the copies it has in flight and returns.
// This file is the body of the kernel.  It is included once per build (MK_NS = namespace, MK_NW_VALUE = consumer
// warps per CTA); everything that does not depend on the number of warps lives in megakernel_types.cuh.
#include <type_traits>

#include "megakernel_types.cuh"

namespace edgefm {
namespace MK_NS {

constexpr int MK_NW = MK_NW_VALUE;               // consumer warps per CTA
#ifndef MK_M_VALUE
#define MK_M_VALUE 1
#endif
// Tokens one call may carry.  1: the plain decode step.  M > 1 (a build of its own): a block of up to M tokens is pushed
// through the step together -- the token to decode and proposed continuations (Sec. 3.11 of the paper: the base model
// verifies a proposed block); the weights are streamed once, every token has its own activation vectors, and the tensor-core
// product carries the tokens side by side in the columns of its B operand (three columns per token).
constexpr int MK_M = MK_M_VALUE;
constexpr int MK_S = mk_splits(MK_M);             // bf16 pieces per activation value in this build
static_assert(MK_M >= 1 && MK_M * MK_S <= 8, "the tokens of a block share the eight columns of one B operand");
constexpr int MK_NT = MK_NW * 32;                // consumer threads
constexpr int MK_THREADS = MK_NT + 32;           // + the L2 prefetch warp

// 1: one-head-per-CTA attention leaves the merge of its chunks to the O projection's prologue (every CTA merges);
// 0: the last CTA of every head merges (atomic ticket) and the O projection stages the finished vector
#ifndef MK_SPLIT_DEFER
#define MK_SPLIT_DEFER 1
#endif
#ifndef MK_ACC_CHAINS
#define MK_ACC_CHAINS 4   // independent tensor-core accumulation chains per warp
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
// One box of a weight matrix through tensor map `map`; the coordinates are listed innermost first.  The innermost one is a
// column (0, or a multiple of 64: x * 2 bytes is a multiple of 16 by construction); no multicast.
__device__ __forceinline__ void tma_load_box(void *dst, const void *map, int x, int y, unsigned long long *bar, unsigned long long policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
// (more dimensions: the 64-column blocks of a row, the partner rows of gate/up and of rotate-half, the heads)
__device__ __forceinline__ void tma_load_box3(void *dst, const void *map, int x, int y, int z, unsigned long long *bar, unsigned long long policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tma_load_box4(void *dst, const void *map, int x, int y, int z, int w, unsigned long long *bar, unsigned long long policy) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4, %5}], [%6], %7;"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(z), "r"(w), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tma_load_box5(void *dst, const void *map, int x, int y, int z, int w, int v, unsigned long long *bar, unsigned long long policy) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4, %5, %6}], [%7], %8;"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(z), "r"(w), "r"(v), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
// all consumer threads of the CTA (the feeding warp never joins)
__device__ __forceinline__ void cta_sync() { asm volatile("bar.sync 1, %0;" ::"n"(MK_NT) : "memory"); }

// Dynamic shared memory: operators | schedule table | tile lists | rings (1 KB-aligned slots) | staged activation vector
// (also the attention scratch).
// (Addresses are recomputed from the kernel parameters where they are used instead of being carried in registers.)
extern __shared__ __align__(1024) unsigned char mk_smem[];
__device__ __forceinline__ MkOp *sm_ops(const MkParams &) { return reinterpret_cast<MkOp *>(mk_smem); }
__device__ __forceinline__ int *sm_tab(const MkParams &p) { return reinterpret_cast<int *>(mk_smem + p.ops_bytes); }
__device__ __forceinline__ uint2 *sm_tiles(const MkParams &p) { return reinterpret_cast<uint2 *>(mk_smem + p.ops_bytes + p.tab_bytes); }
// the CTA's combine entries follow its tiles (16-byte aligned)
__device__ __forceinline__ MkCombine *sm_combines(const MkParams &p) {
    const int nt = sm_tab(p)[MK_NW * MK_WARP_TAB + 11];
    return reinterpret_cast<MkCombine *>(mk_smem + p.ops_bytes + p.tab_bytes + ((nt * 8 + 15) & ~15));
}
__device__ __forceinline__ unsigned char *sm_ring(const MkParams &p, int warp) {
    return mk_smem + p.ops_bytes + p.tab_bytes + p.sched_bytes + warp * (p.slots * p.slot_bytes);
}
__device__ __forceinline__ unsigned char *sm_xbuf(const MkParams &p) { return sm_ring(p, MK_NW); }
// The staged activation vector of an operator with K columns: MK_S (2 or 3) bf16 arrays of Kpad = K rounded up to whole
// 256-column pieces (zero beyond K), xs_stride(K) bytes apart.  Array s holds piece s of every value (value = sum of its
// pieces to 24 bits), columns in tensor-core fragment order (mk_xs_index).
__device__ __forceinline__ int xs_stride(int K) { return (K + MK_TILE_COLS - 1) / MK_TILE_COLS * (MK_TILE_COLS * 2) + MK_XS_PAD; }
// two values -> one bf16x2 word (first value in the low half), round to nearest even
__device__ __forceinline__ unsigned pack_bf16x2(float lo, float hi) {
    unsigned d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
// Split four consecutive values (columns 4 * i4 ..) into their bf16 pieces and store them in fragment order.
__device__ __forceinline__ void stage_piece(unsigned char *xs, int stride, int i4, float4 t) {
    const int idx = mk_xs_index(i4 * 4);          // columns c, c+1 are neighbours; c+2, c+3 follow 8 entries later
    unsigned *dst = reinterpret_cast<unsigned *>(xs) + (idx >> 1);
#pragma unroll
    for (int sp = 0; sp < MK_S; ++sp) {
        const unsigned a = pack_bf16x2(t.x, t.y), b = pack_bf16x2(t.z, t.w);
        dst[0] = a;
        dst[4] = b;
        dst += stride >> 2;
        t.x -= bf16lo(a); t.y -= bf16hi(a); t.z -= bf16lo(b); t.w -= bf16hi(b);   // exact: the remainder is what the next piece holds
    }
}

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

// All consumer threads of all CTAs meet here.  Returns false when the wait expired (step aborted).
__device__ __forceinline__ bool grid_barrier(const MkParams &p, unsigned target, volatile int *abort_flag, int tid, int &prof_idx) {
    cta_sync();
    prof_stamp(p, tid, prof_idx);   // this CTA's share of the operator is done
    if (tid == 0 && !*abort_flag) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.barrier) : "memory");
    if (tid == 0 && !*abort_flag) {
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
    cta_sync();
    prof_stamp(p, tid, prof_idx);   // released by the slowest CTA
    return !*abort_flag;
}

// First weight row of unit u of an operator (its partner row, if any, is `partner` rows further).
__device__ __forceinline__ int unit_row(const MkParams &p, int kind, int u) {
    if (kind == PH_QKV) {
        const int half = p.d >> 1;
        return (u >> p.half_shift) * p.d + (u & (half - 1));
    }
    return u;
}

// ---- fetching a warp's tiles ------------------------------------------------------------------------------------
// Every consumer warp keeps S tiles in flight in its own ring: slot k % S holds tile k of the warp's sequence over the
// whole step (its layer list once per layer, then its output-layer list).  Right after the warp has multiplied a tile,
// its lane 0 fetches the tile S places further into the slot that has just become free -- whatever operator that tile
// belongs to, so the stream runs ahead across operator boundaries.  One lane arms and one warp drains every "full"
// barrier strictly in order, so the one-bit phase parity cannot alias and no "empty" barrier is needed.
struct TileCursor {
    int layer, i;          // next tile: i-th of the layer list (layer < n_layers) or of the output-layer list
    unsigned count;        // tiles passed so far
};
__device__ __forceinline__ void cursor_step(TileCursor &c, int n_layer, int n_layers) {
    ++c.count;
    ++c.i;
    if (c.layer < n_layers && c.i == n_layer) { c.i = 0; ++c.layer; }
}
struct WarpStream {
    int list;                   // next tile to multiply: index into the CTA's tile lists
    TileCursor next;            // next tile to fetch (lane 0's view)
    uint2 nd;                   // its descriptor, read ahead (valid while next.count < total)
    int slot;                   // slot of the next tile to multiply
    unsigned round;
    unsigned consumed;          // tiles multiplied so far
    int fenced_op;
    unsigned total;             // tiles of this warp over the whole step
    int n_layer;                // tiles per layer
    int list_layer, list_lm;    // the warp's two lists in the CTA's tile block
};
// Lane 0 only: fetch tile ws.next into ring slot `slot` (whose previous contents this warp has finished reading).
__device__ __forceinline__ bool fetch_next_tile(const MkParams &p, WarpStream &ws, int slot, volatile int *abort_flag, volatile unsigned *s_issued,
                                                unsigned long long *full_bar, int warp) {
#ifdef EDGEFM_TRACE_OP
    long long fc[6];
    fc[0] = clock64();
#define FSEG(i) fc[i] = clock64()
#else
#define FSEG(i) do {} while (0)
#endif
    if (ws.next.count >= ws.total) return true;          // the whole step has been fetched
    const bool lm = ws.next.layer >= p.n_layers;
    const uint2 d = ws.nd;
    // the operators of a layer are QKV, O, gate/up, down in this order; 4 = the output layer
    const int op = static_cast<int>((d.y >> 20) & 7u);
    const int opi = 4 * ws.next.layer + (lm ? 0 : op);
    const int m = static_cast<int>(d.y & 31u), x = static_cast<int>((d.x >> 20) & 0xffu) * MK_TILE_COLS;
    const int u0 = static_cast<int>(d.x & 0xfffffu);
    const bool paired = op == 0 || op == 2;
    const unsigned bytes = static_cast<unsigned>(m) << (paired ? 10 : 9);   // m rows (and their partners) x 512 bytes
    // (the host made the schedule; a corrupt entry must still not write past the slot)
    if (m < 1 || bytes > static_cast<unsigned>(p.slot_bytes) || (lm ? op != 4 : op > 3)) return diag_fail(p, abort_flag, 1, opi, u0);
    const unsigned char *map = p.maps + (static_cast<size_t>(opi) * MK_MAX_VARIANTS + ((d.x >> 28) & 3u)) * 128;
    if (p.map_fence != 0 && opi != ws.fenced_op && (p.map_fence == 2 || lm)) {
        // the host may have rewritten this operator's tensor maps since the last launch (another vocabulary subset, or a
        // static call with other weights): order the copy engine's view of them behind what is in memory now
        ws.fenced_op = opi;
        for (int v = 0; v < MK_MAX_VARIANTS; ++v)
            asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(p.maps + (static_cast<size_t>(opi) * MK_MAX_VARIANTS + v) * 128) : "memory");
    }
    unsigned char *dst = sm_ring(p, warp) + slot * p.slot_bytes;
    unsigned long long *bar = &full_bar[warp * MK_MAX_SLOTS + slot];
    unsigned long long policy;   // weights are read once per step: first out of L2
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    FSEG(1);
    // the warp read the slot through the generic proxy: order those reads before the asynchronous write
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    FSEG(2);
    mbar_arrive_expect_tx(bar, bytes);
    FSEG(3);
    if (!(d.y & MKT_RAGGED)) {                           // one copy: the tile's four 64-column blocks are a dimension of the map
        const int cb = x >> 6;
        if (op == 0) tma_load_box5(dst, map, 0, u0 & ((p.d >> 1) - 1), 0, u0 >> p.half_shift, cb, bar, policy);
        else if (op == 2) tma_load_box4(dst, map, 0, u0, 0, cb, bar, policy);
        else tma_load_box3(dst, map, 0, u0, cb, bar, policy);
    } else {                                               // K has a ragged last block: block by block (blocks past K read as zero)
        const unsigned blk = bytes >> 2;
#pragma unroll
        for (int cb = 0; cb < MK_TILE_COLS / 64; ++cb) {
            if (op == 0) tma_load_box4(dst + cb * blk, map, x + cb * 64, u0 & ((p.d >> 1) - 1), 0, u0 >> p.half_shift, bar, policy);
            else if (op == 2) tma_load_box3(dst + cb * blk, map, x + cb * 64, u0, 0, bar, policy);
            else tma_load_box(dst + cb * blk, map, x + cb * 64, u0, bar, policy);
        }
    }
    FSEG(4);
    cursor_step(ws.next, ws.n_layer, p.n_layers);
    s_issued[warp] = ws.next.count;     // read by the L2 prefetch warp
    ws.nd = sm_tiles(p)[(ws.next.layer >= p.n_layers ? ws.list_lm : ws.list_layer) + ws.next.i];   // (one entry behind the lists is readable: the combines follow)
#ifdef EDGEFM_TRACE_OP
    FSEG(5);
    if (p.prof && blockIdx.x == 0 && warp == 3 && opi == EDGEFM_TRACE_OP) {
        unsigned long long *o = p.prof + static_cast<size_t>(gridDim.x) * p.prof_stride + MK_NW_MAX * 16 * 4;
        for (int i = 0; i < 5; ++i) o[i] += static_cast<unsigned long long>(fc[i + 1] - fc[i]);
        o[5] += 1;
    }
#endif
    return true;
}

// Attention chunking shared by the attention phase and by the consumer of its partial results.
// mult: tokens of a block that are attended in the same pass (each with its own CTAs); n is then the longest token's length.
__device__ __forceinline__ void att_chunking(const MkParams &p, int n, int hg, int min_chunk, int tile, int ncta, int &nch, int &chunk_len, int mult = 1) {
    const int groups = p.nq / hg * mult;
    nch = (n + min_chunk - 1) / min_chunk;
    nch = min(nch, min(ncta / groups, p.max_chunks));
    if (hg == 1) nch = min(nch, MK_ATT_SPLIT_MAXC);
    nch = max(nch, 1);
    chunk_len = (n + nch - 1) / nch;
    chunk_len = (chunk_len + tile - 1) / tile * tile;
    nch = (n + chunk_len - 1) / chunk_len;
}

// ---- the L2 prefetch warp ------------------------------------------------------------------------------------
// The ring of a consumer warp holds only a few tiles, so HBM would idle whenever the consumers stall (grid barriers,
// attention) and every refill would pay the full HBM latency.  One more warp therefore runs ahead of the rings: lanes w
// and 16 + w walk the tile list of consumer warp w (low rows / partner rows of every tile) and ask L2 for the lines of
// every tile that is at most `pf_tiles` tiles ahead of what the feeding lane of that warp has fetched (plain
// prefetch.global.L2, one 128-byte line per instruction).  The lanes only read counters; nobody ever waits for them,
// and a tile the ring has already fetched is skipped.
__device__ __forceinline__ void prefetch_tiles(const MkParams &p, volatile int *abort_flag, volatile unsigned *s_issued, int lane) {
    const MkOp *s_ops = sm_ops(p);
    const int *s_tab = sm_tab(p);
    const uint2 *s_tiles = sm_tiles(p);
    const int w = lane & 15, half = lane >> 4;
    if (p.pf_tiles > 0 && w >= MK_NW) {
        // The spare lanes pull the K and V rows this CTA's attention will read into L2, a layer ahead: as soon as warp 0's
        // ring has started on the tiles of layer l, the chunk of layer l (one-head-per-CTA chunking only).
        const int n_spare = 2 * (16 - MK_NW), me = (w - MK_NW) * 2 + half;
        const int m_run = MK_M > 1 ? min(max(p.req->m, 1), MK_M) : 1;
        const int n = p.state->cur_len + m_run;
        if (p.kv8 || n > p.att_split_max_n || n < 1 || n > p.max_context) return;
        int nch, chunk_len;
        att_chunking(p, n, 1, p.att_chunk_split, 32 / MK_ATT_LPP_SPLIT, static_cast<int>(gridDim.x), nch, chunk_len, m_run);
        const int cta = static_cast<int>(blockIdx.x);
        if (cta >= nch * p.nq * m_run) return;
        const int qh = MK_M > 1 ? (cta / nch) % p.nq : cta / nch, c = cta - (cta / nch) * nch, g = qh / (p.nq / p.nkv);
        const int t0 = c * chunk_len, t1 = min(n, t0 + chunk_len);
        const int n_lines = ((t1 - t0) * p.d * 2 + 127) / 128;
        const int n_layer0 = s_tab[7];
        for (int layer = 0; layer < p.n_layers; ++layer) {
            unsigned spins = 0;
            while (s_issued[0] < static_cast<unsigned>(layer) * n_layer0) {
                if (*abort_flag || ++spins > (1u << 22)) return;
                __nanosleep(200);
            }
            const size_t off = ((static_cast<size_t>(layer) * p.nkv + g) * p.max_context + t0) * p.d * 2;
            const unsigned char *kb = reinterpret_cast<const unsigned char *>(p.k_cache) + off;
            const unsigned char *vb = reinterpret_cast<const unsigned char *>(p.v_cache) + off;
            for (int i = me; i < n_lines; i += n_spare) {
                asm volatile("prefetch.global.L2 [%0];" ::"l"(kb + static_cast<size_t>(i) * 128));
                asm volatile("prefetch.global.L2 [%0];" ::"l"(vb + static_cast<size_t>(i) * 128));
            }
        }
        return;
    }
    if (p.pf_tiles <= 0 || w >= MK_NW) return;
    const int *tab = s_tab + w * MK_WARP_TAB;
    const int n_layer = tab[1] + tab[2] + tab[3] + tab[4], n_lm = tab[6];
    const uint2 *layer_list = s_tiles + tab[0], *lm_list = s_tiles + tab[5];
    const unsigned total = static_cast<unsigned>(n_layer) * p.n_layers + n_lm;
    unsigned k = 0;              // next tile of this warp's whole-step sequence to ask for
    unsigned idle = 0;
    while (k < total) {
        const unsigned issued = s_issued[w];
        if (k < issued) k = issued;                         // the ring got there first
        if (k >= total) break;
        // (the output layer is one long uninterrupted stream: a deeper look-ahead pays there, and only there)
        if (k >= issued + static_cast<unsigned>(k >= static_cast<unsigned>(n_layer) * p.n_layers ? MK_PF_TILES_LM : p.pf_tiles)) {   // far enough ahead: wait for the ring to move
            if (*abort_flag || ++idle > (1u << 22)) return;  // bounded: give up (prefetching is only a hint)
            __nanosleep(200);
            continue;
        }
        idle = 0;
        const unsigned in_layers = static_cast<unsigned>(n_layer) * p.n_layers;
        const bool lm = k >= in_layers;
        const int layer = lm ? p.n_layers : static_cast<int>(k / n_layer);
        const uint2 d = lm ? lm_list[k - in_layers] : layer_list[k - static_cast<unsigned>(layer) * n_layer];
        const int op = static_cast<int>((d.y >> 20) & 7u);
        const int opi = lm ? 4 * p.n_layers : 4 * layer + op;
        const MkOp &P = s_ops[opi];
        const bool paired = P.kind == PH_QKV || P.kind == PH_SWIGLU;
        const int m = static_cast<int>(d.y & 31u), kcol = static_cast<int>((d.x >> 20) & 0xffu);
        const int u0 = static_cast<int>(d.x & 0xfffffu);
        ++k;
        if (m < 1 || m > MK_TILE_ROWS || u0 + m > P.units_total || kcol * MK_TILE_COLS >= P.K || (lm ? op != 4 : op > 3)) return;
        // rows of this lane: the low box (or rows 0..7), the partner box (or rows 8..)
        int row = unit_row(p, P.kind, u0), n_rows = paired ? m : min(m, 8);
        if (half) {
            if (paired) row += P.kind == PH_QKV ? (p.d >> 1) : p.F;
            else { row += 8; n_rows = m - 8; }
        }
        const int row_bytes = P.K * 2, col0 = kcol * (MK_TILE_COLS * 2);
        const int n_lines = min(MK_TILE_COLS * 2, row_bytes - col0 + 127) / 128;
        const unsigned char *base = reinterpret_cast<const unsigned char *>(p.op_weights[opi]) + static_cast<size_t>(row) * row_bytes + col0;
        for (int r = 0; r < n_rows; ++r)
            for (int l = 0; l < n_lines; ++l) asm volatile("prefetch.global.L2 [%0];" ::"l"(base + static_cast<size_t>(r) * row_bytes + l * 128));
    }
}

struct ItemCtx {             // per token of the call
    float rscale[MK_M];    // deferred RMSNorm factor (1 for plain prologues)
    int slot_row;          // cache slot written by the first token (token t writes slot_row + t)
    int m_run;             // tokens in this call (<= MK_M)
    float best_v[MK_M];    // PH_LMHEAD running argmax of this lane
    int best_i[MK_M];
};

// ---- fused epilogue of one output unit (a row, or a row pair) ------------------------------------------------
// pre: the value the epilogue adds (old residual / the two biases) was fetched ahead into pre_lo, pre_hi.
// tok: the token of the call this value belongs to (0 in the plain step).
__device__ __forceinline__ void apply_epilogue(const MkParams &p, const MkOp &P, ItemCtx &cx, const float *s_rope, int u, float lo, float hi,
                                               bool pre = false, float pre_lo = 0.f, float pre_hi = 0.f, int tok = 0) {
    float *const out = MK_M > 1 ? P.out + static_cast<size_t>(tok) * P.out_tok_stride : P.out;
    if (P.kind == PH_RESID) {
        out[u] = (pre ? pre_lo : __ldcg(out + u)) + lo;
    } else if (P.kind == PH_LMHEAD) {
        float *logits_out = p.req->logits_out;
        if (logits_out) logits_out[(MK_M > 1 ? static_cast<size_t>(tok) * P.units_total : 0) + u] = lo;
#pragma unroll
        for (int t = 0; t < MK_M; ++t)
            if (t == tok && arg_better(lo, u, cx.best_v[t], cx.best_i[t])) { cx.best_v[t] = lo; cx.best_i[t] = u; }
    } else if (P.kind == PH_SWIGLU) {
        const float a = lo / (1.f + expf(-lo)) * hi;
        if (P.flags() & PHF_OUT_SPLIT) {   // the layout the next operator's prologue copies straight into shared memory
            uint16_t *o = reinterpret_cast<uint16_t *>(P.out) + (MK_M > 1 ? static_cast<size_t>(tok) * P.out_tok_stride : 0) + mk_xs_index(u);
            float r = a;
#pragma unroll
            for (int sp = 0; sp < MK_S; ++sp) {
                const uint16_t b = f32_to_bf16_bits(r);
                o[static_cast<size_t>(sp) * ((P.units_total + MK_TILE_COLS - 1) / MK_TILE_COLS * MK_TILE_COLS)] = b;
                r -= bf16_bits_to_f32(b);
            }
        } else {
            out[u] = a;
        }
    } else {  // PH_QKV: bias, rotate-half RoPE of q and k, q to the work buffer, k and v to the cache row of this step
        const int half = p.d >> 1;
        const int head = u >> p.half_shift, i = u & (half - 1);
        struct Publish {   // when the unit's stores are done: one more finished unit of this head (release: the stores come first)
            unsigned *counter;
            __device__ ~Publish() { if (counter) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(counter) : "memory"); }
        } publish{p.head_flags ? p.head_ready + head : nullptr};
        const int row_lo = head * p.d + i, row_hi = row_lo + half;
        if (P.bias) {
            lo += pre ? pre_lo : bf16_bits_to_f32(P.bias[row_lo]);
            hi += pre ? pre_hi : bf16_bits_to_f32(P.bias[row_hi]);
        }
        const size_t layer_off = static_cast<size_t>(P.layer()) * p.nkv * p.max_context * p.d;
        if (head < p.nq + p.nkv) {
            const float c = s_rope[tok * 128 + i], sn = s_rope[tok * 128 + half + i];   // the table of this token's position
            const float rlo = lo * c - hi * sn, rhi = hi * c + lo * sn;
            if (head < p.nq) {
                out[row_lo] = rlo;
                out[row_hi] = rhi;
            } else if (p.kv8) {   // compressed cache: the row is left in fp32 for the attention phase, which compresses it whole
                float *dst = p.kv_stage + static_cast<size_t>(head - p.nq) * p.d;
                dst[i] = rlo;
                dst[i + half] = rhi;
            } else {
                uint16_t *dst = p.k_cache + layer_off + (static_cast<size_t>(head - p.nq) * p.max_context + cx.slot_row + tok) * p.d;
                dst[i] = f32_to_bf16_bits(rlo);
                dst[i + half] = f32_to_bf16_bits(rhi);
            }
        } else if (p.kv8) {
            float *dst = p.kv_stage + static_cast<size_t>(p.nkv + head - p.nq - p.nkv) * p.d;
            dst[i] = lo;
            dst[i + half] = hi;
        } else {
            uint16_t *dst = p.v_cache + layer_off + (static_cast<size_t>(head - p.nq - p.nkv) * p.max_context + cx.slot_row + tok) * p.d;
            dst[i] = f32_to_bf16_bits(lo);
            dst[i + half] = f32_to_bf16_bits(hi);
        }
    }
}

// ---- the consumer side of the weight stream --------------------------------------------------------------------
// Optional fine-grained trace of one operator in CTA 0 (compile with -DEDGEFM_TRACE_OP=<operator index>): lane 0 of every
// consumer warp appends %globaltimer stamps (before the wait, data there, tile multiplied) behind the profile table.
#ifdef EDGEFM_TRACE_OP
#define MK_TRACE(k)                                                                                                           \
    do {                                                                                                                      \
        if (p.prof && (&P - p_ops_base) == EDGEFM_TRACE_OP && blockIdx.x == 0 && lane == 0 && t < 16)                          \
            p.prof[static_cast<size_t>(gridDim.x) * p.prof_stride + ((threadIdx.x >> 5) * 16 + t) * 3 + (k)] = global_ns();     \
    } while (0)
#else
#define MK_TRACE(k) do {} while (0)
#endif
// This warp's `n` tiles of operator P: wait, multiply, release; reduce and finish rows where the schedule says so.
//
// The multiplication runs on the tensor cores, not because the operator has the arithmetic intensity of a GEMM (it is a
// matrix-vector product) but because the scalar form needs 17 instructions per 16 bytes of weights (load, 8 conversions, 8
// FMAs) and the warp's serial wait - multiply - refill chain, not HBM, bounded the stream.  One mma.m16n8k16 multiplies a
// 16-row x 16-column block of bf16 weights (A, read with ldmatrix from the swizzled tile) by B = [16 x 8]: columns 0..2 hold
// the three bf16 pieces of the fp32 activations, columns 3..7 are zero.  Accumulation is fp32; the row sum is the sum of
// columns 0..2.  Products of two bf16 values are exact in fp32, so the result differs from an fp32 FMA chain only in the
// order of the additions.
__device__ __forceinline__ bool consume_tiles(const MkParams &p, const MkOp &P, int n, WarpStream &ws, volatile int *abort_flag, ItemCtx &cx,
                                              float *s_partial, const float *s_rope, volatile unsigned *s_issued, unsigned long long *full_bar, int lane) {
    const int warp = static_cast<int>(threadIdx.x >> 5);
    const MkOp *p_ops_base = sm_ops(p);
    (void)p_ops_base;
    // D fragments: rows lane/4 and lane/4 + 8, columns 2 (lane%4), 2 (lane%4) + 1; one accumulator per 64-column block of a tile,
    // so that four independent chains of tensor-core instructions are in flight
    float acc[MK_ACC_CHAINS][4];
#pragma unroll
    for (int cb = 0; cb < MK_ACC_CHAINS; ++cb) { acc[cb][0] = 0.f; acc[cb][1] = 0.f; acc[cb][2] = 0.f; acc[cb][3] = 0.f; }
    const bool paired = P.kind == PH_QKV || P.kind == PH_SWIGLU;
    // B fragments: lanes 0..11 hold piece (lane / 4) of the activations, k indices by lane % 4; the other lanes multiply by zero.
    // They are read from shared memory block by block while the tile is multiplied: from the staged vector, or (PHF_X_GLOBAL:
    // the vector is in global memory in the same form) from a small buffer of this warp, into which the 1.5 KB of the next
    // tile are copied asynchronously (no registers held) as soon as the current tile has been multiplied.
    const bool xg = (P.flags() & PHF_X_GLOBAL) != 0;
    const int kpad2 = (P.K + MK_TILE_COLS - 1) / MK_TILE_COLS * (MK_TILE_COLS * 2);
    unsigned char *wbuf = sm_xbuf(p) + p.xbuf_bytes + warp * mk_wbuf_bytes(MK_M);   // [token][piece][512 (+ pad) bytes]
    const unsigned char *b_base = xg ? wbuf + (lane >> 2) * mk_wbuf_array_bytes(MK_M) + (lane & 3) * 16
                                     : sm_xbuf(p) + (lane >> 2) * xs_stride(P.K) + (lane & 3) * 16;
    auto request_b = [&](int kcol) {
        const unsigned char *src = reinterpret_cast<const unsigned char *>(P.x_src) + kcol * (MK_TILE_COLS * 2) + lane * 16;
#pragma unroll
        for (int c = 0; c < MK_S * MK_M; ++c)   // array c: piece c % MK_S of token c / MK_S
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(wbuf + c * mk_wbuf_array_bytes(MK_M) + lane * 16)),
                         "l"(src + static_cast<size_t>(c / MK_S) * P.x_tok_stride * 2 + static_cast<size_t>(c % MK_S) * kpad2) : "memory");
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    auto load_b = [&](const unsigned char *at) {
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (lane < 4 * MK_S * MK_M) v = *reinterpret_cast<const uint4 *>(at);
        return v;
    };
    // A fragments: ldmatrix.x4 takes from lane l the address of row l % 8 of matrix l / 8; the four matrices are
    // (rows 0..7 | rows 8..15) x (k 0..7 | k 8..15) of a 16 x 16 block
    const int mrow = (lane & 7) + ((lane >> 3) & 1) * 8, khalf = lane >> 4;
    const uint2 *list = sm_tiles(p) + ws.list;
    uint2 d = n > 0 ? list[0] : make_uint2(0u, 0u);
    if (xg && n > 0) request_b(static_cast<int>((d.x >> 20) & 0xffu));
    for (int t = 0; t < n; ++t) {
        const uint2 dn = t + 1 < n ? list[t + 1] : make_uint2(0u, 0u);
        if (d.x & MKT_FIRST) {
#pragma unroll
            for (int cb = 0; cb < MK_ACC_CHAINS; ++cb) { acc[cb][0] = 0.f; acc[cb][1] = 0.f; acc[cb][2] = 0.f; acc[cb][3] = 0.f; }
        }
        const int m = static_cast<int>(d.y & 31u);
        const unsigned char *bl = b_base + (xg ? 0 : static_cast<int>((d.x >> 20) & 0xffu) * (MK_TILE_COLS * 2));
        MK_TRACE(0);
        if (!mbar_wait(&full_bar[warp * MK_MAX_SLOTS + ws.slot], ws.round & 1u, abort_flag, p.spin_limit)) return false;
        MK_TRACE(1);
        if (xg) {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncwarp();
        }
        uint4 bb0 = load_b(bl), bb1 = load_b(bl + 64);   // two k-steps per 16-byte piece
        // The tile: [4 column blocks][rows_total][128 bytes]; rows_total = m, or the m low rows followed by their m partners.
        // M rows 0..7 are rows 0..7 (low rows), M rows 8..15 are rows 8..15 (partners); rows the tile does not have repeat its
        // last row (their sums are never used).  16-byte chunk j of a row is stored at chunk j ^ (row index in the slot % 8).
        const int rows_total = paired ? 2 * m : m;
        const int tr = paired ? (mrow < 8 ? min(mrow, m - 1) : m + min(mrow - 8, m - 1)) : min(mrow, m - 1);
        const unsigned tile = smem_u32(sm_ring(p, warp) + ws.slot * p.slot_bytes);
#pragma unroll
        for (int cb = 0; cb < MK_TILE_COLS / 64; ++cb) {
            const int blk = cb * rows_total + tr;
            const unsigned row_addr = tile + static_cast<unsigned>(blk) * 128u;
            const unsigned sw = static_cast<unsigned>(blk & 7);
            uint4 nb0 = bb0, nb1 = bb1;
            if (cb + 1 < MK_TILE_COLS / 64) { nb0 = load_b(bl + (cb + 1) * 128); nb1 = load_b(bl + (cb + 1) * 128 + 64); }
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                const int s = cb * 4 + ks;
                const unsigned addr = row_addr + (((static_cast<unsigned>(ks * 2 + khalf)) ^ sw) << 4);
                unsigned a0, a1, a2, a3;
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3) : "r"(addr));
                const uint4 bb = ks < 2 ? bb0 : bb1;
                const unsigned b0 = (s & 1) ? bb.z : bb.x, b1 = (s & 1) ? bb.w : bb.y;
                asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                             : "+f"(acc[s % MK_ACC_CHAINS][0]), "+f"(acc[s % MK_ACC_CHAINS][1]), "+f"(acc[s % MK_ACC_CHAINS][2]), "+f"(acc[s % MK_ACC_CHAINS][3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
            }
            bb0 = nb0; bb1 = nb1;
        }
        __syncwarp();
        MK_TRACE(2);
        if (xg && t + 1 < n) request_b(static_cast<int>((dn.x >> 20) & 0xffu));   // every lane has read the buffer (the sync above)
        if (lane == 0 && !fetch_next_tile(p, ws, ws.slot, abort_flag, s_issued, full_bar, warp)) return false;   // refill the slot
        if (++ws.slot == p.slots) { ws.slot = 0; ++ws.round; }
        ++ws.consumed;
        if (d.x & MKT_FLUSH) {
            // row sums: columns 0, 1 are in the lane with lane % 4 == 0, column 2 in its neighbour; then lanes 2r, 2r+1 take row r
            // (the accumulators start over with the next FIRST tile)
            float d0 = acc[0][0], d1 = acc[0][1], d2 = acc[0][2], d3 = acc[0][3];
#pragma unroll
            for (int c = 1; c < MK_ACC_CHAINS; ++c) { d0 += acc[c][0]; d1 += acc[c][1]; d2 += acc[c][2]; d3 += acc[c][3]; }
#pragma unroll
            for (int tk = 0; tk < MK_M; ++tk) {
                float lo, hi;
                if constexpr (MK_M == 1) {
                    lo = d0 + d1 + __shfl_down_sync(0xffffffffu, d0, 1);
                    hi = d2 + d3 + __shfl_down_sync(0xffffffffu, d2, 1);
                } else {
                    // token tk: columns 3 tk .. 3 tk + 2; column c is register c % 2 of the lane with lane % 4 == c / 2
                    lo = 0.f; hi = 0.f;
#pragma unroll
                    for (int sp = 0; sp < MK_S; ++sp) {
                        const int c = MK_S * tk + sp;
                        lo += __shfl_sync(0xffffffffu, (c & 1) ? d1 : d0, (lane & ~3) + (c >> 1));
                        hi += __shfl_sync(0xffffffffu, (c & 1) ? d3 : d2, (lane & ~3) + (c >> 1));
                    }
                }
                const int src = ((lane >> 1) & 7) * 4;
                const float vlo = __shfl_sync(0xffffffffu, lo, src), vhi = __shfl_sync(0xffffffffu, hi, src);
                const float v = lane < 16 ? vlo : vhi;
                const int j = lane >> 1;
                if (tk >= cx.m_run) continue;     // (uniform over the warp)
                if (d.y & MKT_DIRECT) {
                    const float hi2 = __shfl_down_sync(0xffffffffu, v, 16);   // partner row 8 + j of unit j
                    const int v0 = static_cast<int>((d.y >> 5) & 15u);
                    const int u = static_cast<int>(d.x & 0xfffffu) + j;
                    if (!(lane & 1) && j < m && j >= v0 && (!paired || lane < 16))
                        apply_epilogue(p, P, cx, s_rope, u, v * cx.rscale[tk], hi2 * cx.rscale[tk], false, 0.f, 0.f, tk);
                } else {
                    const int slot = static_cast<int>((d.y >> 10) & 1023u);
                    if (slot >= MK_PARTIAL_SLOTS) return diag_fail(p, abort_flag, 2, slot, 0);
                    if (!(lane & 1)) s_partial[(slot * MK_M + tk) * MK_TILE_ROWS + j] = v;
                }
            }
        }
        d = dn;
    }
    ws.list += n;
    return true;
}

// One weight-streaming operator: prologue (stage the activation vector, RMSNorm folded in: x*w is staged
// and the scalar rsqrt(mean x^2 + eps) is applied to the dot products), then this warp's tiles, then the units
// whose columns were shared between warps.
// merge_attn > 0: the input is the attention output, still split into merge_attn chunk partials per head
// (m, l, unnormalised o); the exact log-sum-exp merge is done here, in chunk order, by every CTA.
__device__ __forceinline__ bool gemv_phase(const MkParams &p, int ph, int op_in_layer, WarpStream &ws, volatile int *abort_flag, float *s_part,
                                           float *s_partial, const float *s_rope, ItemCtx &cx, const int (&tokens)[MK_M], int merge_attn, int tid,
                                           int &prof_idx, volatile unsigned *s_issued, unsigned long long *full_bar) {
    const MkOp &P = sm_ops(p)[ph];
    unsigned char *const xs0 = sm_xbuf(p);
    const int xstride = xs_stride(P.K);
    const int *s_tab = sm_tab(p);
    const int lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x;
    const int n4 = P.K >> 2;
    // Token tk of the call stages its vector into arrays 3 tk .. 3 tk + 2.  The pieces of all tokens form one list of items
    // (token-major) that the threads share, so that the loads of all tokens are in flight together.
    const int m_run = cx.m_run;
    const int n_items = m_run * n4;
    float ss[MK_M];
#pragma unroll
    for (int t = 0; t < MK_M; ++t) ss[t] = 0.f;
    if (merge_attn > 0) {
        const int nch = merge_attn;   // chunks per head of the attention pass, the same for every token of the call
        const int d4 = p.d >> 2;
        const int n_stat = p.nq * nch;
        float *sm_m = s_partial;                     // [token][nq][nch] chunk maxima
        float *sm_l = s_partial + m_run * n_stat;    // [token][nq][nch] chunk denominators
        // A thread merges piece o4 of a token's vector (16 bytes: 4 dims of one head): all its chunk partials are requested at
        // once, before the statistics are waited for.  (Spreading the left-over pieces of a vector longer than the CTA over
        // all threads, parked in shared memory and summed after one more sync, was measured slower twice: 4.6 instead of
        // 3.7 us for this prologue at the 1.5B shape even without spills.)
        float4 ob[MK_ATT_SPLIT_MAXC];
        auto load_partials = [&](int item) {
            const int tk = MK_M > 1 ? item / n4 : 0, o4 = item - tk * n4;
            const int h = o4 / d4, j4 = o4 - h * d4;
            const float4 *po = reinterpret_cast<const float4 *>(p.part_o + (static_cast<size_t>(tk) * p.nq + h) * p.max_chunks * p.d) + j4;
#pragma unroll
            for (int c = 0; c < MK_ATT_SPLIT_MAXC; ++c)
                if (c < nch) ob[c] = __ldcg(po + static_cast<size_t>(c) * d4);
        };
        if (tid < n_items) load_partials(tid);
        for (int i = tid; i < m_run * n_stat; i += MK_NT) {
            const int hh = i / nch, c = i - hh * nch;      // hh = token * nq + head
            sm_m[i] = __ldcg(p.part_m + hh * p.max_chunks + c);
            sm_l[i] = __ldcg(p.part_l + hh * p.max_chunks + c);
        }
        cta_sync();
        for (int item = tid; item < n_items; item += MK_NT) {
            if (item != tid) load_partials(item);
            const int tk = MK_M > 1 ? item / n4 : 0, o4 = item - tk * n4;
            const int h = o4 / d4;
            const float *hm = sm_m + (tk * p.nq + h) * nch, *hl = sm_l + (tk * p.nq + h) * nch;
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
            stage_piece(xs0 + tk * (MK_S * xstride), xstride, o4, acc);
        }
    } else if (P.flags() & PHF_X_GLOBAL) {
        // nothing to stage: the consumer warps read the vector from global memory as they go
    } else {
        constexpr int PU = 4;  // loads in flight per thread
        for (int base = tid; base < n_items; base += MK_NT * PU) {
            float4 v[PU];
            uint2 w[PU];
#pragma unroll
            for (int u = 0; u < PU; ++u) {
                const int item = base + u * MK_NT;
                if (item < n_items) {
                    const int tk = MK_M > 1 ? item / n4 : 0, i4 = item - tk * n4;
                    if (P.x_src) {
                        v[u] = __ldcg(reinterpret_cast<const float4 *>(P.x_src + (MK_M > 1 ? static_cast<size_t>(tk) * P.x_tok_stride : 0)) + i4);
                    } else {  // first operator of the step: the embedding row is the residual stream
                        int token = tokens[0];
#pragma unroll
                        for (int t = 1; t < MK_M; ++t) token = tk == t ? tokens[t] : token;
                        const uint2 e = *reinterpret_cast<const uint2 *>(p.embed + static_cast<size_t>(token) * p.H + i4 * 4);
                        v[u] = make_float4(bf16lo(e.x), bf16hi(e.x), bf16lo(e.y), bf16hi(e.y));
                    }
                    if (P.norm_w) w[u] = *reinterpret_cast<const uint2 *>(P.norm_w + i4 * 4);
                }
            }
#pragma unroll
            for (int u = 0; u < PU; ++u) {
                const int item = base + u * MK_NT;
                if (item < n_items) {
                    const int tk = MK_M > 1 ? item / n4 : 0, i4 = item - tk * n4;
                    float4 t = v[u];
                    if (!P.x_src && cta == 0) reinterpret_cast<float4 *>(p.x + (MK_M > 1 ? static_cast<size_t>(tk) * p.H : 0))[i4] = t;
                    if (P.norm_w) {
                        float sq = 0.f;
                        sq = fmaf(t.x, t.x, sq); sq = fmaf(t.y, t.y, sq); sq = fmaf(t.z, t.z, sq); sq = fmaf(t.w, t.w, sq);
#pragma unroll
                        for (int tt = 0; tt < MK_M; ++tt) ss[tt] += tk == tt ? sq : 0.f;
                        t.x *= bf16lo(w[u].x); t.y *= bf16hi(w[u].x); t.z *= bf16lo(w[u].y); t.w *= bf16hi(w[u].y);
                    }
                    stage_piece(xs0 + tk * (MK_S * xstride), xstride, i4, t);
                }
            }
        }
    }
    if (!(P.flags() & PHF_X_GLOBAL)) {   // columns past K of the last 256-column piece multiply zero-filled weights: the activations there are zero
        const int c1 = (P.K + MK_TILE_COLS - 1) / MK_TILE_COLS * MK_TILE_COLS;
        for (int c = P.K + 2 * tid; c < c1; c += 2 * MK_NT)
#pragma unroll
            for (int sp = 0; sp < MK_S * MK_M; ++sp) *reinterpret_cast<unsigned *>(xs0 + sp * xstride + mk_xs_index(c) * 2) = 0u;
    }
    if (P.norm_w) {
#pragma unroll
        for (int t = 0; t < MK_M; ++t) {
            const float tot = warp_sum(ss[t]);
            if (lane == 0) s_part[t * MK_NW + warp] = tot;
        }
    }
    cta_sync();
    prof_stamp(p, tid, prof_idx);   // activation vector staged
#pragma unroll
    for (int tk = 0; tk < MK_M; ++tk) {
        cx.rscale[tk] = 1.f;
        if (P.norm_w && tk < cx.m_run) {
            float tot = 0.f;
#pragma unroll
            for (int w = 0; w < MK_NW; ++w) tot += s_part[tk * MK_NW + w];
            cx.rscale[tk] = rsqrtf(tot / static_cast<float>(P.K) + p.eps);
        }
    }
    const int *tab = s_tab + warp * MK_WARP_TAB;
    const int n_tiles = op_in_layer < 4 ? tab[1 + op_in_layer] : tab[6];
    // units whose columns are shared between warps are finished after the tiles, one unit per thread; what their epilogue
    // adds (old residual value, biases) is fetched now so that the load latency overlaps the arithmetic
    const int *ctab = s_tab + MK_NW * MK_WARP_TAB + 2 * op_in_layer;
    const int n_comb = ctab[1];
    const MkCombine *cb = sm_combines(p) + ctab[0];
    const bool paired = P.kind == PH_QKV || P.kind == PH_SWIGLU;
    float pre_lo = 0.f, pre_hi = 0.f;
    if (tid < n_comb * MK_TILE_ROWS) {
        const MkCombine e = cb[tid >> 4];
        const int j = tid & 15, m = static_cast<int>(e.y & 0xffu), v0 = static_cast<int>(e.y >> 8);
        if (j < m && j >= v0 && !(paired && j >= 8)) {
            const int u = static_cast<int>(e.x) + j;
            if (P.kind == PH_RESID) {
                pre_lo = __ldcg(P.out + u);
            } else if (P.kind == PH_QKV && P.bias) {
                const int row_lo = unit_row(p, PH_QKV, u);
                pre_lo = bf16_bits_to_f32(P.bias[row_lo]);
                pre_hi = bf16_bits_to_f32(P.bias[row_lo + (p.d >> 1)]);
            }
        }
    }
    bool ok = consume_tiles(p, P, n_tiles, ws, abort_flag, cx, s_partial, s_rope, s_issued, full_bar, lane);
    // their partial sums meet here, slots in order
    if (n_comb > 0) {
        cta_sync();
        if (ok && !*abort_flag) {
            for (int idx = tid; idx < n_comb * MK_TILE_ROWS; idx += MK_NT) {
                const MkCombine e = cb[idx >> 4];
                const int j = idx & 15, m = static_cast<int>(e.y & 0xffu), v0 = static_cast<int>(e.y >> 8);
                if (j >= m || j < v0 || (paired && j >= 8)) continue;
#pragma unroll
                for (int tk = 0; tk < MK_M; ++tk) {
                    if (tk >= cx.m_run) break;
                    float lo = 0.f, hi = 0.f;
                    for (unsigned s = 0; s < e.w; ++s) {
                        const float *sp = s_partial + ((e.z + s) * MK_M + tk) * MK_TILE_ROWS;
                        lo += sp[j];
                        if (paired) hi += sp[8 + j];
                    }
                    // (what the epilogue adds was fetched ahead for the first token only)
                    apply_epilogue(p, P, cx, s_rope, static_cast<int>(e.x) + j, lo * cx.rscale[tk], hi * cx.rscale[tk], idx == tid && (tk == 0 || P.kind == PH_QKV), pre_lo,
                                   pre_hi, tk);
                }
            }
        }
    }
    return ok;
}

// ---- attention -----------------------------------------------------------------------------------------------
// A CTA serves HG query heads of one GQA group over one chunk of the cached positions: HG = G (the whole
// group shares every K/V row read: least traffic, for long contexts) or HG = 1 (every query head has
// its own CTAs: G times more parallelism for short, latency-bound contexts; K/V re-reads hit L2).
// Scores: MK_ATT_LPP lanes per position, each lane reads interleaved 16-byte pieces of the K row from
// global memory; P V: every lane owns d/32 dims.  Shared memory (the idle activation buffer): q,
// probabilities, warp merge area, chunk statistics.  The CTA that arrives last for its head group
// (atomic ticket, no waiting) merges the chunks exactly:  m = max m_c, l = sum l_c e^{m_c - m},
// o = sum o_c e^{m_c - m} / l, in index order.
//
// Q8: the compressed cache (Sec. 3.9 of the paper, KV~ = C(KV) with reconstruction on demand; the paper fixes no C): every
// cached row is d signed 8-bit codes and one fp32 scale (scale = amax / 127).  The codes are turned into fp32 exactly, two
// instructions each (the byte + 128 dropped into the mantissa of 2^23, minus 2^23 + 128); the K scale multiplies the finished
// score, the V scale the probability.  The row this step appends was left in fp32 by the QKV epilogue; the CTA whose chunk
// ends with it compresses it into the cache (two warps, one row each) before anybody reads it.
__device__ __forceinline__ void codes4_to_f32(uint32_t w, float (&f)[4]) {
    const uint32_t u = w ^ 0x80808080u;     // two's complement -> offset binary
    f[0] = __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7440)) - 8388736.f;
    f[1] = __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7441)) - 8388736.f;
    f[2] = __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7442)) - 8388736.f;
    f[3] = __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7443)) - 8388736.f;
}
// wait_heads: there was no grid barrier behind the QKV projection; the CTA waits (bounded) until the heads it reads are
// complete: its query head and, if its chunk ends with the row this step appends, the K and V head of its group.  Every
// finished unit (row pair) of a head adds one to the head's counter (apply_epilogue), d/2 per layer.
template <int D, int HG, int LPP, bool Q8 = false>
__device__ __forceinline__ void attention_phase(const MkParams &p, int layer, int n, int min_chunk, bool defer_merge,
                                                unsigned char *xbuf, int tid, int *s_flag, bool wait_heads = false,
                                                volatile int *abort_flag = nullptr, int *prof_idx = nullptr, int tok = 0, int m_run = 1) {
    static_assert(!(Q8 && MK_M > 1), "blocks of several tokens are built for the plain cache only");
    // token `tok` of a call of m_run tokens: its own queries and partial results; n counts the rows of the tokens before it
    constexpr int TILE = 32 / LPP;   // positions per warp iteration
    constexpr int DV = D / 32, CPR = D / 8, CPL = CPR / LPP;
    constexpr int CPL8 = D / 16 / LPP;                  // 16-byte pieces (16 codes) of a compressed K row per lane
    static_assert(!Q8 || (D / 16) % LPP == 0, "compressed rows are split into whole 16-byte pieces");
    constexpr int MW = MK_NW;                            // every warp publishes its partial: one sync, then one pass
    const int lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x, ncta = gridDim.x;
    const int G = p.nq / p.nkv;
    const int groups = p.nq / HG;                       // head groups served by separate CTAs
    int nch, chunk_len;
    // a block (m_run > 1, tok < 0): all its tokens in this one pass, every (token, head) with CTAs of its own; n is the
    // longest token's length and token t attends to n - (m_run - 1 - t) rows
    const bool all_tokens = MK_M > 1 && tok < 0;
    att_chunking(p, n, HG, min_chunk, TILE, ncta, nch, chunk_len, all_tokens ? m_run : 1);
    if (all_tokens) {
        tok = min(cta / (nch * groups), m_run - 1);
        n -= m_run - 1 - tok;
    }
    if (cta >= nch * groups * (all_tokens ? m_run : 1)) {
        if (wait_heads && (all_tokens || tok == 0)) prof_stamp(p, tid, *prof_idx);
        return;
    }
    const float *const q_tok = p.q + static_cast<size_t>(tok) * p.nq * D;
    float *const attn_tok = p.attn + static_cast<size_t>(tok) * p.nq * D;
    float *const part_o = p.part_o + static_cast<size_t>(tok) * p.nq * p.max_chunks * D;
    float *const part_m = p.part_m + static_cast<size_t>(tok) * p.nq * p.max_chunks, *const part_l = p.part_l + static_cast<size_t>(tok) * p.nq * p.max_chunks;
    const int grp = MK_M > 1 ? (cta / nch) % groups : cta / nch, c = cta - (cta / nch) * nch;
    const int qh0 = grp * HG;                            // first query head of this CTA
    const int g = qh0 / G;                               // its kv head
    const int t0 = c * chunk_len, t1 = min(n, t0 + chunk_len);
    if (wait_heads) {
        if (tid == 0 && !*abort_flag) {
            const unsigned target = static_cast<unsigned>(layer + 1) * (D / 2) * static_cast<unsigned>(m_run);
            const unsigned long long w0 = global_ns();
            for (unsigned it = 0;; ++it) {
                bool ready = ld_acquire_gpu(p.head_ready + qh0) >= target;
                if (ready && t1 > n - 1 - tok) ready = ld_acquire_gpu(p.head_ready + p.nq + g) >= target && ld_acquire_gpu(p.head_ready + p.nq + p.nkv + g) >= target;
                if (ready) break;
                if ((it & 63u) == 63u && global_ns() - w0 > p.spin_limit) { *abort_flag = 1; p.state->status = 6; break; }
            }
        }
        cta_sync();
        if (all_tokens || tok == 0) prof_stamp(p, tid, *prof_idx);   // the heads this CTA reads are complete
    }

    float *qs = reinterpret_cast<float *>(xbuf);               // [HG][D]
    float *ps = qs + HG * D;                                    // [NW][HG][TILE]
    float *mg_m = ps + MK_NW * HG * TILE;                       // [MW][HG]
    float *mg_l = mg_m + MW * HG;                               // [MW][HG]
    float *mg_o = mg_l + MW * HG;                               // [MW][HG][D]
    float *cm = mg_o + MW * HG * D;                             // [HG][max_chunks] chunk maxima
    float *cl = cm + HG * p.max_chunks;                         // [HG][max_chunks] chunk denominators

    const size_t head_off = (static_cast<size_t>(layer) * p.nkv + g) * p.max_context * D;
    const uint16_t *kg = p.k_cache + head_off;
    const uint16_t *vg = p.v_cache + head_off;
    // compressed cache: the same arrays hold one byte per element; the scales are [L][nkv][max_context]
    const unsigned char *kg8 = reinterpret_cast<const unsigned char *>(p.k_cache) + head_off;
    const unsigned char *vg8 = reinterpret_cast<const unsigned char *>(p.v_cache) + head_off;
    const float *ksg = p.k_scale + (static_cast<size_t>(layer) * p.nkv + g) * p.max_context;
    const float *vsg = p.v_scale + (static_cast<size_t>(layer) * p.nkv + g) * p.max_context;
    float *pw = ps + warp * (HG * TILE);
    const int pi = lane / LPP, part = lane % LPP;

    if constexpr (Q8) {
        if (t1 == n && warp < 2) {
            // the row appended by this step: warp 0 compresses k (after RoPE), warp 1 v; every lane DV values
            const float *src = p.kv_stage + (static_cast<size_t>(warp) * p.nkv + g) * D + lane * DV;
            float xv[DV];
            float amax = 0.f;
#pragma unroll
            for (int e = 0; e < DV; ++e) { xv[e] = __ldcg(src + e); amax = fmaxf(amax, fabsf(xv[e])); }
            amax = warp_max(amax);
            const float inv = amax > 0.f ? __fdiv_rn(127.0f, amax) : 0.f;
            uint32_t packed = 0u;
#pragma unroll
            for (int e = 0; e < DV; ++e) {
                const float c = fminf(fmaxf(rintf(__fmul_rn(xv[e], inv)), -127.f), 127.f);
                packed |= (static_cast<uint32_t>(static_cast<int>(c)) & 0xffu) << (8 * e);
            }
            unsigned char *dst = const_cast<unsigned char *>(warp == 0 ? kg8 : vg8) + static_cast<size_t>(n - 1) * D + lane * DV;
            if constexpr (DV == 4) *reinterpret_cast<uint32_t *>(dst) = packed;
            else *reinterpret_cast<uint16_t *>(dst) = static_cast<uint16_t>(packed);
            if (lane == 0) const_cast<float *>(warp == 0 ? ksg : vsg)[n - 1] = amax > 0.f ? __fdiv_rn(amax, 127.0f) : 0.f;
        }
        // (published to the rest of the CTA by the sync that follows the staging of the queries)
    }

    // K and V rows of one warp iteration: K pieces of this lane's position, raw bf16 pairs (or 8-bit codes) of V (converted when
    // used to keep the register footprint small)
    uint4 kk[Q8 ? CPL8 : CPL];
    uint32_t vraw[TILE][Q8 ? 1 : DV / 2];
    float ksc = 0.f, vsc = 0.f;   // scales of this lane's position (compressed cache)
    auto load_kv = [&](int tt) {
        const bool pvalid = tt + pi < t1;
        if constexpr (Q8) {
#pragma unroll
            for (int j = 0; j < CPL8; ++j)
                kk[j] = pvalid ? __ldcg(reinterpret_cast<const uint4 *>(kg8 + static_cast<size_t>(tt + pi) * D) + j * LPP + part)
                               : make_uint4(0u, 0u, 0u, 0u);
            ksc = pvalid ? __ldcg(ksg + tt + pi) : 0.f;
            vsc = pvalid ? __ldcg(vsg + tt + pi) : 0.f;
#pragma unroll
            for (int x = 0; x < TILE; ++x) {
                const int t = tt + x;
                const unsigned char *vp = vg8 + static_cast<size_t>(t) * D + lane * DV;
                if constexpr (DV == 4) vraw[x][0] = t < t1 ? __ldcg(reinterpret_cast<const unsigned *>(vp)) : 0u;
                else vraw[x][0] = t < t1 ? static_cast<unsigned>(__ldcg(reinterpret_cast<const unsigned short *>(vp))) : 0u;
            }
        } else {
#pragma unroll
            for (int j = 0; j < CPL; ++j)
                kk[j] = pvalid ? __ldcg(reinterpret_cast<const uint4 *>(kg + static_cast<size_t>(tt + pi) * D) + j * LPP + part)
                               : make_uint4(0, 0, 0, 0);
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
        }
    };
    int tt = t0 + warp * TILE;
    for (int i = tid; i < HG * D; i += MK_NT) qs[i] = __ldcg(q_tok + static_cast<size_t>(qh0) * D + i) * p.scale;
    cta_sync();

    float m[HG], l[HG], o[HG][DV];
#pragma unroll
    for (int h = 0; h < HG; ++h) {
        m[h] = -INFINITY; l[h] = 0.f;
#pragma unroll
        for (int e = 0; e < DV; ++e) o[h][e] = 0.f;
    }

    while (tt < t1) {
        const bool pvalid = tt + pi < t1;
        load_kv(tt);
        float s[HG];
#pragma unroll
        for (int h = 0; h < HG; ++h) s[h] = 0.f;
        if constexpr (Q8) {
#pragma unroll
            for (int j = 0; j < CPL8; ++j) {
                const int cc = j * LPP + part;
                const uint32_t words[4] = {kk[j].x, kk[j].y, kk[j].z, kk[j].w};
#pragma unroll
                for (int wi = 0; wi < 4; ++wi) {
                    float f[4];
                    codes4_to_f32(words[wi], f);
#pragma unroll
                    for (int h = 0; h < HG; ++h) {
                        const float4 q4 = *reinterpret_cast<const float4 *>(qs + h * D + cc * 16 + wi * 4);
                        s[h] = fmaf(f[0], q4.x, s[h]); s[h] = fmaf(f[1], q4.y, s[h]);
                        s[h] = fmaf(f[2], q4.z, s[h]); s[h] = fmaf(f[3], q4.w, s[h]);
                    }
                }
            }
        } else {
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
        }
#pragma unroll
        for (int h = 0; h < HG; ++h) {
#pragma unroll
            for (int x = 1; x < LPP; x <<= 1) s[h] += __shfl_xor_sync(0xffffffffu, s[h], x);
            if constexpr (Q8) s[h] *= ksc;
            if (!pvalid) s[h] = -INFINITY;
            const float mn = fmaxf(m[h], warp_max(s[h]));
            const float corr = __expf(m[h] - mn);
            const float pr = pvalid ? __expf(s[h] - mn) : 0.f;
            l[h] = l[h] * corr + (part == 0 ? pr : 0.f);
#pragma unroll
            for (int e = 0; e < DV; ++e) o[h][e] *= corr;
            m[h] = mn;
            if (part == 0) pw[h * TILE + pi] = Q8 ? pr * vsc : pr;
        }
        __syncwarp();
#pragma unroll
        for (int tb = 0; tb < TILE; tb += 4) {
            float v[4][DV];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                if constexpr (Q8) {
                    float f[4];
                    codes4_to_f32(vraw[tb + x][0], f);
#pragma unroll
                    for (int e = 0; e < DV; ++e) v[x][e] = f[e];
                } else {
#pragma unroll
                    for (int e = 0; e < DV; e += 2) {
                        v[x][e] = bf16lo(vraw[tb + x][e / 2]);
                        v[x][e + 1] = bf16hi(vraw[tb + x][e / 2]);
                    }
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
        tt += MK_NW * TILE;
    }

    // merge the warps of the CTA: every warp publishes (m, l, o) (idle warps carry m = -inf and weigh 0), one sync, then
    // every output element is merged over the warps in index order.
    float lt[HG];
#pragma unroll
    for (int h = 0; h < HG; ++h) lt[h] = warp_sum(l[h]);
#pragma unroll
    for (int h = 0; h < HG; ++h) {
        if (lane == 0) { mg_m[warp * HG + h] = m[h]; mg_l[warp * HG + h] = lt[h]; }
#pragma unroll
        for (int e = 0; e < DV; ++e) mg_o[(warp * HG + h) * D + lane * DV + e] = o[h][e];
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
            attn_tok[qh * D + j] = oo / ll;
        } else {
            part_o[(static_cast<size_t>(qh) * p.max_chunks + c) * D + j] = oo;
            if (j == 0) { part_m[qh * p.max_chunks + c] = mm; part_l[qh * p.max_chunks + c] = ll; }
        }
    }
    if (nch == 1 || defer_merge) return;   // deferred: the next operator's prologue merges the chunks
    __threadfence();
    cta_sync();
    if (tid == 0) *s_flag = (atomicAdd(p.tickets + grp, 1u) == static_cast<unsigned>(nch - 1)) ? 1 : 0;
    cta_sync();
    if (!*s_flag) return;

    // Last CTA of this head group: merge the chunks.  All loads of a batch (up to CB partial vectors per thread) are
    // issued before any is used.
    __threadfence();
    constexpr int CB = 8;
    for (int i = tid; i < HG * nch; i += MK_NT) {
        const int h = i / nch, cc = i - h * nch;
        cm[h * p.max_chunks + cc] = __ldcg(part_m + (qh0 + h) * p.max_chunks + cc);
        cl[h * p.max_chunks + cc] = __ldcg(part_l + (qh0 + h) * p.max_chunks + cc);
    }
    cta_sync();
    for (int out = tid; out < HG * D / 4; out += MK_NT) {     // output (h, j4) of this thread
        const int oh = out / (D / 4), oj4 = out - oh * (D / 4);
        const float4 *po = reinterpret_cast<const float4 *>(part_o + static_cast<size_t>(qh0 + oh) * p.max_chunks * D) + oj4;
        const float *hm = cm + oh * p.max_chunks, *hl = cl + oh * p.max_chunks;
        float mm = -INFINITY;
        for (int cc = 0; cc < nch; ++cc) mm = fmaxf(mm, hm[cc]);
        float ll = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int c0 = 0; c0 < nch; c0 += CB) {
            float4 ob[CB];
#pragma unroll
            for (int u = 0; u < CB; ++u)
                ob[u] = (c0 + u < nch) ? __ldcg(po + static_cast<size_t>(c0 + u) * (D / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
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
        reinterpret_cast<float4 *>(attn_tok)[(qh0 + oh) * (D / 4) + oj4] = acc;
    }
    if (tid == 0) p.tickets[grp] = 0u;
}

// ---- the kernel -----------------------------------------------------------------------------------------------
// LONG = false: contexts that always run attention with one query head per CTA group (max_context <=
// att_split_max_n); the grouped variant is then not compiled in, which keeps the register footprint small.
// Q8 (long build only): the variant for the compressed cache, a kernel of its own so that the plain cache's attention loop
// keeps its register allocation (one kernel holding both lost 1.6 % at the 7B / 32k shape).
template <int D, int G, bool LONG, bool Q8 = false>
__global__ void __launch_bounds__(MK_THREADS, 1) decode_megakernel(const MkParams p) {
    __shared__ __align__(8) unsigned long long full_bar[MK_NW * MK_MAX_SLOTS];
    __shared__ float s_rope[MK_M * 128];     // per token of the call: cos | sin of its position
    __shared__ float s_part[MK_M * MK_NW];
    __shared__ __align__(16) float s_partial[MK_M * MK_PARTIAL_FLOATS];
    __shared__ float s_bv[MK_M * MK_NW];
    __shared__ int s_bi[MK_M * MK_NW];
    __shared__ int s_flag;
    __shared__ int s_abort;
    __shared__ unsigned s_issued[MK_NW];   // tiles fetched so far per consumer warp (read by the L2 prefetch warp)

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x, ncta = gridDim.x;
    if (tid == 0) {
        for (int i = 0; i < MK_NW * MK_MAX_SLOTS; ++i) mbar_init(&full_bar[i], 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < MK_NW) s_issued[tid] = 0u;
    {
        const int n16 = p.nph * static_cast<int>(sizeof(MkOp) / 16);
        const uint4 *src = reinterpret_cast<const uint4 *>(p.ops);
        uint4 *dst = reinterpret_cast<uint4 *>(sm_ops(p));
        for (int i = tid; i < n16; i += MK_THREADS) dst[i] = src[i];
        const int *tsrc = p.cta_tab + static_cast<size_t>(cta) * p.cta_tab_ints;
        for (int i = tid; i < p.cta_tab_ints; i += MK_THREADS) sm_tab(p)[i] = tsrc[i];
        const int t0 = tsrc[MK_NW * MK_WARP_TAB + 10], nt = min(tsrc[MK_NW * MK_WARP_TAB + 11], p.sched_bytes / 8);
        for (int i = tid; i < nt; i += MK_THREADS) sm_tiles(p)[i] = p.tiles[t0 + i];
        const int c0 = tsrc[MK_NW * MK_WARP_TAB + 12], nc = tsrc[MK_NW * MK_WARP_TAB + 13];
        MkCombine *cdst = reinterpret_cast<MkCombine *>(mk_smem + p.ops_bytes + p.tab_bytes + ((nt * 8 + 15) & ~15));
        if ((nt * 8 + 15) / 16 * 16 + nc * 16 <= p.sched_bytes)
            for (int i = tid; i < nc; i += MK_THREADS) cdst[i] = p.combines[c0 + i];
    }
    __syncthreads();   // the only CTA-wide sync: from here on the prefetch warp and the consumers go separate ways
    volatile int *abort_flag = &s_abort;

    if (warp == MK_NW) {
        prefetch_tiles(p, abort_flag, s_issued, lane);
        return;
    }

    // The small per-layer vectors (norm weights, biases) are read on the critical path right after a grid barrier;
    // ask L2 for all of them now (they stay: the weight stream is evict-first).
    for (int i = cta * MK_NT + tid; i < p.nph * 64; i += ncta * MK_NT) {
        const MkOp &P = sm_ops(p)[i >> 6];
        const int line = i & 63;   // 128-byte line of the vector
        if (P.norm_w && line * 64 < P.K) asm volatile("prefetch.global.L2 [%0];" ::"l"(P.norm_w + line * 64));
        if (P.bias && P.kind == PH_QKV && line * 64 < 2 * P.units_total) asm volatile("prefetch.global.L2 [%0];" ::"l"(P.bias + line * 64));
    }

    WarpStream ws;
    {
        const int *tab = sm_tab(p) + warp * MK_WARP_TAB;
        ws.next = TileCursor{tab[7] == 0 ? p.n_layers : 0, 0, 0u};
        ws.nd = sm_tiles(p)[(tab[7] == 0 ? tab[5] : tab[0])];
        ws.list = tab[0];
        ws.n_layer = tab[7]; ws.list_layer = tab[0]; ws.list_lm = tab[5];
        ws.total = static_cast<unsigned>(tab[7]) * p.n_layers + tab[6];
    }
    ws.slot = 0; ws.round = 0; ws.consumed = 0;
    ws.fenced_op = -1;
    bool ok = true;
    const int rt = p.req->token, rp = p.req->position;
    const int token = rt >= 0 ? rt : p.state->next_token;
    const int pos = rp >= 0 ? rp : p.state->next_position;
    const int slot_row = p.state->cur_len;
    const int half = p.d >> 1;
    // a block: the token above followed by the proposed continuation, at consecutive positions and cache slots
    const int m_run = MK_M > 1 ? min(max(p.req->m, 1), MK_M) : 1;
    int tokens[MK_M];
    tokens[0] = token;
#pragma unroll
    for (int t = 1; t < MK_M; ++t) tokens[t] = t < m_run ? p.req->draft[t - 1] : 0;
    bool tokens_ok = true;
#pragma unroll
    for (int t = 0; t < MK_M; ++t) tokens_ok = tokens_ok && tokens[t] >= 0 && tokens[t] < p.V;
    if (!tokens_ok || slot_row < 0 || slot_row + m_run > p.max_context || pos < 0 || (smem_u32(sm_ring(p, 0)) & 1023u)) {
        if (tid == 0) diag_fail(p, abort_flag, 3, token, slot_row);   // corrupt request/state (or ring slots off their 1 KB boundary): compute nothing
        ok = false;
    }
    if (ok) {  // rotary tables of the tokens' positions; fp64 angle, rounded once
        for (int i = tid; i < m_run * half; i += MK_NT) {
            const int t = i / half, f = i - t * half;
            double sn, cs;
            sincos(static_cast<double>(pos + t) * p.inv_freq[f], &sn, &cs);
            s_rope[t * 128 + f] = static_cast<float>(cs);
            s_rope[t * 128 + half + f] = static_cast<float>(sn);
        }
    }
    if (ok && cta == 0 && tid == 0) { p.state->token = token; p.state->position = pos; }
    if (ok && cta == 1 % ncta && p.nph > 2) {
        // the MLP activation arrays in global memory are read in whole 256-column pieces: columns F.. of the last piece are zero
        // (the gate/up epilogues, grid barriers later, write columns < F only)
        const int fpad = (p.F + MK_TILE_COLS - 1) / MK_TILE_COLS * MK_TILE_COLS;
        uint16_t *a = reinterpret_cast<uint16_t *>(sm_ops(p)[2].out);
        for (int c = p.F + tid; c < fpad; c += MK_NT)
#pragma unroll
            for (int sp = 0; sp < MK_S * MK_M; ++sp) a[static_cast<size_t>(sp) * fpad + mk_xs_index(c)] = 0;   // (the tokens' arrays follow one another)
    }
    // (s_rope is published by the sync of the first prologue)

    // start this warp's weight stream: fill its ring
    if (ok && lane == 0)
        for (int sl = 0; sl < p.slots && ok; ++sl) ok = fetch_next_tile(p, ws, sl, abort_flag, s_issued, full_bar, warp);
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;

    ItemCtx cx;
    cx.slot_row = slot_row; cx.m_run = m_run;
#pragma unroll
    for (int t = 0; t < MK_M; ++t) { cx.rscale[t] = 1.f; cx.best_v[t] = -INFINITY; cx.best_i[t] = 0x7fffffff; }

    unsigned bar_no = 0;
    const unsigned bar_arrivals = static_cast<unsigned>(ncta + p.barrier_extra);
    int prof_idx = 0;
    prof_stamp(p, tid, prof_idx);
    const int n_att = slot_row + 1;
    // (a compressed cache is always attended with one CTA per kv head and chunk: one CTA then owns the row the step appends)
    const bool att_split = !LONG || (!Q8 && n_att <= p.att_split_max_n && static_cast<long long>(p.nq) * MK_ATT_SPLIT_MAXC * 2 <= MK_PARTIAL_FLOATS);
    int merge_chunks = 0;   // chunks per head the O-projection prologue has to merge (split mode)
    if (att_split && MK_SPLIT_DEFER) {
        int cl;
        if constexpr (MK_M > 1) att_chunking(p, n_att + m_run - 1, 1, p.att_chunk_split, 32 / MK_ATT_LPP_SPLIT, ncta, merge_chunks, cl, m_run);
        else att_chunking(p, n_att, 1, p.att_chunk_split, 32 / MK_ATT_LPP_SPLIT, ncta, merge_chunks, cl);
    }
    // One loop over the operators of the step, with a single inlined copy of the streaming operator and of the grid barrier
    // (the code of a step is executed once per layer: a small instruction footprint matters).  Operator 4l+1 (the O
    // projection) is preceded by the attention of layer l.
    const int n_layer_ops = 4 * p.n_layers;
    for (int ph = 0; ph < p.nph && ok; ++ph) {
        const bool layer_op = ph < n_layer_ops;
        const bool after_attention = layer_op && (ph & 3) == 1;
        if (layer_op && (ph & 3) == 0) ws.list = sm_tab(p)[warp * MK_WARP_TAB];          // every layer walks the same list
        if (!layer_op) ws.list = sm_tab(p)[warp * MK_WARP_TAB + 5];
        if (after_attention) {
            const int l = ph >> 2;
            if constexpr (LONG) {
                if (att_split) attention_phase<D, 1, MK_ATT_LPP_SPLIT>(p, l, n_att, p.att_chunk_split, MK_SPLIT_DEFER != 0, sm_xbuf(p), tid, &s_flag);
                else attention_phase<D, G, MK_ATT_LPP, Q8>(p, l, n_att, p.att_chunk_shared, false, sm_xbuf(p), tid, &s_flag);
            } else {
                // (a block: all its tokens in one pass; token t also attends to the rows of the tokens before it)
                if constexpr (MK_M > 1) {
                    attention_phase<D, 1, MK_ATT_LPP_SPLIT>(p, l, n_att + m_run - 1, p.att_chunk_split, MK_SPLIT_DEFER != 0, sm_xbuf(p), tid, &s_flag,
                                                            p.head_flags != 0, abort_flag, &prof_idx, -1, m_run);
                } else {
                    attention_phase<D, 1, MK_ATT_LPP_SPLIT>(p, l, n_att, p.att_chunk_split, MK_SPLIT_DEFER != 0, sm_xbuf(p), tid, &s_flag,
                                                            p.head_flags != 0, abort_flag, &prof_idx);
                }
            }
            ok = grid_barrier(p, ++bar_no * bar_arrivals, abort_flag, tid, prof_idx) && ok;
            if (!ok) break;
        }
        ok = gemv_phase(p, ph, layer_op ? (ph & 3) : 4, ws, abort_flag, s_part, s_partial, s_rope, cx, tokens, after_attention ? merge_chunks : 0, tid,
                        prof_idx, s_issued, full_bar);
        if (!LONG && p.head_flags && layer_op && (ph & 3) == 0) {
            // no grid barrier behind the QKV projection: the attention phase waits for the heads it reads (the CTA-wide sync
            // keeps the attention scratch, which shares the staged vector's memory, from being written under slower warps)
            cta_sync();
            prof_stamp(p, tid, prof_idx);
            ok = ok && !*abort_flag;
        } else if (layer_op) {
            ok = grid_barrier(p, ++bar_no * bar_arrivals, abort_flag, tid, prof_idx) && ok;
        }
    }
    prof_stamp(p, tid, prof_idx);
    if (!ok || *abort_flag) {
        // aborted: wait (bounded) for the copies still in flight into this warp's ring, then leave
        *abort_flag = 1;
        if (tid == 0 && p.state->status == 0) p.state->status = 6;
        const unsigned issued = __shfl_sync(0xffffffffu, ws.next.count, 0);
        for (unsigned k = ws.consumed; k < issued; ++k) {
            const unsigned long long t1 = global_ns();
            while (!mbar_try_wait(&full_bar[warp * MK_MAX_SLOTS + ws.slot], ws.round & 1u))
                if (global_ns() - t1 > p.spin_limit) break;
            if (++ws.slot == p.slots) { ws.slot = 0; ++ws.round; }
        }
        return;
    }

    // ---- greedy sampling: warp -> CTA -> last CTA reduces all partials, then the state advances -------------
    // (a block: one greedy token per token of the call; partials of token t at [t][cta])
#pragma unroll
    for (int t = 0; t < MK_M; ++t) {
        float bv = cx.best_v[t];
        int bi = cx.best_i[t];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (arg_better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
        }
        if (lane == 0) { s_bv[t * MK_NW + warp] = bv; s_bi[t * MK_NW + warp] = bi; }
    }
    cta_sync();
    if (tid == 0) {
#pragma unroll
        for (int t = 0; t < MK_M; ++t) {
            float bv = s_bv[t * MK_NW];
            int bi = s_bi[t * MK_NW];
            for (int w = 1; w < MK_NW; ++w)
                if (arg_better(s_bv[t * MK_NW + w], s_bi[t * MK_NW + w], bv, bi)) { bv = s_bv[t * MK_NW + w]; bi = s_bi[t * MK_NW + w]; }
            p.lm_part_val[t * ncta + cta] = bv;
            p.lm_part_idx[t * ncta + cta] = bi;
        }
        __threadfence();
        s_flag = (atomicAdd(p.tickets + p.nq, 1u) == static_cast<unsigned>(ncta - 1)) ? 1 : 0;
    }
    cta_sync();
    if (!s_flag) return;
    __threadfence();
    if (warp == 0) {
        int greedy[MK_M];
#pragma unroll
        for (int t = 0; t < MK_M; ++t) {
            float bv = -INFINITY;
            int bi = 0x7fffffff;
            for (int i = lane; i < ncta; i += 32) {
                const float v = __ldcg(p.lm_part_val + t * ncta + i);
                const int ix = __ldcg(p.lm_part_idx + t * ncta + i);
                if (arg_better(v, ix, bv, bi)) { bv = v; bi = ix; }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (arg_better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
            }
            if (bi == 0x7fffffff) bi = 0;
            if (sm_ops(p)[p.nph - 1].flags() & PHF_REMAP) bi = p.vocab_ids[bi];   // pruned vocabulary: row index -> token id
            greedy[t] = bi;
        }
        if (lane == 0) {
            // Verification (Sec. 3.11): proposal t + 1 is accepted if it is the base model's greedy choice after token t;
            // it stops at the first rejection.  The cache advances by the accepted tokens; the rows of the rejected ones
            // stay behind the cache length and are overwritten by the next call.
            int n_acc = 1;
            const bool given = MK_M > 1 && (p.req->flags & 1);   // prompt tokens: nothing to verify
#pragma unroll
            for (int t = 1; t < MK_M; ++t)
                if (t < m_run && n_acc == t && (given || tokens[t] == greedy[t - 1])) n_acc = t + 1;
            int bi = greedy[0];
#pragma unroll
            for (int t = 1; t < MK_M; ++t)
                if (n_acc == t + 1) bi = greedy[t];
            int *nto = p.req->next_token_out;
            if (nto) *nto = bi;
            if (MK_M > 1 && p.req->n_accepted_out) *p.req->n_accepted_out = n_acc;
            p.state->next_token = bi;
            p.state->next_position = pos + n_acc;
            p.state->cur_len = slot_row + n_acc;
            p.state->n_accepted = n_acc;
            p.tickets[p.nq] = 0u;
            *p.barrier = 0u;  // every CTA has passed the last grid barrier
            if (p.head_flags)
                for (int h = 0; h < p.nq + 2 * p.nkv; ++h) p.head_ready[h] = 0u;
        }
    }
}

}  // namespace MK_NS
}  // namespace edgefm
