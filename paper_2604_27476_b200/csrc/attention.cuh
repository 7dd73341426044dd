// GQA decode attention over the bf16 KV cache: split-KV partials + exact log-sum-exp combine.
//
// Grid (max_chunks, n_kv).  CTA (c, g) owns chunk c of the attended positions of kv head g and
// serves all G = n_q / n_kv query heads of the group from one read of K and V.  Each warp walks
// tiles of TILE = 32 / LPP positions:
//   * the K tile is staged in shared memory with 16-byte cp.async (double buffered), rows padded so
//     that LPP lanes per position read it without bank conflicts; each lane accumulates its share of
//     the G dot products with q (pre-scaled by 1/sqrt(d)) broadcast from shared memory;
//   * an online softmax keeps a running maximum m_h and (per lane) partial denominators l_h;
//   * p_h(t) go through shared memory, and o_h += p_h(t) V_t with every lane owning d/32 dims of V,
//     read straight from global memory (coalesced rows).
// Warps are merged in shared memory, the CTA writes one partial (m, l, o) per query head, and the CTA
// that arrives last for its kv head (atomic ticket, no waiting) merges the chunks in index order:
//     m = max_c m_c,  l = sum_c l_c e^{m_c - m},  o = sum_c o_c e^{m_c - m} / l .
// The merge is exact up to rounding, so the result does not depend on the split.
#pragma once
#include "common.cuh"

namespace edgefm {

struct AttnArgs {
    const float *q;           // fp32 [nq][d], rotated
    const uint16_t *k_cache;  // this layer, bf16 [nkv][max_context][d]
    const uint16_t *v_cache;
    float *out;               // fp32 [nq][d]
    float *part_m;            // [nq][max_chunks]
    float *part_l;            // [nq][max_chunks]
    float *part_o;            // [nq][max_chunks][d]
    unsigned *tickets;        // [nkv]
    const StepState *state;
    int max_context;
    int max_chunks;           // gridDim.x
    int min_chunk;            // smallest chunk length worth a CTA (multiple of 32)
    float scale;              // 1/sqrt(d)
};

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src) {
    const unsigned s = static_cast<unsigned>(__cvta_generic_to_shared(smem_dst));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int D, int G, int LPP, int NW>
struct AttnSmem {
    static constexpr int TILE = 32 / LPP;
    static constexpr int ROWB = D * 2 + 16 * LPP;            // padded K row, bytes
    static constexpr int K_BYTES = NW * 2 * TILE * ROWB;      // double buffered per warp
    static constexpr int Q_BYTES = G * D * 4;
    static constexpr int P_BYTES = NW * G * TILE * 4;
    static constexpr int MERGE_BYTES = NW * G * (D + 2) * 4;  // reuses the K region after the loop
    static constexpr int TOTAL = Q_BYTES + P_BYTES + (K_BYTES > MERGE_BYTES ? K_BYTES : MERGE_BYTES);
};

template <int D, int G, int LPP, int NW>
__global__ void __launch_bounds__(NW * 32) attn_kernel(const AttnArgs a) {
    using S = AttnSmem<D, G, LPP, NW>;
    constexpr int TILE = S::TILE, ROWB = S::ROWB;
    constexpr int DV = D / 32;          // V dims per lane
    constexpr int CPR = D / 8;          // 16-byte pieces per K row
    constexpr int CPL = CPR / LPP;      // pieces per lane in the score phase
    static_assert(CPR % LPP == 0 && TILE % 4 == 0, "bad tiling");
    extern __shared__ __align__(16) unsigned char smraw[];
    float *qs = reinterpret_cast<float *>(smraw);                           // [G][D]
    float *ps = reinterpret_cast<float *>(smraw + S::Q_BYTES);              // [NW][G][TILE]
    unsigned char *kbase = smraw + S::Q_BYTES + S::P_BYTES;                 // [NW][2][TILE][ROWB]
    __shared__ int s_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = blockIdx.y, c = blockIdx.x;

    pdl_launch_dependents();
    pdl_wait();

    const int n = a.state->cur_len + 1;  // attended positions, the slot just written included
    int nchunks = (n + a.min_chunk - 1) / a.min_chunk;
    nchunks = nchunks < a.max_chunks ? nchunks : a.max_chunks;
    int chunk_len = (n + nchunks - 1) / nchunks;
    chunk_len = (chunk_len + 31) & ~31;
    nchunks = (n + chunk_len - 1) / chunk_len;
    if (c >= nchunks) return;
    const int t0 = c * chunk_len;
    const int t1 = min(n, t0 + chunk_len);

    for (int i = tid; i < G * D; i += NW * 32) qs[i] = a.q[static_cast<size_t>(g) * G * D + i] * a.scale;
    __syncthreads();

    const uint16_t *kg = a.k_cache + static_cast<size_t>(g) * a.max_context * D;
    const uint16_t *vg = a.v_cache + static_cast<size_t>(g) * a.max_context * D;
    unsigned char *kw = kbase + warp * (2 * TILE * ROWB);
    float *pw = ps + warp * (G * TILE);

    float m[G], l[G], o[G][DV];
#pragma unroll
    for (int h = 0; h < G; ++h) {
        m[h] = -INFINITY; l[h] = 0.f;
#pragma unroll
        for (int e = 0; e < DV; ++e) o[h][e] = 0.f;
    }

    // stage one K tile: TILE rows x CPR pieces, rows beyond t1 are not fetched (and never read)
    auto stage = [&](int tt, int buf) {
        unsigned char *dst = kw + buf * (TILE * ROWB);
        for (int i = lane; i < TILE * CPR; i += 32) {
            const int r = i / CPR, cc = i - r * CPR;
            if (tt + r < t1) cp_async16(dst + r * ROWB + cc * 16, kg + static_cast<size_t>(tt + r) * D + cc * 8);
        }
        cp_async_commit();
    };

    const int pi = lane / LPP, part = lane % LPP;
    int tt = t0 + warp * TILE;
    int buf = 0;
    if (tt < t1) stage(tt, 0);
    for (; tt < t1; tt += NW * TILE, buf ^= 1) {
        const int tnext = tt + NW * TILE;
        if (tnext < t1) { stage(tnext, buf ^ 1); cp_async_wait<1>(); } else { cp_async_wait<0>(); }
        __syncwarp();

        // ---- scores of position tt + pi for the G heads of the group -----------------------------
        const bool pvalid = tt + pi < t1;
        float s[G];
#pragma unroll
        for (int h = 0; h < G; ++h) s[h] = 0.f;
        if (pvalid) {
            const unsigned char *krow = kw + buf * (TILE * ROWB) + pi * ROWB;
#pragma unroll
            for (int j = 0; j < CPL; ++j) {
                const int cc = j * LPP + part;
                const uint4 kk = *reinterpret_cast<const uint4 *>(krow + cc * 16);
#pragma unroll
                for (int h = 0; h < G; ++h) {
                    const float4 q0 = *reinterpret_cast<const float4 *>(qs + h * D + cc * 8);
                    const float4 q1 = *reinterpret_cast<const float4 *>(qs + h * D + cc * 8 + 4);
                    s[h] = dot8(kk, q0, q1, s[h]);
                }
            }
        }
#pragma unroll
        for (int h = 0; h < G; ++h) {
#pragma unroll
            for (int x = 1; x < LPP; x <<= 1) s[h] += __shfl_xor_sync(0xffffffffu, s[h], x);
            if (!pvalid) s[h] = -INFINITY;
            const float mn = fmaxf(m[h], warp_max(s[h]));   // finite: the tile has a valid position
            const float corr = __expf(m[h] - mn);            // m = -inf on the first tile -> 0
            const float p = pvalid ? __expf(s[h] - mn) : 0.f;
            l[h] = l[h] * corr + (part == 0 ? p : 0.f);
#pragma unroll
            for (int e = 0; e < DV; ++e) o[h][e] *= corr;
            m[h] = mn;
            if (part == 0) pw[h * TILE + pi] = p;
        }
        __syncwarp();

        // ---- o_h += p_h(t) * V_t, lane owns dims [lane*DV, lane*DV + DV) ----------------------------
#pragma unroll
        for (int tb = 0; tb < TILE; tb += 4) {
            float v[4][DV];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int t = tt + tb + x;
                if (t < t1) {
                    const uint16_t *vp = vg + static_cast<size_t>(t) * D + lane * DV;
                    if constexpr (DV == 4) {
                        const uint2 w = ldg_stream8(vp);
                        v[x][0] = bf16lo(w.x); v[x][1] = bf16hi(w.x); v[x][2] = bf16lo(w.y); v[x][3] = bf16hi(w.y);
                    } else {
                        const uint32_t w = ldg_stream4(vp);
                        v[x][0] = bf16lo(w); v[x][1] = bf16hi(w);
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < DV; ++e) v[x][e] = 0.f;
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

    // ---- merge the warps of the CTA ------------------------------------------------------------------
    __syncthreads();  // every warp is done with its K buffers; the region is reused below
    float *mg_m = reinterpret_cast<float *>(kbase);      // [NW][G]
    float *mg_l = mg_m + NW * G;                         // [NW][G]
    float *mg_o = mg_l + NW * G;                         // [NW][G][D]
#pragma unroll
    for (int h = 0; h < G; ++h) {
        const float lt = warp_sum(l[h]);
        if (lane == 0) { mg_m[warp * G + h] = m[h]; mg_l[warp * G + h] = lt; }
#pragma unroll
        for (int e = 0; e < DV; ++e) mg_o[(warp * G + h) * D + lane * DV + e] = o[h][e];
    }
    __syncthreads();
    for (int i = tid; i < G * D; i += NW * 32) {
        const int h = i / D, j = i - h * D;
        float mm = -INFINITY;
#pragma unroll
        for (int w = 0; w < NW; ++w) mm = fmaxf(mm, mg_m[w * G + h]);
        float ll = 0.f, oo = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const float e = __expf(mg_m[w * G + h] - mm);   // idle warps: m = -inf -> weight 0
            ll = fmaf(mg_l[w * G + h], e, ll);
            oo = fmaf(mg_o[(w * G + h) * D + j], e, oo);
        }
        const int qh = g * G + h;
        a.part_o[(static_cast<size_t>(qh) * a.max_chunks + c) * D + j] = oo;
        if (j == 0) { a.part_m[qh * a.max_chunks + c] = mm; a.part_l[qh * a.max_chunks + c] = ll; }
    }

    // ---- last CTA of this kv head merges the chunks ----------------------------------------------
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(a.tickets + g, 1u) == static_cast<unsigned>(nchunks - 1)) ? 1 : 0;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    for (int i = tid; i < G * D; i += NW * 32) {
        const int h = i / D, j = i - h * D;
        const int qh = g * G + h;
        const float *pm = a.part_m + qh * a.max_chunks;
        const float *pl = a.part_l + qh * a.max_chunks;
        float mm = -INFINITY;
        for (int cc = 0; cc < nchunks; ++cc) mm = fmaxf(mm, __ldcg(pm + cc));
        float ll = 0.f, oo = 0.f;
        for (int cc = 0; cc < nchunks; ++cc) {
            const float e = __expf(__ldcg(pm + cc) - mm);
            ll = fmaf(__ldcg(pl + cc), e, ll);
            oo = fmaf(__ldcg(a.part_o + (static_cast<size_t>(qh) * a.max_chunks + cc) * D + j), e, oo);
        }
        a.out[qh * D + j] = oo / ll;
    }
    if (tid == 0) a.tickets[g] = 0u;
}

}  // namespace edgefm
