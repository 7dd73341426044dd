// Weight-streaming bf16 GEMV family: y = W x with the step's element-wise work fused around it.
//
// One CTA owns a tile of TR = RW * WR output rows; its WR x WK warps split the tile's rows (WR) and
// the reduction dimension (WK, in-CTA split-K).  Every lane streams 16-byte (8 x bf16) pieces of
// weight rows straight from HBM into registers, RW * U loads in flight, and multiplies them with the
// fp32 activation vector staged once per CTA in shared memory.  Partial sums are combined with
// warp shuffles, then across the WK warps in a fixed order through shared memory, so the result
// is bit-reproducible.  CTAs loop over tiles with a grid stride.
//
// Prologues (operators named in the hotspot list of Sec. 3.4 of the paper):
//   PRO_PLAIN    x as is
//   PRO_RMSNORM  x_i * rsqrt(mean(x^2) + eps) * w_i
// Epilogues:
//   EPI_QKV      + bias, rotate-half RoPE of q and k, q -> fp32 work buffer, k,v -> bf16 cache row
//                at slot cur_len (the KV-cache write path)
//   EPI_RESIDUAL x[row] += y
//   EPI_SWIGLU   a_i = silu(gate_i) * up_i
//   EPI_LMHEAD   optional logits store, block-wise argmax, last CTA reduces and advances the state
#pragma once
#include "common.cuh"

namespace edgefm {

enum { PRO_PLAIN = 0, PRO_RMSNORM = 1 };
enum { EPI_QKV = 0, EPI_RESIDUAL = 1, EPI_SWIGLU = 2, EPI_LMHEAD = 3 };

struct GemvArgs {
    const uint16_t *W;       // bf16 [rows][K] row-major
    int rows;
    int K;                   // multiple of 8
    const float *x_in;       // fp32 [K]
    const uint16_t *norm_w;  // bf16 [K] (PRO_RMSNORM)
    float eps;
    const uint16_t *bias;    // bf16 [rows] or null (EPI_QKV)
    float *out;              // EPI_QKV: q fp32 [nq*d]; EPI_RESIDUAL: x fp32 [rows] (+=); EPI_SWIGLU: a fp32 [F]
    // EPI_QKV
    uint16_t *k_cache;       // this layer's K cache, bf16 [nkv][max_context][d]
    uint16_t *v_cache;
    int max_context, nq, nkv, d;
    const float *rope_cs;    // fp32 [d/2] cos then [d/2] sin of the current position
    StepState *state;
    // EPI_SWIGLU
    int F;
    // EPI_LMHEAD
    const StepRequest *req;
    float *part_val;         // [gridDim.x]
    int *part_idx;           // [gridDim.x]
    unsigned *ticket;
};

// Row of the weight matrix that tile-local row j of tile `tile` maps to (or -1 when out of range).
// Paired epilogues put row i and its partner (RoPE: i + d/2 in the same head; SwiGLU: i + F) in
// the two halves of the tile so that one thread sees both results.
template <int EPI, int TR>
__device__ __forceinline__ int map_row(const GemvArgs &a, int tile, int j) {
    if constexpr (EPI == EPI_QKV) {
        const int half = a.d >> 1;
        const int u = tile * (TR / 2) + (j % (TR / 2));
        const int head = u / half, i = u - head * half;
        const int row = head * a.d + i + (j >= TR / 2 ? half : 0);
        return row < a.rows ? row : -1;
    } else if constexpr (EPI == EPI_SWIGLU) {
        const int u = tile * (TR / 2) + (j % (TR / 2));
        return u < a.F ? u + (j >= TR / 2 ? a.F : 0) : -1;
    } else {
        const int row = tile * TR + j;
        return row < a.rows ? row : -1;
    }
}

template <int EPI, int TR>
__device__ __forceinline__ int num_tiles(const GemvArgs &a) {
    if constexpr (EPI == EPI_QKV) return (a.rows / 2 + TR / 2 - 1) / (TR / 2);
    else if constexpr (EPI == EPI_SWIGLU) return (a.F + TR / 2 - 1) / (TR / 2);
    else return (a.rows + TR - 1) / TR;
}

template <int PRO, int EPI, int RW, int WR, int WK, int U>
__global__ void __launch_bounds__(WR *WK * 32) gemv_kernel(const GemvArgs a) {
    constexpr int TR = RW * WR;
    constexpr int NT = WR * WK * 32;
    static_assert(TR % 2 == 0 || (EPI != EPI_QKV && EPI != EPI_SWIGLU), "paired epilogues need an even tile");
    extern __shared__ __align__(16) float gemv_smem[];
    float *smem = gemv_smem;
    float *xs = smem;                 // [K]
    float *red = smem + a.K;          // [WK][TR]
    float *yt = red + WK * TR;        // [TR]
    __shared__ float s_red[32];
    __shared__ int s_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wr = warp % WR, wk = warp / WR;

    pdl_launch_dependents();
    pdl_wait();

    // ---- prologue: stage the activation vector -------------------------------------------------
    {
        const float4 *x4 = reinterpret_cast<const float4 *>(a.x_in);
        const int n4 = a.K >> 2;
        if constexpr (PRO == PRO_RMSNORM) {
            float ss = 0.f;
            for (int i = tid; i < n4; i += NT) {
                const float4 v = x4[i];
                ss = fmaf(v.x, v.x, ss); ss = fmaf(v.y, v.y, ss); ss = fmaf(v.z, v.z, ss); ss = fmaf(v.w, v.w, ss);
            }
            ss = warp_sum(ss);
            if (lane == 0) s_red[warp] = ss;
            __syncthreads();
            float tot = 0.f;
#pragma unroll
            for (int w = 0; w < NT / 32; ++w) tot += s_red[w];
            const float r = rsqrtf(tot / static_cast<float>(a.K) + a.eps);
            const uint2 *w2 = reinterpret_cast<const uint2 *>(a.norm_w);
            for (int i = tid; i < n4; i += NT) {
                const float4 v = x4[i];
                const uint2 w = w2[i];
                float4 o;
                o.x = v.x * r * bf16lo(w.x); o.y = v.y * r * bf16hi(w.x);
                o.z = v.z * r * bf16lo(w.y); o.w = v.w * r * bf16hi(w.y);
                reinterpret_cast<float4 *>(xs)[i] = o;
            }
        } else {
            for (int i = tid; i < n4; i += NT) reinterpret_cast<float4 *>(xs)[i] = x4[i];
        }
    }
    __syncthreads();

    const int kc = a.K >> 3;  // 16-byte pieces per row
    const int c0 = static_cast<int>((static_cast<long long>(kc) * wk) / WK);
    const int c1 = static_cast<int>((static_cast<long long>(kc) * (wk + 1)) / WK);
    const int ntiles = num_tiles<EPI, TR>(a);
    const float4 *xs4 = reinterpret_cast<const float4 *>(xs);

    float best_v = -INFINITY;  // EPI_LMHEAD running argmax of thread j < TR
    int best_i = 0x7fffffff;

    for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const uint4 *wrow[RW];
        bool valid[RW];
        float acc[RW];
#pragma unroll
        for (int r = 0; r < RW; ++r) {
            const int row = map_row<EPI, TR>(a, tile, wr * RW + r);
            valid[r] = row >= 0;
            wrow[r] = reinterpret_cast<const uint4 *>(a.W + static_cast<size_t>(valid[r] ? row : 0) * a.K);
            acc[r] = 0.f;
        }
        for (int c = c0 + lane; c < c1; c += 32 * U) {
            uint4 w[U][RW];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int cc = c + 32 * u;
#pragma unroll
                for (int r = 0; r < RW; ++r)
                    w[u][r] = (cc < c1 && valid[r]) ? ldg_stream16(wrow[r] + cc) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int cc = c + 32 * u;
                if (cc < c1) {
                    const float4 x0 = xs4[2 * cc], x1 = xs4[2 * cc + 1];
#pragma unroll
                    for (int r = 0; r < RW; ++r) acc[r] = dot8(w[u][r], x0, x1, acc[r]);
                }
            }
        }
#pragma unroll
        for (int r = 0; r < RW; ++r) {
            const float s = warp_sum(acc[r]);
            if (lane == 0) red[wk * TR + wr * RW + r] = s;
        }
        __syncthreads();
        if (tid < TR) {
            float s = 0.f;
#pragma unroll
            for (int k = 0; k < WK; ++k) s += red[k * TR + tid];
            yt[tid] = s;
        }
        if constexpr (EPI == EPI_QKV || EPI == EPI_SWIGLU) __syncthreads();

        // ---- epilogue --------------------------------------------------------------------------
        if constexpr (EPI == EPI_RESIDUAL) {
            if (tid < TR) {
                const int row = map_row<EPI, TR>(a, tile, tid);
                if (row >= 0) a.out[row] += yt[tid];
            }
        } else if constexpr (EPI == EPI_SWIGLU) {
            if (tid < TR / 2) {
                const int u = tile * (TR / 2) + tid;
                if (u < a.F) {
                    const float g = yt[tid], up = yt[tid + TR / 2];
                    a.out[u] = g / (1.f + expf(-g)) * up;
                }
            }
        } else if constexpr (EPI == EPI_QKV) {
            if (tid < TR / 2) {
                const int row_lo = map_row<EPI, TR>(a, tile, tid);
                if (row_lo >= 0) {
                    const int half = a.d >> 1;
                    const int row_hi = row_lo + half;
                    const int head = row_lo / a.d, i = row_lo - head * a.d;
                    float lo = yt[tid], hi = yt[tid + TR / 2];
                    if (a.bias) { lo += bf16_bits_to_f32(a.bias[row_lo]); hi += bf16_bits_to_f32(a.bias[row_hi]); }
                    const int slot = a.state->cur_len;
                    if (head < a.nq + a.nkv) {
                        const float c = a.rope_cs[i], s = a.rope_cs[half + i];
                        const float rlo = lo * c - hi * s, rhi = hi * c + lo * s;
                        if (head < a.nq) {
                            a.out[row_lo] = rlo;
                            a.out[row_hi] = rhi;
                        } else {
                            uint16_t *dst = a.k_cache + (static_cast<size_t>(head - a.nq) * a.max_context + slot) * a.d;
                            dst[i] = f32_to_bf16_bits(rlo);
                            dst[i + half] = f32_to_bf16_bits(rhi);
                        }
                    } else {
                        uint16_t *dst = a.v_cache + (static_cast<size_t>(head - a.nq - a.nkv) * a.max_context + slot) * a.d;
                        dst[i] = f32_to_bf16_bits(lo);
                        dst[i + half] = f32_to_bf16_bits(hi);
                    }
                }
            }
        } else {  // EPI_LMHEAD
            if (tid < TR) {
                const int row = map_row<EPI, TR>(a, tile, tid);
                if (row >= 0) {
                    const float v = yt[tid];
                    float *lo = a.req->logits_out;
                    if (lo) lo[row] = v;
                    if (arg_better(v, row, best_v, best_i)) { best_v = v; best_i = row; }
                }
            }
        }
        __syncthreads();
    }

    if constexpr (EPI == EPI_LMHEAD) {
        static_assert(TR <= 32, "lm_head tile reduction assumes one warp");
        // block-wise argmax over the CTA's rows
        if (warp == 0) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, best_v, o);
                const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
                if (arg_better(ov, oi, best_v, best_i)) { best_v = ov; best_i = oi; }
            }
            if (lane == 0) {
                a.part_val[blockIdx.x] = best_v;
                a.part_idx[blockIdx.x] = best_i;
                __threadfence();
                s_last = (atomicAdd(a.ticket, 1u) == gridDim.x - 1) ? 1 : 0;
            }
        }
        __syncthreads();
        if (s_last) {  // the CTA that arrives last reduces all partials in index order
            __threadfence();
            float bv = -INFINITY;
            int bi = 0x7fffffff;
            for (int i = tid; i < static_cast<int>(gridDim.x); i += NT) {
                const float v = __ldcg(a.part_val + i);
                const int ix = __ldcg(a.part_idx + i);
                if (arg_better(v, ix, bv, bi)) { bv = v; bi = ix; }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (arg_better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
            }
            __shared__ float s_bv[32];
            __shared__ int s_bi[32];
            if (lane == 0) { s_bv[warp] = bv; s_bi[warp] = bi; }
            __syncthreads();
            if (tid == 0) {
                for (int w = 1; w < NT / 32; ++w)
                    if (arg_better(s_bv[w], s_bi[w], bv, bi)) { bv = s_bv[w]; bi = s_bi[w]; }
                if (bi == 0x7fffffff) bi = 0;  // no finite-or-infinite candidate (all NaN)
                int *nto = a.req->next_token_out;
                if (nto) *nto = bi;
                StepState *st = a.state;  // state advance: the cache grew by one slot
                st->next_token = bi;
                st->next_position = st->position + 1;
                st->cur_len = st->cur_len + 1;
                *a.ticket = 0u;
            }
        }
    }
}

}  // namespace edgefm
