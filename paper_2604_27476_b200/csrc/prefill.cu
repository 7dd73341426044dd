// Prompt processing for sm_100a: KV <- Prefill(x_1:T) (Eq. 3 of the paper).
//
// The T given tokens go through the layers together, so every projection is a dense [T x K] x [K x N] contraction:
//   * prefill_gemm_kernel: one 128 x 128 (gate/up: 128 x 256) output tile per CTA.  A producer thread stages bf16 operand
//     tiles in shared memory by TMA (128-byte swizzle), one thread issues tcgen05.mma with the fp32 accumulator in tensor
//     memory, four warps read the accumulator back (tcgen05.ld) and apply the operator's epilogue:
//       QKV      : + bias, rotate-half RoPE of q and k, q to the work buffer, k and v rows to the cache;
//       O / down : added to the fp32 residual stream;
//       gate/up  : SwiGLU, silu(gate) * up, to the bf16 activation buffer.
//   * prefill_attention_tc_kernel: causal attention of the T queries over the cache rows (prefix + the T new rows), also on
//     tcgen05: S = Q K^T and O = P V in tensor memory, online softmax by warps that own the rows (see the kernel).
//   * rmsnorm / embedding kernels: one row per warp.
// Every activation enters the tensor cores as TWO bf16 pieces (hi + lo, 16 mantissa bits; twice the multiplies, one load of
// the weight tile), because single bf16 activations put the logits of a 28-layer model outside the step's tolerance
// (measured: 3.6e-2 max-abs).  The residual stream stays fp32.
// Every wait on an mbarrier is bounded; a wait that runs out raises PrefillBuffers::error and the CTA drains and returns.
#include "prefill.h"

#include <cuda.h>
#include <cuda_bf16.h>

#include "step_plan.h"

namespace edgefm {
namespace {

// ---- PTX wrappers ----------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after `limit` polls or as soon as another thread of the CTA has given up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag, uint32_t limit) {
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 63u) == 63u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
                     smem_u32(dst)),
                 "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
                 : "memory");
}

// Programmatic dependent launch: every kernel of the prefill chain lets its successor be launched as soon as all of its own CTAs
// have started (pdl_trigger, first statement), and touches global memory only after its predecessor has completed and its writes
// are visible (pdl_wait).  What overlaps is the successor's launch and set-up (barriers, tensor memory, descriptor fetch).
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Descriptor fetch ahead of the first copy that uses the map (the map is a kernel parameter).
__device__ __forceinline__ void prefetch_map(const CUtensorMap *map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T: 128 x N x 16, bf16 operands (both K-major), fp32 accumulator.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The same with the A operand in tensor memory (lane = row, 16-bit elements packed two per column, K along the columns).
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The mbarrier receives one arrival when every tcgen05.mma issued so far by this thread has finished.
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 lanes x 32 columns of fp32: thread i of the warp receives row (lane base + i), columns c .. c + 31.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float *v) {
    uint32_t *r = reinterpret_cast<uint32_t *>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, "
        "%18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float *v) {
    uint32_t *r = reinterpret_cast<uint32_t *>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
template <int N> __device__ __forceinline__ void tmem_ld(uint32_t taddr, float *v) {
    static_assert(N == 16 || N % 32 == 0, "16 columns or a multiple of 32");
    if constexpr (N == 16) {
        tmem_ld16(taddr, v);
    } else {
#pragma unroll
        for (int c = 0; c < N / 32; ++c) tmem_ld32(taddr + c * 32, v + c * 32);
    }
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float *v) {
    const uint32_t *r = reinterpret_cast<const uint32_t *>(v);
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, "
        "%19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]),
        "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]),
        "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float *v) {
    const uint32_t *r = reinterpret_cast<const uint32_t *>(v);
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]),
        "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
template <int N> __device__ __forceinline__ void tmem_st(uint32_t taddr, const float *v) {
    static_assert(N == 16 || N % 32 == 0, "16 columns or a multiple of 32");
    if constexpr (N == 16) {
        tmem_st16(taddr, v);
    } else {
#pragma unroll
        for (int c = 0; c < N / 32; ++c) tmem_st32(taddr + c * 32, v + c * 32);
    }
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 tile written by TMA with the 128-byte swizzle: rows of 64 elements
// (128 bytes), groups of 8 rows 1024 bytes apart.  Fields: start address >> 4 (bits 0-13), leading byte offset >> 4 (16-29;
// 1, unused with this swizzle), stride byte offset >> 4 (32-45) = 64, descriptor version 1 (46-47), layout 2 = 128-byte
// swizzle (61-63).  A step of 16 elements along K inside the 128-byte row adds 32 bytes to the start address.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
    return static_cast<uint64_t>((smem_addr >> 4) & 0x3fffu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: fp32 accumulator (bits 4-5 = 1), A and B bf16 (7-9 = 1, 10-12 = 1), both K-major (15, 16 = 0),
// N >> 3 (17-22), M >> 4 (24-28).
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int m, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
    return static_cast<uint32_t>(f32_to_bf16_bits(lo)) | (static_cast<uint32_t>(f32_to_bf16_bits(hi)) << 16);
}

// An fp32 activation as two bf16 pieces, hi = bf16(x), lo = bf16(x - hi): 16 mantissa bits enter the tensor cores (the
// weights are bf16 exactly), so a contraction's operand rounding stays below 2^-17 relative.
__device__ __forceinline__ void split2(float x, uint16_t &hi, uint16_t &lo) {
    hi = f32_to_bf16_bits(x);
    lo = f32_to_bf16_bits(x - bf16_bits_to_f32(hi));
}
__device__ __forceinline__ void split2x2(float a, float b, uint32_t &hi, uint32_t &lo) {
    uint16_t ah, al, bh, bl;
    split2(a, ah, al);
    split2(b, bh, bl);
    hi = static_cast<uint32_t>(ah) | (static_cast<uint32_t>(bh) << 16);
    lo = static_cast<uint32_t>(al) | (static_cast<uint32_t>(bl) << 16);
}

// The same split by truncation (hi = the upper 16 bits of x, lo = the upper 16 bits of x - hi; x - hi is exact): no conversion
// instruction, which shares the special-function pipe with exp2 in the attention loop.  Error below 2^-16 relative.
__device__ __forceinline__ void split2x2_trunc(float a, float b, uint32_t &hi, uint32_t &lo) {
    const uint32_t ab = __float_as_uint(a), bb = __float_as_uint(b);
    hi = __byte_perm(ab, bb, 0x7632);
    const float ra = a - __uint_as_float(ab & 0xffff0000u), rb = b - __uint_as_float(bb & 0xffff0000u);
    lo = __byte_perm(__float_as_uint(ra), __float_as_uint(rb), 0x7632);
}

// ---- small kernels -----------------------------------------------------------------------------------------------------
// (cos, sin) of angle (position + t) * theta^(-2 j / d), evaluated in double and rounded once.
__global__ void __launch_bounds__(256) prefill_rope_kernel(float2 *rope, int n, int half, int position, double theta) {
    pdl_trigger();
    pdl_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n * half) return;
    const int t = i / half, j = i % half;
    const double inv = pow(theta, -static_cast<double>(j) / static_cast<double>(half));
    double sn, cs;
    sincos(static_cast<double>(position + t) * inv, &sn, &cs);
    rope[i] = make_float2(static_cast<float>(cs), static_cast<float>(sn));
}

// One CTA of 128 threads per row: y = x * rsqrt(mean(x^2) + eps) * w, stored as two bf16 planes (hi, lo; `plane` elements apart).  With `embed` the row is first fetched from the embedding
// table (bf16 -> fp32) and written to the residual stream.  Thread 0 of the grid also records the new cache length.
__global__ void __launch_bounds__(128) prefill_norm_kernel(float *resid, uint16_t *xn, size_t plane, const uint16_t *w, const uint16_t *embed,
                                                           const int *tokens, int n, int H, float eps, StepState *st, int new_len,
                                                           int new_pos, const float *part, int splits, size_t part_plane) {
    pdl_trigger();
    pdl_wait();
    if (st && blockIdx.x == 0 && threadIdx.x == 0) {
        st->cur_len = new_len;
        st->next_position = new_pos;
        st->status = 0;
    }
    __shared__ float red[4];
    const int row = blockIdx.x, tid = threadIdx.x;
    float *x = resid + static_cast<size_t>(row) * H;
    uint16_t *y = xn + static_cast<size_t>(row) * H;
    // H is a multiple of 8: eight values per lane and round, 16- and 32-byte accesses
    const uint16_t *e = embed ? embed + static_cast<size_t>(tokens[row]) * H : nullptr;
    float ss = 0.f;
    for (int j = tid * 8; j < H; j += 1024) {
        float v[8];
        if (e) {
            const uint4 b = *reinterpret_cast<const uint4 *>(e + j);
            v[0] = bf16lo(b.x); v[1] = bf16hi(b.x); v[2] = bf16lo(b.y); v[3] = bf16hi(b.y);
            v[4] = bf16lo(b.z); v[5] = bf16hi(b.z); v[6] = bf16lo(b.w); v[7] = bf16hi(b.w);
            *reinterpret_cast<float4 *>(x + j) = make_float4(v[0], v[1], v[2], v[3]);
            *reinterpret_cast<float4 *>(x + j + 4) = make_float4(v[4], v[5], v[6], v[7]);
        } else {
            const float4 a = *reinterpret_cast<const float4 *>(x + j), c = *reinterpret_cast<const float4 *>(x + j + 4);
            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = c.x; v[5] = c.y; v[6] = c.z; v[7] = c.w;
            if (splits > 1) {   // the K-split partial sums of the contraction before: added in plane order, written back
                for (int sp = 0; sp < splits; ++sp) {
                    const float *q = part + sp * part_plane + static_cast<size_t>(row) * H + j;
                    const float4 pa = *reinterpret_cast<const float4 *>(q), pc = *reinterpret_cast<const float4 *>(q + 4);
                    v[0] += pa.x; v[1] += pa.y; v[2] += pa.z; v[3] += pa.w; v[4] += pc.x; v[5] += pc.y; v[6] += pc.z; v[7] += pc.w;
                }
                *reinterpret_cast<float4 *>(x + j) = make_float4(v[0], v[1], v[2], v[3]);
                *reinterpret_cast<float4 *>(x + j + 4) = make_float4(v[4], v[5], v[6], v[7]);
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) ss = fmaf(v[i], v[i], ss);
    }
    ss = warp_sum(ss);
    if ((tid & 31) == 0) red[tid >> 5] = ss;
    __syncthreads();
    ss = (red[0] + red[1]) + (red[2] + red[3]);
    const float r = rsqrtf(ss / static_cast<float>(H) + eps);
    for (int j = tid * 8; j < H; j += 1024) {
        const float4 a = *reinterpret_cast<const float4 *>(x + j), c = *reinterpret_cast<const float4 *>(x + j + 4);
        const uint4 wb = *reinterpret_cast<const uint4 *>(w + j);
        uint4 hi, lo;
        split2x2(a.x * r * bf16lo(wb.x), a.y * r * bf16hi(wb.x), hi.x, lo.x);
        split2x2(a.z * r * bf16lo(wb.y), a.w * r * bf16hi(wb.y), hi.y, lo.y);
        split2x2(c.x * r * bf16lo(wb.z), c.y * r * bf16hi(wb.z), hi.z, lo.z);
        split2x2(c.z * r * bf16lo(wb.w), c.w * r * bf16hi(wb.w), hi.w, lo.w);
        *reinterpret_cast<uint4 *>(y + j) = hi;
        *reinterpret_cast<uint4 *>(y + plane + j) = lo;
    }
}

// Compressed cache (Sec. 3.9): one warp per new row (k rows, then v rows) of the fp32 staging buffers [nkv][stride / d][d];
// scale = amax / 127, code = clamp(rint(x * (127 / amax))) in fp32 -- the arithmetic of the decode step's own row.
__global__ void __launch_bounds__(256) prefill_quantize_rows_kernel(const float *k, const float *v, long long stage_stride, signed char *kc,
                                                                    signed char *vc, float *ks, float *vs, int nkv, int n, int d,
                                                                    int max_context, int slot0) {
    pdl_trigger();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const long long r = (blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x) >> 5, rows = static_cast<long long>(nkv) * n;
    if (r >= 2 * rows) return;
    const bool is_v = r >= rows;
    const long long rr = is_v ? r - rows : r;
    const int t = static_cast<int>(rr % n), g = static_cast<int>(rr / n);
    const float *src = (is_v ? v : k) + g * stage_stride + static_cast<long long>(t) * d;
    const long long row = static_cast<long long>(g) * max_context + slot0 + t;
    float x[4];                                                              // d <= 128: at most 4 values per lane
    float amax = 0.f;
    for (int e = 0; e < 4; ++e) {
        const int j = lane + 32 * e;
        x[e] = j < d ? src[j] : 0.f;
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

// Output layer for ONE row (the prompt's last token): final RMSNorm, logits = W x over `rows` rows of the output matrix (bf16
// weights, fp32 x and sums), greedy token (larger value wins, equal values -> lower row), and the device state a decode step
// would leave.  A matrix-vector product: bound by the one pass over W.  grid: any; 256 threads; dynamic shared memory H floats.
__global__ void __launch_bounds__(256) prefill_head_kernel(const float *x, const uint16_t *wnorm, const uint16_t *lm, const int *ids, int rows,
                                                           int H, float eps, float *logits_out, int *next_token_out, float *part_val,
                                                           int *part_idx, unsigned *ticket, StepState *st, int token, int pos) {
    extern __shared__ __align__(16) float pf_xs[];
    __shared__ float red[8], bvs[8];
    __shared__ int bis[8], is_last;
    pdl_trigger();
    pdl_wait();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    float ss = 0.f;
    for (int j = tid; j < H; j += 256) ss = fmaf(x[j], x[j], ss);
    ss = warp_sum(ss);
    if (lane == 0) red[warp] = ss;
    __syncthreads();
    ss = ((red[0] + red[1]) + (red[2] + red[3])) + ((red[4] + red[5]) + (red[6] + red[7]));
    const float r = rsqrtf(ss / static_cast<float>(H) + eps);
    for (int j = tid; j < H; j += 256) pf_xs[j] = x[j] * r * bf16_bits_to_f32(wnorm[j]);
    __syncthreads();
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    const int stride = gridDim.x * 8;
    for (int row = blockIdx.x * 8 + warp; row < rows; row += 2 * stride) {   // two rows per round: more loads in flight
        const int row2 = row + stride;
        const uint16_t *w0 = lm + static_cast<size_t>(row) * H, *w1 = lm + static_cast<size_t>(row2 < rows ? row2 : row) * H;
        float a0 = 0.f, a1 = 0.f;
        for (int j = lane * 8; j < H; j += 256) {
            const uint4 u0 = *reinterpret_cast<const uint4 *>(w0 + j), u1 = *reinterpret_cast<const uint4 *>(w1 + j);
            const float4 x0 = *reinterpret_cast<const float4 *>(pf_xs + j), x1 = *reinterpret_cast<const float4 *>(pf_xs + j + 4);
            a0 = dot8(u0, x0, x1, a0);
            a1 = dot8(u1, x0, x1, a1);
        }
        a0 = warp_sum(a0);
        a1 = warp_sum(a1);
        if (lane == 0) {
            if (logits_out) { logits_out[row] = a0; if (row2 < rows) logits_out[row2] = a1; }
            if (arg_better(a0, row, bv, bi)) { bv = a0; bi = row; }
            if (row2 < rows && arg_better(a1, row2, bv, bi)) { bv = a1; bi = row2; }
        }
    }
    if (lane == 0) { bvs[warp] = bv; bis[warp] = bi; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < 8; ++w)
            if (arg_better(bvs[w], bis[w], bv, bi)) { bv = bvs[w]; bi = bis[w]; }
        part_val[blockIdx.x] = bv;
        part_idx[blockIdx.x] = bi;
        __threadfence();
        is_last = atomicAdd(ticket, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (is_last && warp == 0) {      // the last CTA to finish merges the CTAs' candidates
        __threadfence();
        bv = -INFINITY; bi = 0x7fffffff;
        for (int i = lane; i < static_cast<int>(gridDim.x); i += 32) {
            const float v = __ldcg(part_val + i);
            const int ix = __ldcg(part_idx + i);
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
            if (ids) bi = ids[bi];   // pruned vocabulary: row index -> token id
            if (next_token_out) *next_token_out = bi;
            st->token = token;
            st->position = pos;
            st->next_token = bi;
            st->next_position = pos + 1;
            st->n_accepted = 1;
            *ticket = 0u;
        }
    }
}

// Greedy tokens of the m <= PF_VERIFY_MAX rows of a logits matrix [m][rows] and the acceptance rule of a verified block (Sec. 3.11)
// on the device: proposal t + 1 is accepted if tokens[t + 1] equals the greedy token after token t, verification stops at the
// first mismatch; the cache length becomes slot0 + n_accepted (the rows behind it are overwritten later), the next token is the
// greedy token after the last accepted one.  The logits come from a contraction over the output matrix (EPI_LOGITS).
__global__ void __launch_bounds__(256) prefill_verify_pick_kernel(const float *logits, const int *ids, int rows, int m, const int *tokens,
                                                                  float *part_val, int *part_idx, unsigned *ticket, StepState *st, int slot0,
                                                                  int pos, int *n_accepted_out, int *next_token_out) {
    pdl_trigger();
    pdl_wait();
    __shared__ float bvs[8][PF_VERIFY_MAX];
    __shared__ int bis[8][PF_VERIFY_MAX], is_last;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    for (int t = 0; t < m; ++t) {
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        for (int r = blockIdx.x * 256 + tid; r < rows; r += gridDim.x * 256) {
            const float v = logits[static_cast<size_t>(t) * rows + r];
            if (arg_better(v, r, bv, bi)) { bv = v; bi = r; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (arg_better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
        }
        if (lane == 0) { bvs[warp][t] = bv; bis[warp][t] = bi; }
    }
    __syncthreads();
    if (tid < m) {
        float v = bvs[0][tid];
        int ix = bis[0][tid];
        for (int w = 1; w < 8; ++w)
            if (arg_better(bvs[w][tid], bis[w][tid], v, ix)) { v = bvs[w][tid]; ix = bis[w][tid]; }
        part_val[blockIdx.x * PF_VERIFY_MAX + tid] = v;
        part_idx[blockIdx.x * PF_VERIFY_MAX + tid] = ix;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) is_last = atomicAdd(ticket, 1u) == gridDim.x - 1;
    __syncthreads();
    if (is_last && warp == 0) {
        __threadfence();
        int greedy = 0;
        if (lane < m) {
            float v = -INFINITY;
            int ix = 0x7fffffff;
            for (int i = 0; i < static_cast<int>(gridDim.x); ++i) {
                const float pv = __ldcg(part_val + i * PF_VERIFY_MAX + lane);
                const int pi = __ldcg(part_idx + i * PF_VERIFY_MAX + lane);
                if (arg_better(pv, pi, v, ix)) { v = pv; ix = pi; }
            }
            if (ix == 0x7fffffff) ix = 0;
            greedy = ids ? ids[ix] : ix;
        }
        int n_acc = 1, next = __shfl_sync(0xffffffffu, greedy, 0);
        for (int t = 1; t < m; ++t) {
            const int g_prev = __shfl_sync(0xffffffffu, greedy, t - 1), g_t = __shfl_sync(0xffffffffu, greedy, t);
            if (n_acc == t && tokens[t] == g_prev) { n_acc = t + 1; next = g_t; }
        }
        if (lane == 0) {
            if (next_token_out) *next_token_out = next;
            if (n_accepted_out) *n_accepted_out = n_acc;
            st->token = tokens[0];
            st->position = pos;
            st->next_token = next;
            st->next_position = pos + n_acc;
            st->cur_len = slot0 + n_acc;
            st->n_accepted = n_acc;
            *ticket = 0u;
        }
    }
}

// ---- the contraction -------------------------------------------------------------------------------------------------------
enum { EPI_QKV = 0, EPI_RESID = 1, EPI_SWIGLU = 2, EPI_LOGITS = 3 };   // EPI_LOGITS: plain fp32 store to g.resid [M][N] (output layer)

struct GemmArgs {
    int M, N, K;              // rows (tokens), output features (gate/up: F, each of gate and up), reduction length
    int *error;
    uint32_t wait_limit;      // polls a wait on an mbarrier may take
    uint32_t extra_arrivals;  // 0; 1 (tests): the stage barriers expect an arrival nobody makes, so the first wait runs out
    // QKV
    const uint16_t *bias;     // [N] or null
    const float2 *rope;       // [M][d/2]
    uint16_t *q_out;          // [2][..][nq d]: hi and lo planes
    size_t q_plane;           // elements between the planes
    uint16_t *k_rows, *v_rows;  // the layer's cache at the first new slot: + head * head_stride + row * d
    float *k_stage, *v_stage;   // compressed cache: the rows go here in fp32 instead ([nkv][stage_stride / d rows][d]) and are
    long long stage_stride;     // compressed by prefill_quantize_rows_kernel
    int nq, nkv, d;
    long long head_stride;
    // O / down
    float *resid;             // [M][N]
    int splits;               // K split into this many units per output tile (1 = none).  With a split the units write their
    float *part;              // partial sums to part[split][..][N] (planes `part_plane` elements apart) instead of adding to resid;
    size_t part_plane;        // the norm kernel that follows adds the planes to the residual stream in a fixed order.
    // gate/up
    uint16_t *act;            // [2][..][N]: hi and lo planes
    size_t act_plane;
};

constexpr int PF_BM = 128, PF_BK = 64;
constexpr int PF_SPLIT_MAX = 8;               // K splits of a contraction that adds to the residual stream: up to 4, up to 8 when the
                                             // tokens fit one row tile (short prompts, verified blocks: the grids are smallest there)

// Tile shapes.  PF_NARROW: 128 output columns, 4 stages of 48 KB.  PF_WIDE: 256 output columns, 3 stages of 64 KB: per k-block
// 64 KB of operands feed twice the multiplies of a narrow tile's 48 KB, which matters because operand delivery from L2, not
// the tensor pipe, bounds the narrow tiles.  Gate/up always runs wide: 128 gate columns and their 128 up partners.
// The kernel is persistent (one CTA per SM, tiles dealt round-robin, neighbours sharing a weight tile) with TWO accumulators
// in tensor memory, so that the epilogue of a tile runs under the main loop of the next.
enum { PF_NARROW = 0, PF_WIDE = 2 };
template <int SHAPE> struct GemmCfg {
    static constexpr int BN = SHAPE == PF_WIDE ? 256 : 128;
    static constexpr int STAGES = SHAPE == PF_WIDE ? 3 : 4;
    static constexpr int A_BYTES = PF_BM * PF_BK * 2, B_BYTES = BN * PF_BK * 2;
    static constexpr int STAGE_BYTES = 2 * A_BYTES + B_BYTES;          // A hi, A lo, B
    static constexpr int SMEM = STAGES * STAGE_BYTES + 1024;   // + room to align the first stage to 1024 bytes
};

template <int EPI, int SHAPE>
__global__ void __launch_bounds__(192) prefill_gemm_kernel(const __grid_constant__ CUtensorMap map_a_hi,
                                                           const __grid_constant__ CUtensorMap map_a_lo,
                                                           const __grid_constant__ CUtensorMap map_b, const GemmArgs g) {
    pdl_trigger();
    using C = GemmCfg<SHAPE>;
    static_assert(EPI != EPI_SWIGLU || SHAPE == PF_WIDE, "gate and up share one accumulator");
    constexpr int N_STEP = EPI == EPI_SWIGLU ? 128 : C::BN;   // output columns (of g.N) a CTA covers
    extern __shared__ uint8_t pf_dyn[];
    __shared__ uint64_t full_bar[C::STAGES], empty_bar[C::STAGES], acc_full[2], acc_empty[2], drain_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    uint8_t *tiles = pf_dyn + ((1024u - (smem_u32(pf_dyn) & 1023u)) & 1023u);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m_tiles = (g.M + PF_BM - 1) / PF_BM, n_tiles = (g.N + N_STEP - 1) / N_STEP;
    const int KB = (g.K + PF_BK - 1) / PF_BK;
    const int splits = EPI == EPI_RESID ? g.splits : 1;
    const int my_tiles = (m_tiles * n_tiles * splits - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
    // unit u of the grid-wide list: row tile u % m_tiles (neighbouring CTAs share a weight tile), then the K split, then the column tile
    auto unit_of = [&](int i, int &m0, int &n0, int &kb0, int &kb1) {
        const int u = blockIdx.x + i * gridDim.x, rest = u / m_tiles, sp = rest % splits;
        m0 = (u % m_tiles) * PF_BM;
        n0 = (rest / splits) * N_STEP;
        kb0 = sp * KB / splits;
        kb1 = (sp + 1) * KB / splits;
        return sp;
    };

    if (threadIdx.x == 0) {
        prefetch_map(&map_a_hi); prefetch_map(&map_a_lo); prefetch_map(&map_b);
        for (int s = 0; s < C::STAGES; ++s) { mbar_init(&full_bar[s], 1 + g.extra_arrivals); mbar_init(&empty_bar[s], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], 4); }
        mbar_init(&drain_bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // two accumulators: 2 BN columns of tensor memory, 128 lanes
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(2 * C::BN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    pdl_wait();   // set-up done; from here on the kernel reads what its predecessor wrote

    if (warp == 0 && lane == 0) {            // producer: operand tiles by TMA
        bool ok = true;
        int issued = 0;
        for (int i = 0, it = 0; i < my_tiles && ok; ++i) {
          int m0, n0, kb0, kb1;
          unit_of(i, m0, n0, kb0, kb1);
          for (int kb = kb0; kb < kb1; ++kb, ++it) {
            const int s = it % C::STAGES;
            if (it >= C::STAGES && !mbar_wait(&empty_bar[s], ((it / C::STAGES) - 1) & 1, &abort_flag, g.wait_limit)) { ok = false; break; }
            uint8_t *a = tiles + s * C::STAGE_BYTES, *b = a + 2 * C::A_BYTES;
            mbar_expect_tx(&full_bar[s], C::STAGE_BYTES);
            tma_load_2d(a, &map_a_hi, kb * PF_BK, m0, &full_bar[s]);
            tma_load_2d(a + C::A_BYTES, &map_a_lo, kb * PF_BK, m0, &full_bar[s]);
            tma_load_2d(b, &map_b, kb * PF_BK, n0, &full_bar[s]);
            if (C::BN == 256) tma_load_2d(b + 128 * PF_BK * 2, &map_b, kb * PF_BK, (EPI == EPI_SWIGLU ? g.N : 128) + n0, &full_bar[s]);
            issued = it + 1;
          }
        }
        if (abort_flag) {   // giving up: the copies still in flight must land before the CTA's shared memory is released
            int dummy = 0;
            for (int j = issued > C::STAGES ? issued - C::STAGES : 0; j < issued; ++j)
                mbar_wait(&full_bar[j % C::STAGES], (j / C::STAGES) & 1, &dummy, g.wait_limit);
        }
    } else if (warp == 1 && lane == 0) {     // issuer: per stage 4 tcgen05.mma (K = 16 each) for the hi pieces, 4 for the lo pieces
        constexpr uint32_t idesc = umma_idesc_bf16(PF_BM, C::BN);
        bool ok = true;
        for (int i = 0, it = 0; i < my_tiles && ok; ++i) {
          const int buf = i & 1;
          const uint32_t acc = tmem + buf * C::BN;
          if (i >= 2) ok = mbar_wait(&acc_empty[buf], ((i >> 1) - 1) & 1, &abort_flag, g.wait_limit);   // its epilogue has read it
          if (!ok) break;
          tc_fence_after();
          int m0, n0, kb0, kb1;
          unit_of(i, m0, n0, kb0, kb1);
          for (int kb = kb0; kb < kb1; ++kb, ++it) {
            const int s = it % C::STAGES;
            ok = mbar_wait(&full_bar[s], (it / C::STAGES) & 1, &abort_flag, g.wait_limit);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a = smem_u32(tiles + s * C::STAGE_BYTES), b = a + 2 * C::A_BYTES;
            const uint64_t da = umma_desc_sw128(a), dl = umma_desc_sw128(a + C::A_BYTES), db = umma_desc_sw128(b);
#pragma unroll
            for (int k = 0; k < PF_BK / 16; ++k) umma_bf16(acc, da + 2 * k, db + 2 * k, idesc, ((kb - kb0) | k) != 0);
#pragma unroll
            for (int k = 0; k < PF_BK / 16; ++k) umma_bf16(acc, dl + 2 * k, db + 2 * k, idesc, 1);
            umma_commit(&empty_bar[s]);      // the stage is free again when these have read it
          }
          if (ok) umma_commit(&acc_full[buf]);
        }
        if (!ok) {          // giving up: the multiplies already issued must finish before the tensor memory is freed
            int dummy = 0;
            umma_commit(&drain_bar);
            mbar_wait(&drain_bar, 0, &dummy, g.wait_limit);
        }
    } else if (warp >= 2) {                  // epilogue: warp w may read lanes 32 (w % 4) .. + 31 of tensor memory
      const int quarter = warp & 3;
      for (int i = 0; i < my_tiles; ++i) {
        int m0, n0, kb0, kb1;
        const int sp = unit_of(i, m0, n0, kb0, kb1), buf = i & 1;
        const bool ok = __all_sync(0xffffffffu, mbar_wait(&acc_full[buf], (i >> 1) & 1, &abort_flag, g.wait_limit));   // warp-uniform: tcgen05.ld is .aligned
        if (!ok) break;
        tc_fence_after();
        const int row = m0 + quarter * 32 + lane;
        const bool live = row < g.M;
        const uint32_t trow = tmem + buf * C::BN + (static_cast<uint32_t>(quarter * 32) << 16);
        {
            if (EPI == EPI_RESID) {
                for (int c = 0; c < N_STEP / 32; ++c) {
                    const int n = n0 + c * 32;
                    if (n >= g.N) break;
                    float v[32];
                    tmem_ld32(trow + c * 32, v);
                    tmem_ld_wait();
                    if (live && splits > 1) {   // a partial sum: stored, added to the stream by the norm kernel
                        float4 *p = reinterpret_cast<float4 *>(g.part + sp * g.part_plane + static_cast<size_t>(row) * g.N + n);
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            if (n + 4 * i + 3 < g.N) p[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                    } else if (live) {
                        float4 *p = reinterpret_cast<float4 *>(g.resid + static_cast<size_t>(row) * g.N + n);
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            if (n + 4 * i + 3 < g.N) {
                                float4 o = p[i];
                                o.x += v[4 * i]; o.y += v[4 * i + 1]; o.z += v[4 * i + 2]; o.w += v[4 * i + 3];
                                p[i] = o;
                            }
                    }
                }
            } else if (EPI == EPI_LOGITS) {
                for (int c = 0; c < N_STEP / 32; ++c) {
                    const int n = n0 + c * 32;
                    if (n >= g.N) break;
                    float v[32];
                    tmem_ld32(trow + c * 32, v);
                    tmem_ld_wait();
                    if (live) {                      // N need not be a multiple of 4 (a pruned vocabulary): scalar stores
                        float *p = g.resid + static_cast<size_t>(row) * g.N + n;
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (n + i < g.N) p[i] = v[i];
                    }
                }
            } else if (EPI == EPI_SWIGLU) {
                for (int c = 0; c < 4; ++c) {
                    const int n = n0 + c * 32;
                    if (n >= g.N) break;
                    float gt[32], up[32];
                    tmem_ld32(trow + c * 32, gt);
                    tmem_ld32(trow + 128 + c * 32, up);
                    tmem_ld_wait();
                    if (live) {
                        uint4 *p = reinterpret_cast<uint4 *>(g.act + static_cast<size_t>(row) * g.N + n);
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            if (n + 8 * i + 7 < g.N) {
                                float o[8];
#pragma unroll
                                for (int j = 0; j < 8; ++j) o[j] = gt[8 * i + j] / (1.f + __expf(-gt[8 * i + j])) * up[8 * i + j];
                                uint4 hi, lo;
                                split2x2(o[0], o[1], hi.x, lo.x); split2x2(o[2], o[3], hi.y, lo.y);
                                split2x2(o[4], o[5], hi.z, lo.z); split2x2(o[6], o[7], hi.w, lo.w);
                                p[i] = hi;
                                *reinterpret_cast<uint4 *>(reinterpret_cast<uint16_t *>(p + i) + g.act_plane) = lo;
                            }
                    }
                }
            } else {   // EPI_QKV
                const int half = g.d >> 1;
                for (int off = 0; off < N_STEP; off += g.d) {
                    const int col0 = n0 + off;
                    if (col0 >= g.N) break;
                    const int head = col0 / g.d;
                    if (head < g.nq + g.nkv) {   // q or k: rotate-half pairs (j, j + d/2)
                        const bool is_q = head < g.nq;
                        uint16_t *dst = is_q ? g.q_out + static_cast<size_t>(row) * g.nq * g.d + static_cast<size_t>(head) * g.d
                                                    : g.k_rows + (head - g.nq) * g.head_stride + static_cast<size_t>(row) * g.d;
                        for (int j0 = 0; j0 < half; j0 += 32) {
                            float lo[32], hi[32];
                            tmem_ld32(trow + off + j0, lo);
                            tmem_ld32(trow + off + half + j0, hi);
                            tmem_ld_wait();
                            if (live) {
                                const float2 *cs = g.rope + static_cast<size_t>(row) * half + j0;
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    float a[8], b[8], bx[8], by[8];
                                    if (g.bias) {                        // eight biases per 16-byte load
                                        const uint4 u = *reinterpret_cast<const uint4 *>(g.bias + col0 + j0 + 8 * i);
                                        const uint4 w = *reinterpret_cast<const uint4 *>(g.bias + col0 + half + j0 + 8 * i);
                                        bx[0] = bf16lo(u.x); bx[1] = bf16hi(u.x); bx[2] = bf16lo(u.y); bx[3] = bf16hi(u.y);
                                        bx[4] = bf16lo(u.z); bx[5] = bf16hi(u.z); bx[6] = bf16lo(u.w); bx[7] = bf16hi(u.w);
                                        by[0] = bf16lo(w.x); by[1] = bf16hi(w.x); by[2] = bf16lo(w.y); by[3] = bf16hi(w.y);
                                        by[4] = bf16lo(w.z); by[5] = bf16hi(w.z); by[6] = bf16lo(w.w); by[7] = bf16hi(w.w);
                                    }
#pragma unroll
                                    for (int j = 0; j < 8; j += 2) {
                                        const int e = 8 * i + j;
                                        const float4 t = *reinterpret_cast<const float4 *>(cs + e);   // (cos, sin) of two pairs
                                        float x0 = lo[e], y0 = hi[e], x1 = lo[e + 1], y1 = hi[e + 1];
                                        if (g.bias) { x0 += bx[j]; y0 += by[j]; x1 += bx[j + 1]; y1 += by[j + 1]; }
                                        a[j] = x0 * t.x - y0 * t.y;
                                        b[j] = y0 * t.x + x0 * t.y;
                                        a[j + 1] = x1 * t.z - y1 * t.w;
                                        b[j + 1] = y1 * t.z + x1 * t.w;
                                    }
                                    uint4 ah, al, bh, bl;
                                    split2x2(a[0], a[1], ah.x, al.x); split2x2(a[2], a[3], ah.y, al.y);
                                    split2x2(a[4], a[5], ah.z, al.z); split2x2(a[6], a[7], ah.w, al.w);
                                    split2x2(b[0], b[1], bh.x, bl.x); split2x2(b[2], b[3], bh.y, bl.y);
                                    split2x2(b[4], b[5], bh.z, bl.z); split2x2(b[6], b[7], bh.w, bl.w);
                                    if (!is_q && g.k_stage) {                                  // compressed cache: k in fp32 for the quantiser
                                        float *f = g.k_stage + (head - g.nq) * g.stage_stride + static_cast<size_t>(row) * g.d + j0 + 8 * i;
                                        *reinterpret_cast<float4 *>(f) = make_float4(a[0], a[1], a[2], a[3]);
                                        *reinterpret_cast<float4 *>(f + 4) = make_float4(a[4], a[5], a[6], a[7]);
                                        *reinterpret_cast<float4 *>(f + half) = make_float4(b[0], b[1], b[2], b[3]);
                                        *reinterpret_cast<float4 *>(f + half + 4) = make_float4(b[4], b[5], b[6], b[7]);
                                        continue;
                                    }
                                    *reinterpret_cast<uint4 *>(dst + j0 + 8 * i) = ah;          // k rows: the hi piece IS the bf16 row
                                    *reinterpret_cast<uint4 *>(dst + half + j0 + 8 * i) = bh;
                                    if (is_q) {                                                // queries keep both pieces
                                        *reinterpret_cast<uint4 *>(dst + g.q_plane + j0 + 8 * i) = al;
                                        *reinterpret_cast<uint4 *>(dst + g.q_plane + half + j0 + 8 * i) = bl;
                                    }
                                }
                            }
                        }
                    } else {                     // v: bias only
                        uint16_t *dst = g.v_rows + (head - g.nq - g.nkv) * g.head_stride + static_cast<size_t>(row) * g.d;
                        for (int j0 = 0; j0 < g.d; j0 += 32) {
                            float v[32];
                            tmem_ld32(trow + off + j0, v);
                            tmem_ld_wait();
                            if (live) {
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    float o[8];
#pragma unroll
                                    for (int j = 0; j < 8; ++j)
                                        o[j] = v[8 * i + j] + (g.bias ? bf16_bits_to_f32(g.bias[col0 + j0 + 8 * i + j]) : 0.f);
                                    if (g.v_stage) {
                                        float *f = g.v_stage + (head - g.nq - g.nkv) * g.stage_stride + static_cast<size_t>(row) * g.d + j0 + 8 * i;
                                        *reinterpret_cast<float4 *>(f) = make_float4(o[0], o[1], o[2], o[3]);
                                        *reinterpret_cast<float4 *>(f + 4) = make_float4(o[4], o[5], o[6], o[7]);
                                        continue;
                                    }
                                    *reinterpret_cast<uint4 *>(dst + j0 + 8 * i) =
                                        make_uint4(pack2_bf16(o[0], o[1]), pack2_bf16(o[2], o[3]), pack2_bf16(o[4], o[5]), pack2_bf16(o[6], o[7]));
                                }
                            }
                        }
                    }
                }
            }
        }
        tc_fence_before();           // the accumulator may be overwritten: this warp has read its quarter
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[buf]);
      }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(2 * C::BN) : "memory");
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(g.error, 1);
}

// ---- causal attention on tcgen05 ---------------------------------------------------------------------------------------------
// One CTA = 128 queries of one head (a query = a lane of tensor memory, two softmax threads per query); keys in blocks of 128.
// Per block j:  S_j = Q K_j^T (tcgen05.mma, M 128, N 128, K = D; queries as two bf16 pieces) into one of two S buffers in
// tensor memory;  the softmax warps read their part of the row twice (tcgen05.ld; once for the maximum, once for the
// exponentials), mask on diagonal blocks, update the running maximum and sum, and store the probabilities as two bf16 pieces
// into tensor memory (tcgen05.st, two keys per column);  O_j = P_j V_j (M 128, N = D, K = 128 keys; P from tensor memory, V straight
// from its cache rows as an MN-major B operand), accumulated over the blocks in tensor memory;  the exponentials are taken
// against a reference maximum that moves only when a row's maximum has grown by more than 2^8 (then the row of O and the row
// sum are rescaled once, tcgen05.ld / tcgen05.st).  The scores and P V are issued by two threads (warps 1 and 2), the K and V
// tiles have barriers of their own.
//   tensor memory: S0 [0, 128), S1 [128, 256), O [256, 256 + D), P hi [384, 448), P lo [448, 512)
//   shared memory: Q 2 x D/64 x 16 KB | 2 stages x (K D/64 x 16 KB, V D/64 x 16 KB)   (compressed cache: one stage + landing areas)
#ifndef AT_PARTS_VALUE
#define AT_PARTS_VALUE 2
#endif
constexpr int AT_BM = 128, AT_BN = 128, AT_PARTS = AT_PARTS_VALUE;
constexpr int AT_KVS_MAX = 2;  // stages of the K / V tiles: two on the bf16 cache, one on the compressed cache (whose tiles are
                               // expanded in place)
constexpr int AT_PB = 2;       // the probabilities of a block live in tensor memory as two halves of 64 keys with barriers of their own:
                               // P V of the first half runs while the softmax still works on the second
constexpr int AT_SPLIT_MAX = 8; // CTAs that share the key blocks of a lone query tile
constexpr int AT_CW = 4;       // compressed cache: warps that expand the codes (AT_BN / AT_CW rows of a tile each)
constexpr int AT_THREADS = 96 + 128 * AT_PARTS;   // producer, two issuers, softmax warps

// B operand in MN-major form for P V: the V tile is D/64 blocks of [64 keys][64 d] (128-byte rows, 128-byte swizzle).  N (= d)
// runs along a row, K (= keys) across rows: groups of 8 keys are 1024 bytes apart (stride byte offset), the 64-column blocks
// `lbo` bytes apart (leading byte offset).
__device__ __forceinline__ uint64_t umma_desc_sw128_mn(uint32_t smem_addr, uint32_t lbo) {
    return static_cast<uint64_t>((smem_addr >> 4) & 0x3fffu) | (static_cast<uint64_t>((lbo >> 4) & 0x3fffu) << 16) | (64ull << 32) |
           (1ull << 46) | (2ull << 61);
}

template <int D> struct AttnCfg {
    static constexpr int KBLK = D / 64;                        // 64-column blocks of a row of q, k, v
    static constexpr int Q_BYTES = 2 * KBLK * AT_BM * 128;     // two pieces
    static constexpr int K_BYTES = KBLK * AT_BN * 128, V_BYTES = K_BYTES;
    static constexpr int SMEM = Q_BYTES + 2 * (K_BYTES + V_BYTES) + 1024;     // bf16 cache: two stages of K and V
    // compressed cache: the 8-bit K tile has a landing area of its own, so that it can load while the scores of the block
    // before still read the operand tile; the V tile lands in the first half of its operand tile's own place when a row of
    // codes is as long as a 128-byte operand row (D = 128: every row is then expanded in place; there is no room for a second
    // landing area), D = 64 gets one
    static constexpr int RAW_BYTES = AT_BN * D;
    static constexpr int SMEM_Q8 = Q_BYTES + (K_BYTES + V_BYTES) + (D == 128 ? 1 : 2) * RAW_BYTES + 1024;
    static constexpr int TMEM_COLS = 2 * AT_BN + 2 * D <= 256 ? 256 : 512;   // S0, S1, O0, O1
};

template <int D, bool Q8>
__global__ void __launch_bounds__(AT_THREADS + (Q8 ? 32 * AT_CW : 0)) prefill_attention_tc_kernel(const __grid_constant__ CUtensorMap map_q_hi,
                                                                   const __grid_constant__ CUtensorMap map_q_lo,
                                                                   const __grid_constant__ CUtensorMap map_k,
                                                                   const __grid_constant__ CUtensorMap map_v, uint16_t *out, size_t plane,
                                                                   int T, int slot0, int nq, int group, int max_context,
                                                                   float scale_log2, uint32_t wait_limit, int *error, const float *k_scale,
                                                                   const float *v_scale, float *part_o, float *part_ml) {
    // Q8: the cache holds 8-bit codes and a scale per row (k_scale, v_scale: this layer's [nkv][max_context]); map_k / map_v then
    // describe byte matrices; two more warps expand the codes to bf16 (exactly) into the operand layout, the softmax multiplies
    // the scores by the keys' scales and folds the values' scales into the probabilities.
    pdl_trigger();
    using C = AttnCfg<D>;
    extern __shared__ uint8_t at_tc_dyn[];
    __shared__ uint64_t kraw_full, kraw_empty, vraw_full;
    __shared__ __align__(16) float sc_k[Q8 ? 4 : 1][AT_BN], sc_v[Q8 ? 4 : 1][AT_BN];   // scales of the last four key blocks
    constexpr int AT_KVS = Q8 ? 1 : 2;
    __shared__ uint64_t q_full, k_full[AT_KVS_MAX], k_empty[AT_KVS_MAX], v_full[AT_KVS_MAX], v_empty[AT_KVS_MAX], s_full[2], s_empty[2], p_full[AT_PB], p_empty[AT_PB], o_full[2], o_empty[2], drain_bar[2], pair_bar[4];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ float xchg[2][AT_PARTS][AT_BM];      // row maxima / sums passed between the two threads of a row
    uint8_t *base = at_tc_dyn + ((1024u - (smem_u32(at_tc_dyn) & 1023u)) & 1023u);
    uint8_t *sq = base, *skv = sq + C::Q_BYTES, *sraw = skv + AT_KVS * (C::K_BYTES + C::V_BYTES);   // sraw: landing area of the codes (Q8)
    const uint32_t tmem_p_off = 2 * AT_BN + 128;             // P in tensor memory: hi piece 64 columns (128 keys, two per column), then lo
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // grid (heads, query tiles): CTAs start in linear order, so every head's longest tile (the last queries) starts first
    const int t0 = (gridDim.y - 1 - blockIdx.y) * AT_BM;
    const int h = blockIdx.x, hk = h / group;
    const int last_key = slot0 + min(t0 + AT_BM - 1, T - 1);
    // gridDim.z > 1 (few queries behind a long cache): the key blocks are shared out among gridDim.z CTAs; each leaves its
    // unnormalised row of O, its reference maximum and its row sum in part_o / part_ml, prefill_attention_merge_kernel adds them
    const int nb_total = last_key / AT_BN + 1, splits = gridDim.z;
    const int j0 = static_cast<int>(blockIdx.z) * nb_total / splits;          // first key block of this CTA
    const int nb = (static_cast<int>(blockIdx.z) + 1) * nb_total / splits - j0;   // its key blocks (indices below are local)

    if (threadIdx.x == 0) {
        prefetch_map(&map_q_hi); prefetch_map(&map_q_lo); prefetch_map(&map_k); prefetch_map(&map_v);
        mbar_init(&q_full, 1);
        for (int i = 0; i < AT_KVS; ++i) { mbar_init(&k_full[i], Q8 ? AT_CW : 1); mbar_init(&k_empty[i], 1); mbar_init(&v_full[i], Q8 ? AT_CW : 1); mbar_init(&v_empty[i], 1); }
        mbar_init(&kraw_full, 1); mbar_init(&kraw_empty, AT_CW); mbar_init(&vraw_full, 1);
        for (int i = 0; i < AT_PB; ++i) { mbar_init(&p_full[i], 4 * AT_PARTS); mbar_init(&p_empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&s_full[i], 1); mbar_init(&s_empty[i], 4 * AT_PARTS); mbar_init(&o_full[i], 1); mbar_init(&o_empty[i], 4 * AT_PARTS); }
        mbar_init(&drain_bar[0], 1); mbar_init(&drain_bar[1], 1);
        for (int i = 0; i < 4; ++i) mbar_init(&pair_bar[i], AT_PARTS);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(C::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    pdl_wait();   // set-up done; from here on the kernel reads what its predecessor wrote

    if (warp == 0 && lane == 0) {            // producer: the query tile once, then the K and V rows of every key block
        mbar_expect_tx(&q_full, C::Q_BYTES);
        for (int kb = 0; kb < C::KBLK; ++kb) {
            tma_load_2d(sq + kb * AT_BM * 128, &map_q_hi, h * D + kb * 64, t0, &q_full);
            tma_load_2d(sq + (C::KBLK + kb) * AT_BM * 128, &map_q_lo, h * D + kb * 64, t0, &q_full);
        }
        // K and V of a block have barriers of their own: the K tile is free again as soon as S_j is done, a block earlier than
        // the V tile, and the next scores need only K.  Order of issue: K_0, then K_{j+1} before V_j, so that the wait for V's
        // tile (P V of the block before) never holds the next K tile back.
        int nk = 0, nv = 0;
        auto load_k = [&](int j) {
            const int st = j % AT_KVS;
            uint8_t *k = skv + st * (C::K_BYTES + C::V_BYTES);
            if (j >= AT_KVS && !mbar_wait(Q8 ? &kraw_empty : &k_empty[st], ((j / AT_KVS) - 1) & 1, &abort_flag, wait_limit)) return false;
            if constexpr (Q8) {
                mbar_expect_tx(&kraw_full, C::RAW_BYTES);
                tma_load_2d(sraw, &map_k, 0, hk * max_context + (j0 + j) * AT_BN, &kraw_full);
            } else {
                mbar_expect_tx(&k_full[st], C::K_BYTES);
                for (int kb = 0; kb < C::KBLK; ++kb) tma_load_2d(k + kb * AT_BN * 128, &map_k, kb * 64, hk * max_context + (j0 + j) * AT_BN, &k_full[st]);
            }
            nk = j + 1;
            return true;
        };
        auto load_v = [&](int j) {
            const int st = j % AT_KVS;
            uint8_t *v = skv + st * (C::K_BYTES + C::V_BYTES) + C::K_BYTES;
            if (j >= AT_KVS && !mbar_wait(&v_empty[st], ((j / AT_KVS) - 1) & 1, &abort_flag, wait_limit)) return false;
            if constexpr (Q8) {
                mbar_expect_tx(&vraw_full, C::RAW_BYTES);
                tma_load_2d(D == 128 ? v : sraw + C::RAW_BYTES, &map_v, 0, hk * max_context + (j0 + j) * AT_BN, &vraw_full);
            } else {
                mbar_expect_tx(&v_full[st], C::V_BYTES);
                for (int kb = 0; kb < C::KBLK; ++kb) tma_load_2d(v + kb * AT_BN * 128, &map_v, kb * 64, hk * max_context + (j0 + j) * AT_BN, &v_full[st]);
            }
            nv = j + 1;
            return true;
        };
        bool ok = load_k(0);
        for (int j = 0; j < nb && ok; ++j) {
            if (j + 1 < nb) ok = load_k(j + 1);
            if (ok) ok = load_v(j);
        }
        if (abort_flag) {   // giving up: the copies in flight must land before the shared memory is released
            int dummy = 0;
            mbar_wait(&q_full, 0, &dummy, wait_limit);
            for (int j = nk > AT_KVS ? nk - AT_KVS : 0; j < nk; ++j) mbar_wait(Q8 ? &kraw_full : &k_full[j % AT_KVS], (j / AT_KVS) & 1, &dummy, wait_limit);
            for (int j = nv > AT_KVS ? nv - AT_KVS : 0; j < nv; ++j) mbar_wait(Q8 ? &vraw_full : &v_full[j % AT_KVS], (j / AT_KVS) & 1, &dummy, wait_limit);
        }
    } else if (warp == 1 && lane == 0) {     // issuer of the scores: S_j = Q K_j^T, hi pieces then lo pieces
        // (two issuing threads, scores here and P V in warp 2: a tcgen05.mma takes about 40 ns to issue, and one thread issuing
        // both, with its six waits per block, was what bounded the kernel: 2.3 us per block)
        constexpr uint32_t idesc_s = umma_idesc_bf16(AT_BM, AT_BN);
        bool ok = mbar_wait(&q_full, 0, &abort_flag, wait_limit);
        for (int j = 0; j < nb && ok; ++j) {
            const int st = j % AT_KVS, sb = j & 1;
            ok = mbar_wait(&k_full[st], (j / AT_KVS) & 1, &abort_flag, wait_limit);
            if (ok && j >= 2) ok = mbar_wait(&s_empty[sb], ((j >> 1) - 1) & 1, &abort_flag, wait_limit);   // the softmax has read S_{j-2}
            if (!ok) break;
            tc_fence_after();
            const uint32_t k = smem_u32(skv + st * (C::K_BYTES + C::V_BYTES)), acc = tmem + sb * AT_BN;
#pragma unroll
            for (int piece = 0; piece < 2; ++piece)
#pragma unroll
                for (int kb = 0; kb < C::KBLK; ++kb) {
                    const uint64_t da = umma_desc_sw128(smem_u32(sq) + (piece * C::KBLK + kb) * AT_BM * 128);
                    const uint64_t db = umma_desc_sw128(k + kb * AT_BN * 128);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) umma_bf16(acc, da + 2 * kk, db + 2 * kk, idesc_s, (piece | kb | kk) != 0);
                }
            umma_commit(&s_full[sb]);
            umma_commit(&k_empty[st]);       // the K rows are free when these have read them
        }
        if (!ok) {
            int dummy = 0;
            umma_commit(&drain_bar[0]);
            mbar_wait(&drain_bar[0], 0, &dummy, wait_limit);
        }
    } else if (warp == 2 && lane == 0) {     // issuer of O_j = P_j V_j
        constexpr uint32_t idesc_o = umma_idesc_bf16(AT_BM, D) | (1u << 16);   // B (= V) is MN-major
        bool ok = true;
        for (int j = 0; j < nb && ok; ++j) {
            const int st = j % AT_KVS;
            ok = mbar_wait(&v_full[st], (j / AT_KVS) & 1, &abort_flag, wait_limit);
            const uint32_t v = smem_u32(skv + st * (C::K_BYTES + C::V_BYTES) + C::K_BYTES);
#pragma unroll
            for (int h = 0; h < 2 && ok; ++h) {          // the two 64-key halves of the block
                ok = mbar_wait(&p_full[h], j & 1, &abort_flag, wait_limit);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int piece = 0; piece < 2; ++piece)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)       // 16 keys: 8 columns of P in tensor memory, 2048 bytes of the V tile
                        umma_bf16_ts(tmem + 2 * AT_BN, tmem + tmem_p_off + h * 64 + piece * 32 + kk * 8,
                                     umma_desc_sw128_mn(v + (h * 4 + kk) * 2048, AT_BN * 128), idesc_o, (j | h | piece | kk) != 0);   // O accumulates
                umma_commit(&p_empty[h]);
            }
            if (!ok) break;
            umma_commit(&o_full[0]);
            umma_commit(&v_empty[st]);
        }
        if (!ok) {
            int dummy = 0;
            umma_commit(&drain_bar[1]);
            mbar_wait(&drain_bar[1], 0, &dummy, wait_limit);
        }
    }
    else if (Q8 && warp >= AT_THREADS / 32) {   // compressed cache: expand the 8-bit tiles to bf16 operand tiles (AT_CW warps, AT_BN / AT_CW rows each)
        static_assert(!Q8 || AT_KVS == 1, "one raw tile of K and of V in flight");
        const int cw = warp - AT_THREADS / 32;
        constexpr int LPR = D / 16, RPS = 32 / LPR;       // lanes per row of codes (16 codes each), rows per step
        constexpr int ROWS = AT_BN / AT_CW;               // rows of a tile this warp expands
        auto warp_wait = [&](uint64_t *bar, int parity) {
            int r = 1;
            if (lane == 0) r = mbar_wait(bar, parity, &abort_flag, wait_limit) ? 1 : 0;
            return __shfl_sync(0xffffffffu, r, 0) != 0;
        };
        // 16 codes -> 16 bf16, exactly: byte b of (code + 128) under the exponent of 2^23 is the float 8388608 + code + 128
        auto expand = [&](uint4 c, uint4 &lo8, uint4 &hi8) {
            uint32_t w[4] = {c.x ^ 0x80808080u, c.y ^ 0x80808080u, c.z ^ 0x80808080u, c.w ^ 0x80808080u};
            uint32_t o[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float f0 = __uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7650)) - 8388736.f;
                const float f1 = __uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7651)) - 8388736.f;
                const float f2 = __uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7652)) - 8388736.f;
                const float f3 = __uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7653)) - 8388736.f;
                o[2 * i] = __byte_perm(__float_as_uint(f0), __float_as_uint(f1), 0x7632);
                o[2 * i + 1] = __byte_perm(__float_as_uint(f2), __float_as_uint(f3), 0x7632);
            }
            lo8 = make_uint4(o[0], o[1], o[2], o[3]);
            hi8 = make_uint4(o[4], o[5], o[6], o[7]);
        };
        auto expand_tile = [&](uint8_t *tile, const uint8_t *raw) {
            // a lane takes 16 codes of a row per step; the warp loads the codes of ALL its rows before it stores anything (D = 128:
            // the operand rows overwrite the codes they came from), which also lets the loads overlap
            uint4 codes[ROWS / RPS];
#pragma unroll
            for (int step = 0; step < ROWS / RPS; ++step)
                codes[step] = *reinterpret_cast<const uint4 *>(raw + (cw * ROWS + step * RPS + lane / LPR) * D + (lane % LPR) * 16);
            __syncwarp();
#pragma unroll
            for (int step = 0; step < ROWS / RPS; ++step) {
                const int row = cw * ROWS + step * RPS + lane / LPR, c = lane % LPR;
                uint4 a, b;
                expand(codes[step], a, b);
                uint8_t *dst = tile + (c >> 2) * AT_BN * 128 + row * 128;
                *reinterpret_cast<uint4 *>(dst + (((2 * (c & 3)) ^ (row & 7)) << 4)) = a;
                *reinterpret_cast<uint4 *>(dst + (((2 * (c & 3) + 1) ^ (row & 7)) << 4)) = b;
            }
        };
        uint8_t *k = skv, *v = k + C::K_BYTES;
        auto expand_k = [&](int j) {
            if (!(warp_wait(&kraw_full, j & 1) && (j == 0 || warp_wait(&k_empty[0], (j - 1) & 1)))) return false;   // the codes are here, the operand tile is free
            expand_tile(k, sraw);
            __syncwarp();
            if (lane == 0) mbar_arrive(&kraw_empty);       // the next K tile may land
            for (int i = lane; i < ROWS; i += 32) {        // the scales of this block's keys (both kinds: they are in memory already)
                const int key = min((j0 + j) * AT_BN + cw * ROWS + i, last_key);
                sc_k[j & 3][cw * ROWS + i] = k_scale[static_cast<size_t>(hk) * max_context + key];
                sc_v[j & 3][cw * ROWS + i] = v_scale[static_cast<size_t>(hk) * max_context + key];
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&k_full[0]);
            return true;
        };
        bool ok = expand_k(0);
        for (int j = 0; j < nb && ok; ++j) {              // like the producer: the next K tile before this block's V tile
            if (j + 1 < nb) ok = expand_k(j + 1);
            if (!ok) break;
            ok = warp_wait(&vraw_full, j & 1);
            if (!ok) break;
            expand_tile(v, D == 128 ? v : sraw + C::RAW_BYTES);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&v_full[0]);
        }
    }
    else if (warp >= 3) {                    // softmax: AT_PARTS threads per query row (= lane of tensor memory), AT_BN / AT_PARTS keys of a block each
        const int quarter = warp & 3, part = (warp - 3) >> 2, row = quarter * 32 + lane;
        const uint32_t trow = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
        const int qi = slot0 + t0 + row;     // cache slot of this query: it sees the keys 0 .. qi
        constexpr int DP = D / AT_PARTS;     // this thread's columns of the output row
        // The output row accumulates in tensor memory over the blocks (P V with accumulation).  The exponentials are taken
        // against a reference maximum m_ref that moves only when the row's maximum has grown by more than 2^8 in the
        // exponent (or at the first block); then the row of O and the row sum are rescaled once.  In between the
        // probabilities may reach 2^8, which fp32 sums and the two bf16 pieces carry without loss.
        float m_ref = -INFINITY, l_run = 0.f;
        bool ok = true;
        // one lane waits / arrives for its warp (an mbarrier operation per thread would cost more than the arithmetic)
        auto warp_wait = [&](uint64_t *bar, int parity) {
            int r = 1;
            if (lane == 0) r = mbar_wait(bar, parity, &abort_flag, wait_limit) ? 1 : 0;
            return __shfl_sync(0xffffffffu, r, 0) != 0;
        };
        auto warp_arrive = [&](uint64_t *bar) {
            __syncwarp();
            if (lane == 0) mbar_arrive(bar);
        };
        auto row_sync = [&](int round) {     // the AT_PARTS warps of a quarter meet (bounded like every other wait)
            warp_arrive(&pair_bar[quarter]);
            return warp_wait(&pair_bar[quarter], round & 1);
        };
        for (int j = 0; j < nb; ++j) {
            ok = warp_wait(&s_full[j & 1], (j >> 1) & 1);
            if (!ok) break;
            tc_fence_after();
            const bool diagonal = (j0 + j) * AT_BN + AT_BN - 1 > slot0 + t0;   // some query of the tile does not see the whole block
            // this thread's keys: 32 of the block's first half (chunk 0), 32 of its second half (chunk 1)
            static_assert(AT_PARTS == 2 && AT_BN == 128, "two threads per row, 2 x 32 keys each");
            const uint32_t srow = trow + (j & 1) * AT_BN + part * 32;
            auto load_chunk = [&](int c, float *v) {    // scores of chunk c, scaled (Q8) and masked
                tmem_ld32(srow + c * 64, v);
                tmem_ld_wait();
                if constexpr (Q8) {                   // scores of codes -> scores: the keys' scales (16-byte shared-memory reads)
                    const float4 *sk = reinterpret_cast<const float4 *>(&sc_k[j & 3][c * 64 + part * 32]);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float4 f = sk[i];
                        v[4 * i] *= f.x; v[4 * i + 1] *= f.y; v[4 * i + 2] *= f.z; v[4 * i + 3] *= f.w;
                    }
                }
                if (diagonal) {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if ((j0 + j) * AT_BN + c * 64 + part * 32 + i > qi) v[i] = -INFINITY;
                }
            };
            float mx = -INFINITY;
#pragma unroll
            for (int c = 0; c < 2; ++c) {         // pass 1: the maximum over this thread's keys the query sees
                float v[32];
                load_chunk(c, v);
#pragma unroll
                for (int i = 0; i < 32; i += 4) mx = fmaxf(mx, fmaxf(fmaxf(v[i], v[i + 1]), fmaxf(v[i + 2], v[i + 3])));
            }
            xchg[j & 1][part][row] = mx;     // the row maximum needs the other threads' keys
            ok = row_sync(j);
            if (!ok) break;
            mx = m_ref;
#pragma unroll
            for (int q = 0; q < AT_PARTS; ++q) mx = fmaxf(mx, xchg[j & 1][q][row]);
            if (j == 0) {
                m_ref = fmaxf(mx, -1e30f);   // nothing accumulated yet (a row that sees none of this CTA's keys keeps a finite reference)
            } else if (__any_sync(0xffffffffu, (mx - m_ref) * scale_log2 > 8.f)) {
                // some row of this warp has outgrown its reference (both warps of a quarter see the same rows and maxima, so they
                // decide alike): every row moves its reference to its maximum and rescales its sum and its part of O, once the
                // multiplies of the blocks before are done (the next one waits for this block's probabilities)
                ok = warp_wait(&o_full[0], (j - 1) & 1);
                if (!ok) break;
                tc_fence_after();
                const float f = fast_exp2((m_ref - mx) * scale_log2);
                l_run *= f;
                {
                    float v[DP];
                    tmem_ld<DP>(trow + 2 * AT_BN + part * DP, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < DP; ++i) v[i] *= f;
                    tmem_st<DP>(trow + 2 * AT_BN + part * DP, v);
                }
                tmem_st_wait();
                tc_fence_before();
                m_ref = mx;
            }
            const float neg = -m_ref * scale_log2;
            float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
            for (int c = 0; c < 2; ++c) {         // pass 2: probabilities as two bf16 pieces, half by half
                float v[32];
                load_chunk(c, v);
                if (c == 1) {
                    tc_fence_before();
                    warp_arrive(&s_empty[j & 1]);     // S_j has been read for the last time
                }
                uint32_t phi[16], plo[16];        // two keys per word
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const float p0 = fast_exp2(fmaf(v[i], scale_log2, neg)), p1 = fast_exp2(fmaf(v[i + 1], scale_log2, neg));
                    sum0 += p0;
                    sum1 += p1;
                    if constexpr (Q8) {               // the values' scales ride on the probabilities
                        const float2 f = *reinterpret_cast<const float2 *>(&sc_v[j & 3][c * 64 + part * 32 + i]);
                        split2x2_trunc(p0 * f.x, p1 * f.y, phi[i / 2], plo[i / 2]);
                    } else {
                        split2x2_trunc(p0, p1, phi[i / 2], plo[i / 2]);
                    }
                }
                if (j >= 1) {                     // this half's multiply of the block before is done
                    ok = warp_wait(&p_empty[c], (j - 1) & 1);
                    if (!ok) break;
                }
                // P as the A operand in tensor memory: lane = query row, a column holds two consecutive keys (bf16)
                tmem_st16(trow + tmem_p_off + c * 64 + part * 16, reinterpret_cast<const float *>(phi));
                tmem_st16(trow + tmem_p_off + c * 64 + 32 + part * 16, reinterpret_cast<const float *>(plo));
                tmem_st_wait();
                tc_fence_before();
                warp_arrive(&p_full[c]);
            }
            if (!ok) break;
            l_run += sum0 + sum1;
        }
        float o[DP];
        if (ok) ok = warp_wait(&o_full[0], (nb - 1) & 1);   // the last block's multiply
        if (ok) {
            tc_fence_after();
            tmem_ld<DP>(trow + 2 * AT_BN + part * DP, o);
            tmem_ld_wait();
        }
        if (ok) {
            xchg[nb & 1][part][row] = l_run; // the parts of the row sum
            ok = row_sync(nb);
            l_run = 0.f;
#pragma unroll
            for (int q = 0; q < AT_PARTS; ++q) l_run += xchg[nb & 1][q][row];
        }
        const int t = t0 + row;
        if (ok && t < T && splits > 1) {     // partial result of this CTA's key blocks
            const size_t slot = (static_cast<size_t>(blockIdx.z) * AT_BM + row) * nq + h;
            float *dst = part_o + slot * D + part * DP;
#pragma unroll
            for (int i = 0; i < DP; i += 4) *reinterpret_cast<float4 *>(dst + i) = make_float4(o[i], o[i + 1], o[i + 2], o[i + 3]);
            if (part == 0) { part_ml[slot * 2] = m_ref; part_ml[slot * 2 + 1] = l_run; }
        } else if (ok && t < T) {
            const float inv = 1.f / l_run;
            uint16_t *dst = out + static_cast<size_t>(t) * nq * D + static_cast<size_t>(h) * D + part * DP;
#pragma unroll
            for (int i = 0; i < DP; i += 8) {
                uint4 hi, lo;
                split2x2(o[i] * inv, o[i + 1] * inv, hi.x, lo.x); split2x2(o[i + 2] * inv, o[i + 3] * inv, hi.y, lo.y);
                split2x2(o[i + 4] * inv, o[i + 5] * inv, hi.z, lo.z); split2x2(o[i + 6] * inv, o[i + 7] * inv, hi.w, lo.w);
                *reinterpret_cast<uint4 *>(dst + i) = hi;
                *reinterpret_cast<uint4 *>(dst + plane + i) = lo;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(AttnCfg<D>::TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(error, 1);
}

// Adds the partial results of a query tile whose key blocks were shared out among `splits` CTAs: for row t and head h,
// M = max m_s, O = sum O_s 2^((m_s - M) c), L = sum l_s 2^((m_s - M) c), out = O / L as two bf16 planes.  grid (T, nq), D / 4 threads.
template <int D>
__global__ void __launch_bounds__(D / 4) prefill_attention_merge_kernel(const float *part_o, const float *part_ml, int splits, uint16_t *out,
                                                                        size_t plane, int nq, float scale_log2) {
    pdl_trigger();
    pdl_wait();
    const int t = blockIdx.x, h = blockIdx.y, i = threadIdx.x * 4;
    float mmax = -INFINITY;
    for (int s = 0; s < splits; ++s) mmax = fmaxf(mmax, part_ml[((static_cast<size_t>(s) * AT_BM + t) * nq + h) * 2]);
    float l = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < splits; ++s) {
        const size_t slot = (static_cast<size_t>(s) * AT_BM + t) * nq + h;
        const float w = fast_exp2((part_ml[slot * 2] - mmax) * scale_log2);
        const float4 o = *reinterpret_cast<const float4 *>(part_o + slot * D + i);
        l = fmaf(part_ml[slot * 2 + 1], w, l);
        acc.x = fmaf(o.x, w, acc.x); acc.y = fmaf(o.y, w, acc.y); acc.z = fmaf(o.z, w, acc.z); acc.w = fmaf(o.w, w, acc.w);
    }
    const float inv = 1.f / l;
    uint2 hi, lo;
    split2x2(acc.x * inv, acc.y * inv, hi.x, lo.x);
    split2x2(acc.z * inv, acc.w * inv, hi.y, lo.y);
    uint16_t *dst = out + static_cast<size_t>(t) * nq * D + static_cast<size_t>(h) * D + i;
    *reinterpret_cast<uint2 *>(dst) = hi;
    *reinterpret_cast<uint2 *>(dst + plane) = lo;
}

// Launch with the programmatic-stream-serialization attribute (see pdl_trigger / pdl_wait) for passes of up to 1024 tokens:
// there the kernels are short and the launch gaps are 3 - 5 % of a prompt (512 tokens: 4.37 -> 4.17 ms); longer passes lose 1 - 3 %
// with it (7B shape, 2048 tokens: 44.8 -> 46.5 ms), so they are launched the plain way (the kernels' griddepcontrol
// instructions are then no-ops).
thread_local bool g_pdl = false;
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args &&...args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- host side ---------------------------------------------------------------------------------------------------------------
// Map of a row-major bf16 [rows][K] matrix; a box is box_rows rows x 64 columns (one 128-byte swizzled row each); rows and
// columns outside the matrix read as zero.  (No multicast is used with these maps.)
bool encode_operand_map(CUtensorMap *m, const void *base, long long rows, int K, int box_rows = 128) {
    TensorMapEncodeFn enc = tensor_map_encoder();
    if (!enc) return false;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(K) * 2};
    const cuuint32_t box[2] = {PF_BK, static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t es[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int EPI, int SHAPE>
const char *launch_gemm_cfg(const CUtensorMap &ma, const CUtensorMap &ml, const CUtensorMap &mb, const GemmArgs &g, int num_sms, cudaStream_t s) {
    using C = GemmCfg<SHAPE>;
    if (cudaFuncSetAttribute(prefill_gemm_kernel<EPI, SHAPE>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM) != cudaSuccess)
        return "cudaFuncSetAttribute failed";
    const int n_step = EPI == EPI_SWIGLU ? 128 : C::BN;
    const int units = ((g.N + n_step - 1) / n_step) * ((g.M + PF_BM - 1) / PF_BM) * (EPI == EPI_RESID ? g.splits : 1);
    launch_pdl(prefill_gemm_kernel<EPI, SHAPE>, dim3(units < num_sms ? units : num_sms), dim3(192), C::SMEM, s, ma, ml, mb, g);
    return cudaGetLastError() == cudaSuccess ? nullptr : "prefill GEMM launch failed";
}

// Shape and K split.  Cost model: the rounds the SMs need (units / SMs, rounded up) times the cost of a unit; a wide tile does
// twice the work of a narrow one for 1.33 x the operand traffic (1.6), a K split divides a unit's cost and adds a little for
// the partial sums (5 %).  Only the contractions that add to the residual stream split (their partial sums are added by the
// norm kernel that follows, in a fixed order); a split keeps at least 12 k-blocks per unit and is considered only when the
// unsplit tiles do not fill the SMs once (with more tiles the partial-sum traffic costs more than the better balance gains:
// 7B shape, 2048 tokens, 48.0 -> 50.7 ms).
template <int EPI>
const char *launch_gemm(const uint16_t *a, size_t a_plane, const void *w, long long w_rows, GemmArgs &g, int num_sms, cudaStream_t s) {
    CUtensorMap ma, ml, mb;
    if (!encode_operand_map(&ma, a, g.M, g.K) || !encode_operand_map(&ml, a + a_plane, g.M, g.K) || !encode_operand_map(&mb, w, w_rows, g.K))
        return "cuTensorMapEncodeTiled failed";
    int wide = 1;
    prefill_plan_contraction(EPI, g.M, g.N, g.K, num_sms, &wide, &g.splits);
    if constexpr (EPI == EPI_SWIGLU) {
        return launch_gemm_cfg<EPI, PF_WIDE>(ma, ml, mb, g, num_sms, s);
    } else {
        return wide ? launch_gemm_cfg<EPI, PF_WIDE>(ma, ml, mb, g, num_sms, s) : launch_gemm_cfg<EPI, PF_NARROW>(ma, ml, mb, g, num_sms, s);
    }
}

// Map of a byte matrix [rows][row_bytes] (the codes of a compressed cache); a box is box_rows whole rows, unswizzled.
bool encode_bytes_map(CUtensorMap *m, const void *base, long long rows, int row_bytes, int box_rows) {
    TensorMapEncodeFn enc = tensor_map_encoder();
    if (!enc) return false;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(row_bytes), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(row_bytes)};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(row_bytes), static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t es[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// kc / vc: this layer's cache, bf16 rows or (k_scale != nullptr) rows of 8-bit codes with their scales.
// A single query tile behind a long cache (a short suffix behind a prefix, a verified block) would run on n_q CTAs only: its key
// blocks are then shared out among up to AT_SPLIT_MAX CTAs per head and the partial results merged (part_o / part_ml: room for
// AT_SPLIT_MAX x 128 rows).
template <int D>
const char *launch_attention_tc(const uint16_t *q, const void *kc, const void *vc, const float *k_scale, const float *v_scale, uint16_t *out,
                                size_t plane, int T, int slot0, int nq, int nkv, int max_context, uint32_t wait_limit, int *error,
                                float *part_o, float *part_ml, int num_sms, cudaStream_t s) {
    CUtensorMap mqh, mql, mk, mv;
    const long long kv_rows = static_cast<long long>(nkv) * max_context;
    const bool q8 = k_scale != nullptr;
    if (!encode_operand_map(&mqh, q, T, nq * D) || !encode_operand_map(&mql, q + plane, T, nq * D)) return "cuTensorMapEncodeTiled failed";
    if (q8 ? (!encode_bytes_map(&mk, kc, kv_rows, D, AT_BN) || !encode_bytes_map(&mv, vc, kv_rows, D, AT_BN))
           : (!encode_operand_map(&mk, kc, kv_rows, D, AT_BN) || !encode_operand_map(&mv, vc, kv_rows, D, AT_BN)))
        return "cuTensorMapEncodeTiled failed";
    const float scale_log2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(D)));
    int splits = 1;
    if (T <= AT_BM) {
        const int blocks = (slot0 + T - 1) / AT_BN + 1;
        splits = num_sms / nq;                       // CTAs per head that still fit the SMs once
        if (splits > AT_SPLIT_MAX) splits = AT_SPLIT_MAX;
        if (splits > blocks / 2) splits = blocks / 2;   // at least two key blocks per CTA
        if (splits < 1) splits = 1;
    }
    const dim3 grid(nq, (T + AT_BM - 1) / AT_BM, splits);
    if (q8) {
        if (cudaFuncSetAttribute(prefill_attention_tc_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnCfg<D>::SMEM_Q8) != cudaSuccess)
            return "cudaFuncSetAttribute failed";
        launch_pdl(prefill_attention_tc_kernel<D, true>, grid, dim3(AT_THREADS + 32 * AT_CW), AttnCfg<D>::SMEM_Q8, s, mqh, mql, mk, mv, out, plane, T,
                   slot0, nq, nq / nkv, max_context, scale_log2, wait_limit, error, k_scale, v_scale, part_o, part_ml);
    } else {
        if (cudaFuncSetAttribute(prefill_attention_tc_kernel<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnCfg<D>::SMEM) != cudaSuccess)
            return "cudaFuncSetAttribute failed";
        launch_pdl(prefill_attention_tc_kernel<D, false>, grid, dim3(AT_THREADS), AttnCfg<D>::SMEM, s, mqh, mql, mk, mv, out, plane, T, slot0, nq,
                   nq / nkv, max_context, scale_log2, wait_limit, error, static_cast<const float *>(nullptr), static_cast<const float *>(nullptr), part_o,
                   part_ml);
    }
    if (splits > 1)
        launch_pdl(prefill_attention_merge_kernel<D>, dim3(T, nq), dim3(D / 4), 0, s, static_cast<const float *>(part_o),
                   static_cast<const float *>(part_ml), splits, out, plane, nq, scale_log2);
    return cudaGetLastError() == cudaSuccess ? nullptr : "prefill attention launch failed";
}

}  // namespace

void prefill_plan_contraction(int epilogue, int M, int N, int K, int num_sms, int *wide, int *splits) {
    const int m_tiles = (M + PF_BM - 1) / PF_BM, kb = (K + PF_BK - 1) / PF_BK;
    *wide = 1;
    *splits = 1;
    if (epilogue == EPI_SWIGLU) return;
    const int tiles[2] = {((N + 127) / 128) * m_tiles, ((N + 255) / 256) * m_tiles};
    const double cost[2] = {1.0, 1.6};
    int best_shape = 0, best_split = 1;
    double best = 1e30;
    for (int shape = 0; shape < 2; ++shape)
        for (int sp = 1; sp <= (epilogue == EPI_RESID ? (m_tiles == 1 ? PF_SPLIT_MAX : 4) : 1); ++sp) {
            if (sp > 1 && (kb / sp < 12 || tiles[shape] > num_sms)) break;   // split only grids that leave SMs idle in their one round
            const int units = tiles[shape] * sp;
            const double t = ((units + num_sms - 1) / num_sms) * cost[shape] / sp * (sp > 1 ? 1.05 : 1.0);
            if (t < best - 1e-9) { best = t; best_shape = shape; best_split = sp; }
        }
    *wide = best_shape;
    *splits = best_split;
}

size_t prefill_buffer_bytes(const edgefm_shape &sh, int chunk) {
    const size_t c = static_cast<size_t>(chunk), qd = static_cast<size_t>(sh.n_q_heads) * sh.head_dim;
    return c * sh.hidden * 4 * (1 + PF_SPLIT_MAX) + c * sh.hidden * 4 + 2 * c * qd * 4 + c * sh.ffn * 4 + c * (sh.head_dim / 2) * 8 + c * 4 + 256;
}

cudaError_t prefill_alloc(PrefillBuffers *b, const edgefm_shape &sh, int chunk, bool kv8) {
    const size_t c = static_cast<size_t>(chunk), qd = static_cast<size_t>(sh.n_q_heads) * sh.head_dim;
    cudaError_t e;
    if ((e = cudaMalloc(&b->resid, c * sh.hidden * 4)) != cudaSuccess) return e;
    if ((e = cudaMalloc(&b->xn, c * sh.hidden * 4)) != cudaSuccess) return e;
    if ((e = cudaMalloc(&b->part, c * sh.hidden * 4 * PF_SPLIT_MAX)) != cudaSuccess) return e;
    if ((e = cudaMalloc(&b->q, c * qd * 4)) != cudaSuccess) return e;
    if ((e = cudaMalloc(&b->attn, c * qd * 4)) != cudaSuccess) return e;
    if ((e = cudaMalloc(&b->act, c * sh.ffn * 4)) != cudaSuccess) return e;
    if ((e = cudaMalloc(&b->rope, c * (sh.head_dim / 2) * sizeof(float2))) != cudaSuccess) return e;
    if (kv8 && (e = cudaMalloc(&b->kv_stage, 2 * c * sh.n_kv_heads * sh.head_dim * sizeof(float))) != cudaSuccess) return e;
    if ((e = cudaMalloc(&b->tokens, c * 4)) != cudaSuccess) return e;
    if ((e = cudaMalloc(&b->error, 4)) != cudaSuccess) return e;
    b->logits_rows = sh.vocab;
    if ((e = cudaMalloc(&b->logits, static_cast<size_t>(PF_VERIFY_MAX) * sh.vocab * 4)) != cudaSuccess) return e;
    if ((e = cudaMalloc(&b->att_o, static_cast<size_t>(AT_SPLIT_MAX) * AT_BM * qd * 4)) != cudaSuccess) return e;
    if ((e = cudaMalloc(&b->att_ml, static_cast<size_t>(AT_SPLIT_MAX) * AT_BM * sh.n_q_heads * 2 * 4)) != cudaSuccess) return e;
    if ((e = cudaMalloc(&b->head_val, PF_HEAD_GRID_MAX * PF_VERIFY_MAX * 4)) != cudaSuccess) return e;
    if ((e = cudaMalloc(&b->head_idx, PF_HEAD_GRID_MAX * PF_VERIFY_MAX * 4)) != cudaSuccess) return e;
    if ((e = cudaMalloc(&b->head_ticket, 4)) != cudaSuccess) return e;
    if ((e = cudaMemset(b->head_ticket, 0, 4)) != cudaSuccess) return e;
    if ((e = cudaMemset(b->error, 0, 4)) != cudaSuccess) return e;
    b->chunk = chunk;
    return cudaSuccess;
}

void prefill_free(PrefillBuffers *b) {
    cudaFree(b->resid); cudaFree(b->xn); cudaFree(b->part); cudaFree(b->kv_stage); cudaFree(b->q); cudaFree(b->attn); cudaFree(b->act); cudaFree(b->rope);
    cudaFree(b->tokens); cudaFree(b->error); cudaFree(b->logits); cudaFree(b->att_o); cudaFree(b->att_ml); cudaFree(b->head_val); cudaFree(b->head_idx); cudaFree(b->head_ticket);
    *b = PrefillBuffers{};
}

const char *prefill_run(const PrefillModel &m, PrefillBuffers *b, const int32_t *tokens, int n, int slot0, int position, bool whole_last_layer,
                        cudaStream_t s, int *launches) {
    const edgefm_shape &sh = m.shape;
    const int H = sh.hidden, F = sh.ffn, d = sh.head_dim, nq = sh.n_q_heads, nkv = sh.n_kv_heads, qd = nq * d;
    const int n_qkv = (nq + 2 * nkv) * d;
    const long long head_stride = static_cast<long long>(m.max_context) * d;
    const size_t cap = static_cast<size_t>(b->chunk), x_plane = cap * H, q_plane = cap * qd, f_plane = cap * F;   // hi / lo planes
    int count = 0;
    g_pdl = n <= 1024;
    if (cudaMemcpyAsync(b->tokens, tokens, static_cast<size_t>(n) * 4, cudaMemcpyHostToDevice, s) != cudaSuccess) return "token upload failed";
    launch_pdl(prefill_rope_kernel, dim3((n * (d / 2) + 255) / 256), dim3(256), 0, s, b->rope, n, d / 2, position, static_cast<double>(sh.rope_theta));
    const int norm_grid = n;
    launch_pdl(prefill_norm_kernel, dim3(norm_grid), dim3(128), 0, s, b->resid, b->xn, x_plane, static_cast<const uint16_t *>(m.layers[0].input_norm),
                                                  static_cast<const uint16_t *>(m.embed), b->tokens, n, H, sh.rms_eps, m.state,
                                                  slot0 + n, position + n, nullptr, 0, 0);
    count += 2;
    for (int l = 0; l < sh.n_layers; ++l) {
        const edgefm_layer_weights &w = m.layers[l];
        const bool kv8 = m.k_scale != nullptr;   // compressed cache: one byte per element and a scale per row
        const size_t layer_rows = static_cast<size_t>(l) * nkv * m.max_context;
        uint16_t *kc = m.k_cache + static_cast<size_t>(l) * nkv * head_stride, *vc = m.v_cache + static_cast<size_t>(l) * nkv * head_stride;
        signed char *kc8 = reinterpret_cast<signed char *>(m.k_cache) + layer_rows * d, *vc8 = reinterpret_cast<signed char *>(m.v_cache) + layer_rows * d;
        GemmArgs g{};
        g.M = n; g.error = b->error; g.wait_limit = b->wait_limit; g.extra_arrivals = b->extra_arrivals;
        g.N = n_qkv; g.K = H;
        g.bias = sh.qkv_bias ? static_cast<const uint16_t *>(w.bqkv) : nullptr;
        if (g.bias && (reinterpret_cast<uintptr_t>(g.bias) & 15u)) return "edgefm_prefill reads bqkv in 16-byte pieces: the vector must be 16-byte aligned";
        g.rope = b->rope; g.q_out = b->q; g.q_plane = q_plane;
        g.k_rows = kc + static_cast<size_t>(slot0) * d; g.v_rows = vc + static_cast<size_t>(slot0) * d;
        g.nq = nq; g.nkv = nkv; g.d = d; g.head_stride = head_stride;
        if (kv8) { g.k_stage = b->kv_stage; g.v_stage = b->kv_stage + cap * nkv * d; g.stage_stride = static_cast<long long>(cap) * d; }
        if (const char *e = launch_gemm<EPI_QKV>(b->xn, x_plane, w.wqkv, n_qkv, g, m.num_sms, s)) return e;
        ++count;
        if (kv8) {   // the new rows, compressed into their cache slots (attention reads them from there, like every other row)
            launch_pdl(prefill_quantize_rows_kernel, dim3((2 * nkv * n + 7) / 8), dim3(256), 0, s, g.k_stage, g.v_stage, g.stage_stride, kc8, vc8, m.k_scale + layer_rows,
                                                                              m.v_scale + layer_rows, nkv, n, d, m.max_context, slot0);
            ++count;
        }
        if (l == sh.n_layers - 1 && !whole_last_layer) break;   // the rest of the last layer feeds nothing that is kept
        const void *ka = kv8 ? static_cast<const void *>(kc8) : kc, *va = kv8 ? static_cast<const void *>(vc8) : vc;
        const float *ksc = kv8 ? m.k_scale + layer_rows : nullptr, *vsc = kv8 ? m.v_scale + layer_rows : nullptr;
        const char *e = d == 64 ? launch_attention_tc<64>(b->q, ka, va, ksc, vsc, b->attn, q_plane, n, slot0, nq, nkv, m.max_context, b->wait_limit, b->error, b->att_o, b->att_ml, m.num_sms, s)
                                : launch_attention_tc<128>(b->q, ka, va, ksc, vsc, b->attn, q_plane, n, slot0, nq, nkv, m.max_context, b->wait_limit, b->error, b->att_o, b->att_ml, m.num_sms, s);
        if (e) return e;
        g.N = H; g.K = qd; g.resid = b->resid; g.part = b->part; g.part_plane = x_plane;
        if ((e = launch_gemm<EPI_RESID>(b->attn, q_plane, w.wo, H, g, m.num_sms, s))) return e;
        launch_pdl(prefill_norm_kernel, dim3(norm_grid), dim3(128), 0, s, b->resid, b->xn, x_plane, static_cast<const uint16_t *>(w.post_norm), nullptr, nullptr, n, H,
                                                      sh.rms_eps, nullptr, 0, 0, b->part, g.splits, x_plane);
        g.N = F; g.K = H; g.act = b->act; g.act_plane = f_plane;
        if ((e = launch_gemm<EPI_SWIGLU>(b->xn, x_plane, w.w_gate_up, 2LL * F, g, m.num_sms, s))) return e;
        g.N = H; g.K = F;
        if ((e = launch_gemm<EPI_RESID>(b->act, f_plane, w.w_down, H, g, m.num_sms, s))) return e;
        // (behind the last layer the norm weights do not matter: the kernel runs for the K-split partial sums of the down projection)
        launch_pdl(prefill_norm_kernel, dim3(norm_grid), dim3(128), 0, s, b->resid, b->xn, x_plane, static_cast<const uint16_t *>(m.layers[l + 1 < sh.n_layers ? l + 1 : l].input_norm),
                                                      nullptr, nullptr, n, H, sh.rms_eps, nullptr, 0, 0, b->part, g.splits, x_plane);
        count += 6;
    }
    if (cudaGetLastError() != cudaSuccess) return "prefill kernel launch failed";
    if (launches) *launches = count;
    return nullptr;
}

const char *prefill_head(const PrefillModel &m, PrefillBuffers *b, int row, const void *final_norm, const void *lm, const int *ids, int rows,
                         float *logits_out, int *next_token_out, int token, int pos, cudaStream_t s) {
    const int H = m.shape.hidden;
    int grid = 2 * m.num_sms;
    if (grid > PF_HEAD_GRID_MAX) grid = PF_HEAD_GRID_MAX;
    if (grid * 8 > rows) grid = (rows + 7) / 8;
    if (H * 4 > 40 * 1024 &&
        cudaFuncSetAttribute(prefill_head_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, H * 4) != cudaSuccess)
        return "cudaFuncSetAttribute failed";
    launch_pdl(prefill_head_kernel, dim3(grid), dim3(256), static_cast<size_t>(H) * 4, s, b->resid + static_cast<size_t>(row) * H, static_cast<const uint16_t *>(final_norm),
                                                                     static_cast<const uint16_t *>(lm), ids, rows, H, m.shape.rms_eps, logits_out,
                                                                     next_token_out, b->head_val, b->head_idx, b->head_ticket, m.state, token, pos);
    return cudaGetLastError() == cudaSuccess ? nullptr : "prefill output layer launch failed";
}

const char *prefill_verify_head(const PrefillModel &m, PrefillBuffers *b, int n, const void *final_norm, const void *lm, const int *ids, int rows,
                                float *logits_out, int *n_accepted_out, int *next_token_out, int slot0, int pos, cudaStream_t s) {
    // final norm of the block's rows (two bf16 planes), the logits of all rows as ONE contraction over the output matrix on the
    // tensor cores (into the caller's buffer or the work buffer), then the greedy tokens and the acceptance rule
    const int H = m.shape.hidden;
    const size_t x_plane = static_cast<size_t>(b->chunk) * H;
    float *logits = logits_out ? logits_out : b->logits;
    if (!logits_out && rows > b->logits_rows) return "block verification: the work buffer for the logits is too small";
    launch_pdl(prefill_norm_kernel, dim3(n), dim3(128), 0, s, b->resid, b->xn, x_plane, static_cast<const uint16_t *>(final_norm),
               static_cast<const uint16_t *>(nullptr), static_cast<const int *>(nullptr), n, H, m.shape.rms_eps, static_cast<StepState *>(nullptr), 0, 0,
               static_cast<const float *>(nullptr), 0, static_cast<size_t>(0));
    GemmArgs g{};
    g.M = n; g.N = rows; g.K = H; g.error = b->error; g.wait_limit = b->wait_limit; g.extra_arrivals = b->extra_arrivals;
    g.resid = logits;
    if (const char *e = launch_gemm<EPI_LOGITS>(b->xn, x_plane, lm, rows, g, m.num_sms, s)) return e;
    int grid = m.num_sms;
    if (grid > PF_HEAD_GRID_MAX) grid = PF_HEAD_GRID_MAX;
    if (grid * 256 > rows) grid = (rows + 255) / 256;
    launch_pdl(prefill_verify_pick_kernel, dim3(grid), dim3(256), 0, s, static_cast<const float *>(logits), ids, rows, n, static_cast<const int *>(b->tokens),
               b->head_val, b->head_idx, b->head_ticket, m.state, slot0, pos, n_accepted_out, next_token_out);
    return cudaGetLastError() == cudaSuccess ? nullptr : "block verification output layer launch failed";
}

}  // namespace edgefm
