// Shared device helpers of the decode-step kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace edgefm {

// Device-resident dynamic parameters of the step graph (Sec. 3.10 of the paper: dynamic
// parameters live in GPU buffers so that one fixed graph serves every decode iteration).
struct StepState {
    int token;          // input token of the step in flight
    int position;       // its rotary position
    int cur_len;        // filled cache slots before the step == slot the step writes
    int next_token;     // greedy result of the last finished step
    int next_position;  // position the next step uses when the caller passes -1
    int status;         // 0 = ok (reserved for bounded-wait failures)
    int pad[2];
    int n_accepted;     // tokens of the last block the cache was advanced by (1 for a plain step)
    int reserved[3];
};

// What the host asks of the next step; uploaded only when it differs from the previous request.
struct StepRequest {
    int token;          // >= 0 explicit, -1 = StepState::next_token
    int position;       // >= 0 explicit, -1 = StepState::next_position
    float *logits_out;  // device fp32[V] (a block of m tokens: [m][V]) or null
    int *next_token_out;  // device int32[1] or null
    int m;              // tokens in this call: 1 = a plain decode step; > 1 = a block to verify (Sec. 3.11): `token` followed by
    int draft[3];       // ... the proposed continuation draft[0 .. m-2]
    int flags;          // bit 0: the tokens are given, not proposed (prompt tokens): all m enter the cache
    int pad_;
    int *n_accepted_out;  // device int32[1] or null: how many of the m tokens entered the cache (1 + accepted proposals)
};

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ float bf16_bits_to_f32(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }
__device__ __forceinline__ uint16_t f32_to_bf16_bits(float f) { return __bfloat16_as_ushort(__float2bfloat16_rn(f)); }

// acc += <8 bf16 weights, 8 fp32 activations>
__device__ __forceinline__ float dot8(uint4 w, float4 x0, float4 x1, float acc) {
    acc = fmaf(bf16lo(w.x), x0.x, acc);
    acc = fmaf(bf16hi(w.x), x0.y, acc);
    acc = fmaf(bf16lo(w.y), x0.z, acc);
    acc = fmaf(bf16hi(w.y), x0.w, acc);
    acc = fmaf(bf16lo(w.z), x1.x, acc);
    acc = fmaf(bf16hi(w.z), x1.y, acc);
    acc = fmaf(bf16lo(w.w), x1.z, acc);
    acc = fmaf(bf16hi(w.w), x1.w, acc);
    return acc;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// (value, index) ordering of the greedy sampler: larger value wins, equal values -> lower index.
__device__ __forceinline__ bool arg_better(float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); }

}  // namespace edgefm
