// river_quantize_w4: the exit layers' weights from the backbone's, on the GPU (sm_100a).
//
// River-LLM builds an exit layer by copying a backbone block and quantising its Attention and FFN matrices with a
// training-free 4-bit weight-only method, HQQ (paper Section 4.1).  One thread owns one group of `group` inputs of a
// weight row: the scale comes from the group's range ((max - min) / 15, stored as bf16); the zero-point starts at
// -min / s and is refined by HQQ's half-quadratic iteration - quantise, shrink the residual with the generalised soft
// threshold of an l_p norm (p = 0.7), re-solve the zero-point in closed form as the group mean of W_q - (W - W_e) / s,
// beta growing by 1.01 per round - and is stored as bf16; the codes are then taken against the stored scale and zero,
// so that (q - z) s is the best the stored triple can give.  refine_iters = 0 leaves the plain min/max grid.
// Every arithmetic step is a single fp32 operation in a fixed order (no fused multiply-add, sums sequential over the
// group), because it decides integers: a reference that follows the same order reproduces the codes bit for bit.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "../../include/river.h"

namespace {

constexpr int kMaxGroup = 128;

__device__ __forceinline__ float bf16_round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

template <int G>
__global__ void __launch_bounds__(128) quantize_w4_kernel(const __nv_bfloat16 *w, long long n_groups, int refine_iters,
                                                          uint8_t *codes, __nv_bfloat16 *scale, __nv_bfloat16 *zero) {
    const long long gi = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (gi >= n_groups) return;
    float x[G];
    const uint4 *src = reinterpret_cast<const uint4 *>(w + gi * G);
#pragma unroll
    for (int i = 0; i < G / 8; ++i) {
        const uint4 v = src[i];
        const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            x[8 * i + 2 * j] = __uint_as_float(u[j] << 16);
            x[8 * i + 2 * j + 1] = __uint_as_float(u[j] & 0xffff0000u);
        }
    }
    float mn = x[0], mx = x[0];
#pragma unroll
    for (int i = 1; i < G; ++i) { mn = fminf(mn, x[i]); mx = fmaxf(mx, x[i]); }
    const bool constant = mx == mn;
    float s = bf16_round(__fdiv_rn(__fsub_rn(mx, mn), 15.0f));
    if (constant || s == 0.f) s = 1.f;
    float z = __fdiv_rn(-mn, s);
    float beta = 10.0f;
    for (int it = 0; it < refine_iters; ++it) {
        const float inv_beta = __fdiv_rn(1.0f, beta);
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < G; ++i) {
            const float q = fminf(fmaxf(rintf(__fadd_rn(__fdiv_rn(x[i], s), z)), 0.f), 15.f);
            const float e = __fsub_rn(x[i], __fmul_rn(__fsub_rn(q, z), s));
            const float ae = fabsf(e);
            float we = 0.f;
            if (ae > 0.f) {
                const float t = __fsub_rn(ae, __fmul_rn(inv_beta, powf(ae, 0.7f - 1.0f)));
                we = copysignf(fmaxf(t, 0.f), e);
            }
            sum = __fadd_rn(sum, __fsub_rn(q, __fdiv_rn(__fsub_rn(x[i], we), s)));
        }
        z = __fdiv_rn(sum, (float)G);
        beta = __fmul_rn(beta, 1.01f);
    }
    float zb = bf16_round(z);
    if (constant) zb = bf16_round(-mn);
    uint32_t packed[G / 8];
#pragma unroll
    for (int i = 0; i < G / 8; ++i) {
        uint32_t p = 0u;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float q = fminf(fmaxf(rintf(__fadd_rn(__fdiv_rn(x[8 * i + j], s), zb)), 0.f), 15.f);
            if (constant) q = 0.f;
            p |= (uint32_t)q << (4 * j);  // low nibble = even input
        }
        packed[i] = p;
    }
    uint32_t *dst = reinterpret_cast<uint32_t *>(codes + gi * (G / 2));
#pragma unroll
    for (int i = 0; i < G / 8; ++i) dst[i] = packed[i];
    scale[gi] = __float2bfloat16_rn(s);
    zero[gi] = __float2bfloat16_rn(zb);
}

}  // namespace

extern "C" int river_quantize_w4(const void *w, int out, int in, int group, int refine_iters, void *codes, void *scale,
                                 void *zero, void *cuda_stream) {
    if (!w || !codes || !scale || !zero || out <= 0 || in <= 0 || refine_iters < 0 || refine_iters > 1000) return RIVER_E_BADARG;
    if (!(group == 32 || group == 64 || group == kMaxGroup) || in % group) return RIVER_E_SHAPE;
    if (((uintptr_t)w | (uintptr_t)codes) & 15) return RIVER_E_BADARG;  // 16-byte loads / 4-byte stores of whole groups
    const long long n_groups = (long long)out * (in / group);
    const unsigned grid = (unsigned)((n_groups + 127) / 128);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const __nv_bfloat16 *wp = static_cast<const __nv_bfloat16 *>(w);
    uint8_t *cp = static_cast<uint8_t *>(codes);
    __nv_bfloat16 *sp = static_cast<__nv_bfloat16 *>(scale), *zp = static_cast<__nv_bfloat16 *>(zero);
    if (group == 32) quantize_w4_kernel<32><<<grid, 128, 0, st>>>(wp, n_groups, refine_iters, cp, sp, zp);
    else if (group == 64) quantize_w4_kernel<64><<<grid, 128, 0, st>>>(wp, n_groups, refine_iters, cp, sp, zp);
    else quantize_w4_kernel<128><<<grid, 128, 0, st>>>(wp, n_groups, refine_iters, cp, sp, zp);
    return cudaGetLastError() == cudaSuccess ? RIVER_OK : RIVER_E_DEVICE;
}
