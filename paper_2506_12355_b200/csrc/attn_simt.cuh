// CUDA-core cross-check kernel for the attention operator of Section 2.2: one warp per
// query row, fp32 arithmetic, online softmax over chunks of 32 keys.  No tensor cores, no
// TMA, no shared-memory tiling of K/V: it is deliberately simple so that it can stand
// beside the tcgen05 kernel as an independent on-device check.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <stdint.h>

namespace attn_simt {

// DTYPE 0 / 1: fp16 / bf16 inputs and output; DTYPE 2: E4M3 inputs (one byte each), bf16 output.
template <int DTYPE>
__device__ __forceinline__ float load16(const void* base, int64_t idx) {
    if constexpr (DTYPE == 0) {
        return __half2float(reinterpret_cast<const __half*>(base)[idx]);
    } else if constexpr (DTYPE == 1) {
        return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(base)[idx]);
    } else {
        const __half_raw h = __nv_cvt_fp8_to_halfraw(reinterpret_cast<const __nv_fp8_storage_t*>(base)[idx], __NV_E4M3);
        return __half2float(__half(h));   // every E4M3 value is exact in binary16
    }
}

template <int DTYPE>
__device__ __forceinline__ void store16(void* base, int64_t idx, float x) {
    if constexpr (DTYPE == 0)
        reinterpret_cast<__half*>(base)[idx] = __float2half_rn(x);
    else
        reinterpret_cast<__nv_bfloat16*>(base)[idx] = __float2bfloat16_rn(x);
}

constexpr int kWarpsPerBlock = 4;

template <int D, int DTYPE>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
attn_fwd_simt_kernel(const void* __restrict__ q, const void* __restrict__ k,
                     const void* __restrict__ v, void* __restrict__ o, float* __restrict__ lse,
                     int Sq, int Sk, float scale, int causal, int H, int Hkv, int k_offset, float o_scale) {
    constexpr int CPL = D / 32;  // output columns per lane
    __shared__ float qs[kWarpsPerBlock][D];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t bh = blockIdx.y;
    const int64_t i = static_cast<int64_t>(blockIdx.x) * kWarpsPerBlock + warp;
    if (i >= Sq) return;

    const int64_t qrow = (bh * Sq + i) * D;
    const int64_t kv_bh = (bh / H) * Hkv + (bh % H) / (H / Hkv);  // grouped-query attention
    const int64_t kvbase = kv_bh * static_cast<int64_t>(Sk) * D;
    for (int d = lane; d < D; d += 32) qs[warp][d] = load16<DTYPE>(q, qrow + d);
    __syncwarp();

    // visible keys: all, or (causal) those with k_offset + j <= i
    int64_t n_vis = Sk;
    if (causal) {
        n_vis = i + 1 - k_offset;
        if (n_vis < 0) n_vis = 0;
        if (n_vis > Sk) n_vis = Sk;
    }
    float m = -INFINITY, l = 0.f;
    float acc[CPL];
#pragma unroll
    for (int c = 0; c < CPL; ++c) acc[c] = 0.f;

    for (int64_t j0 = 0; j0 < n_vis; j0 += 32) {
        const int64_t j = j0 + lane;
        float s = -INFINITY;
        if (j < n_vis) {
            float dot = 0.f;
            for (int d = 0; d < D; ++d) dot = fmaf(qs[warp][d], load16<DTYPE>(k, kvbase + j * D + d), dot);
            s = dot * scale;
        }
        float mx = s;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        const float m_new = fmaxf(m, mx);  // finite: the chunk holds at least one visible key
        const float alpha = expf(m - m_new);
        const float p = (j < n_vis) ? expf(s - m_new) : 0.f;
        float ps = p;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, off);
        l = l * alpha + ps;
#pragma unroll
        for (int c = 0; c < CPL; ++c) acc[c] *= alpha;
        const int nj = (n_vis - j0 < 32) ? static_cast<int>(n_vis - j0) : 32;
        for (int jj = 0; jj < nj; ++jj) {
            const float pj = __shfl_sync(0xffffffffu, p, jj);
            const int64_t vrow = kvbase + (j0 + jj) * D + lane * CPL;
#pragma unroll
            for (int c = 0; c < CPL; ++c) acc[c] = fmaf(pj, load16<DTYPE>(v, vrow + c), acc[c]);
        }
        m = m_new;
    }

    const float inv = (l > 0.f) ? o_scale / l : 0.f;
#pragma unroll
    for (int c = 0; c < CPL; ++c) store16<DTYPE>(o, qrow + lane * CPL + c, acc[c] * inv);
    if (lane == 0) lse[bh * Sq + i] = (l > 0.f) ? m + logf(l) : -INFINITY;
}

// O = 0, LSE = -inf for problems without keys.
__global__ void attn_fill_empty_kernel(uint16_t* __restrict__ o, float* __restrict__ lse,
                                       int64_t n_o, int64_t n_lse) {
    const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t e = t; e < n_o; e += stride) o[e] = 0;
    for (int64_t e = t; e < n_lse; e += stride) lse[e] = -INFINITY;
}

}  // namespace attn_simt
