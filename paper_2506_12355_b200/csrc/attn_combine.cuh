// Merge of partial attention results computed over disjoint K/V shards.
//
// For every query row, shard r delivers a normalised O_r and LSE_r = ln(sum of exponentials over the
// shard's visible keys).  Softmax over the union of the shards is then exactly
//     LSE = ln sum_r exp(LSE_r),      O = sum_r exp(LSE_r - LSE) * O_r,
// the same rescaling identity the online softmax of the attention kernels applies tile by tile.
// Shards in which a row sees no key carry LSE_r = -inf and drop out.  Memory-bound elementwise work.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace attn_merge {

template <int DTYPE>
__device__ __forceinline__ void unpack8(const uint4& w, float* f) {
    const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if constexpr (DTYPE == 0) {
            const __half2 h = *reinterpret_cast<const __half2*>(&u[i]);
            f[2 * i] = __low2float(h);
            f[2 * i + 1] = __high2float(h);
        } else {
            const __nv_bfloat162 h = *reinterpret_cast<const __nv_bfloat162*>(&u[i]);
            f[2 * i] = __low2float(h);
            f[2 * i + 1] = __high2float(h);
        }
    }
}

template <int DTYPE>
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    if constexpr (DTYPE == 0) {
        __half2 h = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&h);
    } else {
        __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&h);
    }
}

// The merge of rows [row0, row0 + n_rows) of the flattened (batch, head, query) axis; one thread per 8
// consecutive output elements (16 bytes).  `src` says where shard r's partial result lies: src.lse(r, row)
// and src.o(r, row, seg) (seg: 16-byte piece of the row).  o: [rows_total, D]; lse: [rows_total].
template <int DTYPE, int BATCH, class Src>
__device__ __forceinline__ void merge_rows(const Src src, int n_parts, uint4* __restrict__ o, float* __restrict__ lse,
                                           int64_t row0, int64_t n_rows, int segs_per_row) {
    const int64_t total = n_rows * segs_per_row;
    for (int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; idx < total;
         idx += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t local_row = idx / segs_per_row;
        const int seg = static_cast<int>(idx - local_row * segs_per_row);
        const int64_t row = row0 + local_row;
        float mx = -INFINITY;
        for (int r = 0; r < n_parts; ++r) mx = fmaxf(mx, src.lse(r, row));
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        float total_lse = -INFINITY;
        if (mx != -INFINITY) {
            float sum = 0.f;
            for (int r = 0; r < n_parts; ++r) sum += expf(src.lse(r, row) - mx);
            total_lse = mx + logf(sum);
            // BATCH shards at a time: all loads of a batch are issued before their results are used
            for (int r0 = 0; r0 < n_parts; r0 += BATCH) {
                uint4 v[BATCH];
                float w[BATCH];
#pragma unroll
                for (int i = 0; i < BATCH; ++i) {
                    const int r = r0 + i < n_parts ? r0 + i : n_parts - 1;   // tail: re-read the last shard, weight 0
                    v[i] = src.o(r, row, seg);
                    w[i] = r0 + i < n_parts ? expf(src.lse(r, row) - total_lse) : 0.f;
                }
#pragma unroll
                for (int i = 0; i < BATCH; ++i) {
                    float f[8];
                    unpack8<DTYPE>(v[i], f);
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[e] = fmaf(w[i], f[e], acc[e]);
                }
            }
        }
        uint4 w;
        w.x = pack2<DTYPE>(acc[0], acc[1]);
        w.y = pack2<DTYPE>(acc[2], acc[3]);
        w.z = pack2<DTYPE>(acc[4], acc[5]);
        w.w = pack2<DTYPE>(acc[6], acc[7]);
        o[row * segs_per_row + seg] = w;
        if (seg == 0) lse[row] = total_lse;
    }
}

// Shards stacked in one allocation of this GPU: o_parts [n_parts, rows, D] 16-bit, lse_parts [n_parts, rows] fp32
// (read through the read-only path).
struct StackedParts {
    const uint4* __restrict__ o_parts;
    const float* __restrict__ lse_parts;
    int64_t rows;
    int segs_per_row;
    __device__ __forceinline__ float lse(int r, int64_t row) const { return lse_parts[r * rows + row]; }
    __device__ __forceinline__ uint4 o(int r, int64_t row, int seg) const {
        return __ldg(o_parts + (r * rows + row) * segs_per_row + seg);
    }
};

template <int DTYPE, int BATCH>
__global__ void __launch_bounds__(256)
attn_combine_kernel(const uint4* __restrict__ o_parts, const float* __restrict__ lse_parts, int n_parts,
                    uint4* __restrict__ o, float* __restrict__ lse, int64_t rows, int segs_per_row) {
    merge_rows<DTYPE, BATCH>(StackedParts{o_parts, lse_parts, rows, segs_per_row}, n_parts, o, lse, 0, rows, segs_per_row);
}

// Every shard's partial result behind its own base pointer (a table passed by value).  The pointers may be peer
// memory: a rank of a K/V-sharded run merges its slice of the rows by reading the other ranks' partial results
// over NVLink in place, so the exchange and the merge are one kernel and nothing is gathered first.
// Plain loads only: no TMA, no cluster multicast, no read-only-path loads of memory a peer may rewrite.
constexpr int kMaxGatherParts = 32;
struct GatherTable {
    const uint4* o[kMaxGatherParts];      // each [rows_total, D] 16-bit
    const float* lse[kMaxGatherParts];    // each [rows_total] fp32
};

struct TableParts {
    const GatherTable& tab;
    int segs_per_row;
    __device__ __forceinline__ float lse(int r, int64_t row) const { return tab.lse[r][row]; }
    __device__ __forceinline__ uint4 o(int r, int64_t row, int seg) const { return tab.o[r][row * segs_per_row + seg]; }
};

template <int DTYPE, int BATCH>
__global__ void __launch_bounds__(256)
attn_combine_gather_kernel(const GatherTable tab, int n_parts, uint4* __restrict__ o, float* __restrict__ lse,
                           int64_t row0, int64_t n_rows, int segs_per_row) {
    merge_rows<DTYPE, BATCH>(TableParts{tab, segs_per_row}, n_parts, o, lse, row0, n_rows, segs_per_row);
}

}  // namespace attn_merge
