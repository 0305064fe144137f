// Definitions shared by the tensor-core attention kernels.
#pragma once
#include "sm100_ptx.cuh"

namespace attn_tc {

using namespace sm100;

constexpr int kStatusTimeout = 9;  // ATTN_ERR_DEVICE_TIMEOUT

// Last key (index inside this K/V shard) that query row `row` may see, or a negative number when it
// sees none: all Sk keys without a mask; with the causal mask key j of a shard that starts at global
// key index k_offset is visible iff k_offset + j <= row.
__device__ __forceinline__ int last_visible_key(int row, int Sk, int causal, int k_offset) {
    const int all = Sk - 1;
    if (!causal) return all;
    const int c = row - k_offset;
    return c < all ? c : all;
}

}  // namespace attn_tc
