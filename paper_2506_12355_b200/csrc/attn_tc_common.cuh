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

// End of a persistent kernel, executed by one thread per CTA after the CTA's last draw from the work
// counter: reports a timed-out wait, and hands the counter back zeroed.  counter[0] is the next work
// item, counter[1] the number of CTAs that have finished; the CTA that finishes last resets both, so
// the next launch that uses this counter (launches that share one are ordered on one stream) starts
// from zero without a memset.  Every CTA reaches this point, also after a timed-out wait.
__device__ __forceinline__ void finish_cta(int* status, bool timed_out, unsigned int* counter) {
    if (timed_out) atomicExch(status, kStatusTimeout);
    if (counter) {
        __threadfence();
        if (atomicAdd(counter + 1, 1u) == gridDim.x - 1) {
            counter[0] = 0u;
            counter[1] = 0u;
            __threadfence();
        }
    }
}

}  // namespace attn_tc
