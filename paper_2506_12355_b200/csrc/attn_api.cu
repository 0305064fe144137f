// C ABI of the attention forward library (declared in include/attn_fwd.h):
// host-side validation, TMA tensor-map construction and kernel dispatch.
// There is no CPU fallback anywhere in this file.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <functional>
#include <map>
#include <mutex>
#include <thread>
#include <utility>
#include <vector>

#include "../../include/attn_fwd.h"
#include "attn_bwd.cuh"
#include "attn_combine.cuh"
#include "attn_simt.cuh"
#include "attn_tc_qtmem.cuh"
#include "attn_tc_pipe.cuh"

// Share of the exponentials evaluated by a polynomial on the FMA pipe instead of the special-function
// unit (POLY_NUM of every POLY_DEN element pairs).
#ifndef ATTN_POLY_NUM
#define ATTN_POLY_NUM 1
#define ATTN_POLY_DEN 8
#endif

#ifndef ATTN_POLY64_NUM
#define ATTN_POLY64_NUM 1
#define ATTN_POLY64_DEN 4
#endif
#ifndef ATTN_FP8_POLY_NUM
#define ATTN_FP8_POLY_NUM 1
#define ATTN_FP8_POLY_DEN 8
#endif
#ifndef ATTN_MERGE_LAST
#define ATTN_MERGE_LAST 3
#endif
#ifndef ATTN_L2_MB
#define ATTN_L2_MB 24
#endif

namespace {

// Device-side status word: 0, or ATTN_ERR_DEVICE_TIMEOUT once a kernel gave up on a wait.
__device__ int g_device_status = 0;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// Rank-3 map over a [BH, S, D] row-major tensor of 16-bit (dtype 0 / 1) or 8-bit (dtype 2) elements;
// box = [1, box_rows, 128 bytes of columns], 128-byte swizzle, out-of-range rows read as zero.
// head_stride_rows: distance between consecutive (batch, head) slices in rows (S for a contiguous tensor; larger
// when the map covers a range of rows of a bigger tensor: a K/V shard addressed in place).
// A tensor map is a pure function of the address and the shape arguments (it does not depend on the
// memory's contents), so encoded maps are kept in a small per-thread direct-mapped cache: a caller
// that passes the same buffers again (a training or serving loop) pays for four look-ups instead of
// four driver calls per launch.
struct MapKey {
    const void* base;
    int64_t BH, S, head_stride_rows;
    int dtype, D, box_rows;
    bool operator==(const MapKey& o) const {
        return base == o.base && BH == o.BH && S == o.S && head_stride_rows == o.head_stride_rows && dtype == o.dtype &&
               D == o.D && box_rows == o.box_rows;
    }
};
struct MapCacheEntry {
    bool valid = false;
    MapKey key;
    CUtensorMap map;
};
constexpr int kMapCacheSize = 64;

bool encode_map(CUtensorMap* map, const void* base, int dtype, int64_t BH, int64_t S, int D, int box_rows,
                int64_t head_stride_rows);

bool make_map(CUtensorMap* map, const void* base, int dtype, int64_t BH, int64_t S, int D, int box_rows,
              int64_t head_stride_rows = -1) {
    thread_local MapCacheEntry cache[kMapCacheSize];
    const MapKey key{base, BH, S, head_stride_rows, dtype, D, box_rows};
    uint64_t h = reinterpret_cast<uintptr_t>(base) >> 8;
    h = (h ^ (static_cast<uint64_t>(S) * 0x9E3779B97F4A7C15ull) ^ (static_cast<uint64_t>(BH) << 17) ^
         (static_cast<uint64_t>(D + 3 * dtype + 7 * box_rows) << 40) ^ static_cast<uint64_t>(head_stride_rows)) *
        0xD6E8FEB86659FD93ull;
    MapCacheEntry& e = cache[(h >> 32) % kMapCacheSize];
    if (e.valid && e.key == key) {
        *map = e.map;
        return true;
    }
    if (!encode_map(map, base, dtype, BH, S, D, box_rows, head_stride_rows)) return false;
    e.valid = true;
    e.key = key;
    e.map = *map;
    return true;
}

bool encode_map(CUtensorMap* map, const void* base, int dtype, int64_t BH, int64_t S, int D, int box_rows,
                int64_t head_stride_rows) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return false;
    const cuuint64_t es = dtype == ATTN_DTYPE_FP8_E4M3 ? 1 : 2;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(S), static_cast<cuuint64_t>(BH)};
    const cuuint64_t hs = static_cast<cuuint64_t>(head_stride_rows < 0 ? S : head_stride_rows);
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(D) * es, hs * D * es};
    cuuint32_t box[3] = {static_cast<cuuint32_t>(128 / es), static_cast<cuuint32_t>(box_rows), 1};
    cuuint32_t estr[3] = {1, 1, 1};
    const CUtensorMapDataType type = dtype == ATTN_DTYPE_FP16   ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                     : dtype == ATTN_DTYPE_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                                                : CU_TENSOR_MAP_DATA_TYPE_UINT8;
    CUresult r = enc(map, type,
                     3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

int check_arch() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ATTN_ERR_CUDA;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return ATTN_ERR_CUDA;
    return major == 10 ? ATTN_OK : ATTN_ERR_UNSUPPORTED_ARCH;
}

constexpr int kMaxSeq = 2147483647 - 256;

// Validation shared by every entry point; no CUDA call happens here.
int validate(const void* q, const void* k, const void* v, const void* o, const void* lse, int B, int H, int Hkv, int Sq,
             int Sk, int D, float scale, int dtype, bool device_pointers) {
    if (B < 0 || H < 0 || Hkv < 0 || Sq < 0 || Sk < 0 || D < 0) return ATTN_ERR_BAD_SHAPE;
    if (H > 0 && (Hkv == 0 || H % Hkv != 0)) return ATTN_ERR_BAD_SHAPE;
    // empty tensors may come with NULL pointers (an allocator returns none for zero bytes)
    const bool no_rows = static_cast<int64_t>(B) * H * Sq == 0, no_keys = static_cast<int64_t>(B) * Hkv * Sk == 0;
    if (!no_rows && (!q || !o || !lse)) return ATTN_ERR_NULL_POINTER;
    if (!no_rows && !no_keys && (!k || !v)) return ATTN_ERR_NULL_POINTER;
    if (Sq > kMaxSeq || Sk > kMaxSeq) return ATTN_ERR_BAD_SHAPE;
    if (static_cast<int64_t>(B) * H > 2147483647LL) return ATTN_ERR_BAD_SHAPE;
    if (D != 64 && D != 128 && D != 256) return ATTN_ERR_UNSUPPORTED_HEAD_DIM;
    if (dtype != ATTN_DTYPE_FP16 && dtype != ATTN_DTYPE_BF16) return ATTN_ERR_UNSUPPORTED_DTYPE;
    if (device_pointers) {
        if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k) | reinterpret_cast<uintptr_t>(v) |
             reinterpret_cast<uintptr_t>(o)) & 15u)
            return ATTN_ERR_MISALIGNED;
        if (reinterpret_cast<uintptr_t>(lse) & 3u) return ATTN_ERR_MISALIGNED;
    }
    if (!isfinite(scale) || scale < 0.f) return ATTN_ERR_BAD_SCALE;
    return ATTN_OK;
}

// Work counters of the persistent kernels.  A counter is two words {next item, CTAs done}; it is zero
// when a launch starts and the kernel zeroes it again when its last CTA exits, so no memset is
// enqueued.  Two launches may share a counter only if they cannot overlap, hence:
//   * an eager launch takes the counter of its stream (launches on one stream are ordered); the
//     per-thread default stream is a different stream in every host thread and is keyed by thread too;
//   * a launch made while its stream is being captured into a CUDA graph takes a counter of its own
//     from a separate region that eager launches never use: a graph may be replayed on any stream,
//     at any time, next to eager launches.  (Replays of one executable graph are ordered by CUDA.)
// Both regions are finite; when one is used up the launch is refused with ATTN_ERR_COUNTER_SLOTS.
constexpr int kStreamSlots = 768;    // distinct streams that may launch counted kernels, per device
constexpr int kCaptureSlots = 256;   // counted launches that may be captured into graphs, per device
__device__ unsigned int g_work_counters[2 * (kStreamSlots + kCaptureSlots)];

constexpr int kMaxDevices = 64;

struct DeviceInfo {
    unsigned int* counters = nullptr;
    int sm_count = 0;
};

struct CounterTable {
    std::mutex mu;
    std::map<std::pair<uintptr_t, size_t>, int> by_stream;
    int captured = 0;
};
CounterTable g_counter_table[kMaxDevices];

// Per-device facts resolved on first use (symbol address of the counters, SM count).
int device_info(DeviceInfo* out, int* dev_out = nullptr) {
    static std::mutex mu;
    static DeviceInfo info[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ATTN_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!info[dev].counters) {
        void* p = nullptr;
        int sms = 0;
        if (cudaGetSymbolAddress(&p, g_work_counters) != cudaSuccess || !p) return ATTN_ERR_CUDA;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
            return ATTN_ERR_CUDA;
        info[dev].counters = static_cast<unsigned int*>(p);
        info[dev].sm_count = sms;
    }
    *out = info[dev];
    if (dev_out) *dev_out = dev;
    return ATTN_OK;
}

// The work counter for a launch on stream `st` of the current device (see above).
int work_counter(const DeviceInfo& di, int dev, cudaStream_t st, unsigned int** out) {
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) return ATTN_ERR_CUDA;
    CounterTable& tab = g_counter_table[dev];
    std::lock_guard<std::mutex> lock(tab.mu);
    int slot;
    if (cap != cudaStreamCaptureStatusNone) {
        if (tab.captured >= kCaptureSlots) return ATTN_ERR_COUNTER_SLOTS;
        slot = kStreamSlots + tab.captured++;
    } else {
        const size_t thread_key = st == cudaStreamPerThread ? std::hash<std::thread::id>()(std::this_thread::get_id()) : 0;
        const auto key = std::make_pair(reinterpret_cast<uintptr_t>(st), thread_key);
        auto it = tab.by_stream.find(key);
        if (it == tab.by_stream.end()) {
            if (tab.by_stream.size() >= static_cast<size_t>(kStreamSlots)) return ATTN_ERR_COUNTER_SLOTS;
            it = tab.by_stream.emplace(key, static_cast<int>(tab.by_stream.size())).first;
        }
        slot = it->second;
    }
    *out = di.counters + 2 * slot;
    return ATTN_OK;
}

// Raises a kernel's dynamic shared-memory limit once per (kernel, device): the attribute belongs to
// the device's context, and one process may drive several GPUs.
bool allow_dynamic_smem(const void* kern, int bytes) {
    static std::mutex mu;
    static std::vector<std::pair<const void*, int>> done;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    std::lock_guard<std::mutex> lock(mu);
    for (const auto& d : done)
        if (d.first == kern && d.second == dev) return true;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    done.emplace_back(kern, dev);
    return true;
}

int* device_status_ptr() {
    int* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_device_status) != cudaSuccess) return nullptr;
    return p;
}

int fill_empty(void* o, float* lse, int64_t n_o, int64_t n_lse, cudaStream_t st) {
    attn_simt::attn_fill_empty_kernel<<<148, 256, 0, st>>>(static_cast<uint16_t*>(o), lse, n_o, n_lse);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

#ifdef ATTN_TEST_HOOKS
int g_test_skip_ring_item = -1;   // test build only: consumed by the next launch of the pipelined kernel
#endif

// Pipelined, warp-specialised kernel (head dims 64 and 128): one CTA per pair of 128-row Q tiles.
template <int D, int DTYPE>
int launch_tc_pipe(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv, int Sq, int Sk,
                   float scale, int causal, int k_offset, cudaStream_t st, float o_scale = 1.f, int64_t kv_stride_rows = -1,
                   int n_splits = 1) {
    // n_splits > 1: the keys are cut into n_splits ranges of whole tiles; range s of a head is a work item of its own
    // and writes its partial result as head s * (B * H) + bh of o and lse, which then hold n_splits partial results
    constexpr int ES = DTYPE == ATTN_DTYPE_FP8_E4M3 ? 1 : 2;                 // bytes per Q/K/V element
    constexpr int ODT = DTYPE == ATTN_DTYPE_FP8_E4M3 ? ATTN_DTYPE_BF16 : DTYPE;   // O storage type
    using C = attn_tc::PipeCfg<D, ES>;
    // share of the exponentials evaluated by the polynomial (measured best): 1 pair in 8 at head dim 128, 1 in 4 at
    // head dim 64, where the tensor core leaves more issue slots to the softmax warps
    constexpr int PN = DTYPE == ATTN_DTYPE_FP8_E4M3 ? ATTN_FP8_POLY_NUM : (D == 64 ? ATTN_POLY64_NUM : ATTN_POLY_NUM);
    constexpr int PD = DTYPE == ATTN_DTYPE_FP8_E4M3 ? ATTN_FP8_POLY_DEN : (D == 64 ? ATTN_POLY64_DEN : ATTN_POLY_DEN);
    auto kern = n_splits > 1 ? attn_tc::attn_fwd_tc_pipe_kernel<D, DTYPE, PN, PD, true> : attn_tc::attn_fwd_tc_pipe_kernel<D, DTYPE, PN, PD, false>;
    if (!allow_dynamic_smem(reinterpret_cast<const void*>(kern), C::SMEM_BYTES)) return ATTN_ERR_CUDA;
    const int64_t BH = static_cast<int64_t>(B) * H;
    const int64_t n_pairs = (static_cast<int64_t>(Sq) + 2 * C::BM - 1) / (2 * C::BM);
    if (n_pairs * BH * n_splits > 2147483647LL) return ATTN_ERR_BAD_SHAPE;
    CUtensorMap mq, mk, mv, mo;
    if (!make_map(&mq, q, DTYPE, BH, Sq, D, C::BM) ||
        !make_map(&mk, k, DTYPE, static_cast<int64_t>(B) * Hkv, Sk, D, C::BN, kv_stride_rows) ||
        !make_map(&mv, v, DTYPE, static_cast<int64_t>(B) * Hkv, Sk, D, C::BN, kv_stride_rows) ||
        !make_map(&mo, o, ODT, BH * n_splits, Sq, D, C::BM))
        return ATTN_ERR_CUDA;
    attn_tc::PipeParams prm;
    prm.o = o;
    prm.lse = lse;
    prm.Sq = Sq;
    prm.Sk = Sk;
    prm.scale = scale;
    prm.scale_log2 = scale * 1.4426950408889634f;
    prm.o_scale = o_scale;
    prm.causal = causal ? 1 : 0;
    prm.status = device_status_ptr();
    if (!prm.status) return ATTN_ERR_CUDA;
    prm.H = H;
    prm.Hkv = Hkv;
    prm.k_offset = k_offset;
    prm.n_pairs = static_cast<int>(n_pairs);
    prm.BH = static_cast<int>(BH);
    // walk together as many heads as keep their K and V (2 * Sk * D * 2 bytes each) inside ~24 MB of L2 (the L2 is split over two dies)
    const int64_t kv_bytes_per_head = 2LL * ES * Sk * D;
    int64_t hpg = (static_cast<int64_t>(ATTN_L2_MB) << 20) / (kv_bytes_per_head > 0 ? kv_bytes_per_head : 1);
    if (hpg < 1) hpg = 1;
    hpg *= H / Hkv;  // the query heads of one K/V head share its footprint
    if (hpg > BH) hpg = BH;
    prm.heads_per_group = static_cast<int>(hpg);
    // under the causal mask the last three groups are merged into one: its items, ordered longest-first, then
    // end with short ones, which keeps the tail of the launch short; without a mask all items are equally long
    // and merging would only enlarge the K/V footprint of the tail beyond what stays in L2
    {
        const int64_t n_groups = (BH + hpg - 1) / hpg;
        const int merge = causal ? ATTN_MERGE_LAST : 1;
        prm.last_group = static_cast<int>(n_groups >= merge ? n_groups - merge : 0);
    }
    prm.n_items = static_cast<int>(n_pairs * BH * n_splits);
    prm.halves_from = 2147483647;
    prm.n_splits = n_splits;
    {
        const int tiles = (Sk + C::BN - 1) / C::BN;
        prm.split_tiles = n_splits > 1 ? (tiles + n_splits - 1) / n_splits : 2147483647 / 2;
    }
#ifdef ATTN_TEST_HOOKS
    prm.test_skip_ring_item = g_test_skip_ring_item;
    g_test_skip_ring_item = -1;
#endif
    // persistent grid: one CTA per SM; the first item of a CTA is its block index, the rest come from
    // a device counter that is zero at launch (the previous kernel that used it left it so)
    DeviceInfo di;
    int dev = 0;
    if (device_info(&di, &dev) != ATTN_OK) return ATTN_ERR_CUDA;
    // Without a mask all items are equally long (whole keys, n_splits == 1): when the last wave would occupy at most
    // half of the CTAs, its items are cut into their two Q tiles (a tile alone runs a step in ~83 % of the time of
    // two in ping-pong, so the launch ends after ~0.83 instead of 1 more item time).
    if (!causal && n_splits == 1 && Sq >= 2 * C::BM && prm.n_items > di.sm_count && prm.n_items < 2147483647 - di.sm_count) {
        const int rem = prm.n_items % di.sm_count;
        if (rem > 0 && 2 * rem <= di.sm_count) {
            prm.halves_from = prm.n_items - rem;
            prm.n_items += rem;
        }
    }
    const unsigned grid = static_cast<unsigned>(prm.n_items < di.sm_count ? prm.n_items : di.sm_count);
    prm.counter = nullptr;   // small problems: every CTA takes exactly one item, no counter
    if (prm.n_items > di.sm_count) {
        const int rc = work_counter(di, dev, st, &prm.counter);
        if (rc != ATTN_OK) return rc;
    }
    kern<<<grid, C::THREADS, C::SMEM_BYTES, st>>>(mq, mk, mv, mo, prm);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

// One Q tile per CTA, Q in tensor memory, double-buffered S: head dim 256 and the 192/128 head shape.
template <int DQK, int DV, int BN, int DTYPE>
int launch_tc_qtmem(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv, int Sq, int Sk,
                    float scale, int causal, int k_offset, cudaStream_t st, int64_t kv_stride_rows = -1) {
    using C = attn_tc::QTmemCfg<DQK, DV, BN>;
    auto kern = attn_tc::attn_fwd_tc_qtmem_kernel<DQK, DV, BN, DTYPE>;
    if (!allow_dynamic_smem(reinterpret_cast<const void*>(kern), C::SMEM_BYTES)) return ATTN_ERR_CUDA;
    const int64_t BH = static_cast<int64_t>(B) * H;
    const int64_t n_qtiles = (static_cast<int64_t>(Sq) + C::BM - 1) / C::BM;
    if (n_qtiles * BH > 2147483647LL) return ATTN_ERR_BAD_SHAPE;
    CUtensorMap mk, mv, mo;
    if (!make_map(&mk, k, DTYPE, static_cast<int64_t>(B) * Hkv, Sk, DQK, C::BN, kv_stride_rows) ||
        !make_map(&mv, v, DTYPE, static_cast<int64_t>(B) * Hkv, Sk, DV, C::BN, kv_stride_rows) || !make_map(&mo, o, DTYPE, BH, Sq, DV, C::BM))
        return ATTN_ERR_CUDA;
    attn_tc::QTmemParams prm;
    prm.q = q;
    prm.o_plain = o;
    prm.lse = lse;
    prm.Sq = Sq;
    prm.Sk = Sk;
    prm.scale = scale;
    prm.scale_log2 = scale * 1.4426950408889634f;
    prm.causal = causal ? 1 : 0;
    prm.status = device_status_ptr();
    if (!prm.status) return ATTN_ERR_CUDA;
    prm.n_qtiles = static_cast<int>(n_qtiles);
    prm.BH = static_cast<int>(BH);
    prm.H = H;
    prm.Hkv = Hkv;
    prm.k_offset = k_offset;
    const int64_t kv_bytes_per_head = 2LL * Sk * (DQK + DV);
    int64_t hpg = (static_cast<int64_t>(ATTN_L2_MB) << 20) / (kv_bytes_per_head > 0 ? kv_bytes_per_head : 1);
    if (hpg < 1) hpg = 1;
    hpg *= H / Hkv;
    if (hpg > BH) hpg = BH;
    prm.heads_per_group = static_cast<int>(hpg);
    {   // merged tail only under the causal mask (see launch_tc_pipe)
        const int64_t n_groups = (BH + hpg - 1) / hpg;
        const int merge = causal ? ATTN_MERGE_LAST : 1;
        prm.last_group = static_cast<int>(n_groups >= merge ? n_groups - merge : 0);
    }
    prm.n_items = static_cast<int>(n_qtiles * BH);
    DeviceInfo di;
    int dev = 0;
    if (device_info(&di, &dev) != ATTN_OK) return ATTN_ERR_CUDA;
    const unsigned grid = static_cast<unsigned>(prm.n_items < di.sm_count ? prm.n_items : di.sm_count);
    prm.counter = nullptr;   // small problems: every CTA takes exactly one item, no counter
    if (prm.n_items > di.sm_count) {
        const int rc = work_counter(di, dev, st, &prm.counter);
        if (rc != ATTN_OK) return rc;
    }
    kern<<<grid, C::THREADS, C::SMEM_BYTES, st>>>(mk, mv, mo, prm);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

template <int D, int DTYPE>
int launch_simt(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv, int Sq, int Sk,
                float scale, int causal, int k_offset, cudaStream_t st, float o_scale = 1.f) {
    const int64_t BH = static_cast<int64_t>(B) * H;
    if (BH > 65535) return ATTN_ERR_BAD_SHAPE;
    dim3 grid(static_cast<unsigned>((static_cast<int64_t>(Sq) + attn_simt::kWarpsPerBlock - 1) / attn_simt::kWarpsPerBlock),
              static_cast<unsigned>(BH));
    attn_simt::attn_fwd_simt_kernel<D, DTYPE><<<grid, attn_simt::kWarpsPerBlock * 32, 0, st>>>(q, k, v, o, lse, Sq, Sk,
                                                                                              scale, causal ? 1 : 0, H, Hkv, k_offset, o_scale);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

enum class Impl { TensorCore, Simt };

template <Impl IMPL>
int dispatch(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv, int Sq, int Sk, int D,
             float scale, int causal, int k_offset, int dtype, void* stream, int64_t kv_stride_rows = -1) {
    int rc = validate(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, scale, dtype, true);
    if (rc != ATTN_OK) return rc;
    if (k_offset < 0 || static_cast<int64_t>(k_offset) + Sk > 2147483647LL) return ATTN_ERR_BAD_SHAPE;
    if (static_cast<int64_t>(B) * H * Sq == 0) return ATTN_OK;
    rc = check_arch();
    if (rc != ATTN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (Sk == 0)
        return fill_empty(o, lse, static_cast<int64_t>(B) * H * Sq * D, static_cast<int64_t>(B) * H * Sq, st);
    // Grouped K/V heads without a mask and with few query rows per head (decoding, short chunks): the H / Hkv
    // query heads of one K/V head lie next to each other in Q, O and LSE, so they ARE one head of (H / Hkv) * Sq
    // rows over the same keys.  Taken that way they share Q tiles (one tile of 128 rows instead of H / Hkv
    // tiles with Sq valid rows each) and K/V is streamed once for the group.
    if (IMPL == Impl::TensorCore && !causal && Hkv < H && Sq < 256 &&
        static_cast<int64_t>(H / Hkv) * Sq <= 2147483647LL - 256) {
        Sq *= H / Hkv;
        H = Hkv;
    }
#define ATTN_CASE(DD, TT)                                                                              \
    if (D == DD && dtype == TT) {                                                                      \
        if (IMPL == Impl::Simt) return launch_simt<DD, TT>(q, k, v, o, lse, B, H, Hkv, Sq, Sk, scale, causal, k_offset, st); \
        if (DD == 256) return launch_tc_qtmem<256, 256, 64, TT>(q, k, v, o, lse, B, H, Hkv, Sq, Sk, scale, causal, k_offset, st, kv_stride_rows); \
        return launch_tc_pipe<(DD == 256 ? 128 : DD), TT>(q, k, v, o, lse, B, H, Hkv, Sq, Sk, scale, causal, k_offset, st, 1.f, kv_stride_rows); \
    }
    ATTN_CASE(64, 0)
    ATTN_CASE(64, 1)
    ATTN_CASE(128, 0)
    ATTN_CASE(128, 1)
    ATTN_CASE(256, 0)
    ATTN_CASE(256, 1)
#undef ATTN_CASE
    return ATTN_ERR_UNSUPPORTED_HEAD_DIM;
}

size_t align256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

// Built-in staging buffer of attn_fwd_host_static.  In host code this name is only a stand-in
// for the symbol: the device address is looked up once per device (below) and that pointer, not
// the name, is what the copies and the kernel are given.
static __device__ __align__(256) unsigned char g_static_workspace[ATTN_STATIC_WORKSPACE_BYTES];

std::mutex g_static_mutex;
void* g_static_workspace_addr[kMaxDevices] = {};

// Device address of the built-in buffer on the current device; resolved on first use per device.
int static_workspace_ptr(void** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ATTN_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return ATTN_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_workspace_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess || !p) return ATTN_ERR_CUDA;
        g_static_workspace_addr[dev] = p;
    }
    *out = g_static_workspace_addr[dev];
    return ATTN_OK;
}

}  // namespace

namespace {

// ---- attn_fwd_host for large problems: groups of heads pipelined over two internal copy streams ----
//
// The caller's stream runs the kernels; one internal stream carries the host-to-device copies, one the
// device-to-host copies, so that the copies of neighbouring groups overlap the kernels and each other
// (PCIe is full duplex).  Streams and events are created once per device, on first use.
constexpr int kHostPipeMaxChunks = 8;
struct HostPipe {
    bool ready = false;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_done = nullptr, ev_in[kHostPipeMaxChunks] = {}, ev_k[kHostPipeMaxChunks] = {};
    std::mutex mu;   // one enqueue sequence at a time: the events are shared by every call on the device
};
HostPipe g_host_pipe[64];

// ---- attn_fwd_splitkv: the K/V shards of one problem as concurrent launches on internal streams ----
constexpr int kSplitStreams = 16;
struct SplitPipe {
    bool ready = false;
    cudaStream_t s[kSplitStreams] = {};
    cudaEvent_t ev_start = nullptr, ev_done[kSplitStreams] = {};
    std::mutex mu;
};
SplitPipe g_split_pipe[64];

// at least 16 MiB to copy in (more than the built-in buffer of attn_fwd_host_static can hold, so that entry point
// never takes this path and keeps its promise to create nothing) and at least 4 heads to split
bool host_pipe_wanted(size_t bh, size_t h2d_bytes) { return bh >= 4 && h2d_bytes >= (static_cast<size_t>(16) << 20); }

int host_pipelined(const void* q_host, const void* k_host, const void* v_host, void* o_host, float* lse_host, int BH, int Sq,
                   int Sk, int D, float scale, int causal, int dtype, uint8_t* dq, uint8_t* dk, uint8_t* dv, uint8_t* d_o,
                   float* dl, cudaStream_t st) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ATTN_ERR_CUDA;
    HostPipe& hp = g_host_pipe[dev];
    std::lock_guard<std::mutex> lock(hp.mu);
    if (!hp.ready) {
        bool ok = cudaStreamCreateWithFlags(&hp.s_in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&hp.s_out, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp.ev_start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp.ev_done, cudaEventDisableTiming) == cudaSuccess;
        for (int c = 0; ok && c < kHostPipeMaxChunks; ++c)
            ok = cudaEventCreateWithFlags(&hp.ev_in[c], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&hp.ev_k[c], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return ATTN_ERR_CUDA;
        hp.ready = true;
    }
    const int n_chunks = BH < kHostPipeMaxChunks ? BH : kHostPipeMaxChunks;
    const size_t q_head = static_cast<size_t>(Sq) * D * 2, kv_head = static_cast<size_t>(Sk) * D * 2, l_head = static_cast<size_t>(Sq) * 4;
    // everything below is ordered after the work already on the caller's stream
    if (cudaEventRecord(hp.ev_start, st) != cudaSuccess) return ATTN_ERR_CUDA;
    if (cudaStreamWaitEvent(hp.s_in, hp.ev_start, 0) != cudaSuccess) return ATTN_ERR_CUDA;
    if (cudaStreamWaitEvent(hp.s_out, hp.ev_start, 0) != cudaSuccess) return ATTN_ERR_CUDA;
    for (int c = 0; c < n_chunks; ++c) {
        const int h0 = static_cast<int>(static_cast<int64_t>(BH) * c / n_chunks);
        const int h1 = static_cast<int>(static_cast<int64_t>(BH) * (c + 1) / n_chunks);
        const size_t nh = static_cast<size_t>(h1 - h0);
        const uint8_t* qh = static_cast<const uint8_t*>(q_host) + h0 * q_head;
        const uint8_t* kh = static_cast<const uint8_t*>(k_host) + h0 * kv_head;
        const uint8_t* vh = static_cast<const uint8_t*>(v_host) + h0 * kv_head;
        if (cudaMemcpyAsync(dq + h0 * q_head, qh, nh * q_head, cudaMemcpyHostToDevice, hp.s_in) != cudaSuccess) return ATTN_ERR_CUDA;
        if (kv_head) {
            if (cudaMemcpyAsync(dk + h0 * kv_head, kh, nh * kv_head, cudaMemcpyHostToDevice, hp.s_in) != cudaSuccess) return ATTN_ERR_CUDA;
            if (cudaMemcpyAsync(dv + h0 * kv_head, vh, nh * kv_head, cudaMemcpyHostToDevice, hp.s_in) != cudaSuccess) return ATTN_ERR_CUDA;
        }
        if (cudaEventRecord(hp.ev_in[c], hp.s_in) != cudaSuccess) return ATTN_ERR_CUDA;
        if (cudaStreamWaitEvent(st, hp.ev_in[c], 0) != cudaSuccess) return ATTN_ERR_CUDA;
        // the heads of a group as one batch element: (batch, head) only enters the kernels as one flat index
        int rc = attn_fwd(dq + h0 * q_head, dk + h0 * kv_head, dv + h0 * kv_head, d_o + h0 * q_head,
                          reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(dl) + h0 * l_head), 1, static_cast<int>(nh), Sq, Sk, D,
                          scale, causal, dtype, st);
        if (rc != ATTN_OK) return rc;
        if (cudaEventRecord(hp.ev_k[c], st) != cudaSuccess) return ATTN_ERR_CUDA;
        if (cudaStreamWaitEvent(hp.s_out, hp.ev_k[c], 0) != cudaSuccess) return ATTN_ERR_CUDA;
        if (cudaMemcpyAsync(static_cast<uint8_t*>(o_host) + h0 * q_head, d_o + h0 * q_head, nh * q_head, cudaMemcpyDeviceToHost,
                            hp.s_out) != cudaSuccess)
            return ATTN_ERR_CUDA;
        if (cudaMemcpyAsync(reinterpret_cast<uint8_t*>(lse_host) + h0 * l_head, reinterpret_cast<uint8_t*>(dl) + h0 * l_head,
                            nh * l_head, cudaMemcpyDeviceToHost, hp.s_out) != cudaSuccess)
            return ATTN_ERR_CUDA;
    }
    // the caller's stream continues only after the last copy back
    if (cudaEventRecord(hp.ev_done, hp.s_out) != cudaSuccess) return ATTN_ERR_CUDA;
    if (cudaStreamWaitEvent(st, hp.ev_done, 0) != cudaSuccess) return ATTN_ERR_CUDA;
    return ATTN_OK;
}

}  // namespace

extern "C" {

#ifdef ATTN_TEST_HOOKS
// Test build only (never part of libattn_fwd.so): the next launch of the pipelined kernel leaves out the load
// of this K/V ring group (group 0 of a work item is K_0, group i is V_{i-1} with K_i), so that the wait for it runs out
// and the kernel returns through its time-out path.
void attn_test_skip_kv_load(int ring_item) { g_test_skip_ring_item = ring_item; }
#endif

int attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Sq, int Sk, int D,
             float scale, int causal, int dtype, void* stream) {
    return dispatch<Impl::TensorCore>(q, k, v, o, lse, B, H, H, Sq, Sk, D, scale, causal, 0, dtype, stream);
}

int attn_fwd_gqa(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv, int Sq, int Sk,
                 int D, float scale, int causal, int dtype, void* stream) {
    return dispatch<Impl::TensorCore>(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, scale, causal, 0, dtype, stream);
}

int attn_fwd_partial(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv, int Sq,
                     int Sk, int D, float scale, int causal, int k_offset, int dtype, void* stream) {
    return dispatch<Impl::TensorCore>(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, scale, causal, k_offset, dtype, stream);
}

int attn_combine(const void* o_parts, const float* lse_parts, int n_parts, void* o, float* lse, int B, int H, int Sq,
                 int D, int dtype, void* stream) {
    if (B < 0 || H < 0 || Sq < 0 || n_parts < 1 || n_parts > 1024) return ATTN_ERR_BAD_SHAPE;
    if (D <= 0 || D % 8 != 0) return ATTN_ERR_UNSUPPORTED_HEAD_DIM;
    if (dtype != ATTN_DTYPE_FP16 && dtype != ATTN_DTYPE_BF16) return ATTN_ERR_UNSUPPORTED_DTYPE;
    const int64_t rows = static_cast<int64_t>(B) * H * Sq;
    if (rows == 0) return ATTN_OK;
    if (!o_parts || !lse_parts || !o || !lse) return ATTN_ERR_NULL_POINTER;
    if ((reinterpret_cast<uintptr_t>(o_parts) | reinterpret_cast<uintptr_t>(o)) & 15u) return ATTN_ERR_MISALIGNED;
    if ((reinterpret_cast<uintptr_t>(lse_parts) | reinterpret_cast<uintptr_t>(lse)) & 3u) return ATTN_ERR_MISALIGNED;
    int rc = check_arch();
    if (rc != ATTN_OK) return rc;
    const int segs = D / 8;
    const int64_t total = rows * segs;
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 64) blocks = 148 * 64;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
#define ATTN_COMBINE(TT, BB)                                                                                 \
    attn_merge::attn_combine_kernel<TT, BB><<<static_cast<unsigned>(blocks), 256, 0, st>>>(                    \
        static_cast<const uint4*>(o_parts), lse_parts, n_parts, static_cast<uint4*>(o), lse, rows, segs)
    // shards are read in batches of 4 (2 or 1 when there are fewer) so that a batch's loads overlap
    if (dtype == ATTN_DTYPE_FP16) {
        if (n_parts >= 3) ATTN_COMBINE(0, 4); else if (n_parts == 2) ATTN_COMBINE(0, 2); else ATTN_COMBINE(0, 1);
    } else {
        if (n_parts >= 3) ATTN_COMBINE(1, 4); else if (n_parts == 2) ATTN_COMBINE(1, 2); else ATTN_COMBINE(1, 1);
    }
#undef ATTN_COMBINE
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

int attn_combine_gather(const void* const* o_parts, const float* const* lse_parts, int n_parts, void* o, float* lse,
                        int B, int H, int Sq, int D, int dtype, long long row_begin, long long row_count, void* stream) {
    if (B < 0 || H < 0 || Sq < 0 || D <= 0 || n_parts < 1 || n_parts > attn_merge::kMaxGatherParts) return ATTN_ERR_BAD_SHAPE;
    if (D % 8 != 0) return ATTN_ERR_UNSUPPORTED_HEAD_DIM;
    if (dtype != ATTN_DTYPE_FP16 && dtype != ATTN_DTYPE_BF16) return ATTN_ERR_UNSUPPORTED_DTYPE;
    const int64_t rows = static_cast<int64_t>(B) * H * Sq;
    if (row_begin < 0 || row_count < 0 || row_begin + row_count > rows) return ATTN_ERR_BAD_SHAPE;
    if (row_count == 0) return ATTN_OK;
    if (!o_parts || !lse_parts || !o || !lse) return ATTN_ERR_NULL_POINTER;
    attn_merge::GatherTable tab;
    for (int r = 0; r < attn_merge::kMaxGatherParts; ++r) {
        const int src = r < n_parts ? r : n_parts - 1;
        if (!o_parts[src] || !lse_parts[src]) return ATTN_ERR_NULL_POINTER;
        if (reinterpret_cast<uintptr_t>(o_parts[src]) & 15u) return ATTN_ERR_MISALIGNED;
        if (reinterpret_cast<uintptr_t>(lse_parts[src]) & 3u) return ATTN_ERR_MISALIGNED;
        tab.o[r] = static_cast<const uint4*>(o_parts[src]);
        tab.lse[r] = lse_parts[src];
    }
    if ((reinterpret_cast<uintptr_t>(o) & 15u) || (reinterpret_cast<uintptr_t>(lse) & 3u)) return ATTN_ERR_MISALIGNED;
    int rc = check_arch();
    if (rc != ATTN_OK) return rc;
    const int segs = D / 8;
    const int64_t total = row_count * segs;
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 64) blocks = 148 * 64;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
#define ATTN_GATHER(TT, BB)                                                                                     \
    attn_merge::attn_combine_gather_kernel<TT, BB><<<static_cast<unsigned>(blocks), 256, 0, st>>>(                \
        tab, n_parts, static_cast<uint4*>(o), lse, static_cast<int64_t>(row_begin), static_cast<int64_t>(row_count), segs)
    if (dtype == ATTN_DTYPE_FP16) {
        if (n_parts >= 3) ATTN_GATHER(0, 4); else if (n_parts == 2) ATTN_GATHER(0, 2); else ATTN_GATHER(0, 1);
    } else {
        if (n_parts >= 3) ATTN_GATHER(1, 4); else if (n_parts == 2) ATTN_GATHER(1, 2); else ATTN_GATHER(1, 1);
    }
#undef ATTN_GATHER
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

size_t attn_fwd_splitkv_workspace_bytes(int B, int H, int Sq, int D, int n_splits) {
    if (B < 0 || H < 0 || Sq < 0 || D <= 0 || n_splits < 1) return 0;
    const size_t rows = static_cast<size_t>(B) * H * Sq;
    return align256(static_cast<size_t>(n_splits) * rows * D * 2) + align256(static_cast<size_t>(n_splits) * rows * 4);
}

int attn_fwd_splitkv(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv, int Sq, int Sk,
                     int D, float scale, int causal, int dtype, int n_splits, void* workspace, size_t workspace_bytes,
                     void* stream) {
    int rc = validate(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, scale, dtype, true);
    if (rc != ATTN_OK) return rc;
    if (n_splits < 1 || n_splits > 64) return ATTN_ERR_BAD_SHAPE;
    const size_t rows = static_cast<size_t>(B) * H * Sq;
    if (rows == 0) return ATTN_OK;
    // shards are whole 128-key tiles; no more shards than tiles
    const int tiles = (Sk + 127) / 128;
    if (n_splits > tiles) n_splits = tiles > 0 ? tiles : 1;
    if (n_splits == 1 || Sk == 0) return attn_fwd_gqa(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, scale, causal, dtype, stream);
    // partial results as attn_combine reads them: [n_splits, rows, D] 16-bit, then [n_splits, rows] fp32
    const size_t part_o = rows * D * 2, part_l = rows * 4;
    const size_t o_all = align256(static_cast<size_t>(n_splits) * part_o), l_all = align256(static_cast<size_t>(n_splits) * part_l);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < o_all + l_all)
        return ATTN_ERR_WORKSPACE;
    rc = check_arch();
    if (rc != ATTN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t* w_o = static_cast<uint8_t*>(workspace);
    uint8_t* w_l = w_o + o_all;
    if (D == 64 || D == 128) {
        // one launch: the key ranges are work items of the persistent kernel (no internal streams needed)
        const int split_tiles = (tiles + n_splits - 1) / n_splits;
        n_splits = (tiles + split_tiles - 1) / split_tiles;   // ranges that are not empty
        int Hq = H, Sqq = Sq;
        if (!causal && Hkv < H && Sq < 256) {                 // grouped query heads as rows of one head (see dispatch)
            Sqq = Sq * (H / Hkv);
            Hq = Hkv;
        }
        float* pl = reinterpret_cast<float*>(w_l);
#define ATTN_SPLIT_CASE(DD, TT)                                                                                          \
    if (D == DD && dtype == TT)                                                                                          \
        rc = launch_tc_pipe<DD, TT>(q, k, v, w_o, pl, B, Hq, Hkv, Sqq, Sk, scale, causal, 0, st, 1.f, -1, n_splits);
        ATTN_SPLIT_CASE(64, 0)
        ATTN_SPLIT_CASE(64, 1)
        ATTN_SPLIT_CASE(128, 0)
        ATTN_SPLIT_CASE(128, 1)
#undef ATTN_SPLIT_CASE
        if (rc != ATTN_OK) return rc;
        return attn_combine(w_o, pl, n_splits, o, lse, B, H, Sq, D, dtype, stream);
    }
    // head dim 256: one launch per key range, concurrent on the library's own streams
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ATTN_ERR_CUDA;
    SplitPipe& sp = g_split_pipe[dev];
    std::lock_guard<std::mutex> lock(sp.mu);
    if (!sp.ready) {
        bool ok = cudaEventCreateWithFlags(&sp.ev_start, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; ok && i < kSplitStreams; ++i)
            ok = cudaStreamCreateWithFlags(&sp.s[i], cudaStreamNonBlocking) == cudaSuccess &&
                 cudaEventCreateWithFlags(&sp.ev_done[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return ATTN_ERR_CUDA;
        sp.ready = true;
    }
    const int n_streams = n_splits < kSplitStreams ? n_splits : kSplitStreams;
    if (cudaEventRecord(sp.ev_start, st) != cudaSuccess) return ATTN_ERR_CUDA;
    for (int i = 0; i < n_streams; ++i)
        if (cudaStreamWaitEvent(sp.s[i], sp.ev_start, 0) != cudaSuccess) return ATTN_ERR_CUDA;
    for (int s = 0; s < n_splits; ++s) {
        const int t0 = static_cast<int>(static_cast<int64_t>(tiles) * s / n_splits);
        const int t1 = static_cast<int>(static_cast<int64_t>(tiles) * (s + 1) / n_splits);
        const int k0 = t0 * 128, k1 = (t1 * 128 < Sk) ? t1 * 128 : Sk;
        // the shard is addressed in place: rows k0 .. k1-1 of every (batch, K/V head), head stride Sk rows
        const uint8_t* ks = static_cast<const uint8_t*>(k) + static_cast<size_t>(k0) * D * 2;
        const uint8_t* vs = static_cast<const uint8_t*>(v) + static_cast<size_t>(k0) * D * 2;
        rc = dispatch<Impl::TensorCore>(q, ks, vs, w_o + s * part_o, reinterpret_cast<float*>(w_l + s * part_l), B, H, Hkv, Sq,
                                        k1 - k0, D, scale, causal, k0, dtype, sp.s[s % n_streams], Sk);
        if (rc != ATTN_OK) return rc;
    }
    for (int i = 0; i < n_streams; ++i) {
        if (cudaEventRecord(sp.ev_done[i], sp.s[i]) != cudaSuccess) return ATTN_ERR_CUDA;
        if (cudaStreamWaitEvent(st, sp.ev_done[i], 0) != cudaSuccess) return ATTN_ERR_CUDA;
    }
    return attn_combine(w_o, reinterpret_cast<const float*>(w_l), n_splits, o, lse, B, H, Sq, D, dtype, stream);
}

int attn_fwd_qkv_dims(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv, int Sq,
                      int Sk, int Dqk, int Dv, float scale, int causal, int dtype, void* stream) {
    if (Dqk == Dv) return attn_fwd_gqa(q, k, v, o, lse, B, H, Hkv, Sq, Sk, Dqk, scale, causal, dtype, stream);
    if (Dqk != 192 || Dv != 128) return ATTN_ERR_UNSUPPORTED_HEAD_DIM;
    // validate with a supported single head dim (the checks do not depend on its value)
    int rc = validate(q, k, v, o, lse, B, H, Hkv, Sq, Sk, 128, scale, dtype, true);
    if (rc != ATTN_OK) return rc;
    if (static_cast<int64_t>(B) * H * Sq == 0) return ATTN_OK;
    rc = check_arch();
    if (rc != ATTN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (Sk == 0)
        return fill_empty(o, lse, static_cast<int64_t>(B) * H * Sq * Dv, static_cast<int64_t>(B) * H * Sq, st);
    if (dtype == ATTN_DTYPE_FP16)
        return launch_tc_qtmem<192, 128, 128, 0>(q, k, v, o, lse, B, H, Hkv, Sq, Sk, scale, causal, 0, st);
    return launch_tc_qtmem<192, 128, 128, 1>(q, k, v, o, lse, B, H, Hkv, Sq, Sk, scale, causal, 0, st);
}

int attn_fwd_fp8(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv, int Sq, int Sk,
                 int D, float scale, float q_factor, float k_factor, float v_factor, int causal, int impl, void* stream) {
    if (D != 128) {
        if (B < 0 || H < 0 || Hkv < 0 || Sq < 0 || Sk < 0 || D < 0) return ATTN_ERR_BAD_SHAPE;
        return ATTN_ERR_UNSUPPORTED_HEAD_DIM;
    }
    // the shared checks, with a 16-bit type standing in (they do not depend on the element size)
    int rc = validate(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, scale, ATTN_DTYPE_BF16, true);
    if (rc != ATTN_OK) return rc;
    if (!isfinite(q_factor) || !isfinite(k_factor) || !isfinite(v_factor) || q_factor <= 0.f || k_factor <= 0.f ||
        v_factor <= 0.f)
        return ATTN_ERR_BAD_SCALE;
    const float s_eff = scale * q_factor * k_factor;   // the factors of Q and K act only through the scores
    if (!isfinite(s_eff)) return ATTN_ERR_BAD_SCALE;
    if (impl != 0 && impl != 1) return ATTN_ERR_UNSUPPORTED_DTYPE;
    if (static_cast<int64_t>(B) * H * Sq == 0) return ATTN_OK;
    rc = check_arch();
    if (rc != ATTN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (Sk == 0)
        return fill_empty(o, lse, static_cast<int64_t>(B) * H * Sq * D, static_cast<int64_t>(B) * H * Sq, st);
    if (impl == 1)
        return launch_simt<128, ATTN_DTYPE_FP8_E4M3>(q, k, v, o, lse, B, H, Hkv, Sq, Sk, s_eff, causal, 0, st, v_factor);
    return launch_tc_pipe<128, ATTN_DTYPE_FP8_E4M3>(q, k, v, o, lse, B, H, Hkv, Sq, Sk, s_eff, causal, 0, st, v_factor);
}

// attn_bwd's workspace: two fp32 row vectors [B*H][Sq_pad], Sq_pad = Sq rounded up to a multiple of 64
size_t bwd_sq_pad(int Sq) { return (static_cast<size_t>(Sq) + 63) / 64 * 64; }

size_t attn_bwd_workspace_bytes(int B, int H, int Sq) {
    if (B < 0 || H < 0 || Sq < 0) return 0;
    return 2 * align256(static_cast<size_t>(B) * H * bwd_sq_pad(Sq) * sizeof(float));
}

int attn_bwd(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* dout, void* dq,
             void* dk, void* dv, int B, int H, int Hkv, int Sq, int Sk, int D, float scale, int causal, int dtype,
             void* workspace, size_t workspace_bytes, void* stream) {
    if (D != 64 && D != 128) {
        if (B < 0 || H < 0 || Hkv < 0 || Sq < 0 || Sk < 0 || D < 0) return ATTN_ERR_BAD_SHAPE;
        return ATTN_ERR_UNSUPPORTED_HEAD_DIM;
    }
    // the shared checks on q, k, v (dq stands in for o, the caller's lse is checked as a float pointer)
    int rc = validate(q, k, v, dq, lse, B, H, Hkv, Sq, Sk, D, scale, dtype, true);
    if (rc != ATTN_OK) return rc;
    const size_t n_q = static_cast<size_t>(B) * H * Sq, n_kv = static_cast<size_t>(B) * Hkv * Sk;
    if (n_q > 0 && (!o || !dout)) return ATTN_ERR_NULL_POINTER;
    if (n_kv > 0 && (!dk || !dv)) return ATTN_ERR_NULL_POINTER;
    if ((reinterpret_cast<uintptr_t>(o) | reinterpret_cast<uintptr_t>(dout) | reinterpret_cast<uintptr_t>(dk) |
         reinterpret_cast<uintptr_t>(dv)) & 15u)
        return ATTN_ERR_MISALIGNED;
    if (n_q == 0 && n_kv == 0) return ATTN_OK;
    if (n_q > 0 && n_kv > 0 &&
        (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < attn_bwd_workspace_bytes(B, H, Sq)))
        return ATTN_ERR_WORKSPACE;
    rc = check_arch();
    if (rc != ATTN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // no queries: nothing reaches K and V; no keys: nothing reaches Q
    if (n_q == 0 || n_kv == 0) {
        if (n_kv > 0 && (cudaMemsetAsync(dk, 0, n_kv * D * 2, st) != cudaSuccess || cudaMemsetAsync(dv, 0, n_kv * D * 2, st) != cudaSuccess))
            return ATTN_ERR_CUDA;
        if (n_q > 0 && cudaMemsetAsync(dq, 0, n_q * D * 2, st) != cudaSuccess) return ATTN_ERR_CUDA;
        return ATTN_OK;
    }
    const int64_t BH = static_cast<int64_t>(B) * H, BHkv = static_cast<int64_t>(B) * Hkv;
    const int64_t n_qtiles = (static_cast<int64_t>(Sq) + 127) / 128, n_ktiles = (static_cast<int64_t>(Sk) + 127) / 128;
    if (n_qtiles * BH > 2147483647LL || n_ktiles * BHkv > 2147483647LL) return ATTN_ERR_BAD_SHAPE;
    const int64_t sq_pad = static_cast<int64_t>(bwd_sq_pad(Sq));
    float* nl2 = static_cast<float*>(workspace);
    float* ndelta = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + align256(static_cast<size_t>(BH) * sq_pad * sizeof(float)));
    attn_grad::BwdParams prm;
    prm.nl2 = nl2;
    prm.ndelta = ndelta;
    prm.Sq_pad = static_cast<int>(sq_pad);
    prm.Sq = Sq;
    prm.Sk = Sk;
    prm.scale = scale;
    prm.scale_log2 = scale * 1.4426950408889634f;
    prm.causal = causal ? 1 : 0;
    prm.H = H;
    prm.Hkv = Hkv;
    prm.n_qtiles = static_cast<int>(n_qtiles);
    prm.n_ktiles = static_cast<int>(n_ktiles);
    prm.status = device_status_ptr();
    if (!prm.status) return ATTN_ERR_CUDA;
    // resident tiles and outputs move in boxes of 128 rows, streamed tiles in boxes of 64 rows
    DeviceInfo di;
    int dev = 0;
    if (device_info(&di, &dev) != ATTN_OK) return ATTN_ERR_CUDA;
    const int sms = di.sm_count;   // persistent grids: one CTA per SM, later tiles from the stream's work counter
    unsigned int* counter = nullptr;
    if (n_qtiles * BH > sms || n_ktiles * BHkv > sms) {
        rc = work_counter(di, dev, st, &counter);
        if (rc != ATTN_OK) return rc;
    }
    CUtensorMap mq, mk, mv, mdo, mq64, mk64, mv64, mdo64, mdq, mdk, mdv;
    if (!make_map(&mq, q, dtype, BH, Sq, D, 128) || !make_map(&mdo, dout, dtype, BH, Sq, D, 128) ||
        !make_map(&mq64, q, dtype, BH, Sq, D, 64) || !make_map(&mdo64, dout, dtype, BH, Sq, D, 64) ||
        !make_map(&mdq, dq, dtype, BH, Sq, D, 128) || !make_map(&mk, k, dtype, BHkv, Sk, D, 128) ||
        !make_map(&mv, v, dtype, BHkv, Sk, D, 128) || !make_map(&mk64, k, dtype, BHkv, Sk, D, 64) ||
        !make_map(&mv64, v, dtype, BHkv, Sk, D, 64) || !make_map(&mdk, dk, dtype, BHkv, Sk, D, 128) ||
        !make_map(&mdv, dv, dtype, BHkv, Sk, D, 128))
        return ATTN_ERR_CUDA;
#define ATTN_BWD_CASE(DD, TT)                                                                                              \
    if (D == DD && dtype == TT) {                                                                                          \
        using CQ = attn_grad::BwdCfg<DD, 0>;                                                                                \
        using CKV = attn_grad::BwdCfg<DD, 1>;                                                                               \
        auto kq = attn_grad::attn_bwd_kernel<DD, TT, 0>;                                                                    \
        auto kkv = attn_grad::attn_bwd_kernel<DD, TT, 1>;                                                                   \
        if (!allow_dynamic_smem(reinterpret_cast<const void*>(kq), CQ::SMEM_BYTES) ||                                      \
            !allow_dynamic_smem(reinterpret_cast<const void*>(kkv), CKV::SMEM_BYTES))                                      \
            return ATTN_ERR_CUDA;                                                                                          \
        const int64_t rows = BH * sq_pad;                                                                                  \
        int64_t blocks = (rows + 7) / 8;                                                                                   \
        if (blocks > 148 * 16) blocks = 148 * 16;                                                                          \
        attn_grad::attn_bwd_rows_kernel<DD, TT><<<static_cast<unsigned>(blocks), 256, 0, st>>>(o, dout, lse, nl2, ndelta, Sq, \
                                                                                              prm.Sq_pad, rows);          \
        prm.out0 = dq;                                                                                                     \
        prm.out1 = nullptr;                                                                                                \
        prm.n_tiles_total = static_cast<int>(n_qtiles * BH);                                                               \
        prm.counter = prm.n_tiles_total > sms ? counter : nullptr;                                                         \
        kq<<<static_cast<unsigned>(prm.n_tiles_total < sms ? prm.n_tiles_total : sms), CQ::THREADS, CQ::SMEM_BYTES, st>>>(  \
            mq, mdo, mk64, mv64, mdq, mdq, prm);                                                                           \
        prm.out0 = dv;                                                                                                     \
        prm.out1 = dk;                                                                                                     \
        prm.n_tiles_total = static_cast<int>(n_ktiles * BHkv);                                                             \
        prm.counter = prm.n_tiles_total > sms ? counter : nullptr;                                                         \
        kkv<<<static_cast<unsigned>(prm.n_tiles_total < sms ? prm.n_tiles_total : sms), CKV::THREADS, CKV::SMEM_BYTES, st>>>( \
            mk, mv, mq64, mdo64, mdv, mdk, prm);                                                                           \
        return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;                                                \
    }
    ATTN_BWD_CASE(64, 0)
    ATTN_BWD_CASE(64, 1)
    ATTN_BWD_CASE(128, 0)
    ATTN_BWD_CASE(128, 1)
#undef ATTN_BWD_CASE
    return ATTN_ERR_UNSUPPORTED_DTYPE;
}

int attn_fwd_simt(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Sq, int Sk,
                  int D, float scale, int causal, int dtype, void* stream) {
    return dispatch<Impl::Simt>(q, k, v, o, lse, B, H, H, Sq, Sk, D, scale, causal, 0, dtype, stream);
}

size_t attn_fwd_host_workspace_bytes(int B, int H, int Sq, int Sk, int D) {
    if (B < 0 || H < 0 || Sq < 0 || Sk < 0 || D <= 0) return 0;
    const size_t bh = static_cast<size_t>(B) * H;
    const size_t qo = align256(bh * Sq * D * 2), kv = align256(bh * Sk * D * 2), ls = align256(bh * Sq * 4);
    return 2 * qo + 2 * kv + ls;
}

int attn_fwd_host(const void* q_host, const void* k_host, const void* v_host, void* o_host, float* lse_host, int B,
                  int H, int Sq, int Sk, int D, float scale, int causal, int dtype, void* workspace,
                  size_t workspace_bytes, void* stream) {
    int rc = validate(q_host, k_host, v_host, o_host, lse_host, B, H, H, Sq, Sk, D, scale, dtype, false);
    if (rc != ATTN_OK) return rc;
    const size_t bh = static_cast<size_t>(B) * H;
    if (bh * Sq == 0) return ATTN_OK;
    const size_t need = attn_fwd_host_workspace_bytes(B, H, Sq, Sk, D);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < need)
        return ATTN_ERR_WORKSPACE;
    const size_t qo_b = bh * Sq * D * 2, kv_b = bh * Sk * D * 2, ls_b = bh * Sq * 4;
    uint8_t* w = static_cast<uint8_t*>(workspace);
    uint8_t* dq = w;
    uint8_t* dk = dq + align256(qo_b);
    uint8_t* dv = dk + align256(kv_b);
    uint8_t* d_o = dv + align256(kv_b);
    float* dl = reinterpret_cast<float*>(d_o + align256(qo_b));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (host_pipe_wanted(bh, qo_b + 2 * kv_b))
        return host_pipelined(q_host, k_host, v_host, o_host, lse_host, static_cast<int>(bh), Sq, Sk, D, scale, causal, dtype,
                              dq, dk, dv, d_o, dl, st);
    if (cudaMemcpyAsync(dq, q_host, qo_b, cudaMemcpyHostToDevice, st) != cudaSuccess) return ATTN_ERR_CUDA;
    if (kv_b) {
        if (cudaMemcpyAsync(dk, k_host, kv_b, cudaMemcpyHostToDevice, st) != cudaSuccess) return ATTN_ERR_CUDA;
        if (cudaMemcpyAsync(dv, v_host, kv_b, cudaMemcpyHostToDevice, st) != cudaSuccess) return ATTN_ERR_CUDA;
    }
    rc = attn_fwd(dq, dk, dv, d_o, dl, B, H, Sq, Sk, D, scale, causal, dtype, stream);
    if (rc != ATTN_OK) return rc;
    if (cudaMemcpyAsync(o_host, d_o, qo_b, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ATTN_ERR_CUDA;
    if (cudaMemcpyAsync(lse_host, dl, ls_b, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ATTN_ERR_CUDA;
    return ATTN_OK;
}

size_t attn_fwd_host_static_capacity(void) { return ATTN_STATIC_WORKSPACE_BYTES; }

int attn_fwd_host_static(const void* q_host, const void* k_host, const void* v_host, void* o_host, float* lse_host,
                         int B, int H, int Sq, int Sk, int D, float scale, int causal, int dtype, void* stream) {
    int rc = validate(q_host, k_host, v_host, o_host, lse_host, B, H, H, Sq, Sk, D, scale, dtype, false);
    if (rc != ATTN_OK) return rc;
    if (static_cast<size_t>(B) * H * Sq == 0) return ATTN_OK;
    const size_t need = attn_fwd_host_workspace_bytes(B, H, Sq, Sk, D);
    if (need > ATTN_STATIC_WORKSPACE_BYTES) return ATTN_ERR_STATIC_CAPACITY;
    rc = check_arch();
    if (rc != ATTN_OK) return rc;
    void* ws = nullptr;
    rc = static_workspace_ptr(&ws);
    if (rc != ATTN_OK) return rc;
    return attn_fwd_host(q_host, k_host, v_host, o_host, lse_host, B, H, Sq, Sk, D, scale, causal, dtype, ws,
                         ATTN_STATIC_WORKSPACE_BYTES, stream);
}

int attn_query_support(int D, int dtype, int causal) {
    (void)causal;
    if (D != 64 && D != 128 && D != 256) return ATTN_ERR_UNSUPPORTED_HEAD_DIM;
    if (dtype != ATTN_DTYPE_FP16 && dtype != ATTN_DTYPE_BF16) return ATTN_ERR_UNSUPPORTED_DTYPE;
    return check_arch();
}

int attn_last_device_status(void* stream) {
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return ATTN_ERR_CUDA;
    int h = 0;
    if (cudaMemcpyFromSymbol(&h, g_device_status, sizeof(int)) != cudaSuccess) return ATTN_ERR_CUDA;
    if (h != 0) {
        int zero = 0;
        if (cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int)) != cudaSuccess) return ATTN_ERR_CUDA;
    }
    return h == 0 ? ATTN_OK : ATTN_ERR_DEVICE_TIMEOUT;
}

const char* attn_status_string(int status) {
    switch (status) {
        case ATTN_OK: return "ATTN_OK";
        case ATTN_ERR_NULL_POINTER: return "ATTN_ERR_NULL_POINTER";
        case ATTN_ERR_BAD_SHAPE: return "ATTN_ERR_BAD_SHAPE";
        case ATTN_ERR_UNSUPPORTED_HEAD_DIM: return "ATTN_ERR_UNSUPPORTED_HEAD_DIM";
        case ATTN_ERR_UNSUPPORTED_DTYPE: return "ATTN_ERR_UNSUPPORTED_DTYPE";
        case ATTN_ERR_MISALIGNED: return "ATTN_ERR_MISALIGNED";
        case ATTN_ERR_BAD_SCALE: return "ATTN_ERR_BAD_SCALE";
        case ATTN_ERR_UNSUPPORTED_ARCH: return "ATTN_ERR_UNSUPPORTED_ARCH";
        case ATTN_ERR_CUDA: return "ATTN_ERR_CUDA";
        case ATTN_ERR_DEVICE_TIMEOUT: return "ATTN_ERR_DEVICE_TIMEOUT";
        case ATTN_ERR_WORKSPACE: return "ATTN_ERR_WORKSPACE";
        case ATTN_ERR_STATIC_CAPACITY: return "ATTN_ERR_STATIC_CAPACITY";
        case ATTN_ERR_COUNTER_SLOTS: return "ATTN_ERR_COUNTER_SLOTS";
        default: return "ATTN_ERR_UNKNOWN";
    }
}

}  // extern "C"
