// Warp-specialised, persistent tcgen05 attention forward kernel with Q in tensor memory and a
// double-buffered S: head dim 256, and heads whose Q/K dim differs from their V dim (192/128).
//
// With D = 256 the O accumulator of one 128-row Q tile already takes 256 of the 512 tensor-memory
// columns, so the two-Q-tile scheme of the D <= 128 kernel does not fit.  Here a work item is ONE
// Q tile of one (batch, head), and the tensor core overlaps with the softmax through two S buffers:
//
//   tensor memory:  O [0, DV)   Q [DV, DV + DQK/2)   S buffer 0 and 1: the last 2 * BN columns
//   steps of BN keys:  S_{g+1} = Q K_{g+1}^T is computed while the softmax works on S_g,
//   then O += P_g V_g; P_g (16-bit) overwrites the first half of its S buffer.
//
// Q is the A operand of the first product FROM TENSOR MEMORY (written there by the softmax
// threads, straight from global memory), so that product reads only the K tile from shared memory:
// with both operands in shared memory an N = 64 instruction would be bound by shared-memory
// bandwidth.
//
//   warps 0-3  softmax group (one thread per row): Q -> tensor memory, S -> P, rare O rescale, epilogue
//   warp  4    MMA issuer
//   warp  5    scheduler + TMA producer: BN-key K and V tiles through a ring of shared-memory slots
//
// Persistence: one CTA per SM; items are ordered longest-first (causal) inside L2-sized groups of
// heads; a CTA's first item is its block index, later ones come from a device counter.  Barriers,
// tensor memory and the ring live across items: the producer runs ahead into the next item, the
// softmax group writes the next item's Q into tensor memory while the last second product of the
// current item still runs, and the MMA warp issues the next item's first S during the epilogue.
//
// Loop structure as in Appendix C, Listings 1-2 of the paper; online softmax with a lazily advanced
// reference maximum as in the D <= 128 kernel.  The (192, 128) instance is the head shape of the
// MLA variant of Section 4.1 (128-dim embedding plus 64-dim RoPE part for Q/K, 128-dim V).
#pragma once
#include "attn_tc_common.cuh"

namespace attn_tc {

template <int DQK, int DV, int BN_>
struct QTmemCfg {
    static constexpr int BM = 128;
    static constexpr int BN = BN_;                              // keys per step
    static constexpr int K_BYTES = BN * DQK * 2;                // one K tile
    static constexpr int V_BYTES = BN * DV * 2;                 // one V tile
    static constexpr int SLOT_BYTES = K_BYTES > V_BYTES ? K_BYTES : V_BYTES;
    static constexpr int OST_BYTES = 2 * BM * 128;              // epilogue staging: two tiles of 128 rows x 64 columns
    static constexpr int NSLOT = (192 * 1024) / SLOT_BYTES > 6 ? 6 : (192 * 1024) / SLOT_BYTES;
    static constexpr int TILE_BYTES = NSLOT * SLOT_BYTES + OST_BYTES;
    static constexpr int MISC_BYTES = 512;
    static constexpr int SMEM_BYTES = 1024 + TILE_BYTES + MISC_BYTES;
    static constexpr int THREADS = 192;
    static constexpr int O_COL = 0, Q_COL = DV, S_COL = 512 - 2 * BN;   // S buffer b at S_COL + BN * b
    static constexpr int TMEM_COLS = 512;
    static_assert(DV + DQK / 2 <= S_COL, "tensor memory budget");
    static_assert(DQK % 64 == 0 && DV % 64 == 0 && (BN == 64 || BN == 128), "tile shapes");
    static_assert(NSLOT >= 4, "K/V ring too shallow");
};

struct QTmemParams {
    const void* q;
    void* o_plain;          // O as a plain pointer (rows without a visible key are zeroed with ordinary stores)
    float* lse;
    int Sq, Sk;
    float scale, scale_log2;
    int causal;
    int* status;
    int n_qtiles;           // 128-row Q tiles per head
    int BH;
    int heads_per_group;
    int last_group;         // index of the final group, which takes all remaining heads
    int H, Hkv;
    int k_offset;           // global index of key 0 of this K/V shard; enters the causal mask
    int n_items;            // n_qtiles * BH
    unsigned int* counter;  // work counter {next item, CTAs done}, zero at launch and again at exit; NULL when n_items <= grid
};

// One work item, decoded identically by every role.
struct QTmemItem {
    int bh, kv_bh, q0;
    int n;   // K/V steps (0: no row of the tile sees a key of this shard)
};

__device__ __forceinline__ QTmemItem qtmem_decode_item(const QTmemParams& prm, int lin, int BM, int BN) {
    QTmemItem it;
    const int full_group = prm.heads_per_group * prm.n_qtiles;
    int g = lin / full_group;
    if (g > prm.last_group) g = prm.last_group;
    const int r = lin - g * full_group;
    const int hg = (g == prm.last_group) ? prm.BH - g * prm.heads_per_group : prm.heads_per_group;
    const int pr = r / hg;
    it.bh = g * prm.heads_per_group + (r - pr * hg);
    const int qt = prm.causal ? prm.n_qtiles - 1 - pr : pr;   // causal: longest rows first
    it.q0 = qt * BM;
    it.kv_bh = (it.bh / prm.H) * prm.Hkv + (it.bh % prm.H) / (prm.H / prm.Hkv);
    const int last_key = last_visible_key(it.q0 + BM - 1, prm.Sk, prm.causal, prm.k_offset);
    it.n = last_key < 0 ? 0 : last_key / BN + 1;
    return it;
}

template <int DQK, int DV, int BN_, int DTYPE>
__global__ void __launch_bounds__(192, 1)
attn_fwd_tc_qtmem_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                         const __grid_constant__ CUtensorMap tmO, const QTmemParams prm) {
    using C = QTmemCfg<DQK, DV, BN_>;
    constexpr int BM = C::BM, BN = C::BN, NSLOT = C::NSLOT;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    auto sKV = [&](int slot) { return smem_base + slot * C::SLOT_BYTES; };
    const uint32_t sOst = smem_base + NSLOT * C::SLOT_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + C::TILE_BYTES);
    const uint32_t bars_u32 = smem_base + C::TILE_BYTES;
    enum {
        B_QREADY = 0,      // Q of the next item is in tensor memory (128 softmax threads)
        B_SFULL = 1,       // [2] S buffer b ready (MMA commit)
        B_PFULL = 3,       // [2] P written into S buffer b (128 softmax threads)
        B_ODONE = 5,       // completes once per step: O += P_g V_g has finished
        B_OFINAL = 6,      // completes once per item: its last second product has finished
        B_OFREE = 7,       // the epilogue has read O out of tensor memory (128 softmax threads)
        B_SCHEDFULL = 8,   // [2] scheduler slot holds the next item, decoded
        B_SCHEDEMPTY = 10, // [2] slot read by the MMA warp and the 4 softmax warps
        B_KVFULL = 12,
        B_KVEMPTY = 12 + NSLOT,
        B_COUNT = 12 + 2 * NSLOT
    };
    auto bar = [&](int i) { return bars_u32 + i * 8; };
    // scheduler slots [2][8]: item index (-1: no more work), bh, kv_bh, q0, n
    volatile int* sched_item = reinterpret_cast<volatile int*>(bars + B_COUNT);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT) + 16;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + B_COUNT) + 17;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar(B_QREADY), 128);
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar(B_SFULL + b), 1);
            mbar_init(bar(B_PFULL + b), 128);
            mbar_init(bar(B_SCHEDFULL + b), 1);
            mbar_init(bar(B_SCHEDEMPTY + b), 5);
        }
        mbar_init(bar(B_ODONE), 1);
        mbar_init(bar(B_OFINAL), 1);
        mbar_init(bar(B_OFREE), 128);
        for (int s = 0; s < NSLOT; ++s) {
            mbar_init(bar(B_KVFULL + s), 1);
            mbar_init(bar(B_KVEMPTY + s), 1);
        }
        fence_barrier_init();
        fence_proxy_async_smem();
    }
    if (warp == 4) {
        tmem_alloc(smem_u32(tmem_slot), C::TMEM_COLS);
        tmem_relinquish();
    }
    if (warp == 5 && elect_one()) {
        prefetch_tensormap(&tmK);
        prefetch_tensormap(&tmV);
        prefetch_tensormap(&tmO);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    // Consumers of the scheduler: wait for the k-th item of this CTA, read it, hand the slot back.
    // (the producer has decoded the item: the index arithmetic is done once per item, not once per thread)
    auto next_item = [&](int k, bool hand_back, QTmemItem& it) -> int {
        const int slot = k & 1;
        if (!mbar_wait(bar(B_SCHEDFULL + slot), (k >> 1) & 1, abort_flag)) return -1;
        volatile int* e = sched_item + slot * 8;
        const int item = e[0];
        it.bh = e[1];
        it.kv_bh = e[2];
        it.q0 = e[3];
        it.n = e[4];
        if (hand_back) mbar_arrive(bar(B_SCHEDEMPTY + slot));
        return item;
    };
    // Ring order inside one work item = consumption order of the MMA warp: K_0, then for every step j:
    // K_{j+1}, V_j.  Index of K_j: j == 0 ? 0 : 2j - 1; of V_j: 2j + 2 (2j + 1 for the last step).
    auto k_item = [](int j) { return j == 0 ? 0 : 2 * j - 1; };
    auto v_item = [](int j, int n) { return (j + 1 < n) ? 2 * j + 2 : 2 * j + 1; };

    if (warp == 5) {
        // =========================== scheduler + TMA producer ===========================
        const bool leader = elect_one();
        int kv_base = 0;   // ring items issued for earlier work items
        for (int k = 0;; ++k) {
            const int slot = k & 1;
            if (!mbar_wait(bar(B_SCHEDEMPTY + slot), ((k >> 1) & 1) ^ 1, abort_flag)) break;
            if (leader) {
                // no counter: the grid covers every item with the CTAs' first draws
                int next = (k == 0) ? static_cast<int>(blockIdx.x)
                           : (prm.counter ? static_cast<int>(gridDim.x + atomicAdd(prm.counter, 1u)) : prm.n_items);
                if (next < 0 || next >= prm.n_items) next = -1;
                volatile int* e = sched_item + slot * 8;
                if (next >= 0) {
                    const QTmemItem d = qtmem_decode_item(prm, next, BM, BN);
                    e[1] = d.bh;
                    e[2] = d.kv_bh;
                    e[3] = d.q0;
                    e[4] = d.n;
                    // its Q tile (rows q0 .. of one head: one contiguous block) on its way into L2 now, so that the
                    // softmax threads' loads of it, a few steps from now, do not pay the latency of HBM
                    if (k > 0 && d.n > 0) {
                        const int nrows = prm.Sq - d.q0 < BM ? prm.Sq - d.q0 : BM;
                        bulk_prefetch_l2(static_cast<const uint8_t*>(prm.q) + (static_cast<int64_t>(d.bh) * prm.Sq + d.q0) * DQK * 2,
                                         static_cast<uint32_t>(nrows) * DQK * 2);
                    }
                }
                e[0] = next;
                mbar_arrive(bar(B_SCHEDFULL + slot));
            }
            QTmemItem it;
            const int item = next_item(k, false, it);
            if (item < 0) break;
            auto load_kv = [&](const CUtensorMap* map, int nbox, int ring_item, int j) -> bool {
                const int s = ring_item % NSLOT;
                const uint32_t use = ring_item / NSLOT;
                if (!mbar_wait(bar(B_KVEMPTY + s), (use & 1) ^ 1, abort_flag)) return false;
                if (leader) {
                    mbar_arrive_expect_tx(bar(B_KVFULL + s), nbox * BN * 128);
                    for (int bx = 0; bx < nbox; ++bx)
                        tma_load_3d(sKV(s) + bx * BN * 128, map, bar(B_KVFULL + s), bx * 64, j * BN, it.kv_bh);
                }
                return true;
            };
            bool ok = it.n == 0 || load_kv(&tmK, DQK / 64, kv_base, 0);
            for (int j = 0; j < it.n && ok; ++j) {
                if (j + 1 < it.n) ok = load_kv(&tmK, DQK / 64, kv_base + k_item(j + 1), j + 1);
                if (ok) ok = load_kv(&tmV, DV / 64, kv_base + v_item(j, it.n), j);
            }
            if (!ok) break;
            kv_base += 2 * it.n;
        }
    } else if (warp == 4) {
        // =========================== MMA issuer ===========================
        const bool leader = elect_one();
        constexpr uint32_t IDESC_S = make_idesc_f16(BM, BN, DTYPE, 0, 0);   // Q (TMEM) and K both K-major
        constexpr uint32_t IDESC_O = make_idesc_f16(BM, DV, DTYPE, 0, 1);   // P (TMEM) K-major, V MN-major
        constexpr uint32_t DESC_HI = smem_desc_hi_sw128(1024);
        const uint32_t k_lo0 = smem_desc_lo(sKV(0), 16);
        const uint32_t v_lo0 = smem_desc_lo(sKV(0), BN * 128);   // distance between the 64-column boxes
        auto kv_full_wait = [&](int ring_item) {
            return mbar_wait(bar(B_KVFULL + ring_item % NSLOT), (ring_item / NSLOT) & 1, abort_flag);
        };
        int kv_base = 0;
        int g_base = 0;   // steps of earlier work items: step j of this item is global step g_base + j
        int uses = 0;     // work items with at least one step so far
        bool ok = true;
        for (int k = 0; ok; ++k) {
            QTmemItem it;
            const int item = next_item(k, leader, it);
            if (item < 0) break;
            if (it.n == 0) continue;
            auto issue_s = [&](int j) {   // S = Q K_j^T into buffer (g_base + j) & 1 : DQK/16 instructions of K = 16
                if (leader) {
                    const int g = g_base + j, ring = kv_base + k_item(j);
                    const uint32_t b0 = k_lo0 + (ring % NSLOT) * (C::SLOT_BYTES >> 4);
#pragma unroll
                    for (int kk = 0; kk < DQK / 16; ++kk) {
                        const uint32_t off = ((kk >> 2) * BN * 128 + (kk & 3) * 32) >> 4;
                        mma_f16_ts_lohi(tmem + C::S_COL + (g & 1) * BN, tmem + C::Q_COL + kk * 8, b0 + off, DESC_HI,
                                        IDESC_S, kk > 0);
                    }
                    mma_commit(bar(B_SFULL + (g & 1)));
                    mma_commit(bar(B_KVEMPTY + ring % NSLOT));
                }
            };
            ok = mbar_wait(bar(B_QREADY), uses & 1, abort_flag) && kv_full_wait(kv_base);
            if (ok) {
                tc_fence_after_sync();
                issue_s(0);
            }
            for (int j = 0; j < it.n && ok; ++j) {
                const int g = g_base + j;
                if (j + 1 < it.n) {
                    if (!(ok = kv_full_wait(kv_base + k_item(j + 1)))) break;
                    tc_fence_after_sync();
                    issue_s(j + 1);
                }
                const int vring = kv_base + v_item(j, it.n);
                if (!(ok = kv_full_wait(vring))) break;
                if (!(ok = mbar_wait(bar(B_PFULL + (g & 1)), (g >> 1) & 1, abort_flag))) break;
                // the epilogue of the previous item must have read O before it is overwritten
                if (j == 0 && uses > 0 && !(ok = mbar_wait(bar(B_OFREE), (uses - 1) & 1, abort_flag))) break;
                tc_fence_after_sync();
                if (leader) {
                    const uint32_t b0 = v_lo0 + (vring % NSLOT) * (C::SLOT_BYTES >> 4);
#pragma unroll
                    for (int kk = 0; kk < BN / 16; ++kk)
                        mma_f16_ts_lohi(tmem + C::O_COL, tmem + C::S_COL + (g & 1) * BN + kk * 8, b0 + ((kk * 16 * 128) >> 4),
                                        DESC_HI, IDESC_O, (j > 0 || kk > 0) ? 1u : 0u);
                    mma_commit(bar(B_KVEMPTY + vring % NSLOT));
                    mma_commit(bar(B_ODONE));
                    if (j + 1 == it.n) mma_commit(bar(B_OFINAL));
                }
            }
            kv_base += 2 * it.n;
            g_base += it.n;
            ++uses;
        }
    } else {
        // =========================== softmax group ===========================
        const int r = tid;                       // row inside the tile
        const uint32_t lane_off = static_cast<uint32_t>(warp * 32) << 16;
        const uint32_t tO = tmem + C::O_COL + lane_off, tQ = tmem + C::Q_COL + lane_off;
        const float c = prm.scale_log2;

        // Q row of an item -> tensor memory (two 16-bit values per column, in memory order)
        auto load_q = [&](const QTmemItem& it) {
            // Coalesced: a warp reads its 32 rows 128 columns at a time, every instruction covering whole rows
            // (consecutive lanes take consecutive 16-byte chunks), parks them in its own 8 KB of the epilogue's
            // staging tiles, and each thread then picks up its row from there (swizzled by row: no bank
            // conflicts either way).  One row per thread straight from global memory would touch 32 lines per
            // instruction.  The staging tiles are free once the previous epilogue's stores have read them.
            if (r == 0) tma_store_wait_read<0>();
            asm volatile("bar.sync 1, 128;" ::: "memory");
            const uint32_t mine = sOst + warp * 8192;
            const int rows_left = prm.Sq - (it.q0 + warp * 32);   // rows of this warp that exist
            const uint8_t* qbase = static_cast<const uint8_t*>(prm.q) +
                                   (static_cast<int64_t>(it.bh) * prm.Sq + it.q0 + warp * 32) * DQK * 2;
#pragma unroll
            for (int c0 = 0; c0 < DQK / 8; c0 += 16) {   // 16-byte chunks of a row, at most 16 per round
                constexpr int TOTAL = DQK / 8;
                const int CH = TOTAL - c0 < 16 ? TOTAL - c0 : 16;   // 16 or 8 (compile-time after unrolling)
                const int RPI = 32 / CH;                            // rows per load instruction
                uint4 x[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    if (i < CH) {
                        const int row_l = i * RPI + lane / CH, ch = lane % CH;
                        x[i] = (row_l < rows_left)
                                   ? __ldg(reinterpret_cast<const uint4*>(qbase + static_cast<int64_t>(row_l) * DQK * 2 + (c0 + ch) * 16))
                                   : make_uint4(0u, 0u, 0u, 0u);
                    }
                }
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    if (i < CH) {
                        const int row_l = i * RPI + lane / CH, ch = lane % CH;
                        const uint32_t dst = mine + row_l * 256 + ((ch ^ (row_l & (CH - 1))) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(x[i].x), "r"(x[i].y), "r"(x[i].z), "r"(x[i].w) : "memory");
                    }
                }
                __syncwarp();
#pragma unroll
                for (int half = 0; half < 2; ++half) {   // 8 chunks = 32 tensor-memory columns per store
                    if (half * 8 < CH) {
                        uint32_t w[32];
#pragma unroll
                        for (int g = 0; g < 8; ++g) {
                            const uint32_t src = mine + lane * 256 + (((half * 8 + g) ^ (lane & (CH - 1))) << 4);
                            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                         : "=r"(w[g * 4 + 0]), "=r"(w[g * 4 + 1]), "=r"(w[g * 4 + 2]), "=r"(w[g * 4 + 3]) : "r"(src) : "memory");
                        }
                        tmem_st_32x32b_x32(tQ + (c0 + half * 8) * 4, w);
                    }
                }
                __syncwarp();
            }
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(bar(B_QREADY));
        };

        int g_base = 0, uses = 0;
        bool ok = true;
        QTmemItem it;
        int item = next_item(0, lane == 0, it);
        if (item >= 0 && it.n > 0) load_q(it);

        for (int k = 0; ok && item >= 0; ++k) {
            const int n = it.n, q0 = it.q0, bh = it.bh;
            const int row = q0 + r;
            const int row_w0 = q0 + warp * 32;       // first row of this warp
            const int64_t grow = static_cast<int64_t>(bh) * prm.Sq + row;
            float m = -INFINITY, l = 0.f;

            if (n == 0 && row < prm.Sq) {
                // (K/V shards under the causal mask) no row of this tile sees a key: O = 0, LSE = -inf
                uint4* orow0 = reinterpret_cast<uint4*>(static_cast<uint8_t*>(prm.o_plain) + grow * DV * 2);
#pragma unroll
                for (int e = 0; e < DV / 8; ++e) orow0[e] = make_uint4(0u, 0u, 0u, 0u);
                prm.lse[grow] = -INFINITY;
            }

            for (int j = 0; j < n; ++j) {
                const int g = g_base + j;
                const uint32_t tS = tmem + C::S_COL + (g & 1) * BN + lane_off;
                if (!(ok = mbar_wait(bar(B_SFULL + (g & 1)), (g >> 1) & 1, abort_flag))) break;
                tc_fence_after_sync();

                // Visibility of this step's keys, per warp: a chunk of 32 keys is FULL (every row of the warp
                // sees all of it), EMPTY (no row sees any of it) or PARTIAL.
                const int kv0 = j * BN;
                const int lim = last_visible_key(row, prm.Sk, prm.causal, prm.k_offset);   // of this row
                const int lim_lo = last_visible_key(row_w0, prm.Sk, prm.causal, prm.k_offset);
                const int lim_hi = last_visible_key(row_w0 + 31, prm.Sk, prm.causal, prm.k_offset);
                auto chunk_full = [&](int ch) { return kv0 + 32 * ch + 31 <= lim_lo; };
                auto chunk_empty = [&](int ch) { return kv0 + 32 * ch > lim_hi; };
                const bool all_full = chunk_full(BN / 32 - 1);

                // Masked steps are brought into the form the fast path expects: hidden scores are overwritten
                // with -inf in tensor memory (their exponential is 0) before the row is loaded.  A zero scale
                // cannot use -inf (-inf * 0 is NaN) and takes the general path instead.
                if (c > 0.f && !all_full) {
    #pragma unroll
                    for (int ch = 0; ch < BN / 32; ++ch) {
                        if (chunk_full(ch)) continue;
                        uint32_t tmp[32];
                        if (chunk_empty(ch)) {
    #pragma unroll
                            for (int e = 0; e < 32; ++e) tmp[e] = 0xff800000u;   // -inf
                        } else {
                            tmem_ld_32x32b_x32(tS + ch * 32, tmp);
                            tmem_ld_wait();
    #pragma unroll
                            for (int e = 0; e < 32; ++e)
                                if (kv0 + ch * 32 + e > lim) tmp[e] = 0xff800000u;
                        }
                        tmem_st_32x32b_x32(tS + ch * 32, tmp);
                    }
                    tmem_st_wait();
                }
                uint32_t sr[BN];
    #pragma unroll
                for (int ch = 0; ch < BN / 32; ++ch) tmem_ld_32x32b_x32(tS + ch * 32, sr + ch * 32);
                tmem_ld_wait();

                bool done = false;
                bool use_fast = j > 0 && all_full;
                if (c > 0.f && !use_fast) {
                    if (j == 0) {   // the first step takes its exact row maximum as the reference
                        float mx0[8];
    #pragma unroll
                        for (int i = 0; i < 8; ++i) mx0[i] = fmaxf(__uint_as_float(sr[2 * i]), __uint_as_float(sr[2 * i + 1]));
    #pragma unroll
                        for (int e = 16; e < BN; e += 16)
    #pragma unroll
                            for (int i = 0; i < 8; ++i)
                                mx0[i] = max3(mx0[i], __uint_as_float(sr[e + 2 * i]), __uint_as_float(sr[e + 2 * i + 1]));
                        const float mxf = fmaxf(fmaxf(fmaxf(mx0[0], mx0[1]), fmaxf(mx0[2], mx0[3])),
                                                fmaxf(fmaxf(mx0[4], mx0[5]), fmaxf(mx0[6], mx0[7])));
                        m = (mxf == -INFINITY) ? 0.f : mxf;
                    }
                    use_fast = true;
                }
                if (use_fast) {
                    // fast path: exponentials against the reference maximum of the earlier steps, this
                    // step's row maximum computed on the side; redone below if a row ran ahead by > 2^8
                    const float mc = m * c;
                    const uint64_t c2 = pack_f32x2(c, c), nmc2 = pack_f32x2(-mc, -mc);
                    uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};
                    float mxs[8];
    #pragma unroll
                    for (int i = 0; i < 8; ++i) mxs[i] = fmaxf(__uint_as_float(sr[2 * i]), __uint_as_float(sr[2 * i + 1]));
    #pragma unroll
                    for (int e = 16; e < BN; e += 16)
    #pragma unroll
                        for (int i = 0; i < 8; ++i)
                            mxs[i] = max3(mxs[i], __uint_as_float(sr[e + 2 * i]), __uint_as_float(sr[e + 2 * i + 1]));
                    uint32_t pk[BN / 2];
    #pragma unroll
                    for (int e = 0; e < BN; e += 2) {
                        const uint64_t s2 = pack_f32x2(__uint_as_float(sr[e]), __uint_as_float(sr[e + 1]));
                        float x0, x1;
                        unpack_f32x2(fma_f32x2(s2, c2, nmc2), x0, x1);
                        const float p0 = ex2_approx(x0), p1 = ex2_approx(x1);
                        acc[(e / 2) & 3] = add_f32x2(acc[(e / 2) & 3], pack_f32x2(p0, p1));
                        pk[e / 2] = pack2<DTYPE>(p0, p1);
                    }
                    const float mx = fmaxf(fmaxf(fmaxf(mxs[0], mxs[1]), fmaxf(mxs[2], mxs[3])),
                                           fmaxf(fmaxf(mxs[4], mxs[5]), fmaxf(mxs[6], mxs[7])));
                    if (!__any_sync(0xffffffffu, (mx - m) * c > 8.f)) {
    #pragma unroll
                        for (int ch = 0; ch < BN / 64; ++ch)
                            tmem_st_32x32b_x32(tS + ch * 32, pk + ch * 32);   // P overwrites the first half of its S buffer
                        float a0, a1, a2, a3;
                        unpack_f32x2(add_f32x2(acc[0], acc[1]), a0, a1);
                        unpack_f32x2(add_f32x2(acc[2], acc[3]), a2, a3);
                        l += (a0 + a1) + (a2 + a3);
                        done = true;
                    }
                }
                if (!done) {
                    // general path: a row maximum that ran ahead, or a zero scale
                    float mx = -INFINITY;
    #pragma unroll
                    for (int e = 0; e < BN; ++e) {
                        const float sv = (kv0 + e <= lim) ? __uint_as_float(sr[e]) : -INFINITY;
                        sr[e] = __float_as_uint(sv);
                        mx = fmaxf(mx, sv);
                    }
                    float alpha = 1.f;
                    if (j == 0) {
                        m = (mx == -INFINITY) ? 0.f : mx;
                    } else if ((mx - m) * c > 8.f) {
                        alpha = ex2_approx((m - mx) * c);
                        m = mx;
                    }
                    if (__any_sync(0xffffffffu, alpha != 1.f)) {
                        // O += P V of step j-1 must have finished before O is rescaled.  S_j was issued
                        // before that product, so its barrier does not cover it; B_ODONE does.  Step j-2's
                        // product IS covered by S_j, hence the barrier is in phase j-1 or j and the parity
                        // wait below cannot alias.
                        if (!(ok = mbar_wait(bar(B_ODONE), (g - 1) & 1, abort_flag))) break;
                        tc_fence_after_sync();
    #pragma unroll
                        for (int ch = 0; ch < DV / 32; ++ch) {
                            uint32_t orr[32];
                            tmem_ld_32x32b_x32(tO + ch * 32, orr);
                            tmem_ld_wait();
    #pragma unroll
                            for (int e = 0; e < 32; ++e) orr[e] = __float_as_uint(__uint_as_float(orr[e]) * alpha);
                            tmem_st_32x32b_x32(tO + ch * 32, orr);
                        }
                    }
                    const float mc = m * c;
                    float rs = 0.f;
                    uint32_t pk[BN / 2];
    #pragma unroll
                    for (int e = 0; e < BN; e += 2) {
                        const float s0 = __uint_as_float(sr[e]), s1 = __uint_as_float(sr[e + 1]);
                        const float p0 = (s0 == -INFINITY) ? 0.f : ex2_approx(fmaf(s0, c, -mc));
                        const float p1 = (s1 == -INFINITY) ? 0.f : ex2_approx(fmaf(s1, c, -mc));
                        rs += p0 + p1;
                        pk[e / 2] = pack2<DTYPE>(p0, p1);
                    }
    #pragma unroll
                    for (int ch = 0; ch < BN / 64; ++ch) tmem_st_32x32b_x32(tS + ch * 32, pk + ch * 32);
                    l = l * alpha + rs;
                }
                tmem_st_wait();
                tc_fence_before_sync();
                mbar_arrive(bar(B_PFULL + (g & 1)));
            }
            if (!ok) break;

            // ---- the next item: its Q goes into tensor memory while the last second product still runs
            // (every S of the current item has finished: the last one was waited for above) ----
            QTmemItem itn;
            const int next = next_item(k + 1, lane == 0, itn);
            if (next >= 0 && itn.n > 0) load_q(itn);

            // ---- epilogue of the current item: O / l and LSE ----
            if (n > 0) {
                if (!(ok = mbar_wait(bar(B_OFINAL), uses & 1, abort_flag))) break;
                tc_fence_after_sync();
                const bool seen = l > 1e-30f;   // rows that saw no key (K/V shards under the causal mask): O = 0, LSE = -inf
                const float inv = seen ? 1.f / l : 0.f;
                // O leaves through a swizzled staging tile in shared memory and a TMA store (full-line
                // writes; rows beyond Sq are clipped by the tensor map), 64 columns at a time.
#pragma unroll
                for (int h = 0; h < DV / 64; ++h) {
                    uint32_t orr[64];
                    tmem_ld_32x32b_x32(tO + h * 64, orr);
                    tmem_ld_32x32b_x32(tO + h * 64 + 32, orr + 32);
                    tmem_ld_wait();
                    if (h == DV / 64 - 1) {   // O is in registers: the next item may overwrite it
                        tc_fence_before_sync();
                        mbar_arrive(bar(B_OFREE));
                    }
                    const uint32_t ost = sOst + (h & 1) * (BM * 128);   // two staging tiles take turns
                    if (r == 0) tma_store_wait_read<1>();          // the store before the previous one has read this tile
                    asm volatile("bar.sync 1, 128;" ::: "memory");
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const uint32_t w0 = pack2<DTYPE>(__uint_as_float(orr[e * 8 + 0]) * inv, __uint_as_float(orr[e * 8 + 1]) * inv);
                        const uint32_t w1 = pack2<DTYPE>(__uint_as_float(orr[e * 8 + 2]) * inv, __uint_as_float(orr[e * 8 + 3]) * inv);
                        const uint32_t w2 = pack2<DTYPE>(__uint_as_float(orr[e * 8 + 4]) * inv, __uint_as_float(orr[e * 8 + 5]) * inv);
                        const uint32_t w3 = pack2<DTYPE>(__uint_as_float(orr[e * 8 + 6]) * inv, __uint_as_float(orr[e * 8 + 7]) * inv);
                        const uint32_t dst = ost + r * 128 + ((e ^ (r & 7)) << 4);   // 128-byte swizzle
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(w0), "r"(w1), "r"(w2), "r"(w3) : "memory");
                    }
                    fence_proxy_async_smem();
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (r == 0) {
                        tma_store_3d(&tmO, ost, h * 64, q0, bh);
                        tma_store_commit();
                    }
                }
                if (row < prm.Sq) prm.lse[grow] = seen ? m * prm.scale + logf(l) : -INFINITY;
                g_base += n;
                ++uses;
            }
            item = next;
            it = itn;
        }
        if (r == 0) tma_store_wait_all<0>();   // the staging tile must outlive its last store
    }

    // ---- teardown (also reached after a timed-out wait) ----
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) finish_cta(prm.status, *abort_flag != 0, prm.counter);
    if (warp == 4) tmem_dealloc(tmem, C::TMEM_COLS);
}

}  // namespace attn_tc
