// Warp-specialised, pipelined, persistent tcgen05 attention forward kernel for head dims 64 and 128.
//
// A work item is one (batch, head) and a PAIR of 128-row Q tiles; a CTA walks the K/V tiles of
// that head for both Q tiles (the loop of Appendix C, Listings 1-2 of the paper, with the prefetch
// of Listing 1 generalised to a multi-stage ring) and then takes the next item:
//
//   warps 0-3   softmax group of Q tile 0: S -> P (online softmax, exp2), rare O rescale, epilogue
//   warps 4-7   softmax group of Q tile 1
//   warp  8     MMA issuer: S_t = Q_t K_j^T and O_t += P_t V_j, accumulators in tensor memory
//   warp  9     scheduler + TMA producer: draws work items, loads Q tiles and the K_j / V_j ring
//   warps 10-11 idle (they complete the third warpgroup so that registers can be re-balanced)
//
// While one softmax group turns S_t into P_t, the tensor core works on the other tile, so the
// exponentials and the MMAs overlap.  P_t is written back into the tensor-memory columns of S_t as
// 16-bit values and is the A operand of the second product, which is this architecture's form of
// the register-level fusion of the two GEMMs in Section 3.2.2.
//
// Persistence: the grid has one CTA per SM.  Items are ordered longest-first (causal) inside
// L2-sized groups of heads; the first item of a CTA is its block index, later ones come from a
// device counter (zero at launch: the last CTA of the previous user resets it).  Barriers, tensor memory and the K/V ring
// live across items, so the producer already loads the next item's Q/K/V and the MMA warp already
// issues its first S while the softmax groups still write the previous item's O.  Without a mask
// (equally long items) a last wave that would fill at most half of the SMs is cut into single-tile
// items, which the host announces through PipeParams::halves_from.
//
// Running maximum: the reference maximum m of a row is only advanced when the true maximum has
// grown by more than 2^8; otherwise the stale m is kept (P values up to 256, exact after the final
// division by l), so the O accumulator rarely needs rescaling.
//
// 8-bit inputs (the FP8 case study of Section 4.4): the same kernel with E4M3 tiles of half the size,
// kind::f8f6f4 MMAs and P written back as E4M3, four values per tensor-memory column; see the
// constants at the top of the kernel.
#pragma once
#include "attn_tc_common.cuh"

namespace attn_tc {

template <int D, int ES = 2>                             // ES: bytes per Q/K/V element (2, or 1 for 8-bit inputs)
struct PipeCfg {
    static constexpr int BM = 128;                       // rows of one Q tile
    static constexpr int BN = 128;                       // keys per K/V tile
    static constexpr int NBOX = D * ES / 128;            // 128-byte wide TMA boxes per tile row
    static constexpr int BOX_COLS = 128 / ES;            // elements per box row
    static constexpr int Q_BYTES = BM * D * ES;
    static constexpr int KV_BYTES = BN * D * ES;
    static constexpr int NSLOT = (KV_BYTES == 32768) ? 4 : 8;   // ring tile slots (each holds one K or V tile); two of them form a group slot: V_j and K_{j+1}
    static_assert(NBOX >= 1 && (D * ES) % 128 == 0, "tile rows must be whole 128-byte boxes");
    static constexpr int OST_BYTES = BM * 128;           // epilogue staging per Q tile: 128 rows x 64 columns
    static constexpr int TILE_BYTES = 2 * Q_BYTES + NSLOT * KV_BYTES + 2 * OST_BYTES;
    static constexpr int MISC_BYTES = 512;               // barriers, scheduler slots, TMEM slot, abort flag
    static constexpr int SMEM_BYTES = 1024 + TILE_BYTES + MISC_BYTES;
    static constexpr int TMEM_COLS = 512;
    static constexpr int THREADS = 384;
    __host__ __device__ static constexpr int s_col(int t) { return t * 128; }
    __host__ __device__ static constexpr int o_col(int t) { return 256 + t * D; }
};

struct PipeParams {
    void* o;
    float* lse;
    int Sq, Sk;
    float scale, scale_log2;
    float o_scale;          // factor on O (1 for 16-bit inputs; the V dequantisation factor for 8-bit inputs)
    int causal;
    int* status;
    int n_pairs;            // 256-row Q tile pairs per head
    int BH;                 // batch * query heads
    int heads_per_group;    // heads whose K/V are walked together (L2 residency)
    int last_group;         // index of the final group, which takes all remaining heads
    int H, Hkv;             // query heads and key/value heads per batch element (H % Hkv == 0)
    int k_offset;           // global index of key 0 of this K/V shard (0 for whole problems); enters the causal mask
    int n_items;            // work items: n_pairs * BH * n_splits, plus one for every item at or beyond halves_from
    int halves_from;        // items from this index on are cut into their two Q tiles (each half a work item of its own,
                            // consecutive indices); INT_MAX: none.  Used when the last wave of a launch of equally long
                            // items would leave more than half of the CTAs without work.
    int n_splits;           // key ranges per (head, Q tile pair): 1, or more for split-KV decoding, where range s of
    int split_tiles;        // split_tiles K/V tiles writes its partial result as head s * BH + bh of o and lse
    unsigned int* counter;  // work counter {next item, CTAs done}, zero at launch and again at exit:
                            // item = gridDim.x + atomicAdd(counter, 1); NULL when n_items <= grid
#ifdef ATTN_TEST_HOOKS
    int test_skip_ring_item;  // test build only: the K/V ring group whose loads the producer leaves out (-1: none)
#endif
};

// Register re-balancing: 384 threads start with 168 registers each (64512 of the SM's 65536); the
// service warpgroup drops to 64 (frees 13312) and the two softmax warpgroups rise to 216 (need 12288).
__device__ __forceinline__ void reg_inc_softmax() { asm volatile("setmaxnreg.inc.sync.aligned.u32 216;"); }
__device__ __forceinline__ void reg_dec_service() { asm volatile("setmaxnreg.dec.sync.aligned.u32 64;"); }

// One work item, decoded identically by every role.
struct PipeItem {
    int bh, kv_bh, q0;
    int k_tile0;   // first K/V tile of this item's key range (0 unless the keys are split)
    int o_bh;      // head index of the item's rows in o and lse (bh unless the keys are split)
    int n_kv0, n_kv1;   // K/V tiles each Q tile needs (0: tile beyond Sq, or no visible key; -1: the tile belongs to
                        // another work item and nothing of it is touched).  Two scalars, not an
                        // array: an array indexed by a run-time tile number puts the whole item into local memory,
                        // and the MMA warp then reads its loop bounds from there on every step.
    __device__ __forceinline__ int nkv(int t) const { return t ? n_kv1 : n_kv0; }
    int n_max;
};

__device__ __forceinline__ PipeItem pipe_decode_item(const PipeParams& prm, int lin_all, int BM, int BN) {
    PipeItem it;
    // the tail of the item order may consist of half items: two consecutive indices per (head, Q tile pair)
    int only_tile = -1;
    if (lin_all >= prm.halves_from) {
        const int h = lin_all - prm.halves_from;
        only_tile = h & 1;
        lin_all = prm.halves_from + (h >> 1);
    }
    // the key ranges of one (head, Q tile pair) are neighbours in the item order
    const int split = lin_all % prm.n_splits;
    const int lin = lin_all / prm.n_splits;
    const int full_group = prm.heads_per_group * prm.n_pairs;
    int g = lin / full_group;
    if (g > prm.last_group) g = prm.last_group;
    const int r = lin - g * full_group;
    const int hg = (g == prm.last_group) ? prm.BH - g * prm.heads_per_group : prm.heads_per_group;
    const int pr = r / hg;
    it.bh = g * prm.heads_per_group + (r - pr * hg);
    const int pair = prm.causal ? prm.n_pairs - 1 - pr : pr;   // causal: longest rows first
    it.q0 = pair * 2 * BM;
    // grouped-query attention: H / Hkv consecutive query heads read the same K/V head
    it.kv_bh = (it.bh / prm.H) * prm.Hkv + (it.bh % prm.H) / (prm.H / prm.Hkv);
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int qs = it.q0 + t * BM;
        int n = 0;
        if (qs < prm.Sq) {
            const int last_key = last_visible_key(qs + BM - 1, prm.Sk, prm.causal, prm.k_offset);
            n = last_key < 0 ? 0 : last_key / BN + 1;   // 0: no row of the tile sees a key of this shard
        }
        // the part of those tiles that lies in this item's key range
        int in_range = n - split * prm.split_tiles;
        if (in_range > prm.split_tiles) in_range = prm.split_tiles;
        n = in_range < 0 ? 0 : in_range;
        if (only_tile >= 0 && only_tile != t) n = -1;
        if (t == 0) it.n_kv0 = n; else it.n_kv1 = n;
    }
    it.k_tile0 = split * prm.split_tiles;
    it.o_bh = split * prm.BH + it.bh;
    it.n_max = it.n_kv0 > it.n_kv1 ? it.n_kv0 : it.n_kv1;
    return it;
}

// SPLITS: the instance for problems whose keys are cut into ranges (split-KV decoding); the plain instance does not
// carry the range's tile offset and output head through its loops.
template <int D, int DTYPE, int POLY_NUM, int POLY_DEN, bool SPLITS = false>
__global__ void __launch_bounds__(384, 1)
attn_fwd_tc_pipe_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                        const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                        const PipeParams prm) {
    // DTYPE 0 / 1: fp16 / bf16 inputs and output.  DTYPE 2: E4M3 inputs (the FP8 case of Section 4.4,
    // Table 6), bf16 output: both products run as kind::f8f6f4 MMAs and P goes back to tensor memory as
    // E4M3, four values per column.  To keep small probabilities out of that format's subnormal range, P
    // carries a factor 2^P_OFF (l carries it too, so O / l is unchanged and the LSE subtracts it), and the
    // reference maximum may lag the true one by at most 2^LAG so that P stays below the format's 448.
    constexpr bool FP8 = (DTYPE == 2);
    constexpr int ES = FP8 ? 1 : 2;              // bytes per Q/K/V element
    constexpr int ODT = FP8 ? 1 : DTYPE;         // storage type of O
    constexpr int KSTEP = 32 / ES;               // contraction elements per MMA instruction (32 bytes)
    constexpr int PCOLS = 32 * ES / 4;           // tensor-memory columns of 32 P values
    constexpr float P_OFF = FP8 ? 5.f : 0.f;
    constexpr float LAG = FP8 ? 3.f : 8.f;
    using C = PipeCfg<D, ES>;
    constexpr int BM = C::BM, BN = C::BN, NBOX = C::NBOX, NSLOT = C::NSLOT;
    constexpr int NGRP = NSLOT / 2;   // ring groups in flight (two tile slots each)

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    auto sQ = [&](int t) { return smem_base + t * C::Q_BYTES; };
    auto sKV = [&](int slot) { return smem_base + 2 * C::Q_BYTES + slot * C::KV_BYTES; };
    auto sOst = [&](int t) { return smem_base + 2 * C::Q_BYTES + NSLOT * C::KV_BYTES + t * C::OST_BYTES; };

    // misc area: barriers, then scheduler slots, TMEM base, abort flag
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + C::TILE_BYTES);
    const uint32_t bars_u32 = smem_base + C::TILE_BYTES;
    enum {
        B_QFULL = 0,      // [2] Q tile t loaded (TMA bytes)
        B_QEMPTY = 2,     // [2] every S MMA of tile t of the current item has finished: Q_t may be overwritten
        B_SFULL = 4,      // [2] S_t ready (MMA commit)
        B_PFULL = 6,      // [2] first three quarters of P_t written (128 softmax threads)
        B_PFULL2 = 8,     // [2] rest of P_t written
        B_OFINAL = 10,    // [2] last O_t += P_t V of the item has finished
        B_OFREE = 12,     // [2] the epilogue has read O_t out of tensor memory (128 softmax threads)
        B_SCHEDFULL = 14, // [4] scheduler slot holds a decoded item
        B_SCHEDEMPTY = 18,// [4] slot read by the MMA warp and the 8 softmax warps
        B_KVFULL = 22,
        B_KVEMPTY = 22 + NSLOT,
        B_COUNT = 22 + 2 * NSLOT
    };
    auto bar = [&](int i) { return bars_u32 + i * 8; };
    // scheduler slots [4][8]: item index (-1: no more work), bh, kv_bh, q0, n_kv0, n_kv1
    volatile int* sched_item = reinterpret_cast<volatile int*>(bars + B_COUNT);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT) + 32;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + B_COUNT) + 33;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        *abort_flag = 0;
        for (int t = 0; t < 2; ++t) {
            mbar_init(bar(B_QFULL + t), 1);
            mbar_init(bar(B_QEMPTY + t), 1);
            mbar_init(bar(B_SFULL + t), 1);
            mbar_init(bar(B_PFULL + t), 128);
            mbar_init(bar(B_PFULL2 + t), 128);
            mbar_init(bar(B_OFINAL + t), 1);
            mbar_init(bar(B_OFREE + t), 128);
            mbar_init(bar(B_SCHEDFULL + t), 1);
            mbar_init(bar(B_SCHEDFULL + 2 + t), 1);
            mbar_init(bar(B_SCHEDEMPTY + t), 9);
            mbar_init(bar(B_SCHEDEMPTY + 2 + t), 9);
        }
        for (int s = 0; s < NSLOT; ++s) {
            mbar_init(bar(B_KVFULL + s), 1);
            mbar_init(bar(B_KVEMPTY + s), 1);
        }
        fence_barrier_init();
        fence_proxy_async_smem();
    }
    if (warp == 8) {
        tmem_alloc(smem_u32(tmem_slot), C::TMEM_COLS);
        tmem_relinquish();
    }
    if (warp == 9 && lane == 0) {
        prefetch_tensormap(&tmQ);
        prefetch_tensormap(&tmK);
        prefetch_tensormap(&tmV);
        prefetch_tensormap(&tmO);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    // Consumers of the scheduler: wait for the k-th item of this CTA, read it (the producer has decoded it:
    // the index arithmetic is done once per item, not once per thread), hand the slot back.
    auto next_item = [&](int k, bool hand_back, PipeItem& it) -> int {
        const int slot = k & 3;
        if (!mbar_wait(bar(B_SCHEDFULL + slot), (k >> 2) & 1, abort_flag)) return -1;
        volatile int* e = sched_item + slot * 8;
        const int item = e[0];
        it.bh = e[1];
        it.kv_bh = e[2];
        it.q0 = e[3];
        it.n_kv0 = e[4];
        it.n_kv1 = e[5];
        it.k_tile0 = SPLITS ? e[6] : 0;
        it.o_bh = SPLITS ? e[7] : it.bh;
        it.n_max = it.n_kv0 > it.n_kv1 ? it.n_kv0 : it.n_kv1;
        if (hand_back) mbar_arrive(bar(B_SCHEDEMPTY + slot));
        return item;
    };

    if (warp >= 8) {
        reg_dec_service();
        // Both service warps run their loops with all 32 lanes (uniform control flow keeps the
        // address arithmetic on the uniform datapath); one elected lane issues the TMA / MMA
        // instructions.
        if (warp == 9) {
            // =========================== scheduler + TMA producer ===========================
            const bool leader = elect_one();
            int kv_base = 0;            // ring groups issued for earlier work items
            int q_uses[2] = {0, 0};     // work items that loaded Q tile t so far
            // Draws the k-th work item of this CTA, decodes it and publishes it in scheduler slot k & 3.
            // (Drawing one item ahead was measured and is slower: the CTAs finish less evenly.)
            auto publish = [&](int k) -> bool {
                const int slot = k & 3;
                if (!mbar_wait(bar(B_SCHEDEMPTY + slot), ((k >> 2) & 1) ^ 1, abort_flag)) return false;
                if (leader) {
                    // no counter: the grid covers every item with the CTAs' first draws
                    int next = (k == 0) ? static_cast<int>(blockIdx.x)
                               : (prm.counter ? static_cast<int>(gridDim.x + atomicAdd(prm.counter, 1u)) : prm.n_items);
                    if (next < 0 || next >= prm.n_items) next = -1;
                    volatile int* e = sched_item + slot * 8;
                    if (next >= 0) {
                        const PipeItem d = pipe_decode_item(prm, next, BM, BN);
                        e[1] = d.bh;
                        e[2] = d.kv_bh;
                        e[3] = d.q0;
                        e[4] = d.n_kv0;
                        e[5] = d.n_kv1;
                        e[6] = d.k_tile0;
                        e[7] = d.o_bh;
                    }
                    e[0] = next;
                    mbar_arrive(bar(B_SCHEDFULL + slot));
                }
                return true;
            };
            for (int k = 0;; ++k) {
                if (!publish(k)) break;
                PipeItem it;
                const int item = next_item(k, false, it);
                if (item < 0) break;

                auto load_q = [&](int t) -> bool {
                    // the previous item's S MMAs on this Q buffer must have finished
                    if (!mbar_wait(bar(B_QEMPTY + t), (q_uses[t] & 1) ^ 1, abort_flag)) return false;
                    if (leader) {
                        mbar_arrive_expect_tx(bar(B_QFULL + t), C::Q_BYTES);
#pragma unroll
                        for (int bx = 0; bx < NBOX; ++bx)
                            tma_load_3d(sQ(t) + bx * BM * 128, &tmQ, bar(B_QFULL + t), bx * C::BOX_COLS, it.q0 + t * BM, it.bh);
                    }
                    ++q_uses[t];
                    return true;
                };
                // Ring group i of an item (n = n_max steps): {K_0} for i = 0, {V_{i-1}, K_i} for 0 < i < n, {V_{n-1}} for
                // i = n: what the MMA warp needs together for step i - 1 (O += P V_{i-1}, then S = Q K_i^T).  One full
                // and one empty barrier per group; group slot g holds V in tile slot 2 g and K in tile slot 2 g + 1.
                auto load_group = [&](int group, int i) -> bool {
                    const int g = group % NGRP;
                    const uint32_t use = group / NGRP;
                    if (!mbar_wait(bar(B_KVEMPTY + g), (use & 1) ^ 1, abort_flag)) return false;
#ifdef ATTN_TEST_HOOKS
                    if (group == prm.test_skip_ring_item) return true;   // this group's "full" barrier never completes
#endif
                    if (leader) {
                        const bool has_v = i > 0, has_k = i < it.n_max;
                        mbar_arrive_expect_tx(bar(B_KVFULL + g), (has_v ? C::KV_BYTES : 0) + (has_k ? C::KV_BYTES : 0));
                        if (has_v) {
#pragma unroll
                            for (int bx = 0; bx < NBOX; ++bx)
                                tma_load_3d(sKV(2 * g) + bx * BN * 128, &tmV, bar(B_KVFULL + g), bx * C::BOX_COLS, (it.k_tile0 + i - 1) * BN, it.kv_bh);
                        }
                        if (has_k) {
#pragma unroll
                            for (int bx = 0; bx < NBOX; ++bx)
                                tma_load_3d(sKV(2 * g + 1) + bx * BN * 128, &tmK, bar(B_KVFULL + g), bx * C::BOX_COLS, (it.k_tile0 + i) * BN, it.kv_bh);
                        }
                    }
                    return true;
                };
                bool ok = true;
                if (it.n_kv0 > 0) ok = load_q(0);
                if (it.n_max > 0) {
                    for (int i = 0; i <= it.n_max && ok; ++i) {
                        ok = load_group(kv_base + i, i);
                        if (ok && i == 0 && it.n_kv1 > 0) ok = load_q(1);
                    }
                }
                if (!ok) break;
                if (it.n_max > 0) kv_base += it.n_max + 1;
            }
        } else if (warp == 8) {
            // =========================== MMA issuer ===========================
            const bool leader = elect_one();
            constexpr uint32_t IDESC_S = make_idesc_f16(BM, BN, FP8 ? 0 : DTYPE, 0, 0);   // format 0 of kind::f8f6f4 is E4M3
            constexpr uint32_t IDESC_O = make_idesc_f16(BM, D, FP8 ? 0 : DTYPE, 0, 1);
            constexpr uint32_t DESC_HI = smem_desc_hi_sw128(1024);
            const uint32_t q_lo[2] = {smem_desc_lo(sQ(0), 16), smem_desc_lo(sQ(1), 16)};
            const uint32_t k_lo0 = smem_desc_lo(sKV(0), 16);          // K tile in slot 0 (K-major)
            const uint32_t v_lo0 = smem_desc_lo(sKV(0), BN * 128);    // V tile in slot 0 (MN-major)
            auto issue_s = [&](int t, int s) {   // S_t = Q_t K^T : one instruction per 32 bytes of the head dim
                if (leader) {
                    const uint32_t a0 = q_lo[t], b0 = k_lo0 + s * (C::KV_BYTES >> 4);
#pragma unroll
                    for (int kk = 0; kk < D / KSTEP; ++kk) {
                        const uint32_t off = ((kk >> 2) * 128 * 128 + (kk & 3) * 32) >> 4;
                        if constexpr (FP8)
                            mma_f8_ss_lohi(tmem + C::s_col(t), a0 + off, b0 + off, DESC_HI, IDESC_S, kk > 0);
                        else
                            mma_f16_ss_lohi(tmem + C::s_col(t), a0 + off, b0 + off, DESC_HI, IDESC_S, kk > 0);
                    }
                }
            };
            auto issue_pv = [&](int t, int s, bool accumulate, int kk_begin, int kk_end) {
                if (leader) {                    // O_t += P_t V : KSTEP keys (8 columns of P) per instruction
                    const uint32_t b0 = v_lo0 + s * (C::KV_BYTES >> 4);
#pragma unroll
                    for (int kk = kk_begin; kk < kk_end; ++kk) {
                        if constexpr (FP8)
                            mma_f8_ts_lohi(tmem + C::o_col(t), tmem + C::s_col(t) + kk * 8, b0 + ((kk * KSTEP * 128) >> 4),
                                           DESC_HI, IDESC_O, (accumulate || kk > 0) ? 1u : 0u);
                        else
                            mma_f16_ts_lohi(tmem + C::o_col(t), tmem + C::s_col(t) + kk * 8, b0 + ((kk * KSTEP * 128) >> 4),
                                            DESC_HI, IDESC_O, (accumulate || kk > 0) ? 1u : 0u);
                    }
                }
            };
            auto commit = [&](int b) {
                if (leader) mma_commit(bar(b));
            };
            auto kv_full_wait = [&](int group) {   // both tiles of a ring group are loaded
                return mbar_wait(bar(B_KVFULL + group % NGRP), (group / NGRP) & 1, abort_flag);
            };
            int kv_base = 0;
            int it_base[2] = {0, 0};   // K/V steps tile t has gone through in earlier work items
            int uses[2] = {0, 0};      // work items in which tile t took part
            bool ok = true;
            for (int k = 0; ok; ++k) {
                PipeItem it;
                const int item = next_item(k, leader, it);
                if (item < 0) break;
                // ---- first S of both tiles ----
                if (it.n_max > 0) ok = kv_full_wait(kv_base);
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if (ok && it.nkv(t) > 0) {
                        ok = mbar_wait(bar(B_QFULL + t), uses[t] & 1, abort_flag);
                        if (ok) {
                            tc_fence_after_sync();
                            issue_s(t, 2 * (kv_base % NGRP) + 1);
                            commit(B_SFULL + t);
                            if (it.nkv(t) == 1) commit(B_QEMPTY + t);
                        }
                    }
                }
                if (ok && it.n_max > 0) commit(B_KVEMPTY + kv_base % NGRP);
                for (int j = 0; j < it.n_max && ok; ++j) {
                    // V_j and K_{j+1} are one ring group: one wait, one release
                    const int gslot = (kv_base + j + 1) % NGRP;
                    const int vslot = 2 * gslot, kslot = 2 * gslot + 1;
                    if (!(ok = kv_full_wait(kv_base + j + 1))) break;
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        if (j < it.nkv(t)) {
                            const uint32_t par = (it_base[t] + j) & 1;
                            if (!(ok = mbar_wait(bar(B_PFULL + t), par, abort_flag))) break;
                            // the epilogue of the previous item must have read O_t before it is overwritten
                            if (j == 0 && uses[t] > 0 && !(ok = mbar_wait(bar(B_OFREE + t), (uses[t] - 1) & 1, abort_flag))) break;
                            tc_fence_after_sync();
                            issue_pv(t, vslot, j > 0, 0, 3 * (BN / KSTEP) / 4);
                            if (!(ok = mbar_wait(bar(B_PFULL2 + t), par, abort_flag))) break;
                            tc_fence_after_sync();
                            issue_pv(t, vslot, true, 3 * (BN / KSTEP) / 4, BN / KSTEP);
                            if (j + 1 == it.nkv(t)) commit(B_OFINAL + t);
                        }
                        if (j + 1 < it.nkv(t)) {
                            tc_fence_after_sync();
                            issue_s(t, kslot);
                            commit(B_SFULL + t);
                            if (j + 2 == it.nkv(t)) commit(B_QEMPTY + t);   // that was the last S of this item
                        }
                    }
                    if (ok) commit(B_KVEMPTY + gslot);
                }
                if (it.n_max > 0) kv_base += it.n_max + 1;
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    it_base[t] += it.nkv(t) > 0 ? it.nkv(t) : 0;
                    uses[t] += it.nkv(t) > 0 ? 1 : 0;
                }
            }
        }
    } else {
        // =========================== softmax groups ===========================
        reg_inc_softmax();
        const int t = warp >> 2;                       // Q tile of this group
        const int r = tid & 127;                       // row inside the tile
        const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + C::s_col(t) + lane_off, tO = tmem + C::o_col(t) + lane_off;
        const float c = prm.scale_log2;
        int it_base = 0, uses = 0;
        bool ok = true;
        // 32 values of P -> their tensor-memory columns (two 16-bit or four 8-bit values per column)
        auto store_p = [&](int ch, const uint32_t* pk) {
            if constexpr (FP8)
                tmem_st_32x32b_x8(tS + ch * PCOLS, pk);
            else
                tmem_st_32x32b_x16(tS + ch * PCOLS, pk);
        };

        for (int k = 0; ok; ++k) {
            PipeItem it;
            const int item = next_item(k, lane == 0, it);
            if (item < 0) break;
            const int n = it.nkv(t);
            const int q0 = it.q0;
            const int row = q0 + t * BM + r;
            if (n <= 0) {
                // beyond Sq, or (K/V shards under the causal mask) rows that see no key: O = 0, LSE = -inf;
                // n < 0: the tile is another work item's
                if (n == 0 && row < prm.Sq) {
                    const int64_t grow0 = static_cast<int64_t>(it.o_bh) * prm.Sq + row;
                    uint4* orow0 = reinterpret_cast<uint4*>(static_cast<uint8_t*>(prm.o) + grow0 * D * 2);
#pragma unroll
                    for (int g = 0; g < D / 8; ++g) orow0[g] = make_uint4(0u, 0u, 0u, 0u);
                    prm.lse[grow0] = -INFINITY;
                }
                continue;
            }
            const int row_w0 = q0 + t * BM + (warp & 3) * 32;   // first row of this warp
            float m = -INFINITY, l = 0.f;

            for (int j = 0; j < n; ++j) {
                if (!(ok = mbar_wait(bar(B_SFULL + t), (it_base + j) & 1, abort_flag))) break;
                tc_fence_after_sync();
                // Visibility of this K/V tile, per warp (rows 32 w .. 32 w + 31 of the Q tile): a chunk of
                // 32 keys is FULL (every row sees all of it), EMPTY (no row sees any of it) or PARTIAL.
                const int kv0 = (it.k_tile0 + j) * BN;
                const int lim = last_visible_key(row, prm.Sk, prm.causal, prm.k_offset);   // of this row
                const int lim_lo = last_visible_key(row_w0, prm.Sk, prm.causal, prm.k_offset);
                const int lim_hi = last_visible_key(row_w0 + 31, prm.Sk, prm.causal, prm.k_offset);
                auto chunk_full = [&](int ch) { return kv0 + 32 * ch + 31 <= lim_lo; };
                auto chunk_empty = [&](int ch) { return kv0 + 32 * ch > lim_hi; };
                const bool all_full = chunk_full(BN / 32 - 1);

                // Masked (diagonal / ragged) tiles are brought into the form the fast path expects, so that
                // they run the same (instruction-cache resident) code as every other tile: hidden scores are
                // overwritten with -inf in tensor memory (their exponential is 0) before the row is loaded.
                // A zero scale cannot use -inf (-inf * 0 is NaN): it takes the general path instead.
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
                // With a positive scale every tile takes the fast path: masked tiles were pre-masked above,
                // and the first tile takes its exact row maximum as the reference first.
                bool use_fast = j > 0 && all_full;
                if (c > 0.f && !use_fast) {
                    if (j == 0) {
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
                    // ---- fast path: exponentials against the reference maximum of the previous tiles,
                    // the row maximum of this tile computed on the side.  Valid when no row of the warp
                    // has grown by more than 2^8; otherwise everything is redone by the general path.
                    const float nmc = P_OFF - m * c;
                    const uint64_t c2 = pack_f32x2(c, c), nmc2 = pack_f32x2(nmc, nmc);
                    uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};   // 8 partial row sums
                    float mxs[8];
    #pragma unroll
                    for (int i = 0; i < 8; ++i) mxs[i] = fmaxf(__uint_as_float(sr[2 * i]), __uint_as_float(sr[2 * i + 1]));
                    auto exp_chunk = [&](int ch) {
                        uint32_t pk[PCOLS];
    #pragma unroll
                        for (int e4 = 0; e4 < 32; e4 += 4) {
                            float p[4];
    #pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                const int e = e4 + 2 * h;
                                const uint64_t s2 = pack_f32x2(__uint_as_float(sr[ch * 32 + e]), __uint_as_float(sr[ch * 32 + e + 1]));
                                const uint64_t x2 = fma_f32x2(s2, c2, nmc2);
                                float x0, x1, p0, p1;
                                unpack_f32x2(x2, x0, x1);
                                if (((ch * 16 + e / 2) % POLY_DEN) < POLY_NUM) {   // this pair: polynomial on the FMA pipe
                                    ex2_poly_f32x2(pack_f32x2(fmaxf(x0, -126.f), fmaxf(x1, -126.f)), p0, p1);
                                } else {                                           // this pair: special-function unit
                                    p0 = ex2_approx(x0);
                                    p1 = ex2_approx(x1);
                                }
                                acc[(e / 2) & 3] = add_f32x2(acc[(e / 2) & 3], pack_f32x2(p0, p1));
                                p[2 * h] = p0;
                                p[2 * h + 1] = p1;
                            }
                            if constexpr (FP8) {
                                pk[e4 / 4] = pack4_e4m3(p[0], p[1], p[2], p[3]);
                            } else {
                                pk[e4 / 2] = pack2<DTYPE>(p[0], p[1]);
                                pk[e4 / 2 + 1] = pack2<DTYPE>(p[2], p[3]);
                            }
                        }
                        store_p(ch, pk);   // P overwrites the S columns already in registers
                    };
    #pragma unroll
                    for (int ch = 0; ch < BN / 32 - 1; ++ch) {
                        exp_chunk(ch);
                        // a third of the row maximum per chunk, off the critical path of the exponentials
    #pragma unroll
                        for (int g = 0; g < 7; ++g) {
                            const int e = 16 + (ch * 7 + g) * 16;
                            if (e < BN) {
    #pragma unroll
                                for (int i = 0; i < 8; ++i)
                                    mxs[i] = max3(mxs[i], __uint_as_float(sr[e + 2 * i]), __uint_as_float(sr[e + 2 * i + 1]));
                            }
                        }
                    }
                    const float mx = fmaxf(fmaxf(fmaxf(mxs[0], mxs[1]), fmaxf(mxs[2], mxs[3])),
                                           fmaxf(fmaxf(mxs[4], mxs[5]), fmaxf(mxs[6], mxs[7])));
                    if (!__any_sync(0xffffffffu, (mx - m) * c > LAG)) {
                        tmem_st_wait();
                        tc_fence_before_sync();
                        mbar_arrive(bar(B_PFULL + t));          // first three quarters of P are in place
                        exp_chunk(BN / 32 - 1);
                        float a0, a1, a2, a3;
                        unpack_f32x2(add_f32x2(acc[0], acc[1]), a0, a1);
                        unpack_f32x2(add_f32x2(acc[2], acc[3]), a2, a3);
                        l += (a0 + a1) + (a2 + a3);
                        done = true;
                    }
                }

                if (!done) {
                    // ---- general path: first tile, masked tile, or a row maximum that ran ahead.
                    // Exact row maximum over the visible keys first, then the exponentials chunk by chunk.
                    float alpha = 1.f;
                    {
                        float mxs[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) mxs[i] = -INFINITY;
#pragma unroll
                        for (int ch = 0; ch < BN / 32; ++ch) {
                            if (chunk_full(ch)) {
#pragma unroll
                                for (int e = 0; e < 32; e += 16)
#pragma unroll
                                    for (int i = 0; i < 8; ++i)
                                        mxs[i] = max3(mxs[i], __uint_as_float(sr[ch * 32 + e + 2 * i]),
                                                      __uint_as_float(sr[ch * 32 + e + 2 * i + 1]));
                            } else if (!chunk_empty(ch)) {
#pragma unroll
                                for (int e = 0; e < 32; ++e)
                                    mxs[e & 7] = fmaxf(mxs[e & 7], (kv0 + ch * 32 + e <= lim) ? __uint_as_float(sr[ch * 32 + e]) : -INFINITY);
                            }
                        }
                        const float mx = fmaxf(fmaxf(fmaxf(mxs[0], mxs[1]), fmaxf(mxs[2], mxs[3])),
                                               fmaxf(fmaxf(mxs[4], mxs[5]), fmaxf(mxs[6], mxs[7])));
                        // advance the reference maximum only when the true one ran ahead by more than 2^LAG
                        if (j == 0) {
                            m = (mx == -INFINITY) ? 0.f : mx;
                        } else if ((mx - m) * c > LAG) {
                            alpha = ex2_approx((m - mx) * c);
                            m = mx;
                        }
                    }
                    // rare: rescale the running O (its last update finished before S_j was produced)
                    if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
                        for (int ch = 0; ch < D / 32; ++ch) {
                            uint32_t orr[32];
                            tmem_ld_32x32b_x32(tO + ch * 32, orr);
                            tmem_ld_wait();
#pragma unroll
                            for (int e = 0; e < 32; ++e) orr[e] = __float_as_uint(__uint_as_float(orr[e]) * alpha);
                            tmem_st_32x32b_x32(tO + ch * 32, orr);
                        }
                    }
                    const float nmc = P_OFF - m * c;
                    const uint64_t c2 = pack_f32x2(c, c), nmc2 = pack_f32x2(nmc, nmc);
                    uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};   // 8 partial row sums (FULL chunks)
                    float rs = 0.f;                                // row sum of PARTIAL chunks
#pragma unroll
                    for (int ch = 0; ch < BN / 32; ++ch) {
                        uint32_t pk[PCOLS];
                        float pv[32];   // the chunk's probabilities
                        if (chunk_full(ch)) {
#pragma unroll
                            for (int e = 0; e < 32; e += 2) {
                                const uint64_t s2 = pack_f32x2(__uint_as_float(sr[ch * 32 + e]), __uint_as_float(sr[ch * 32 + e + 1]));
                                float x0, x1;
                                unpack_f32x2(fma_f32x2(s2, c2, nmc2), x0, x1);
                                pv[e] = ex2_approx(x0);
                                pv[e + 1] = ex2_approx(x1);
                                acc[(e / 2) & 3] = add_f32x2(acc[(e / 2) & 3], pack_f32x2(pv[e], pv[e + 1]));
                            }
                        } else if (!chunk_empty(ch)) {
#pragma unroll
                            for (int e = 0; e < 32; ++e) {
                                const int key = kv0 + ch * 32 + e;
                                pv[e] = (key <= lim) ? ex2_approx(fmaf(__uint_as_float(sr[ch * 32 + e]), c, nmc)) : 0.f;
                                rs += pv[e];
                            }
                        } else {
#pragma unroll
                            for (int e = 0; e < 32; ++e) pv[e] = 0.f;
                        }
#pragma unroll
                        for (int w = 0; w < PCOLS; ++w) {
                            if constexpr (FP8)
                                pk[w] = pack4_e4m3(pv[4 * w], pv[4 * w + 1], pv[4 * w + 2], pv[4 * w + 3]);
                            else
                                pk[w] = pack2<DTYPE>(pv[2 * w], pv[2 * w + 1]);
                        }
                        store_p(ch, pk);   // P overwrites the S columns already in registers
                        if (ch == BN / 32 - 2) {
                            tmem_st_wait();
                            tc_fence_before_sync();
                            mbar_arrive(bar(B_PFULL + t));          // first three quarters of P are in place
                        }
                    }
                    float a0, a1, a2, a3;
                    unpack_f32x2(add_f32x2(acc[0], acc[1]), a0, a1);
                    unpack_f32x2(add_f32x2(acc[2], acc[3]), a2, a3);
                    l = l * alpha + (((a0 + a1) + (a2 + a3)) + rs);
                }
                tmem_st_wait();
                tc_fence_before_sync();
                mbar_arrive(bar(B_PFULL2 + t));
            }
            if (!ok) break;

            // ---- epilogue: O / l and LSE ----
            if (!(ok = mbar_wait(bar(B_OFINAL + t), uses & 1, abort_flag))) break;
            tc_fence_after_sync();
            // A row that saw at least one key has l >= 2^-8 (its maximum contributed 1 when it was taken as the
            // reference).  Rows that saw none (possible for K/V shards under the causal mask) only collected
            // the 2^-126 floor of the polynomial exponential: they give O = 0, LSE = -inf.
            const bool seen = l > 1e-30f;
            const float inv = seen ? prm.o_scale / l : 0.f;
            const int64_t grow = static_cast<int64_t>(it.o_bh) * prm.Sq + row;
            // O leaves through a swizzled staging tile in shared memory and a TMA store (full-line writes;
            // rows beyond Sq are clipped by the tensor map), 64 columns at a time.
            const uint32_t ost = sOst(t);
#pragma unroll
            for (int h = 0; h < D / 64; ++h) {
                uint32_t orr[64];
                tmem_ld_32x32b_x32(tO + h * 64, orr);
                tmem_ld_32x32b_x32(tO + h * 64 + 32, orr + 32);
                tmem_ld_wait();
                if (h == D / 64 - 1) {   // O_t is in registers: the next item may overwrite it
                    tc_fence_before_sync();
                    mbar_arrive(bar(B_OFREE + t));
                }
                if (r == 0) tma_store_wait_read<0>();          // the previous store has read the staging tile
                asm volatile("bar.sync %0, 128;" ::"r"(1 + t) : "memory");
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    const uint32_t w0 = pack2<ODT>(__uint_as_float(orr[g * 8 + 0]) * inv, __uint_as_float(orr[g * 8 + 1]) * inv);
                    const uint32_t w1 = pack2<ODT>(__uint_as_float(orr[g * 8 + 2]) * inv, __uint_as_float(orr[g * 8 + 3]) * inv);
                    const uint32_t w2 = pack2<ODT>(__uint_as_float(orr[g * 8 + 4]) * inv, __uint_as_float(orr[g * 8 + 5]) * inv);
                    const uint32_t w3 = pack2<ODT>(__uint_as_float(orr[g * 8 + 6]) * inv, __uint_as_float(orr[g * 8 + 7]) * inv);
                    const uint32_t dst = ost + r * 128 + ((g ^ (r & 7)) << 4);   // 128-byte swizzle
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(w0), "r"(w1), "r"(w2), "r"(w3) : "memory");
                }
                fence_proxy_async_smem();
                asm volatile("bar.sync %0, 128;" ::"r"(1 + t) : "memory");
                if (r == 0) {
                    tma_store_3d(&tmO, ost, h * 64, q0 + t * BM, it.o_bh);
                    tma_store_commit();
                }
            }
            if (row < prm.Sq) prm.lse[grow] = seen ? m * prm.scale + (logf(l) - P_OFF * 0.6931471805599453f) : -INFINITY;
            it_base += n;
            ++uses;
        }
        if (r == 0) tma_store_wait_all<0>();   // the staging tile must outlive its last store
    }

    // ---- teardown (also reached after a timed-out wait) ----
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) finish_cta(prm.status, *abort_flag != 0, prm.counter);
    if (warp == 8) tmem_dealloc(tmem, C::TMEM_COLS);
}

}  // namespace attn_tc
