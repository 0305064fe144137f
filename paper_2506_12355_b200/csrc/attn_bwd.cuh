// Backward pass of the attention operator on tcgen05 tensor cores (head dims 64 and 128).
//
// Gradients of O = Softmax(Mask(scale Q K^T)) V (Section 2.2 of the paper; the paper itself measures the
// forward pass only) for an upstream gradient dO, from Q, K, V, O, dO and the forward pass's per-row
// logsumexp L:
//
//     P  = exp(scale Q K^T - L)           dP = dO V^T            delta_i = sum_d dO_id O_id
//     dS = P o (dP - delta)               dV = P^T dO            dQ = scale dS K        dK = scale dS^T Q
//
// Two passes over the score tiles, each the forward loop of Appendix C's listings with other operands (one
// tile resident, the other side streamed through a TMA ring, the S x S matrices never leave the SM):
//
//   MODE 0 (dQ):      CTA = one 128-row Q tile; Q_i, dO_i resident; K_j, V_j streamed.
//                     S = Q_i K_j^T and dP = dO_i V_j^T -> tensor memory; one thread per query row turns them
//                     into dS (16-bit, tensor memory); dQ += dS K_j with K_j as the MN-major operand.
//   MODE 1 (dK, dV):  CTA = one 128-key K/V tile; K_j, V_j resident; Q_i, dO_i streamed (all query heads of
//                     the K/V head's group).  The TRANSPOSED tiles S^T = K_j Q_i^T and dP^T = V_j dO_i^T are
//                     computed, so that P^T and dS^T land in tensor memory with keys on the lanes, which is
//                     the A operand that dV += P^T dO_i and dK += dS^T Q_i need; one thread per key row, the
//                     per-query -L log2(e) and -delta arrive in shared memory with the streamed tiles.
//
// Recomputing S and dP in both passes costs 7 tile products instead of 5 but needs no atomics and no
// cross-CTA reduction, so the results are deterministic.  A small kernel first prepares the two row vectors
// (-L log2(e) and -delta) in the caller's workspace.  Where the 512 tensor-memory columns allow it (everywhere but
// MODE 1 at D = 128) the resident tiles are copied into tensor memory once and are the A operand of the S / dP
// products from there; with both operands in shared memory those products are paced by shared-memory bandwidth.
//
// The streamed side advances 64 rows per step.  The fp32 dP tile of a step (128 lanes x 64 columns) has ONE place
// in tensor memory, the S tile one or (wherever 64 columns are left: everywhere but MODE 1 at D = 128) two, which an
// element-wise group frees as soon as it has the tiles in registers; the 16-bit operands it makes from them go to one
// of two small operand regions.  So while a group computes, the tensor core already produces S and dP of the next
// step for the other group (with two S buffers the next S directly behind the current dP, before the current step has
// even been read), and the accumulating products of a step run whenever its operands are ready.
//
//   warps 0-3  element-wise group of the even steps (one thread per tensor-memory lane); both groups then run the
//   warps 4-7  element-wise group of the odd steps                                          epilogue together
//   warp  8    MMA issuer of the S and dP products
//   warp  9    TMA producer
//   warp  10   MMA issuer of the accumulating products (two issuers: a tcgen05.mma issue holds its thread while the
//              tensor core's queue is full, and a single issuer's barrier polls between the two kinds of product
//              left the queue running empty ~30 % of the time)
//   warp  11   idle (it completes the third warpgroup so that registers can be re-balanced: an element-wise thread
//              holds a whole S and dP row of a step, 128 registers, while it computes)
//
// Persistent grid: one CTA per SM; its first tile is its block index, later ones come from a device counter (tiles of
// one head are neighbours in the order, so that their streamed tiles meet in L2, and under the causal mask a head's
// heaviest tiles come first, so the launch ends on light ones).  The producer warp draws a tile a few steps before the
// current one ends and publishes it to the other roles through scheduler slots in shared memory.  Barriers, tensor memory
// and the streamed ring live across tiles: the producer loads the next tile's resident tiles while the current tile
// still computes, the element-wise warps copy them into tensor memory right after their last step, and the S / dP
// products of the next tile's first step run while the accumulators of the current tile drain.
//
// Every wait is bounded (see sm100_ptx.cuh); a timed-out wait ends the CTA through the normal exit.
#pragma once
#include <type_traits>

#include "attn_tc_common.cuh"

namespace attn_grad {

using namespace sm100;
using attn_tc::finish_cta;

template <int D, int MODE>
struct BwdCfg {
    static constexpr int BT = 128;                          // rows of the resident tiles = tensor-memory lanes
    static constexpr int BS = 64;                           // rows of the streamed tiles = columns of one step
    static constexpr int NBOX = D / 64;                     // 128-byte wide TMA boxes per tile row
    static constexpr int RES_BYTES = BT * D * 2;            // one resident tile
    static constexpr int STR_BYTES = BS * D * 2;            // one streamed tile
    static constexpr int NACC = MODE == 0 ? 1 : 2;          // accumulators: dQ, or dV and dK
    static constexpr int OST_BYTES = BT * 128;              // one epilogue staging tile: 128 rows x 64 columns
    static constexpr int STG_BYTES = NACC * (D / 64) * OST_BYTES;   // a staging tile for every 64-column piece of the output
    // ring stages, each holds the two streamed tiles (three where the staging tiles leave no room for four)
    static constexpr int NSTAGE = D == 64 ? 6 : (MODE == 0 ? 4 : 3);
    static constexpr int VEC_BYTES = MODE == 1 ? NSTAGE * 2 * BS * 4 : 0;   // -L log2(e) and -delta of a stage's 64 query rows
    static constexpr int TILE_BYTES = 2 * RES_BYTES + NSTAGE * 2 * STR_BYTES + STG_BYTES + VEC_BYTES;
    static constexpr int MISC_BYTES = 512;                  // barriers (up to 34), scheduler slots, TMEM slot, abort flag
    static constexpr int SMEM_BYTES = 1024 + TILE_BYTES + MISC_BYTES;
    static_assert(SMEM_BYTES <= 232448, "shared memory budget");
    static_assert((22 + 2 * NSTAGE) * 8 + 32 <= MISC_BYTES, "barrier area");
    static constexpr int THREADS = 384;
    // tensor memory: fp32 S in columns 0 .. 63, fp32 dP in 64 .. 127; operand region g (steps u = g mod 2): first
    // 16-bit operand (dS in MODE 0, P^T in MODE 1) in its columns 0 .. 31, second (MODE 1: dS^T) in 32 .. 63.
    // Wherever 64 more columns are free (everywhere but the dK/dV pass at D = 128), S has a second buffer: the S of
    // step u + 1 is then computed while the element-wise group still holds the dP columns of step u, and only the dP
    // product is left between "S and dP of step u are in registers" and "S and dP of step u + 1 are ready".
    static constexpr bool S2BUF = !(MODE == 1 && D == 128);
    static constexpr int S_COL = 0, DP_COL = 64;
    __host__ __device__ static constexpr int op_col(int g) { return MODE == 0 ? 128 + 32 * g : 128 + 64 * g; }
    __host__ __device__ static constexpr int s_col(int b) { return (S2BUF && b) ? (MODE == 0 ? 192 : 384) : S_COL; }
    static constexpr int ACC0_COL = 256, ACC1_COL = 256 + D;
    // the resident tiles as 16-bit A operands in tensor memory (where the columns allow it): tile w in D / 2 columns
    __host__ __device__ static constexpr int rt_col(int w) { return 512 - D + w * (D / 2); }
    static constexpr int TMEM_COLS = 512;
    static_assert(D == 64 || D == 128, "head dims 64 and 128");
    static_assert(!S2BUF || MODE == 0 || 384 + 64 <= 512 - D, "second S buffer below the resident operands");
    static_assert(ACC0_COL + NACC * D <= (MODE == 0 ? 512 - D : (D == 64 ? 384 : 512)), "accumulators end below what follows them");
};

struct BwdParams {
    // Row vectors prepared by attn_bwd_rows_kernel, [B*H][Sq_pad] fp32 each (Sq_pad: Sq rounded up to a multiple
    // of 64, the padding rows hold 0, so that 64 rows from any multiple of 64 are one aligned, in-bounds block):
    const float* nl2;       // -LSE * log2(e)   (-inf for rows without a visible key: their P is 0)
    const float* ndelta;    // -rowsum(dO o O)
    int Sq_pad;
    void* out0;             // plain pointers of the outputs, for tiles that no step touches (zero fill):
    void* out1;             //   MODE 0: dq, unused;  MODE 1: dv, dk
    int Sq, Sk;
    float scale, scale_log2;
    int causal;
    int H, Hkv;
    int n_qtiles, n_ktiles; // 128-row tiles of the query and of the key axis
    int n_tiles_total;      // tiles of this pass over all heads
    unsigned int* counter;  // work counter {next tile, CTAs done}, zero at launch and again at exit:
                            // tile = gridDim.x + atomicAdd(counter, 1); NULL when the grid covers every tile
    int* status;
};

__device__ __forceinline__ void zero_rows(void* base, int64_t first_row, int rows, int D, int tid, int nthreads) {
    uint4* p = reinterpret_cast<uint4*>(static_cast<uint8_t*>(base) + first_row * D * 2);
    const int n = rows * D / 8;
    for (int i = tid; i < n; i += nthreads) p[i] = make_uint4(0u, 0u, 0u, 0u);
}

// Per query row, one warp per row: ndelta = -sum_d dO_id * O_id and nl2 = -LSE * log2(e), written with the row
// stride Sq_pad (padding rows: 0).  `rows` counts padded rows: B * H * Sq_pad.
template <int D, int DTYPE>
__global__ void attn_bwd_rows_kernel(const void* __restrict__ o, const void* __restrict__ dout, const float* __restrict__ lse,
                                     float* __restrict__ nl2, float* __restrict__ ndelta, int Sq, int Sq_pad, int64_t rows) {
    const int lane = threadIdx.x & 31;
    const int64_t warps = static_cast<int64_t>(gridDim.x) * (blockDim.x >> 5);
    for (int64_t prow = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); prow < rows; prow += warps) {
        const int64_t bh = prow / Sq_pad;
        const int i = static_cast<int>(prow - bh * Sq_pad);
        if (i >= Sq) {
            if (lane == 0) {
                nl2[prow] = 0.f;
                ndelta[prow] = 0.f;
            }
            continue;
        }
        const int64_t row = bh * Sq + i;
        float acc = 0.f;
        if constexpr (D == 128) {
            const uint2 a = reinterpret_cast<const uint2*>(static_cast<const uint8_t*>(o) + row * D * 2)[lane];
            const uint2 b = reinterpret_cast<const uint2*>(static_cast<const uint8_t*>(dout) + row * D * 2)[lane];
            const uint32_t aw[2] = {a.x, a.y}, bw[2] = {b.x, b.y};
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                float a0, a1, b0, b1;
                if constexpr (DTYPE == 0) {
                    const float2 fa = __half22float2(*reinterpret_cast<const __half2*>(&aw[i]));
                    const float2 fb = __half22float2(*reinterpret_cast<const __half2*>(&bw[i]));
                    a0 = fa.x; a1 = fa.y; b0 = fb.x; b1 = fb.y;
                } else {
                    const float2 fa = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&aw[i]));
                    const float2 fb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&bw[i]));
                    a0 = fa.x; a1 = fa.y; b0 = fb.x; b1 = fb.y;
                }
                acc = fmaf(a0, b0, acc);
                acc = fmaf(a1, b1, acc);
            }
        } else {
            const uint32_t a = reinterpret_cast<const uint32_t*>(static_cast<const uint8_t*>(o) + row * D * 2)[lane];
            const uint32_t b = reinterpret_cast<const uint32_t*>(static_cast<const uint8_t*>(dout) + row * D * 2)[lane];
            float2 fa, fb;
            if constexpr (DTYPE == 0) {
                fa = __half22float2(*reinterpret_cast<const __half2*>(&a));
                fb = __half22float2(*reinterpret_cast<const __half2*>(&b));
            } else {
                fa = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&a));
                fb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&b));
            }
            acc = fmaf(fa.x, fb.x, fa.y * fb.y);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) {
            const float l = lse[row];
            nl2[prow] = (l == -INFINITY) ? -INFINITY : -l * 1.4426950408889634f;
            ndelta[prow] = -acc;
        }
    }
}

// One tile of a pass, decoded identically by every role.
struct BwdTile {
    int tile, bh_res;       // index of the 128-row tile inside its head; (batch, head) of the resident tensors
    int sub_lo, sub_hi;     // range of 64-row tiles of the streamed axis
    int n_steps;            // 0: nothing reaches this tile (its gradients are zero)
    int kv_bh_of_q;         // MODE 0: K/V head of this query head
};

// tmR0 / tmR1: maps of the resident tiles, boxes of 128 rows (MODE 0: Q, dO; MODE 1: K, V); tmT0 / tmT1: maps of
// the streamed tiles, boxes of 64 rows (MODE 0: K, V; MODE 1: Q, dO); tmOut0 / tmOut1: MODE 0: dQ, unused;
// MODE 1: dV, dK (boxes of 128 rows).
template <int D, int DTYPE, int MODE>
__global__ void __launch_bounds__(384, 1)
attn_bwd_kernel(const __grid_constant__ CUtensorMap tmR0, const __grid_constant__ CUtensorMap tmR1,
                const __grid_constant__ CUtensorMap tmT0, const __grid_constant__ CUtensorMap tmT1,
                const __grid_constant__ CUtensorMap tmOut0, const __grid_constant__ CUtensorMap tmOut1,
                const BwdParams prm) {
    using C = BwdCfg<D, MODE>;
    constexpr int BT = C::BT, BS = C::BS, NBOX = C::NBOX, NSTAGE = C::NSTAGE, NACC = C::NACC;
    // The S and dP products read their resident operand (A) from tensor memory wherever 512 columns allow it: with both
    // operands in shared memory an M 128 x N 64 instruction is paced by shared-memory bandwidth (6 KB per 32 tensor
    // cycles), with A in tensor memory it reads 2 KB.  The dK/dV pass at D = 128 has no columns left for it.
    constexpr bool A_TMEM = !(MODE == 1 && D == 128);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    auto sR = [&](int w) { return smem_base + w * C::RES_BYTES; };                                          // resident tile w
    auto sT = [&](int stage, int w) { return smem_base + 2 * C::RES_BYTES + (2 * stage + w) * C::STR_BYTES; };  // streamed tile w
    constexpr int STG_OFF = 2 * C::RES_BYTES + 2 * NSTAGE * C::STR_BYTES;
    const uint32_t sStg = smem_base + STG_OFF;                                                              // staging tiles
    constexpr int VEC_OFF = STG_OFF + C::STG_BYTES;
    float* vec = reinterpret_cast<float*>(smem_gen + VEC_OFF);   // [stage][-L log2 e | -delta][BS]
    const uint32_t sVec = smem_base + VEC_OFF;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + C::TILE_BYTES);
    const uint32_t bars_u32 = smem_base + C::TILE_BYTES;
    // Per-tile barriers complete once per (non-empty) tile of this CTA, per-step barriers once per step of their
    // group or stage; every role counts tiles (kk) and steps (gs) the same way, across tiles.
    enum {
        B_RFULL = 0,      // tile: resident tiles loaded (TMA bytes)
        B_RTMEM = 1,      // tile: resident tiles copied into tensor memory (256 element-wise threads)
        B_SLAST = 2,      // tile: its last S / dP product has finished (MMA commit): resident operand no longer read
        B_ACCFINAL = 3,   // tile: its last accumulating product has finished (MMA commit)
        B_ACCFREE = 4,    // tile: the accumulators are in registers, the next tile may overwrite them (256 threads)
        B_ESYNC = 5,      // barrier among all 256 element-wise threads (epilogue)
        B_SFULL = 6,      // [2] step: S and dP of a step of group g are in tensor memory (MMA commit)
        B_SREAD = 8,      // [2] step: group g has them in registers: S and dP may be overwritten (128 threads)
        B_PFULL = 10,     // [2] step: the 16-bit operands of a step are in operand region g (128 threads)
        B_OPFREE = 12,    // [2] step: the accumulating products of a step have read operand region g (MMA commit)
        B_SCHEDFULL = 14, // [4] scheduler slot holds the CTA's next tile index (-1: no more)
        B_SCHEDEMPTY = 18,// [4] slot read by the two MMA warps and the 8 element-wise warps
        B_TFULL = 22,     // [NSTAGE] step: streamed tiles (and, MODE 1, their row vectors) loaded
        B_TEMPTY = 22 + NSTAGE,
        B_COUNT = 22 + 2 * NSTAGE
    };
    auto bar = [&](int i) { return bars_u32 + i * 8; };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + B_COUNT) + 1;
    volatile int* sched_slot = reinterpret_cast<volatile int*>(bars + B_COUNT) + 2;   // [4]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // ---- the tiles of this CTA ----
    // Tiles of one head are neighbours in the order (their streamed tiles are shared in L2).
    // MODE 0: 128-row Q tile (causal: longest first) of a (batch, query head); steps = 64-key K/V tiles.
    // MODE 1: 128-key K/V tile (the first has the most steps) of a (batch, K/V head);
    //         steps = (query head of the group, 64-row Q tile) pairs.
    const int group = prm.H / prm.Hkv;
    const int tiles_per_head = MODE == 0 ? prm.n_qtiles : prm.n_ktiles;
    auto decode = [&](int lin) {
        BwdTile t;
        const int bid_tile = lin % tiles_per_head;
        t.bh_res = lin / tiles_per_head;
        if constexpr (MODE == 0) {
            t.tile = prm.causal ? prm.n_qtiles - 1 - bid_tile : bid_tile;
            const int last_key = attn_tc::last_visible_key(t.tile * BT + BT - 1, prm.Sk, prm.causal, 0);
            t.sub_lo = 0;
            t.sub_hi = last_key < 0 ? 0 : last_key / BS + 1;
            t.n_steps = t.sub_hi;
        } else {
            t.tile = bid_tile;
            t.sub_lo = prm.causal ? (t.tile * BT) / BS : 0;     // first 64-row Q tile with a row that sees key tile * BT
            t.sub_hi = (prm.Sq + BS - 1) / BS;
            if (t.sub_lo > t.sub_hi) t.sub_lo = t.sub_hi;
            t.n_steps = (t.sub_hi - t.sub_lo) * group;
        }
        t.kv_bh_of_q = (t.bh_res / prm.H) * prm.Hkv + (t.bh_res % prm.H) / group;
        return t;
    };
    // streamed tile of step u of tile t: (head index in its tensor, index of the 64-row tile)
    auto step_head = [&](const BwdTile& t, int u) {
        if constexpr (MODE == 0) return t.kv_bh_of_q;
        else return (t.bh_res / prm.Hkv) * prm.H + (t.bh_res % prm.Hkv) * group + u / (t.sub_hi - t.sub_lo);
    };
    auto step_sub = [&](const BwdTile& t, int u) {
        if constexpr (MODE == 0) return u;
        else return t.sub_lo + u % (t.sub_hi - t.sub_lo);
    };
    // Consumers of the scheduler: the tile index at position p of this CTA's walk (-1: no more); the slot is handed
    // back at once (the caller keeps what it needs in registers).
    auto fetch = [&](int p, bool hand_back) -> int {
        const int slot = p & 3;
        if (!mbar_wait(bar(B_SCHEDFULL + slot), (p >> 2) & 1, abort_flag)) return -1;
        const int lin = sched_slot[slot];
        if (hand_back) mbar_arrive(bar(B_SCHEDEMPTY + slot));
        return lin;
    };
    // the next tile with work at or after position p (-1: none); tiles that nothing reaches are skipped
    auto next_work = [&](int p, bool hand_back, BwdTile& t) {
        for (;; ++p) {
            const int lin = fetch(p, hand_back);
            if (lin < 0) return -1;
            t = decode(lin);
            if (t.n_steps > 0) return p;
        }
    };

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar(B_RFULL), 1);
        mbar_init(bar(B_RTMEM), 256);
        mbar_init(bar(B_SLAST), 1);
        mbar_init(bar(B_ACCFINAL), 1);
        mbar_init(bar(B_ACCFREE), 256);
        mbar_init(bar(B_ESYNC), 256);
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar(B_SFULL + b), 1);
            mbar_init(bar(B_SREAD + b), 128);
            mbar_init(bar(B_PFULL + b), 128);
            mbar_init(bar(B_OPFREE + b), 1);
        }
        for (int s = 0; s < NSTAGE; ++s) {
            mbar_init(bar(B_TFULL + s), 1);
            mbar_init(bar(B_TEMPTY + s), 1);
        }
        for (int s = 0; s < 4; ++s) {
            mbar_init(bar(B_SCHEDFULL + s), 1);
            mbar_init(bar(B_SCHEDEMPTY + s), 10);
        }
        fence_barrier_init();
        fence_proxy_async_smem();
    }
    if (warp == 8) {
        tmem_alloc(smem_u32(tmem_slot), C::TMEM_COLS);
        tmem_relinquish();
    }
    if (warp == 9 && elect_one()) {
        prefetch_tensormap(&tmR0);
        prefetch_tensormap(&tmR1);
        prefetch_tensormap(&tmT0);
        prefetch_tensormap(&tmT1);
        prefetch_tensormap(&tmOut0);
        if constexpr (MODE == 1) prefetch_tensormap(&tmOut1);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    // Register re-balancing: 384 threads start with 168 registers each; the service warpgroup (warps 8-11) drops
    // to 64 and the two element-wise warpgroups rise to 216.
    if (warp >= 8) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
      if (warp == 9) {
        // =========================== TMA producer ===========================
        const bool leader = elect_one();
        BwdTile t;
        int gs = 0, kk = 0;   // steps and tiles (with work) so far
        bool ok = true;
        for (int p = 0; ok; ++p) {
            // draw the tile at position p of this CTA's walk and publish it
            const int slot = p & 3;
            if (!(ok = mbar_wait(bar(B_SCHEDEMPTY + slot), ((p >> 2) & 1) ^ 1, abort_flag))) break;
            int lin = -1;
            if (leader) {
                lin = (p == 0) ? static_cast<int>(blockIdx.x)
                      : (prm.counter ? static_cast<int>(gridDim.x + atomicAdd(prm.counter, 1u)) : prm.n_tiles_total);
                if (lin < 0 || lin >= prm.n_tiles_total) lin = -1;
                sched_slot[slot] = lin;
                mbar_arrive(bar(B_SCHEDFULL + slot));
            }
            lin = fetch(p, false);   // all lanes of the warp read it back
            if (lin < 0) break;
            t = decode(lin);
            if (t.n_steps == 0) continue;
            // the resident tiles' shared memory is free once the previous tile's have been copied into tensor memory
            // or, where they are read in place, once its last S / dP product has finished
            if (kk > 0 && !(ok = mbar_wait(bar(A_TMEM ? B_RTMEM : B_SLAST), (kk - 1) & 1, abort_flag))) break;
            if (leader) {
                mbar_arrive_expect_tx(bar(B_RFULL), 2 * C::RES_BYTES);
#pragma unroll
                for (int bx = 0; bx < NBOX; ++bx) {
                    tma_load_3d(sR(0) + bx * BT * 128, &tmR0, bar(B_RFULL), bx * 64, t.tile * BT, t.bh_res);
                    tma_load_3d(sR(1) + bx * BT * 128, &tmR1, bar(B_RFULL), bx * 64, t.tile * BT, t.bh_res);
                }
            }
            for (int u = 0; u < t.n_steps; ++u, ++gs) {
                const int st = gs % NSTAGE;
                if (!(ok = mbar_wait(bar(B_TEMPTY + st), ((gs / NSTAGE) & 1) ^ 1, abort_flag))) break;
                if (leader) {
                    mbar_arrive_expect_tx(bar(B_TFULL + st), 2 * C::STR_BYTES + (MODE == 1 ? 2 * BS * 4 : 0));
                    const int head = step_head(t, u), row0 = step_sub(t, u) * BS;
                    if constexpr (MODE == 1) {
                        // the prepared row vectors of the 64 streamed query rows (aligned and in bounds by construction)
                        const int64_t off = static_cast<int64_t>(head) * prm.Sq_pad + row0;
                        bulk_load_1d(sVec + st * 2 * BS * 4, prm.nl2 + off, BS * 4, bar(B_TFULL + st));
                        bulk_load_1d(sVec + st * 2 * BS * 4 + BS * 4, prm.ndelta + off, BS * 4, bar(B_TFULL + st));
                    }
#pragma unroll
                    for (int bx = 0; bx < NBOX; ++bx) {
                        tma_load_3d(sT(st, 0) + bx * BS * 128, &tmT0, bar(B_TFULL + st), bx * 64, row0, head);
                        tma_load_3d(sT(st, 1) + bx * BS * 128, &tmT1, bar(B_TFULL + st), bx * 64, row0, head);
                    }
                }
            }
            ++kk;
        }
      } else if (warp == 8 || warp == 10) {
        // =========================== MMA issuers ===========================
        const bool leader = elect_one();
        constexpr uint32_t IDESC_S = make_idesc_f16(BT, BS, DTYPE, 0, 0);    // both operands K-major (contraction over D)
        constexpr uint32_t IDESC_ACC = make_idesc_f16(BT, D, DTYPE, 0, 1);   // A from tensor memory, B MN-major (N = D)
        constexpr uint32_t DESC_HI = smem_desc_hi_sw128(1024);
        const uint32_t r_lo[2] = {smem_desc_lo(sR(0), 16), smem_desc_lo(sR(1), 16)};
        // S (or S^T) = R0 T0^T, dP (or dP^T) = R1 T1^T of global step gs : D / 16 instructions each (M 128, N 64, K 16)
        // product w of global step gs: w = 0: S into the S buffer of the step's parity, w = 1: dP
        auto issue_prod = [&](int gs, int w) {
            if (leader) {
                const int st = gs % NSTAGE;
                const uint32_t b0 = smem_desc_lo(sT(st, w), 16);
                const uint32_t dcol = tmem + (w == 0 ? C::s_col(gs & 1) : C::DP_COL);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t offa = ((kk >> 2) * BT * 128 + (kk & 3) * 32) >> 4;
                    const uint32_t offb = ((kk >> 2) * BS * 128 + (kk & 3) * 32) >> 4;
                    if constexpr (A_TMEM)
                        mma_f16_ts_lohi(dcol, tmem + C::rt_col(w) + kk * 8, b0 + offb, DESC_HI, IDESC_S, kk > 0);
                    else
                        mma_f16_ss_lohi(dcol, r_lo[w] + offa, b0 + offb, DESC_HI, IDESC_S, kk > 0);
                }
            }
        };
        // accumulating products of global step gs, step u of its tile (contraction step kk, 16 values = 8 columns,
        // starts at column 8 kk of its operand); afterwards its streamed tiles and its operand region are free
        auto issue_acc = [&](int gs, int u) {
            if (leader) {
                const int st = gs % NSTAGE;
                const uint32_t op = tmem + C::op_col(gs & 1);
                if constexpr (MODE == 0) {
                    // dQ += dS K_j : dS from tensor memory, K_j MN-major
                    const uint32_t b0 = smem_desc_lo(sT(st, 0), BS * 128);
#pragma unroll
                    for (int kk = 0; kk < BS / 16; ++kk)
                        mma_f16_ts_lohi(tmem + C::ACC0_COL, op + kk * 8, b0 + ((kk * 16 * 128) >> 4), DESC_HI,
                                        IDESC_ACC, (u > 0 || kk > 0) ? 1u : 0u);
                } else {
                    // dV += P^T dO_i, dK += dS^T Q_i; dO_i and Q_i MN-major
                    const uint32_t bdo = smem_desc_lo(sT(st, 1), BS * 128), bq = smem_desc_lo(sT(st, 0), BS * 128);
#pragma unroll
                    for (int kk = 0; kk < BS / 16; ++kk)
                        mma_f16_ts_lohi(tmem + C::ACC0_COL, op + kk * 8, bdo + ((kk * 16 * 128) >> 4), DESC_HI,
                                        IDESC_ACC, (u > 0 || kk > 0) ? 1u : 0u);
#pragma unroll
                    for (int kk = 0; kk < BS / 16; ++kk)
                        mma_f16_ts_lohi(tmem + C::ACC1_COL, op + 32 + kk * 8, bq + ((kk * 16 * 128) >> 4), DESC_HI,
                                        IDESC_ACC, (u > 0 || kk > 0) ? 1u : 0u);
                }
                mma_commit(bar(B_TEMPTY + st));
                mma_commit(bar(B_OPFREE + (gs & 1)));
            }
        };
        BwdTile t;
        int gs = 0, kk = 0;
        bool ok = true;
        if (warp == 8) {
            // dP of a step as soon as the previous step's S and dP are in its group's registers (also across tiles).
            // With two S buffers the S of a step was issued one step earlier, behind the previous dP (the first step of
            // a tile excepted: its resident operand is only then in place); the buffer it goes into was read two
            // steps ago.  With one buffer S and dP are issued together.
            for (int k = next_work(0, leader, t); k >= 0 && ok; k = next_work(k + 1, leader, t), ++kk) {
                if (!(ok = mbar_wait(bar(A_TMEM ? B_RTMEM : B_RFULL), kk & 1, abort_flag))) break;
                for (int u = 0; u < t.n_steps; ++u, ++gs) {
                    if (gs > 0 && !(ok = mbar_wait(bar(B_SREAD + ((gs - 1) & 1)), ((gs - 1) >> 1) & 1, abort_flag))) break;
                    const bool s_pending = !C::S2BUF || u == 0;
                    if (s_pending && !(ok = mbar_wait(bar(B_TFULL + gs % NSTAGE), (gs / NSTAGE) & 1, abort_flag))) break;
                    tc_fence_after_sync();
                    if (s_pending) issue_prod(gs, 0);
                    issue_prod(gs, 1);
                    if (leader) mma_commit(bar(B_SFULL + (gs & 1)));
                    if (u + 1 == t.n_steps) {
                        if (leader) mma_commit(bar(B_SLAST));
                    } else if (C::S2BUF) {
                        if (!(ok = mbar_wait(bar(B_TFULL + (gs + 1) % NSTAGE), ((gs + 1) / NSTAGE) & 1, abort_flag))) break;
                        issue_prod(gs + 1, 0);
                    }
                }
            }
        } else {
            // the accumulating products of a step as soon as its operands are in tensor memory (its streamed tiles
            // were loaded before its S and dP; this warp observes that barrier itself all the same); the first of a
            // tile overwrites the accumulators, which the previous tile's epilogue must have read
            for (int k = next_work(0, leader, t); k >= 0 && ok; k = next_work(k + 1, leader, t), ++kk) {
                for (int u = 0; u < t.n_steps; ++u, ++gs) {
                    if (!(ok = mbar_wait(bar(B_TFULL + gs % NSTAGE), (gs / NSTAGE) & 1, abort_flag))) break;
                    if (!(ok = mbar_wait(bar(B_PFULL + (gs & 1)), (gs >> 1) & 1, abort_flag))) break;
                    if (u == 0 && kk > 0 && !(ok = mbar_wait(bar(B_ACCFREE), (kk - 1) & 1, abort_flag))) break;
                    tc_fence_after_sync();
                    issue_acc(gs, u);
                    if (u + 1 == t.n_steps && leader) mma_commit(bar(B_ACCFINAL));
                }
            }
        }
      }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
        // =========================== element-wise groups + epilogue ===========================
        // Group g (warps 4g .. 4g+3) takes the steps with an even (g = 0) or odd (g = 1) global index: always operand
        // region g.  While one group waits for its tile or for tensor memory, the other computes.
        const int grp = warp >> 2;
        const int half = grp;                                // epilogue: which 32 of every 64 output columns
        const int r = (warp & 3) * 32 + lane;                // tensor-memory lane: query row (MODE 0) / key row (MODE 1)
        const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + C::s_col(grp) + lane_off, tDP = tmem + C::DP_COL + lane_off;   // own S buffer: steps of parity grp
        const uint32_t tOP = tmem + C::op_col(grp) + lane_off;
        const float c = prm.scale_log2;
        const uint64_t c2 = pack_f32x2(c, c);
        bool ok = true;
        // The barrier among the element-wise threads is an mbarrier with the same bounded wait as everything else (a
        // plain bar.sync would wait forever for a thread that has left through the time-out path).
        uint32_t esync_phase = 0;
        auto all_sync = [&]() -> bool {
            mbar_arrive(bar(B_ESYNC));
            const bool done = mbar_wait(bar(B_ESYNC), esync_phase & 1, abort_flag);
            ++esync_phase;
            return done;
        };
        // Group g copies resident tile g of the kk-th tile from shared memory (rows of 128 bytes per 64-column box,
        // 16-byte chunks swizzled by row) into tensor memory: lane = row, two 16-bit values per column in memory order.
        auto copy_resident = [&](int kk) -> bool {
            if (!mbar_wait(bar(B_RFULL), kk & 1, abort_flag)) return false;
            const uint32_t src = sR(grp) + r * 128;
#pragma unroll
            for (int bx = 0; bx < NBOX; ++bx) {
                uint32_t w[32];
#pragma unroll
                for (int g8 = 0; g8 < 8; ++g8)
                    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(w[g8 * 4 + 0]), "=r"(w[g8 * 4 + 1]), "=r"(w[g8 * 4 + 2]), "=r"(w[g8 * 4 + 3])
                                 : "r"(src + bx * BT * 128 + ((g8 ^ (r & 7)) << 4)) : "memory");
                tmem_st_32x32b_x32(tmem + C::rt_col(grp) + bx * 32 + lane_off, w);
            }
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(bar(B_RTMEM));
            return true;
        };

        // the next tile with work at or after position p; tiles on the way that nothing reaches (keys that no query
        // sees) get their zero gradients here
        auto next_tile = [&](int p, BwdTile& t) {
            for (;; ++p) {
                const int lin = fetch(p, lane == 0);
                if (lin < 0) return -1;
                t = decode(lin);
                if (t.n_steps > 0) return p;
                const int rows_total = MODE == 0 ? prm.Sq : prm.Sk;
                const int rows = rows_total - t.tile * BT < BT ? rows_total - t.tile * BT : BT;
                if (rows > 0) {
                    const int64_t first = static_cast<int64_t>(t.bh_res) * rows_total + t.tile * BT;
                    zero_rows(prm.out0, first, rows, D, tid, 256);
                    if constexpr (MODE == 1) zero_rows(prm.out1, first, rows, D, tid, 256);
                }
            }
        };
        BwdTile t, tn;
        int gs0 = 0, kk = 0;   // global index of the tile's first step; tiles so far
        int k = next_tile(0, t);
        if (A_TMEM && k >= 0) ok = copy_resident(0);
        for (; k >= 0 && ok; ++kk) {
            const int my_row = t.tile * BT + r;                  // global query row (MODE 0) or key index (MODE 1)
            float my_nl2 = 0.f, my_ndelta = 0.f;                 // MODE 0: minus this row's L * log2(e), minus its delta
            if constexpr (MODE == 0) {
                if (my_row < prm.Sq) {
                    my_nl2 = prm.nl2[static_cast<int64_t>(t.bh_res) * prm.Sq_pad + my_row];
                    my_ndelta = prm.ndelta[static_cast<int64_t>(t.bh_res) * prm.Sq_pad + my_row];
                }
            }
            for (int u = (gs0 + grp) & 1; u < t.n_steps && ok; u += 2) {     // own steps: global index gs0 + u = grp mod 2
                const int gs = gs0 + u;
                const int ts = step_sub(t, u);
                // MODE 1: -L log2(e) and -delta of the step's 64 query rows arrived with its streamed tiles
                const float* vnl2 = vec + (gs % NSTAGE) * 2 * BS;
                const float* vndl = vnl2 + BS;
                if constexpr (MODE == 1) {   // observe the bulk copies' barrier ourselves (it completed before S was issued)
                    if (!(ok = mbar_wait(bar(B_TFULL + gs % NSTAGE), (gs / NSTAGE) & 1, abort_flag))) break;
                }
                if (!(ok = mbar_wait(bar(B_SFULL + grp), (gs >> 1) & 1, abort_flag))) break;
                tc_fence_after_sync();
                // does any element of this step need the mask?  (uniform over the CTA)
                //   MODE 0: rows tile*128 .. +127, keys ts*64 .. +63;  MODE 1: keys tile*128 .. +127, rows ts*64 .. +63
                const int key0 = MODE == 0 ? ts * BS : t.tile * BT, nkeys = MODE == 0 ? BS : BT;
                const int row0 = MODE == 0 ? t.tile * BT : ts * BS;
                const bool partial = (key0 + nkeys > prm.Sk) || (prm.causal && key0 + nkeys - 1 > row0);
                // the whole S and dP row of this step into registers, then tensor memory is free for the next step
                uint32_t sr[BS], dpr[BS];
#pragma unroll
                for (int ch = 0; ch < BS / 32; ++ch) {
                    tmem_ld_32x32b_x32(tS + 32 * ch, sr + 32 * ch);
                    tmem_ld_32x32b_x32(tDP + 32 * ch, dpr + 32 * ch);
                }
                tmem_ld_wait();
                tc_fence_before_sync();
                mbar_arrive(bar(B_SREAD + grp));
                // operand region `grp` was last read by the accumulating products of global step gs - 2
                bool op_free = gs < 2;
                // Two instances of the arithmetic: steps that need the mask (diagonal and ragged tiles) and all others,
                // whose code then carries no trace of the mask (predicated-off mask code more than doubled its time).
                auto make_operands = [&](auto masked_tag) {
                constexpr bool MASKED = decltype(masked_tag)::value;
#pragma unroll
                for (int ch = 0; ch < BS / 32; ++ch) {
                    uint32_t pk_p[16], pk_ds[16];
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        const int col = 32 * ch + e;
                        uint64_t nl2_2, ndl_2;
                        if constexpr (MODE == 0) {
                            nl2_2 = pack_f32x2(my_nl2, my_nl2);
                            ndl_2 = pack_f32x2(my_ndelta, my_ndelta);
                        } else {
                            const float2 a = *reinterpret_cast<const float2*>(vnl2 + col);
                            const float2 d = *reinterpret_cast<const float2*>(vndl + col);
                            nl2_2 = pack_f32x2(a.x, a.y);
                            ndl_2 = pack_f32x2(d.x, d.y);
                        }
                        float x0, x1;
                        unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sr[col]), __uint_as_float(sr[col + 1])), c2, nl2_2), x0, x1);
                        float p0 = ex2_approx(x0), p1 = ex2_approx(x1);
                        if constexpr (MASKED) {
                            bool v0, v1;
                            if constexpr (MODE == 0) {
                                v0 = key0 + col < prm.Sk && (!prm.causal || key0 + col <= my_row);
                                v1 = key0 + col + 1 < prm.Sk && (!prm.causal || key0 + col + 1 <= my_row);
                            } else {
                                v0 = my_row < prm.Sk && (!prm.causal || my_row <= row0 + col);
                                v1 = my_row < prm.Sk && (!prm.causal || my_row <= row0 + col + 1);
                            }
                            p0 = v0 ? p0 : 0.f;
                            p1 = v1 ? p1 : 0.f;
                        }
                        float d0, d1;
                        unpack_f32x2(mul_f32x2(pack_f32x2(p0, p1),
                                               add_f32x2(pack_f32x2(__uint_as_float(dpr[col]), __uint_as_float(dpr[col + 1])), ndl_2)), d0, d1);
                        if constexpr (MODE == 1) pk_p[e / 2] = pack2<DTYPE>(p0, p1);
                        pk_ds[e / 2] = pack2<DTYPE>(d0, d1);
                    }
                    // 32 values -> 16 columns of this group's operand region
                    if (!op_free) {
                        if (!(ok = mbar_wait(bar(B_OPFREE + grp), ((gs >> 1) - 1) & 1, abort_flag))) break;
                        tc_fence_after_sync();
                        op_free = true;
                    }
                    if constexpr (MODE == 0) {
                        tmem_st_32x32b_x16(tOP + 16 * ch, pk_ds);
                    } else {
                        tmem_st_32x32b_x16(tOP + 16 * ch, pk_p);
                        tmem_st_32x32b_x16(tOP + 32 + 16 * ch, pk_ds);
                    }
                }
                };
                if (partial) make_operands(std::true_type{}); else make_operands(std::false_type{});
                if (!ok) break;
                tmem_st_wait();
                tc_fence_before_sync();
                mbar_arrive(bar(B_PFULL + grp));
            }
            if (!ok) break;

            // ---- tile boundary ----
            // first the next tile's resident operand into tensor memory (its columns are free once this tile's last
            // S / dP product has finished), so that the next tile's first products run while this tile's accumulators drain
            const int kn = next_tile(k + 1, tn);
            if (A_TMEM && kn >= 0) {
                if (!(ok = mbar_wait(bar(B_SLAST), kk & 1, abort_flag))) break;
                tc_fence_after_sync();
                if (!(ok = copy_resident(kk + 1))) break;
            }
            // ---- epilogue: accumulators -> 16-bit -> swizzled staging tiles -> TMA stores (rows beyond the tensor clipped);
            // every 64-column piece of the output has a staging tile of its own: one barrier, then all stores at once ----
            if (!(ok = mbar_wait(bar(B_ACCFINAL), kk & 1, abort_flag))) break;
            tc_fence_after_sync();
            if (tid == 0) tma_store_wait_read<0>();              // the previous tile's stores have read the staging tiles
            if (!(ok = all_sync())) break;
#pragma unroll
            for (int a = 0; a < NACC; ++a) {
                // MODE 0: dQ (x scale).  MODE 1: accumulator 0 = dV, accumulator 1 = dK (x scale).
                const float f = (MODE == 0 || a == 1) ? prm.scale : 1.f;
                const uint32_t tA = tmem + (a == 0 ? C::ACC0_COL : C::ACC1_COL) + lane_off;
#pragma unroll
                for (int h = 0; h < D / 64; ++h) {
                    // 64 output columns per staging tile; this thread converts the 32 of its column half
                    uint32_t acc[32];
                    tmem_ld_32x32b_x32(tA + h * 64 + 32 * half, acc);
                    tmem_ld_wait();
                    if (a == NACC - 1 && h == D / 64 - 1) {      // the accumulators are in registers: the next tile may start
                        tc_fence_before_sync();
                        mbar_arrive(bar(B_ACCFREE));
                    }
                    const uint32_t ost = sStg + (a * (D / 64) + h) * C::OST_BYTES;
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        const uint32_t w0 = pack2<DTYPE>(__uint_as_float(acc[g * 8 + 0]) * f, __uint_as_float(acc[g * 8 + 1]) * f);
                        const uint32_t w1 = pack2<DTYPE>(__uint_as_float(acc[g * 8 + 2]) * f, __uint_as_float(acc[g * 8 + 3]) * f);
                        const uint32_t w2 = pack2<DTYPE>(__uint_as_float(acc[g * 8 + 4]) * f, __uint_as_float(acc[g * 8 + 5]) * f);
                        const uint32_t w3 = pack2<DTYPE>(__uint_as_float(acc[g * 8 + 6]) * f, __uint_as_float(acc[g * 8 + 7]) * f);
                        const uint32_t dst = ost + r * 128 + (((4 * half + g) ^ (r & 7)) << 4);   // 128-byte swizzle
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(w0), "r"(w1), "r"(w2), "r"(w3) : "memory");
                    }
                }
            }
            fence_proxy_async_smem();
            if (!(ok = all_sync())) break;
            if (tid == 0) {
#pragma unroll
                for (int a = 0; a < NACC; ++a)
#pragma unroll
                    for (int h = 0; h < D / 64; ++h)
                        tma_store_3d(a == 0 ? &tmOut0 : &tmOut1, sStg + (a * (D / 64) + h) * C::OST_BYTES, h * 64, t.tile * BT, t.bh_res);
                tma_store_commit();
            }
            gs0 += t.n_steps;
            k = kn;
            t = tn;
        }
        if (tid == 0) tma_store_wait_all<0>();   // the staging tiles must outlive their stores

    }

    // ---- teardown (also reached after a timed-out wait) ----
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) finish_cta(prm.status, *abort_flag != 0, prm.counter);
    if (warp == 8) tmem_dealloc(tmem, C::TMEM_COLS);
}

}  // namespace attn_grad
