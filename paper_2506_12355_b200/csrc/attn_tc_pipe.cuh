// Warp-specialised, pipelined tcgen05 attention forward kernel for head dims 64 and 128.
//
// One CTA owns TWO 128-row Q tiles of one (batch, head) and walks the K/V tiles of that head
// (the loop of Appendix C, Listings 1-2, with the prefetch of Listing 1 generalised to a
// multi-stage ring):
//
//   warps 0-3   softmax group of Q tile 0: S -> P (online softmax, exp2), rare O rescale, epilogue
//   warps 4-7   softmax group of Q tile 1
//   warp  8     MMA issuer: S_t = Q_t K_j^T and O_t += P_t V_j, accumulators in tensor memory
//   warp  9     TMA producer: Q tiles once, K_j / V_j tiles through a ring of shared-memory slots
//   warps 10-11 idle (they complete the third warpgroup so that registers can be re-balanced)
//
// While one softmax group turns S_t into P_t, the tensor core works on the other tile, so the
// exponentials and the MMAs overlap.  P_t is written back into the tensor-memory columns of
// S_t as 16-bit values and is the A operand of the second product, which is this
// architecture's form of the register-level fusion of the two GEMMs in Section 3.2.2.
//
// Running maximum: the reference maximum m of a row is only advanced when the true maximum
// has grown by more than 2^8; otherwise the stale m is kept (P values up to 256, exact after
// the final division by l), so the O accumulator rarely needs rescaling.
#pragma once
#include "attn_tc_basic.cuh"

namespace attn_tc {

template <int D>
struct PipeCfg {
    static constexpr int BM = 128;                       // rows of one Q tile
    static constexpr int BN = 128;                       // keys per K/V tile
    static constexpr int NBOX = D / 64;
    static constexpr int Q_BYTES = BM * D * 2;
    static constexpr int KV_BYTES = BN * D * 2;
    static constexpr int NSLOT = (D == 128) ? 5 : 8;     // ring slots (each holds one K or V tile)
    static constexpr int TILE_BYTES = 2 * Q_BYTES + NSLOT * KV_BYTES;
    static constexpr int MISC_BYTES = 512;               // barriers, TMEM slot, abort flag
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
    int causal;
    int* status;
    int n_pairs;          // 256-row Q tile pairs per head
    int BH;               // batch * heads
    int heads_per_group;  // heads whose K/V are walked together (L2 residency)
    int H, Hkv;           // query heads and key/value heads per batch element (H % Hkv == 0)
#ifdef ATTN_TC_PROFILE
    long long* prof;      // [grid][32] cycle sums per phase (development builds only)
#endif
};

#ifndef ATTN_SUM_MODE
#define ATTN_SUM_MODE 0
#endif
#ifndef ATTN_MAX3
#define ATTN_MAX3 0
#endif

#ifndef ATTN_PROF_ROW
#define ATTN_PROF_ROW 0
#endif
#ifdef ATTN_TC_PROFILE
#define PROF_DECL(n) long long prof_t0 = clock64(), prof_acc[n] = {}
#define PROF_LAP(i) do { const long long prof_t1 = clock64(); prof_acc[i] += prof_t1 - prof_t0; prof_t0 = prof_t1; } while (0)
#define PROF_STAMP(cond, slot) do { if (cond) prm.prof[blockIdx.x * 32 + (slot)] = clock64(); } while (0)
#define PROF_FLUSH(base, n) do { for (int i_ = 0; i_ < (n); ++i_) prm.prof[blockIdx.x * 32 + (base) + i_] = prof_acc[i_]; } while (0)
#else
#define PROF_DECL(n)
#define PROF_LAP(i)
#define PROF_STAMP(cond, slot)
#define PROF_FLUSH(base, n)
#endif

__device__ __forceinline__ void reg_inc_224() { asm volatile("setmaxnreg.inc.sync.aligned.u32 224;"); }
__device__ __forceinline__ void reg_dec_56() { asm volatile("setmaxnreg.dec.sync.aligned.u32 56;"); }

template <int D, int DTYPE, int POLY_NUM, int POLY_DEN>
__global__ void __launch_bounds__(384, 1)
attn_fwd_tc_pipe_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                        const __grid_constant__ CUtensorMap tmV, const PipeParams prm) {
    using C = PipeCfg<D>;
    constexpr int BM = C::BM, BN = C::BN, NBOX = C::NBOX, NSLOT = C::NSLOT;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    auto sQ = [&](int t) { return smem_base + t * C::Q_BYTES; };
    auto sKV = [&](int slot) { return smem_base + 2 * C::Q_BYTES + slot * C::KV_BYTES; };

    // misc area: barriers
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + C::TILE_BYTES);
    const uint32_t bars_u32 = smem_base + C::TILE_BYTES;
    enum { B_Q = 0, B_SFULL = 2, B_PFULL = 4, B_PFULL2 = 6, B_OFINAL = 8, B_KVFULL = 10, B_KVEMPTY = 10 + NSLOT,
           B_COUNT = 10 + 2 * NSLOT };
    auto bar = [&](int i) { return bars_u32 + i * 8; };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + B_COUNT) + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // ---- which work item ----
    int pair, bh;
    {
        const int lin = blockIdx.x;
        const int full_group = prm.heads_per_group * prm.n_pairs;
        const int g = lin / full_group, r = lin - g * full_group;
        int hg = prm.BH - g * prm.heads_per_group;
        if (hg > prm.heads_per_group) hg = prm.heads_per_group;
        const int pr = r / hg;
        bh = g * prm.heads_per_group + (r - pr * hg);
        pair = prm.causal ? prm.n_pairs - 1 - pr : pr;  // causal: longest rows first
    }
    const int q0 = pair * 2 * BM;
    // grouped-query attention: H / Hkv consecutive query heads read the same K/V head
    const int kv_bh = (bh / prm.H) * prm.Hkv + (bh % prm.H) / (prm.H / prm.Hkv);

    // K/V tiles each Q tile needs
    int n_kv[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int qs = q0 + t * BM;
        if (qs >= prm.Sq) {
            n_kv[t] = 0;
        } else {
            int last_key = prm.Sk - 1;
            if (prm.causal && qs + BM - 1 < last_key) last_key = qs + BM - 1;
            n_kv[t] = last_key / BN + 1;
        }
    }
    const int n_max = n_kv[0] > n_kv[1] ? n_kv[0] : n_kv[1];

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar(B_Q + 0), 1);
        mbar_init(bar(B_Q + 1), 1);
        for (int t = 0; t < 2; ++t) {
            mbar_init(bar(B_SFULL + t), 1);
            mbar_init(bar(B_PFULL + t), 128);    // first three quarters of P_t written
            mbar_init(bar(B_PFULL2 + t), 128);   // rest of P_t written
            mbar_init(bar(B_OFINAL + t), 1);
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
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    if (warp >= 8) {
        reg_dec_56();
        // Both service warps run their loops with all 32 lanes (uniform control flow keeps the
        // address arithmetic on the uniform datapath); one elected lane issues the TMA / MMA
        // instructions.
        if (warp == 9) {
            // =========================== TMA producer ===========================
            const bool leader = elect_one();
            PROF_DECL(2);
            auto load_q = [&](int t) {
                if (leader) {
                    mbar_arrive_expect_tx(bar(B_Q + t), C::Q_BYTES);
#pragma unroll
                    for (int bx = 0; bx < NBOX; ++bx)
                        tma_load_3d(sQ(t) + bx * BM * 128, &tmQ, bar(B_Q + t), bx * 64, q0 + t * BM, bh);
                }
            };
            auto load_kv = [&](const CUtensorMap* map, int item, int j) -> bool {
                const int slot = item % NSLOT;
                const uint32_t use = item / NSLOT;
                if (!mbar_wait(bar(B_KVEMPTY + slot), (use & 1) ^ 1, abort_flag)) return false;
                PROF_LAP(0);
                if (leader) {
                    mbar_arrive_expect_tx(bar(B_KVFULL + slot), C::KV_BYTES);
#pragma unroll
                    for (int bx = 0; bx < NBOX; ++bx)
                        tma_load_3d(sKV(slot) + bx * BN * 128, map, bar(B_KVFULL + slot), bx * 64, j * BN, kv_bh);
                }
                return true;
            };
            if (n_kv[0] > 0) load_q(0);
            for (int j = 0; j < n_max; ++j) {
                if (!load_kv(&tmK, 2 * j, j)) break;
                if (j == 0 && n_kv[1] > 0) load_q(1);
                if (!load_kv(&tmV, 2 * j + 1, j)) break;
                PROF_LAP(1);
            }
#ifdef ATTN_TC_PROFILE
            if (leader) PROF_FLUSH(24, 2);
#endif
        } else if (warp == 8) {
            // =========================== MMA issuer ===========================
            const bool leader = elect_one();
            constexpr uint32_t IDESC_S = make_idesc_f16(BM, BN, DTYPE, 0, 0);
            constexpr uint32_t IDESC_O = make_idesc_f16(BM, D, DTYPE, 0, 1);
            constexpr uint32_t DESC_HI = smem_desc_hi_sw128(1024);
            const uint32_t q_lo[2] = {smem_desc_lo(sQ(0), 16), smem_desc_lo(sQ(1), 16)};
            const uint32_t k_lo0 = smem_desc_lo(sKV(0), 16);          // K tile in slot 0 (K-major)
            const uint32_t v_lo0 = smem_desc_lo(sKV(0), BN * 128);    // V tile in slot 0 (MN-major)
            auto issue_s = [&](int t, int slot) {   // S_t = Q_t K^T : D/16 instructions of K = 16
                if (leader) {
                    const uint32_t a0 = q_lo[t], b0 = k_lo0 + slot * (C::KV_BYTES >> 4);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t off = ((kk >> 2) * 128 * 128 + (kk & 3) * 32) >> 4;
                        mma_f16_ss_lohi(tmem + C::s_col(t), a0 + off, b0 + off, DESC_HI, IDESC_S, kk > 0);
                    }
                }
            };
            auto issue_pv = [&](int t, int slot, bool accumulate, int kk_begin, int kk_end) {
                if (leader) {                       // O_t += P_t V : K = 16 keys per instruction
                    const uint32_t b0 = v_lo0 + slot * (C::KV_BYTES >> 4);
#pragma unroll
                    for (int kk = kk_begin; kk < kk_end; ++kk)
                        mma_f16_ts_lohi(tmem + C::o_col(t), tmem + C::s_col(t) + kk * 8, b0 + ((kk * 16 * 128) >> 4),
                                        DESC_HI, IDESC_O, (accumulate || kk > 0) ? 1u : 0u);
                }
            };
            auto commit = [&](int b) {
                if (leader) mma_commit(bar(b));
            };
            auto kv_full_wait = [&](int item) {
                return mbar_wait(bar(B_KVFULL + item % NSLOT), (item / NSLOT) & 1, abort_flag);
            };
            bool ok = true;
            if (n_max > 0) {
                if (n_kv[0] > 0) ok = mbar_wait(bar(B_Q + 0), 0, abort_flag);
                ok = ok && kv_full_wait(0);
                if (ok && n_kv[0] > 0) {
                    tc_fence_after_sync();
                    issue_s(0, 0);
                    commit(B_SFULL + 0);
                }
                if (ok && n_kv[1] > 0) {
                    ok = mbar_wait(bar(B_Q + 1), 0, abort_flag);
                    if (ok) {
                        tc_fence_after_sync();
                        issue_s(1, 0);
                        commit(B_SFULL + 1);
                    }
                }
                if (ok) commit(B_KVEMPTY + 0);
            }
            PROF_DECL(12);
            for (int j = 0; j < n_max && ok; ++j) {
                const int vitem = 2 * j + 1, kitem = 2 * j + 2;
                const int vslot = vitem % NSLOT, kslot = kitem % NSLOT;
                const uint32_t par = j & 1;
                // both tiles of this step are normally long loaded: check them off the P -> S critical path
                if (!(ok = kv_full_wait(vitem))) break;
                bool k_ready = false;
                if (j + 1 < n_max) {
                    if (!(ok = kv_full_wait(kitem))) break;
                    k_ready = true;
                }
                PROF_LAP(0);
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if (j < n_kv[t]) {
                        if (!(ok = mbar_wait(bar(B_PFULL + t), par, abort_flag))) break;
                        PROF_LAP(1 + 5 * t);
                        tc_fence_after_sync();
                        issue_pv(t, vslot, j > 0, 0, 3 * BN / 64);
                        if (!(ok = mbar_wait(bar(B_PFULL2 + t), par, abort_flag))) break;
                        PROF_STAMP(leader && t == 0 && j == 64, 27);
                        PROF_LAP(2 + 5 * t);
                        tc_fence_after_sync();
                        issue_pv(t, vslot, true, 3 * BN / 64, BN / 16);
                        if (j + 1 == n_kv[t]) commit(B_OFINAL + t);
                    }
                    if (t == 1) commit(B_KVEMPTY + vslot);
                    PROF_LAP(3 + 5 * t);
                    if (j + 1 < n_kv[t]) {
                        if (!k_ready) {
                            if (!(ok = kv_full_wait(kitem))) break;
                            k_ready = true;
                        }
                        PROF_LAP(4 + 5 * t);
                        tc_fence_after_sync();
                        issue_s(t, kslot);
                        commit(B_SFULL + t);
                        PROF_STAMP(leader && t == 0 && j == 64, 28);
                    }
                    PROF_LAP(5 + 5 * t);
                }
                if (ok && j + 1 < n_max) commit(B_KVEMPTY + kslot);
            }
#ifdef ATTN_TC_PROFILE
            if (leader) PROF_FLUSH(0, 12);
#endif
        }
    } else {
        // =========================== softmax groups ===========================
        reg_inc_224();
        const int t = warp >> 2;                       // Q tile of this group
        const int r = tid & 127;                       // row inside the tile
        const int row = q0 + t * BM + r;
        const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + C::s_col(t) + lane_off, tO = tmem + C::o_col(t) + lane_off;
        const float c = prm.scale_log2;
        const int n = n_kv[t];
        float m = -INFINITY, l = 0.f;
        bool ok = true;

        PROF_DECL(6);
        for (int j = 0; j < n; ++j) {
            if (!(ok = mbar_wait(bar(B_SFULL + t), j & 1, abort_flag))) break;
            PROF_STAMP(t == 0 && r == 0 && j == 65, 29);
            PROF_LAP(0);
            tc_fence_after_sync();
            uint32_t sr[BN];
#pragma unroll
            for (int ch = 0; ch < BN / 32; ++ch) tmem_ld_32x32b_x32(tS + ch * 32, sr + ch * 32);
            tmem_ld_wait();
            PROF_LAP(1);

            const int kv0 = j * BN;
            const bool need_mask = (kv0 + BN > prm.Sk) || (prm.causal && kv0 + BN - 1 > q0 + t * BM);
            bool done = false;

            if (j > 0 && !need_mask) {
                // ---- fast path: exponentials against the reference maximum of the previous tiles,
                // the row maximum of this tile computed on the side.  Valid when no row of the warp
                // has grown by more than 2^8; otherwise everything is redone by the general path.
                const float mc = m * c;
                const uint64_t c2 = pack_f32x2(c, c), nmc2 = pack_f32x2(-mc, -mc);
#if ATTN_SUM_MODE == 0
                uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};   // 8 partial row sums
#else
                float accs[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#endif
                float mxs[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) mxs[i] = fmaxf(__uint_as_float(sr[2 * i]), __uint_as_float(sr[2 * i + 1]));
                auto exp_chunk = [&](int ch) {
                    uint32_t pk[16];
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
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
#if ATTN_SUM_MODE == 0
                        acc[(e / 2) & 3] = add_f32x2(acc[(e / 2) & 3], pack_f32x2(p0, p1));
#else
                        accs[e & 7] += p0;
                        accs[(e & 7) + 1] += p1;
#endif
                        pk[e / 2] = pack2<DTYPE>(p0, p1);
                    }
                    tmem_st_32x32b_x16(tS + ch * 16, pk);   // P overwrites the S columns already in registers
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
                if (!__any_sync(0xffffffffu, (mx - m) * c > 8.f)) {
                    tmem_st_wait();
                    tc_fence_before_sync();
                    mbar_arrive(bar(B_PFULL + t));          // first three quarters of P are in place
                    PROF_LAP(2);
                    exp_chunk(BN / 32 - 1);
#if ATTN_SUM_MODE == 0
                    float a0, a1, a2, a3;
                    unpack_f32x2(add_f32x2(acc[0], acc[1]), a0, a1);
                    unpack_f32x2(add_f32x2(acc[2], acc[3]), a2, a3);
                    l += (a0 + a1) + (a2 + a3);
#else
                    l += ((accs[0] + accs[1]) + (accs[2] + accs[3])) + ((accs[4] + accs[5]) + (accs[6] + accs[7]));
#endif
                    done = true;
                }
            }

            if (!done) {
                // ---- general path: first tile, diagonal / ragged tile, or a row maximum that ran ahead
                const int lim = !need_mask ? 0x7fffffff
                                           : ((prm.causal && row < prm.Sk - 1) ? row : prm.Sk - 1);  // last visible key
                float mx = -INFINITY;
#pragma unroll
                for (int e = 0; e < BN; ++e) {
                    const float sv = (kv0 + e <= lim) ? __uint_as_float(sr[e]) : -INFINITY;
                    sr[e] = __float_as_uint(sv);
                    mx = fmaxf(mx, sv);
                }
                // advance the reference maximum only when the true one ran ahead by more than 2^8
                float alpha = 1.f;
                if (j == 0) {
                    m = (mx == -INFINITY) ? 0.f : mx;
                } else if ((mx - m) * c > 8.f) {
                    alpha = ex2_approx((m - mx) * c);
                    m = mx;
                }
                // rescale the running O (its last update finished before S_j was produced)
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
                const float mc = m * c;
                float rs = 0.f;
#pragma unroll
                for (int ch = 0; ch < BN / 32; ++ch) {
                    uint32_t pk[16];
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        const float s0 = __uint_as_float(sr[ch * 32 + e]), s1 = __uint_as_float(sr[ch * 32 + e + 1]);
                        // masked entries are -inf; keep them 0 also for a zero scale (-inf * 0 = NaN)
                        const float p0 = (s0 == -INFINITY) ? 0.f : ex2_approx(fmaf(s0, c, -mc));
                        const float p1 = (s1 == -INFINITY) ? 0.f : ex2_approx(fmaf(s1, c, -mc));
                        rs += p0 + p1;
                        pk[e / 2] = pack2<DTYPE>(p0, p1);
                    }
                    tmem_st_32x32b_x16(tS + ch * 16, pk);
                    if (ch == BN / 32 - 2) {
                        tmem_st_wait();
                        tc_fence_before_sync();
                        mbar_arrive(bar(B_PFULL + t));
                    }
                }
                l = l * alpha + rs;
            }
            PROF_LAP(3);
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(bar(B_PFULL2 + t));
            PROF_STAMP(t == 0 && r == 0 && j == 64, 26);
            PROF_LAP(4);
        }
#ifdef ATTN_TC_PROFILE
        if (r == ATTN_PROF_ROW) PROF_FLUSH(12 + 6 * t, 6);
#endif

        // ---- epilogue: O / l and LSE ----
        if (ok && n > 0) ok = mbar_wait(bar(B_OFINAL + t), 0, abort_flag);
        if (ok && n > 0) {
            tc_fence_after_sync();
            const float inv = (l > 0.f) ? 1.f / l : 0.f;
            const int64_t grow = static_cast<int64_t>(bh) * prm.Sq + row;
            uint4* orow = reinterpret_cast<uint4*>(static_cast<uint8_t*>(prm.o) + grow * D * 2);
#pragma unroll
            for (int ch = 0; ch < D / 32; ++ch) {
                uint32_t orr[32];
                tmem_ld_32x32b_x32(tO + ch * 32, orr);
                tmem_ld_wait();
                if (row < prm.Sq) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        uint4 w;
                        w.x = pack2<DTYPE>(__uint_as_float(orr[g * 8 + 0]) * inv, __uint_as_float(orr[g * 8 + 1]) * inv);
                        w.y = pack2<DTYPE>(__uint_as_float(orr[g * 8 + 2]) * inv, __uint_as_float(orr[g * 8 + 3]) * inv);
                        w.z = pack2<DTYPE>(__uint_as_float(orr[g * 8 + 4]) * inv, __uint_as_float(orr[g * 8 + 5]) * inv);
                        w.w = pack2<DTYPE>(__uint_as_float(orr[g * 8 + 6]) * inv, __uint_as_float(orr[g * 8 + 7]) * inv);
                        orow[ch * 4 + g] = w;
                    }
                }
            }
            if (row < prm.Sq) prm.lse[grow] = (l > 0.f) ? m * prm.scale + logf(l) : -INFINITY;
        }
    }

    // ---- teardown (also reached after a timed-out wait) ----
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0 && *abort_flag != 0) atomicExch(prm.status, kStatusTimeout);
    if (warp == 8) tmem_dealloc(tmem, C::TMEM_COLS);
}

}  // namespace attn_tc
