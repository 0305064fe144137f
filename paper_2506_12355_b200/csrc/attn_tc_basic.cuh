// Basic tcgen05 attention forward kernel (no warp specialisation).
//
// One CTA of 128 threads owns one 128-row Q tile of one (batch, head) and walks the
// K/V tiles of that head (the loop of Appendix C, Listings 1-2):
//
//     S   = Q K_j^T           tcgen05.mma, operands in shared memory, S in tensor memory
//     P,l = online softmax    one thread per row; exp2 with the scale folded in
//     O  += P V_j             tcgen05.mma, P read from tensor memory, V_j from shared memory
//
// K_j/V_j tiles arrive through a two-stage TMA ring so that the next tile loads while the
// current one is processed.  Everything else is serial inside the CTA: this kernel is the
// correctness baseline of the tensor-core path and the fallback for shapes the pipelined
// kernel does not take.
#pragma once
#include "sm100_ptx.cuh"

namespace attn_tc {

using namespace sm100;

constexpr int kStatusTimeout = 9;  // ATTN_ERR_DEVICE_TIMEOUT

template <int D>
struct BasicCfg {
    static constexpr int BM = 128;
    static constexpr int BN = (D == 256) ? 64 : 128;
    static constexpr int NSTAGE = 2;
    static constexpr int NBOX = D / 64;                 // 64-column (128-byte) boxes per row
    static constexpr int Q_BYTES = BM * D * 2;
    static constexpr int KV_BYTES = BN * D * 2;         // one K tile or one V tile
    static constexpr int SMEM_BYTES = Q_BYTES + NSTAGE * 2 * KV_BYTES + 1024;  // + alignment slack
    static constexpr int S_COL = 0;                     // S: BN fp32 columns
    static constexpr int P_COL = BN;                    // P: BN/2 columns (two 16-bit values each)
    static constexpr int O_COL = (D == 64) ? 192 : 256; // O: D fp32 columns
    static constexpr int TMEM_COLS = (D == 64) ? 256 : 512;
};

struct Params {
    void* o;
    float* lse;
    int Sq, Sk;
    float scale;        // multiplies Q K^T
    float scale_log2;   // scale * log2(e)
    int causal;
    int* status;        // device status word
    int H, Hkv;         // query heads and key/value heads per batch element (H % Hkv == 0)
};

template <int D, int DTYPE>
__global__ void __launch_bounds__(128, 1)
attn_fwd_tc_basic_kernel(const __grid_constant__ CUtensorMap tmQ,
                         const __grid_constant__ CUtensorMap tmK,
                         const __grid_constant__ CUtensorMap tmV, const Params prm) {
    using C = BasicCfg<D>;
    constexpr int BM = C::BM, BN = C::BN, NBOX = C::NBOX;

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_q, bar_kv[C::NSTAGE], bar_mma, bar_p;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5;
    const int q0 = blockIdx.x * BM;
    const int bh = blockIdx.y;
    const int kv_bh = (bh / prm.H) * prm.Hkv + (bh % prm.H) / (prm.H / prm.Hkv);  // grouped-query attention

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;
    auto sK = [&](int st) { return smem_base + C::Q_BYTES + st * 2 * C::KV_BYTES; };
    auto sV = [&](int st) { return smem_base + C::Q_BYTES + st * 2 * C::KV_BYTES + C::KV_BYTES; };

    const uint32_t b_q = smem_u32(&bar_q), b_mma = smem_u32(&bar_mma), b_p = smem_u32(&bar_p);
    auto b_kv = [&](int st) { return smem_u32(&bar_kv[st]); };

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(b_q, 1);
        for (int st = 0; st < C::NSTAGE; ++st) mbar_init(b_kv(st), 1);
        mbar_init(b_mma, 1);
        mbar_init(b_p, 128);
        fence_barrier_init();
        fence_proxy_async_smem();
        prefetch_tensormap(&tmQ);
        prefetch_tensormap(&tmK);
        prefetch_tensormap(&tmV);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), C::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    const uint32_t lane_off = static_cast<uint32_t>(warp * 32) << 16;  // this warp's TMEM lanes
    const uint32_t tS = tmem + C::S_COL, tP = tmem + C::P_COL, tO = tmem + C::O_COL;

    // number of K/V tiles this Q tile needs
    int last_key = prm.Sk - 1;
    if (prm.causal && q0 + BM - 1 < last_key) last_key = q0 + BM - 1;
    const int n_kv = last_key / BN + 1;

    auto load_kv = [&](int j) {
        const int st = j % C::NSTAGE;
        mbar_arrive_expect_tx(b_kv(st), 2 * C::KV_BYTES);
        for (int bx = 0; bx < NBOX; ++bx) {
            tma_load_3d(sK(st) + bx * BN * 128, &tmK, b_kv(st), bx * 64, j * BN, kv_bh);
            tma_load_3d(sV(st) + bx * BN * 128, &tmV, b_kv(st), bx * 64, j * BN, kv_bh);
        }
    };

    constexpr uint32_t IDESC_S = make_idesc_f16(BM, BN, DTYPE, 0, 0);  // Q, K_j both K-major
    constexpr uint32_t IDESC_O = make_idesc_f16(BM, D, DTYPE, 0, 1);   // P K-major (TMEM), V_j MN-major

    auto issue_s = [&](int st) {  // S = Q K_j^T : D/16 instructions of K = 16
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = (kk >> 2) * 128 * 128 + (kk & 3) * 32;
            const uint32_t offk = (kk >> 2) * BN * 128 + (kk & 3) * 32;
            mma_f16_ss(tS, make_smem_desc_sw128(sQ + off, 16, 1024),
                       make_smem_desc_sw128(sK(st) + offk, 16, 1024), IDESC_S, kk > 0);
        }
    };
    auto issue_o = [&](int st, bool accumulate) {  // O += P V_j : BN/16 instructions of K = 16
#pragma unroll
        for (int kk = 0; kk < BN / 16; ++kk) {
            mma_f16_ts(tO, tP + kk * 8, make_smem_desc_sw128(sV(st) + kk * 16 * 128, BN * 128, 1024),
                       IDESC_O, (accumulate || kk > 0) ? 1u : 0u);
        }
    };

    float m = -INFINITY, l = 0.f;
    const int row = q0 + tid;
    const float c = prm.scale_log2;
    uint32_t ph_mma = 0, ph_p = 0;
    bool ok = true;

    if (tid == 0) {
        mbar_arrive_expect_tx(b_q, C::Q_BYTES);
        for (int bx = 0; bx < NBOX; ++bx) tma_load_3d(sQ + bx * BM * 128, &tmQ, b_q, bx * 64, q0, bh);
        load_kv(0);
        ok = mbar_wait(b_q, 0, &abort_flag) && mbar_wait(b_kv(0), 0, &abort_flag);
        if (ok) {
            tc_fence_after_sync();
            issue_s(0);
            mma_commit(b_mma);
        }
    }
    __syncwarp();
    if (warp == 0) ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;

    for (int j = 0; j < n_kv && ok; ++j) {
        const int st = j % C::NSTAGE;

        // ---- S_j ready (also: O += P V_{j-1} finished, so its stage is free again) ----
        if (!(ok = mbar_wait(b_mma, ph_mma, &abort_flag))) break;
        ph_mma ^= 1;
        if (tid == 0 && j + 1 < n_kv) load_kv(j + 1);
        __syncwarp();
        tc_fence_after_sync();

        uint32_t sr[BN];
#pragma unroll
        for (int ch = 0; ch < BN / 32; ++ch) tmem_ld_32x32b_x32(tS + lane_off + ch * 32, sr + ch * 32);
        tmem_ld_wait();

        const int kv0 = j * BN;
        const bool need_mask = (kv0 + BN > prm.Sk) || (prm.causal && kv0 + BN - 1 > q0);
        float mx = -INFINITY;
        if (need_mask) {
            const int lim = (prm.causal && row < prm.Sk - 1) ? row : prm.Sk - 1;  // last visible key
#pragma unroll
            for (int e = 0; e < BN; ++e) {
                const float s = (kv0 + e <= lim) ? __uint_as_float(sr[e]) : -INFINITY;
                sr[e] = __float_as_uint(s);
                mx = fmaxf(mx, s);
            }
        } else {
#pragma unroll
            for (int e = 0; e < BN; ++e) mx = fmaxf(mx, __uint_as_float(sr[e]));
        }
        const float m_new = fmaxf(m, mx);
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
        const float mc = m_use * c;
        const float alpha = (m == -INFINITY) ? 0.f : ex2_approx(fmaf(m, c, -mc));
        float rs = 0.f;
        uint32_t pk[BN / 2];
#pragma unroll
        for (int e = 0; e < BN; e += 2) {
            float s0 = __uint_as_float(sr[e]), s1 = __uint_as_float(sr[e + 1]);
            // masked entries are -inf; keep them 0 also when the scale is 0 (-inf * 0 = NaN)
            float p0 = (s0 == -INFINITY) ? 0.f : ex2_approx(fmaf(s0, c, -mc));
            float p1 = (s1 == -INFINITY) ? 0.f : ex2_approx(fmaf(s1, c, -mc));
            rs += p0 + p1;
            pk[e / 2] = pack2<DTYPE>(p0, p1);
        }
        l = l * alpha + rs;
        m = m_new;

#pragma unroll
        for (int ch = 0; ch < BN / 64; ++ch) tmem_st_32x32b_x32(tP + lane_off + ch * 32, pk + ch * 32);

        if (j > 0) {  // rescale the running O
#pragma unroll
            for (int ch = 0; ch < D / 32; ++ch) {
                uint32_t orr[32];
                tmem_ld_32x32b_x32(tO + lane_off + ch * 32, orr);
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 32; ++e) orr[e] = __float_as_uint(__uint_as_float(orr[e]) * alpha);
                tmem_st_32x32b_x32(tO + lane_off + ch * 32, orr);
            }
        }
        tmem_st_wait();
        tc_fence_before_sync();
        mbar_arrive(b_p);

        if (tid == 0) {
            ok = mbar_wait(b_p, ph_p, &abort_flag);
            if (ok) {
                tc_fence_after_sync();
                issue_o(st, j > 0);
                if (j + 1 < n_kv)
                    ok = mbar_wait(b_kv((j + 1) % C::NSTAGE), ((j + 1) / C::NSTAGE) & 1, &abort_flag);
                if (ok) {
                    if (j + 1 < n_kv) {
                        tc_fence_after_sync();
                        issue_s((j + 1) % C::NSTAGE);
                    }
                    mma_commit(b_mma);
                }
            }
        }
        ph_p ^= 1;
        __syncwarp();
        if (warp == 0) ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    }

    // ---- epilogue: O / l, LSE ----
    if (ok) ok = mbar_wait(b_mma, ph_mma, &abort_flag);
    if (ok) {
        tc_fence_after_sync();
        const float inv = (l > 0.f) ? 1.f / l : 0.f;
        const int64_t grow = static_cast<int64_t>(bh) * prm.Sq + row;
        uint4* orow = reinterpret_cast<uint4*>(static_cast<uint8_t*>(prm.o) + grow * D * 2);
#pragma unroll
        for (int ch = 0; ch < D / 32; ++ch) {
            uint32_t orr[32];
            tmem_ld_32x32b_x32(tO + lane_off + ch * 32, orr);
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

    // ---- teardown (also reached after a timed-out wait) ----
    tc_fence_before_sync();
    __syncthreads();
    if (abort_flag != 0 && tid == 0) atomicExch(prm.status, kStatusTimeout);
    if (warp == 0) tmem_dealloc(tmem, C::TMEM_COLS);
}

}  // namespace attn_tc
