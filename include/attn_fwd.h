/*
 * attn_fwd.h -- C ABI of the fused attention forward operator for NVIDIA B200 (sm_100a).
 *
 * The operator is the one defined in Section 2.2 of the paper,
 *
 *     Attention(Q, K, V) = Softmax(Mask(Q K^T / sqrt(d))) V ,
 *
 * evaluated FlashAttention-style (Section 2.2 / the kernel loop of Appendix C's
 * listings: a Q tile stays on chip, K/V tiles stream through shared memory, the
 * softmax is computed online with a running maximum and running sum, and the
 * S x S score matrix never reaches global memory).  In addition to O the library
 * returns the per-row logsumexp of the scaled, masked scores.
 *
 * Conventions
 *   - All tensors are row-major and contiguous:  Q, O: [B, H, Sq, D];  K, V: [B, H, Sk, D];
 *     LSE: [B, H, Sq] in fp32.  Q, K, V, O share one 16-bit type (attn_dtype_t).
 *   - scale multiplies Q K^T (the paper uses 1/sqrt(d)); it must be finite and >= 0.
 *   - causal != 0 applies the lower-triangular mask aligned to the top-left corner:
 *     key j is visible to query i iff j <= i, also when Sq != Sk.
 *   - LSE[i] = ln( sum over visible j of exp(scale * <q_i, k_j>) )   (natural log).
 *   - A row without any visible key (Sk == 0, or a K/V shard that the causal mask hides from the
 *     row) gives O = 0, LSE = -inf.
 *   - Accumulation is fp32; the probabilities are rounded to the 16-bit input type
 *     before the second product; O is rounded once at the end.
 *
 * Ownership and asynchrony
 *   - The caller owns every buffer.  The library allocates no device memory.  (attn_fwd_host and
 *     attn_fwd_splitkv create a few streams and events of their own on first use, see there.)
 *   - Device entry points only enqueue work on `stream` (a cudaStream_t, may be NULL for
 *     the default stream) and return; they never synchronise.
 *   - Nothing throws; every entry point returns an attn_status_t (0 = success).
 *   - Q, K, V must not alias O or LSE.
 *
 * Streams and CUDA graphs
 *   - Launches may be issued on any number of streams at once.  A problem with more work items
 *     than the GPU has multiprocessors draws its items from a device-side work counter that lives in
 *     the library image; the kernel leaves it zeroed, so nothing but the kernel is enqueued.  Eager
 *     launches use the counter of their stream: at most 768 distinct streams per device may launch
 *     such problems over the life of the process (the per-thread default stream counts once per
 *     host thread); a stream handle that is destroyed and handed out again keeps its counter.
 *   - Every entry point that takes a `stream` may be captured into a CUDA graph, provided the first
 *     call for that device, head dim and type was made outside capture (one-time set-up).  Each
 *     captured launch of such a problem takes a counter of its own that eager launches never use,
 *     so a graph can be replayed on any stream while eager launches run elsewhere; at most 256 such
 *     launches can be captured per device and process.  Two executable graphs instantiated from the
 *     SAME capture share its counters and must not run at the same time.
 *   - When either limit is exhausted the launch is refused with ATTN_ERR_COUNTER_SLOTS.
 *
 * There is no CPU fallback: on a device that is not compute capability 10.x the entry
 * points return ATTN_ERR_UNSUPPORTED_ARCH.
 */
#ifndef ATTN_FWD_H_
#define ATTN_FWD_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ATTN_DTYPE_FP8_E4M3 names the 8-bit input format of attn_fwd_fp8 only; every entry point with a
 * `dtype` argument accepts the two 16-bit types and answers ATTN_ERR_UNSUPPORTED_DTYPE otherwise. */
typedef enum { ATTN_DTYPE_FP16 = 0, ATTN_DTYPE_BF16 = 1, ATTN_DTYPE_FP8_E4M3 = 2 } attn_dtype_t;

typedef enum {
    ATTN_OK = 0,
    ATTN_ERR_NULL_POINTER = 1,         /* a required pointer is NULL */
    ATTN_ERR_BAD_SHAPE = 2,            /* negative extent, or an extent/product out of range */
    ATTN_ERR_UNSUPPORTED_HEAD_DIM = 3, /* D is not 64, 128 or 256 */
    ATTN_ERR_UNSUPPORTED_DTYPE = 4,    /* dtype is not an attn_dtype_t */
    ATTN_ERR_MISALIGNED = 5,           /* q/k/v/o not 16-byte aligned, lse not 4-byte aligned */
    ATTN_ERR_BAD_SCALE = 6,            /* scale is NaN, infinite or negative */
    ATTN_ERR_UNSUPPORTED_ARCH = 7,     /* current device is not compute capability 10.x */
    ATTN_ERR_CUDA = 8,                 /* a CUDA runtime/driver call failed */
    ATTN_ERR_DEVICE_TIMEOUT = 9,       /* a kernel gave up on a bounded on-chip wait */
    ATTN_ERR_WORKSPACE = 10,           /* workspace missing, misaligned or too small */
    ATTN_ERR_STATIC_CAPACITY = 11,     /* problem does not fit the library's built-in staging buffer */
    ATTN_ERR_COUNTER_SLOTS = 12        /* no work counter left for this launch (see "Streams and CUDA graphs") */
} attn_status_t;

/*
 * attn_fwd -- the hot path (Section 2.2; kernel loop as in Appendix C, Listings 1-2).
 *
 * q, k, v : device pointers, 16-byte aligned, layouts above, element type `dtype`.
 * o       : device pointer, 16-byte aligned, [B,H,Sq,D], element type `dtype` (written).
 * lse     : device pointer, [B,H,Sq] fp32 (written).
 * B, H, Sq, Sk >= 0;  D in {64, 128, 256};  B*H <= 2^31-1, Sq, Sk <= 2^31-1-256.
 * B*H*Sq == 0 is a successful no-op.  Sk == 0 writes O = 0 and LSE = -inf.
 * Pointers of tensors without elements may be NULL (q, o, lse when B*H*Sq == 0; k, v when
 * B*H*Sk == 0); every other pointer must be non-NULL.
 * Runs on sm_100a tensor cores (tcgen05 MMAs with TMEM accumulators, TMA tile loads).
 * Validation happens on the host before anything is enqueued; on an error nothing is
 * launched.
 */
int attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Sq,
             int Sk, int D, float scale, int causal, int dtype, void* stream);

/*
 * attn_fwd_gqa -- grouped-query / multi-query attention (the GQA and MQA variants of Section 2.2
 * and Table 1): K and V carry Hkv heads, [B, Hkv, Sk, D], and query head h reads key/value head
 * h / (H / Hkv).  H must be a multiple of Hkv (Hkv == H is attn_fwd, Hkv == 1 is MQA); otherwise
 * ATTN_ERR_BAD_SHAPE.  Everything else -- layouts of Q, O, LSE, mask, scale, errors, asynchrony --
 * is as for attn_fwd.  The query heads of one K/V head are scheduled next to each other so that
 * their K/V tiles are shared through L2.
 */
int attn_fwd_gqa(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv,
                 int Sq, int Sk, int D, float scale, int causal, int dtype, void* stream);

/*
 * attn_fwd_partial -- attention of all queries over ONE SHARD of the keys and values (split-KV
 * decoding in the manner of FlashDecoding, which the paper cites in its related work, and key/value
 * sharding across GPUs).  k, v: [B, Hkv, Sk, D] hold the keys with GLOBAL indices
 * k_offset .. k_offset + Sk - 1; with the causal mask key (k_offset + j) is visible to query i iff
 * k_offset + j <= i.  o: [B,H,Sq,D] and lse: [B,H,Sq] receive the shard's own normalised result
 * O_r and LSE_r; rows that see no key of the shard get O_r = 0 and LSE_r = -inf.  k_offset >= 0.
 * With k_offset == 0 and the whole key range this is attn_fwd_gqa.  Merge shards with attn_combine.
 */
int attn_fwd_partial(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv,
                     int Sq, int Sk, int D, float scale, int causal, int k_offset, int dtype, void* stream);

/*
 * attn_combine -- merges the partial results of n_parts disjoint K/V shards (1 <= n_parts <= 1024):
 *     LSE = ln sum_r exp(LSE_r),    O = sum_r exp(LSE_r - LSE) O_r,
 * the rescaling identity of the online softmax applied across shards.
 * o_parts: device, [n_parts, B, H, Sq, D] (16-bit, `dtype`), 16-byte aligned; lse_parts: device,
 * [n_parts, B, H, Sq] fp32; o: [B,H,Sq,D]; lse: [B,H,Sq].  D must be a multiple of 8.  Rows for which
 * every shard reports -inf give O = 0, LSE = -inf.  Memory-bound; enqueued on `stream`.
 */
int attn_combine(const void* o_parts, const float* lse_parts, int n_parts, void* o, float* lse, int B, int H,
                 int Sq, int D, int dtype, void* stream);

/*
 * attn_combine_gather -- attn_combine with every shard's partial result behind its own pointer, for a range
 * of rows: the merge step of a K/V-sharded run across GPUs as ONE kernel that reads the other ranks'
 * partial results in place.  o_parts, lse_parts: HOST arrays of n_parts (1..32) DEVICE pointers; part r is
 * [B,H,Sq,D] in `dtype` (16-byte aligned) and [B,H,Sq] fp32.  The pointers may refer to peer GPUs' memory
 * (peer access enabled, or a symmetric-memory / IPC mapping): the kernel reads them with plain loads over
 * NVLink (no TMA, no multicast), so nothing has to be all-gathered first.  row_begin, row_count: the rows of
 * the flattened (batch, head, query) axis this call merges (a rank usually takes its own slice); o, lse:
 * device, full-size [B,H,Sq,D] / [B,H,Sq], of which only those rows are written.  The caller orders the call
 * after the producers of every part (a barrier across the ranks on `stream`) and keeps the parts alive until it
 * has finished.  The pointer arrays are read before the call returns.  Errors as attn_combine, plus
 * ATTN_ERR_BAD_SHAPE for n_parts or a row range out of bounds.
 */
int attn_combine_gather(const void* const* o_parts, const float* const* lse_parts, int n_parts, void* o, float* lse,
                        int B, int H, int Sq, int D, int dtype, long long row_begin, long long row_count, void* stream);

/*
 * attn_fwd_splitkv -- attn_fwd_gqa with the keys split into n_splits ranges that are computed side by
 * side, followed by the merge of attn_combine: split-KV decoding in the manner of FlashDecoding,
 * which the paper cites in its related work.  For problems with few query rows (a handful of heads,
 * one or a few queries each) and many keys, one launch has too few work items to fill the GPU;
 * splitting the keys gives every range its own items.  Arguments and conventions as attn_fwd_gqa,
 * plus: n_splits in 1..64 (clamped to the number of 128-key tiles; 1 is plain attn_fwd_gqa);
 * workspace: caller-owned DEVICE buffer of at least attn_fwd_splitkv_workspace_bytes(...) bytes,
 * 256-byte aligned, which receives the ranges' partial results ([n_splits,B,H,Sq,D] in `dtype`, then
 * [n_splits,B,H,Sq] fp32).  K and V are read in place (no copies).  For head dims 64 and 128 the key
 * ranges are work items of ONE launch of the persistent kernel on `stream`; for head dim 256 they
 * are one launch each, on up to 16 streams of the library's own (created with their events on the
 * first such call on a device), ordered after the work already on `stream`.  The merge runs on
 * `stream` after them.
 * The partial outputs are rounded to `dtype` before the merge, so O carries one more 16-bit rounding
 * than attn_fwd_gqa.  Errors: as attn_fwd_gqa, plus ATTN_ERR_BAD_SHAPE for n_splits outside 1..64
 * and ATTN_ERR_WORKSPACE.
 */
int attn_fwd_splitkv(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv,
                     int Sq, int Sk, int D, float scale, int causal, int dtype, int n_splits, void* workspace,
                     size_t workspace_bytes, void* stream);

/* Bytes of device workspace attn_fwd_splitkv needs (0 for an invalid shape). */
size_t attn_fwd_splitkv_workspace_bytes(int B, int H, int Sq, int D, int n_splits);

/*
 * attn_fwd_qkv_dims -- attention whose Q/K head dim differs from its V/O head dim: the MLA head
 * shape of Section 4.1 / Table 2 (embedding dimension 128 plus RoPE dimension 64 for Q and K,
 * 128 for V).  q: [B,H,Sq,Dqk], k: [B,Hkv,Sk,Dqk], v: [B,Hkv,Sk,Dv], o: [B,H,Sq,Dv], lse: [B,H,Sq].
 * Supported: (Dqk, Dv) = (192, 128), and Dqk == Dv in {64, 128, 256} (then identical to
 * attn_fwd_gqa); anything else returns ATTN_ERR_UNSUPPORTED_HEAD_DIM.  Grouped K/V heads, mask,
 * scale, errors and asynchrony as for attn_fwd_gqa.
 */
int attn_fwd_qkv_dims(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv,
                      int Sq, int Sk, int Dqk, int Dv, float scale, int causal, int dtype, void* stream);

/*
 * attn_fwd_fp8 -- the operator on 8-bit inputs: the FP8 case study of Section 4.4 (Table 6: causal
 * MHA, head dim 128).  The paper reports throughput only and fixes neither the 8-bit format nor a
 * scaling scheme; this entry point takes E4M3 (1 sign, 4 exponent bits with bias 7, 3 fraction bits,
 * no infinities, largest finite value 448) with one positive dequantisation factor per tensor:
 *
 *     O = Softmax(Mask(scale * (q_factor Q)(k_factor K)^T)) (v_factor V),
 *     LSE[i] = ln sum over visible j of exp(scale * q_factor * k_factor * <q_i, k_j>).
 *
 * q: device, [B,H,Sq,D] bytes; k, v: device, [B,Hkv,Sk,D] bytes (H % Hkv == 0); o: device,
 * [B,H,Sq,D] bf16; lse: device, [B,H,Sq] fp32.  D must be 128 (ATTN_ERR_UNSUPPORTED_HEAD_DIM
 * otherwise).  q, k, v, o 16-byte aligned.  scale finite and >= 0; the factors finite and > 0
 * (ATTN_ERR_BAD_SCALE otherwise).  Inputs must be finite: the bytes 0x7f and 0xff are NaN in this
 * format, and a NaN in K or V can reach rows from which the mask hides that key.
 * impl 0: tensor-core kernel -- both products are 8-bit MMAs with fp32 accumulation; the
 * probabilities are rounded to E4M3 (with a power-of-two factor that keeps them in the format's
 * normal range) for the second product, which is the one approximation beyond the 16-bit path:
 * each probability carries a relative rounding error of at most 2^-4, so
 * |O - O_exact| <= 2^-4 * sum_j p_j |v_factor v_j| elementwise, and typically ~4 % of O's own
 * root-mean-square size; LSE is not affected (the row sum is taken in fp32 before rounding).
 * impl 1: the CUDA-core cross-check kernel of attn_fwd_simt on the same inputs (fp32 throughout,
 * no rounding of the probabilities).  Other values: ATTN_ERR_UNSUPPORTED_DTYPE.
 * Mask, empty-row convention, ownership, errors and asynchrony as for attn_fwd_gqa.
 */
int attn_fwd_fp8(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv, int Sq,
                 int Sk, int D, float scale, float q_factor, float k_factor, float v_factor, int causal, int impl,
                 void* stream);

/*
 * attn_bwd -- backward pass: the gradients of the operator of Section 2.2,
 * O = Softmax(Mask(scale Q K^T)) V, with respect to Q, K and V for an upstream gradient dO = dL/dO.
 * (The paper measures the forward pass only; this is the chain rule applied to its definition.)
 *
 *     P = exp(scale Q K^T - LSE)  (visible keys; 0 elsewhere)      dP = dO V^T
 *     dS = P o (dP - rowsum(dO o O))       dV = P^T dO       dQ = scale dS K       dK = scale dS^T Q
 *
 * q, o, dout : device, [B,H,Sq,D] (`dtype`), 16-byte aligned; o and lse are the OUTPUTS of the forward call
 *              (attn_fwd / attn_fwd_gqa) on the same q, k, v, scale and mask.
 * k, v       : device, [B,Hkv,Sk,D]; H % Hkv == 0 (grouped heads as in attn_fwd_gqa).
 * lse        : device, [B,H,Sq] fp32.
 * dq         : device, [B,H,Sq,D] (written);  dk, dv: device, [B,Hkv,Sk,D] (written; with grouped heads
 *              they hold the sum over the query heads of the group).  Same 16-bit type as the inputs.
 * D in {64, 128} (otherwise ATTN_ERR_UNSUPPORTED_HEAD_DIM); top-left causal mask as in attn_fwd.
 * workspace  : device, 256-byte aligned, at least attn_bwd_workspace_bytes(B,H,Sq) bytes (it holds two
 *              fp32 values per query row, -LSE log2(e) and -rowsum(dO o O), rows padded to a multiple
 *              of 64 per head); owned by the caller, may be reused as soon as the stream has passed
 *              this call.  Missing, misaligned or too small: ATTN_ERR_WORKSPACE.
 * Rows of dq whose query sees no key, and rows of dk, dv whose key no query sees, are zero.  Empty
 * tensors may come with NULL pointers.  Three kernels are enqueued on `stream` (the row sums, the dQ
 * pass, the dK/dV pass); nothing is synchronised; the results are deterministic (no atomics).
 * Accumulation is fp32; P and dS are rounded to the 16-bit type before their second products.
 * Errors: as attn_fwd_gqa, plus the above.
 */
int attn_bwd(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* dout,
             void* dq, void* dk, void* dv, int B, int H, int Hkv, int Sq, int Sk, int D, float scale, int causal,
             int dtype, void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of device workspace attn_bwd needs (0 for an invalid shape). */
size_t attn_bwd_workspace_bytes(int B, int H, int Sq);

/*
 * attn_fwd_simt -- same operator, same arguments, same conventions, computed by a plain
 * CUDA-core kernel (one warp per query row, fp32 arithmetic, online softmax).  It is one to
 * two orders of magnitude slower than attn_fwd and exists as an on-device cross-check that
 * uses none of the tensor-core machinery.
 */
int attn_fwd_simt(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H,
                  int Sq, int Sk, int D, float scale, int causal, int dtype, void* stream);

/*
 * attn_fwd_host -- attn_fwd for HOST buffers.  q, k, v, o, lse are host pointers (pinned
 * memory makes the copies asynchronous); `workspace` is a caller-owned DEVICE buffer of at
 * least attn_fwd_host_workspace_bytes(...) bytes, 256-byte aligned.  Enqueues on `stream`:
 * three host-to-device copies, the attention kernel, two device-to-host copies.  The results
 * are valid once the caller has synchronised `stream`.
 * Large problems (at least 16 MiB of Q, K, V and at least 4 heads) are split into up to 8 groups
 * of heads: the kernels of the groups run on `stream`, the copies on two streams of the library's
 * own (created with their events on the first such call on a device), so that copies in both
 * directions overlap the kernels.  Everything is ordered after the work already on `stream`, and
 * `stream` waits for the last copy back, so the caller sees the same ordering as for the small
 * case.  Calls from several host threads are serialised while they enqueue.
 * Errors: as attn_fwd, plus ATTN_ERR_WORKSPACE.
 */
int attn_fwd_host(const void* q_host, const void* k_host, const void* v_host, void* o_host,
                  float* lse_host, int B, int H, int Sq, int Sk, int D, float scale, int causal,
                  int dtype, void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of device workspace attn_fwd_host needs for this problem (0 for an invalid shape). */
size_t attn_fwd_host_workspace_bytes(int B, int H, int Sq, int Sk, int D);

/*
 * attn_fwd_host_static -- attn_fwd_host for callers that cannot allocate device memory.
 * (The paper has no counterpart to this entry point; it is a convenience of this library.)
 *
 * Who needs it: code that holds host buffers but may not call cudaMalloc or any allocating
 * routine at the point of the call -- for example a plug-in running inside a host application
 * that owns the device memory budget, a real-time loop where an allocation (an implicit
 * device-wide synchronisation) is not acceptable, or a process whose memory pool is already
 * committed.  attn_fwd_host asks such a caller for a device workspace it has no means to
 * provide; this variant stages Q, K, V, O and LSE in a buffer that is part of the library image
 * itself: a file-scope `static __device__` array of ATTN_STATIC_WORKSPACE_BYTES (16 MiB), which
 * every GPU that loads the library holds from module load until the process exits.
 *
 * Arguments, layouts, conventions and asynchrony are those of attn_fwd_host without the
 * workspace pair; q, k, v, o, lse are HOST pointers and the results are valid once `stream`
 * has been synchronised.  The call allocates nothing: no cudaMalloc, cudaFree or allocating
 * library routine is reached on this path.
 *
 * Limit: attn_fwd_host_workspace_bytes(B,H,Sq,Sk,D) must not exceed
 * attn_fwd_host_static_capacity(); larger problems are refused with ATTN_ERR_STATIC_CAPACITY
 * before anything is enqueued.  Other errors: as attn_fwd_host.
 *
 * Set-up: the first call on each device looks up the device address of the built-in buffer
 * (once per device, with that device current).  Make that first call outside any stream
 * capture; later calls on the same device do no set-up.
 *
 * Sharing: there is ONE buffer per device and every call uses it from offset 0.  It keeps the
 * previous call's bytes; nothing in it has to start at zero, because each call overwrites every
 * region before reading it (Q, K, V by the host-to-device copies, O and LSE by the kernel).
 * Two calls whose work overlaps on the GPU (different streams, or several host threads)
 * race on the buffer and corrupt each other's results: issue the calls on one stream, or
 * otherwise order them.
 */
#define ATTN_STATIC_WORKSPACE_BYTES (16u << 20)
int attn_fwd_host_static(const void* q_host, const void* k_host, const void* v_host, void* o_host,
                         float* lse_host, int B, int H, int Sq, int Sk, int D, float scale,
                         int causal, int dtype, void* stream);

/* Capacity in bytes of the built-in staging buffer used by attn_fwd_host_static. */
size_t attn_fwd_host_static_capacity(void);

/* ATTN_OK if attn_fwd supports (D, dtype, causal) on the current device, otherwise the
 * status attn_fwd would return.  Launches nothing. */
int attn_query_support(int D, int dtype, int causal);

/* Synchronises `stream`, then returns and clears the device-side status word of the current
 * device: ATTN_OK, or ATTN_ERR_DEVICE_TIMEOUT if any kernel since the last call gave up on a
 * bounded wait (its output is then undefined).  ATTN_ERR_CUDA if the synchronisation fails. */
int attn_last_device_status(void* stream);

/* Static, human-readable name of a status code. */
const char* attn_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* ATTN_FWD_H_ */
