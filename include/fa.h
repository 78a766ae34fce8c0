/*
 * fa.h — C ABI of the B200 (sm_100a) fused attention library.
 *
 * Exact scaled-dot-product attention as defined in the paper's Section 2.1:
 *     S = scale * Q K^T,  P = softmax_rows(S + causal mask),  O = P V        (forward)
 *     dV = P^T dO, dP = dO V^T, dS = dsoftmax(dP), dQ = scale dS K, dK = scale dS^T Q   (backward)
 * computed in BF16 with FP32 accumulation and an FP32 log-sum-exp per query row.
 *
 * Conventions shared by every entry point
 *   - All data pointers are DEVICE pointers on the current CUDA device, 16-byte aligned,
 *     dense and contiguous; the caller owns every buffer, the library allocates no device
 *     memory and keeps no reference after the call's work has finished on `stream`.
 *   - q, o, d_o, dq : [B, Sq, H,   D] bfloat16     (token-major: one token's heads are adjacent)
 *     k, v, dk, dv  : [B, Sk, Hkv, D] bfloat16
 *     lse           : [B, H, Sq]      float32, natural logarithm of the row's sum of exp(S)
 *   - Grouped-query attention: H % Hkv == 0; query head h reads key/value head h / (H / Hkv).
 *   - causal != 0: key j is visible to query i iff j <= i + (Sk - Sq).  A query without any
 *     visible key gets O = 0, LSE = -inf and contributes nothing to the gradients.
 *   - Supported: D in {64, 128}; B, H, Hkv, Sq, Sk >= 1; scale finite and > 0.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls enqueue work
 *     and return; they never synchronise.  Return value: FA_OK or an error code below; on any
 *     error nothing has been launched.
 *   - Every device-side wait is bounded.  If one gives up, the kernel records
 *     FA_ERR_DEVICE_TIMEOUT in a device status word, releases its tensor memory and exits;
 *     the outputs of THAT call are then undefined, and its other thread blocks stop waiting too.
 *     fa_last_device_status() reads (and clears) the word.  Calls made after a timeout, read or
 *     not, run normally: a recorded failure is tied to the launch that caused it.
 *   - Host-side cost: the TMA tensor maps of a call (4 to 9, a microsecond or so each) are
 *     encoded on every call; nothing is cached per pointer.  Per-device set-up (shared-memory
 *     opt-in of the kernels, architecture check) is done once per device ordinal, so one process
 *     may use the library on several GPUs (the device current at the call is the one used).
 */
#ifndef FA_B200_H_
#define FA_B200_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  FA_OK = 0,
  FA_ERR_INVALID_ARGUMENT = 1, /* null/misaligned pointer, non-positive size, bad scale, H % Hkv != 0 */
  FA_ERR_UNSUPPORTED = 2,      /* head dimension or GPU architecture not supported */
  FA_ERR_CUDA = 3,             /* a CUDA runtime/driver call failed (launch, tensor-map encode) */
  FA_ERR_WORKSPACE = 4,        /* workspace pointer null, misaligned or too small */
  FA_ERR_DEVICE_TIMEOUT = 5    /* a bounded device-side wait expired (see fa_last_device_status) */
};

/*
 * Forward pass (paper Section 2.1, first display; kernel design Section 3.1).
 * Reads q, k, v; overwrites o (bfloat16) and lse (float32).  One kernel launch on `stream`: short key
 * sequences (and D = 64 at most lengths) get a kernel with one 128-row tile per thread block and two
 * blocks per SM, the others one with two tiles per block that take turns on the tensor cores; both
 * compute the same thing (FA_FWD_TILE=0 or 1 in the environment, read at the first call, forces the
 * second or the first kernel for every call; FA_EMU_PER8=0..3 likewise fixes how many of every eight
 * exponentials are computed by the polynomial of Section 3.1.3 instead of the hardware unit).
 * Forward results are bit-reproducible from run to run.
 * Arithmetic: scores and all accumulation in FP32; the probabilities enter the second product
 * rounded to 16 bits, scaled by 2^-(running maximum) with the maximum refreshed only when it grew
 * by more than a factor 256 (Section 3.1.4); O is divided by the FP32 sum of the unrounded
 * probabilities, so |O - exact| <= 2^-8 * max|v| plus the rounding of O itself.
 */
int fa_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
           int B, int H, int Hkv, int Sq, int Sk, int D, float scale, int causal, void* stream);

/*
 * Bytes of scratch fa_bwd needs for these sizes: two FP32 row vectors [B, H, Sq_padded] (row dot
 * products of dO and O, and the log-sum-exp in base 2) plus an FP32 dQ accumulator of
 * B * H * Sq_padded * D elements (Sq_padded = Sq rounded up to 128).  Returns 0 for unsupported
 * sizes.  Host-only; launches nothing.
 */
size_t fa_bwd_workspace_bytes(int B, int H, int Hkv, int Sq, int Sk, int D);

/*
 * Forward pass with different query/key and value head dimensions (Section 5 benchmarks head
 * dimensions (192, 128) beside 64 and 128).  q: [B, Sq, H, Dqk], k: [B, Sk, Hkv, Dqk],
 * v: [B, Sk, Hkv, Dv], o: [B, Sq, H, Dv], lse: [B, H, Sq]; everything else as fa_fwd, including the
 * definition of scale (the caller passes it; 1/sqrt(Dqk) is customary) and the status codes.
 * Supported: (Dqk, Dv) = (192, 128); Dqk == Dv is forwarded to fa_fwd.  Other pairs return
 * FA_ERR_UNSUPPORTED.  There is no backward pass for (192, 128).
 */
int fa_fwd_hdim(const void* q, const void* k, const void* v, void* o, float* lse,
                int B, int H, int Hkv, int Sq, int Sk, int Dqk, int Dv, float scale, int causal,
                void* stream);

/*
 * Forward pass over a packed batch of sequences of different lengths (Section 3.3, variable
 * sequence length).  Sequences are concatenated along the token axis:
 *   q, o: [total_q, H, D]   k, v: [total_k, Hkv, D]   (bfloat16, device, 16-byte aligned)
 *   lse:  [H, total_q] float32
 *   cu_seqlens_q, cu_seqlens_k: device int32 [batch + 1], non-decreasing, first entry 0, last entry
 *     total_q / total_k; sequence b owns query tokens [cu_seqlens_q[b], cu_seqlens_q[b+1]) and key
 *     tokens [cu_seqlens_k[b], cu_seqlens_k[b+1]).  They are read on the device only and NOT
 *     checked: entries that break these rules give undefined results.
 *   max_seqlen_q: an upper bound of every query length (it sizes the grid); query rows beyond it
 *     would not be computed.
 *   order: device int32 [batch] permutation giving the sequences longest-first (output of
 *     fa_varlen_lpt_order), or NULL for index order.  With the longest sequences launched first the
 *     tail of the grid is short work (the paper sorts the batch the same way and caches the result;
 *     the array can be reused for as long as the lengths stay the same).
 * Each sequence is an independent attention problem with the semantics of fa_fwd (causal mask
 * aligned bottom-right per sequence; an empty key range gives O = 0, LSE = -inf).  D in {64, 128}.
 * Values of k and v must be finite everywhere (rows of a neighbouring sequence are multiplied by
 * exact zeros).  The backward pass is fa_bwd_varlen.  Status codes as fa_fwd.
 */
int fa_fwd_varlen(const void* q, const void* k, const void* v, void* o, float* lse,
                  const int* cu_seqlens_q, const int* cu_seqlens_k, const int* order,
                  int batch, int total_q, int total_k, int max_seqlen_q, int H, int Hkv, int D,
                  float scale, int causal, void* stream);

/*
 * Backward pass over a packed batch (the counterpart of fa_fwd_varlen; same packing, same rules for
 * cu_seqlens_q / cu_seqlens_k, which are read on the device and not checked).  q, o, d_o, dq:
 * [total_q, H, D]; k, v, dk, dv: [total_k, Hkv, D]; lse: [H, total_q] as written by fa_fwd_varlen.
 * max_seqlen_q / max_seqlen_k: upper bounds of the sequences' lengths (key tiles beyond
 * max_seqlen_k would not be processed).  D = 128 only.  `workspace`: at least
 * fa_bwd_varlen_workspace_bytes(batch, total_q, H, D) bytes, 256-byte aligned, caller-owned.
 * dq is accumulated with floating-point reductions of no fixed order (as in fa_bwd); dk, dv are
 * reproducible.  Four kernel launches on `stream`.  Status codes as fa_bwd.
 */
size_t fa_bwd_varlen_workspace_bytes(int batch, int total_q, int H, int D);
int fa_bwd_varlen(const void* q, const void* k, const void* v, const void* o, const float* lse,
                  const void* d_o, void* dq, void* dk, void* dv,
                  const int* cu_seqlens_q, const int* cu_seqlens_k, int batch, int total_q, int total_k,
                  int max_seqlen_q, int max_seqlen_k, int H, int Hkv, int D, float scale, int causal,
                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * Writes into order[0..batch) (device int32) the sequence indices sorted by decreasing work
 * (visible score area, ties by index) - the longest-processing-time-first order of Section 3.3.
 * batch <= 16384 (the sort is a quadratic rank sort); asynchronous on `stream`.
 */
int fa_varlen_lpt_order(const int* cu_seqlens_q, const int* cu_seqlens_k, int batch, int causal,
                        int* order, void* stream);

/*
 * Backward pass (paper Section 2.1, second display; kernel design Section 3.2).
 * Reads q, k, v, o, lse (as written by fa_fwd for the same arguments) and d_o; overwrites
 * dq, dk, dv (bfloat16; not accumulated into).  `workspace` is caller-owned device scratch of
 * at least fa_bwd_workspace_bytes(...) bytes, 256-byte aligned; its contents on entry are
 * ignored and on return are unspecified.  Three kernel launches on `stream`.
 * Default path (D = 64 and 128): dq is summed across key/value tiles with floating-point reductions
 * whose order is not fixed, so dq is not bit-reproducible; dk and dv are.  When the environment
 * variable FA_BWD_IMPL=split is set before the first call: a reduction-free two-kernel path whose
 * dq, dk and dv are all bit-reproducible (slower; it is what fa_bwd_deterministic runs).
 * FA_BWD_IMPL=pair (D = 128) runs the default path's main kernel on clusters of two thread blocks
 * (Section 3.2, 2-CTA backward); same results up to the order of the dq reductions.
 */
int fa_bwd(const void* q, const void* k, const void* v, const void* o, const float* lse,
           const void* d_o, void* dq, void* dk, void* dv,
           int B, int H, int Hkv, int Sq, int Sk, int D, float scale, int causal,
           void* workspace, size_t workspace_bytes, void* stream);

/*
 * Deterministic backward pass (paper Section 3.2, deterministic mode): same arguments, results and
 * errors as fa_bwd, but dq, dk and dv are bit-identical from run to run for every supported D.
 * The paper orders the dq reductions with per-tile semaphores; here the pass is split into a
 * dK/dV kernel and a dQ kernel that need no cross-block reduction at all (three launches; S and dP
 * are recomputed once more).  A workspace of fa_bwd_workspace_bytes(...) bytes is sufficient.
 */
int fa_bwd_deterministic(const void* q, const void* k, const void* v, const void* o, const float* lse,
                         const void* d_o, void* dq, void* dk, void* dv,
                         int B, int H, int Hkv, int Sq, int Sk, int D, float scale, int causal,
                         void* workspace, size_t workspace_bytes, void* stream);

/*
 * FP16 variants (the paper's kernels take FP16 or BF16 inputs, Section 5): q, k, v, o, d_o, dq,
 * dk, dv hold IEEE half-precision elements instead of bfloat16; everything else - layouts, lse,
 * workspace, stream, status codes - is as in fa_fwd / fa_bwd.  Both support D in {64, 128} (a
 * process running with FA_BWD_IMPL=pair gets FA_ERR_UNSUPPORTED from fa_bwd_f16).  Probabilities
 * are stored as FP16 (they are at most 256, the rescaling threshold), accumulation stays FP32.
 */
int fa_fwd_f16(const void* q, const void* k, const void* v, void* o, float* lse,
               int B, int H, int Hkv, int Sq, int Sk, int D, float scale, int causal, void* stream);
int fa_bwd_f16(const void* q, const void* k, const void* v, const void* o, const float* lse,
               const void* d_o, void* dq, void* dk, void* dv,
               int B, int H, int Hkv, int Sq, int Sk, int D, float scale, int causal,
               void* workspace, size_t workspace_bytes, void* stream);
/* fa_bwd_deterministic on FP16 elements (D in {64, 128}). */
int fa_bwd_deterministic_f16(const void* q, const void* k, const void* v, const void* o, const float* lse,
                             const void* d_o, void* dq, void* dk, void* dv,
                             int B, int H, int Hkv, int Sq, int Sk, int D, float scale, int causal,
                             void* workspace, size_t workspace_bytes, void* stream);

/* Static, human-readable name of a status code. */
const char* fa_status_string(int status);

/*
 * Synchronises `stream`, then returns FA_OK, FA_ERR_DEVICE_TIMEOUT if any kernel of this
 * library gave up on a wait since the last call (the word is cleared), or FA_ERR_CUDA if the
 * synchronisation itself failed.
 */
int fa_last_device_status(void* stream);

/*
 * Test hook for the software 2^x of the paper's Section 3.1.3: y[i] = emulated 2^x[i] for
 * n float32 device values, using exactly the device function the forward kernel uses.
 */
int fa_exp2_emulated(const float* x, float* y, size_t n, void* stream);

/*
 * Test hook, host only (no GPU needed): exercises the per-device bookkeeping behind the
 * "once per device ordinal" set-up named in the conventions above.  Returns FA_OK if flags of
 * different ordinals are independent and out-of-range ordinals are ignored.
 */
int fa_selftest_per_device_flags(void);

/*
 * Test hook for the bounded waits: launches one warp that waits on a barrier nobody arrives on.  The
 * wait gives up after its limit (about half a second), the kernel ends normally, and the next
 * fa_last_device_status() returns FA_ERR_DEVICE_TIMEOUT once; the context stays usable.
 */
int fa_selftest_unsatisfied_wait(void* stream);

/*
 * Backward pass for callers that must not allocate device memory.  (The paper has no counterpart
 * for this entry point; it exists for the way this library gets embedded.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a framework's allocator
 * callbacks or a memory-pool that forbids nested allocation, in a process whose device memory
 * was handed out in full at start-up, or in real-time loops where an allocation's implicit
 * synchronisation is not acceptable.  Such callers cannot supply fa_bwd's `workspace` either,
 * so this variant keeps the scratch inside the library: a file-scope device array of
 * FA_BWD_NOALLOC_MAX_BYTES, reserved on every GPU that loads the library until the process exits.
 *
 * Same arguments, layouts, results and error codes as fa_bwd, minus the workspace pair.
 *   - Sizes whose scratch need, fa_bwd_workspace_bytes(...), exceeds FA_BWD_NOALLOC_MAX_BYTES are
 *     refused with FA_ERR_WORKSPACE and nothing is launched.
 *   - The call allocates nothing: no cudaMalloc / cudaFree and no allocating library routine.
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  Make that first call outside any CUDA stream capture.
 *   - Every call on a device shares the one array, which still holds the previous call's
 *     contents; the part that must start from zero (the dQ accumulator) is cleared by the
 *     call's own first kernel.  Two calls that overlap on the GPU (different streams, no
 *     ordering between them) race on the array: serialise them.
 */
#define FA_BWD_NOALLOC_MAX_BYTES (40u * 1024u * 1024u)
int fa_bwd_noalloc(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o,
                   void* dq, void* dk, void* dv, int B, int H, int Hkv, int Sq, int Sk, int D, float scale,
                   int causal, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* FA_B200_H_ */
