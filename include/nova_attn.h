/*
 * nova_attn.h - C ABI of libnova_attn: fused causal multi-head attention for NVIDIA B200 (sm_100a).
 *
 * The library implements, as hand-written CUDA, the attention sub-graph that the Nova compiler
 * collapses into single kernels (paper Section 4.2, "Attention as a First-Class Lowering"):
 *   forward  - scores = scale * Q K^T, causal mask from indices, online base-2 softmax, O = P V,
 *              log-sum-exp of every row saved for the backward pass;
 *   backward - P recomputed from the saved log-sum-exp (never stored), dV, dP, dS, dQ, dK.
 *
 * Conventions shared by every entry point
 *   - All tensor pointers are DEVICE pointers on the current CUDA device, owned by the caller, and
 *     must be 16-byte aligned, non-overlapping, and stay valid until the work enqueued on `stream`
 *     has finished.  Inputs are never modified; outputs are fully overwritten.
 *   - Q, K, V, O, dO, dQ, dK, dV: bf16, shape [B, H, T, D], contiguous (D fastest).
 *     LSE, Delta: fp32, shape [B, H, T].
 *   - D must be 64 or 128.  Any T >= 1 is accepted (partial tiles are handled inside).  Self
 *     attention only (queries and keys share T); no dropout, bias or grouped heads.
 *   - `scale` multiplies Q K^T before the softmax and must be finite and > 0.
 *   - `causal` != 0 keeps key j for query i iff j <= i; 0 keeps every key.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls only
 *     enqueue work on that stream: they never synchronise the device and never allocate device
 *     memory.
 *   - Return value: NOVA_ATTN_OK (0) or a negative nova_attn_status.  Arguments are validated on the
 *     host before anything is launched; a failed call has launched nothing.
 *   - Every wait inside the kernels is bounded.  If one expires, or a kernel finds at start-up that it
 *     cannot run as built (both indicate a bug or a broken device, never a property of the input), the
 *     kernel records NOVA_ATTN_ERR_TIMEOUT in a device status word, releases what it holds and returns;
 *     nova_attn_poll_device_status() reads the word.
 *   - Because calls only enqueue, a sequence of them may be captured into a CUDA graph and replayed
 *     (pointers, shapes and the workspace are baked into the graph); call each entry point once on the
 *     device before capturing, so that its one-time set-up is not part of the capture.
 *   - Kernels are launched so that each may begin its set-up while the previous kernel in `stream` is
 *     still draining (programmatic dependent launch); each waits for its predecessor before it reads or
 *     writes global memory, so stream order is what the caller observes.
 */
#ifndef NOVA_ATTN_H_
#define NOVA_ATTN_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum nova_attn_status {
    NOVA_ATTN_OK = 0,
    NOVA_ATTN_ERR_NULL = -1,        /* a required pointer is NULL */
    NOVA_ATTN_ERR_SHAPE = -2,       /* B, H or T <= 0, or B*H*T*D overflows the supported range */
    NOVA_ATTN_ERR_UNSUPPORTED = -3, /* D not in {64, 128}, or the device is not sm_100 */
    NOVA_ATTN_ERR_ALIGNMENT = -4,   /* a tensor pointer is not 16-byte aligned */
    NOVA_ATTN_ERR_SCALE = -5,       /* scale is not finite or not > 0 */
    NOVA_ATTN_ERR_WORKSPACE = -6,   /* workspace is NULL or smaller than nova_attn_bwd_workspace_bytes */
    NOVA_ATTN_ERR_CUDA = -7,        /* a CUDA runtime/driver call failed; see nova_attn_last_cuda_error */
    NOVA_ATTN_ERR_TIMEOUT = -8      /* a bounded device-side wait expired (reported by the poll call) */
} nova_attn_status;

/*
 * Forward pass (paper Section 4.2: the nova.online_attention loop - score contraction, index mask,
 * running max / sum in base 2, value contraction, causal loop clamp, 1/sum in the epilogue, and
 * "saves the log-sum-exp of each row for the backward pass").
 *   Q, K, V : in,  bf16 [B,H,T,D]
 *   O       : out, bf16 [B,H,T,D]   O_i = sum_j softmax_j(scale * q_i.k_j) v_j over the kept keys
 *   LSE     : out, fp32 [B,H,T]     natural-log log-sum-exp of the kept scaled scores of row i
 * bf16 operands feed the tensor cores, accumulation and all softmax arithmetic are fp32 (Section 4.3).
 */
int nova_attn_fwd(const void* Q, const void* K, const void* V, void* O, float* LSE,
                  int B, int H, int T, int D, float scale, int causal, void* stream);

/*
 * Backward preprocess: Delta_i = sum_d dO[i,d] * O[i,d], the row term of the softmax Jacobian
 * (equal to sum_j P_ij dP_ij).  The paper's backward (Section 4.2, "The Backward Pass") does not
 * spell this step out; it is the standard way to obtain dS = P * (dP - Delta) without a second
 * reduction over keys.  Memory bound: reads O and dO once.
 *   O, dO : in,  bf16 [B,H,T,D]   (O as written by nova_attn_fwd)
 *   Delta : out, fp32 [B,H,T]
 */
int nova_attn_bwd_preprocess(const void* O, const void* dO, float* Delta,
                             int B, int H, int T, int D, void* stream);

/*
 * Exact variant of the preprocess: Delta_i = sum_j P_ij * (dO_i . V_j) over the kept keys, with P
 * rebuilt from LSE inside the kernel (paper Section 4.2, "The Backward Pass": the probability matrix
 * is recomputed from the cached log-sum-exp, never stored).  Mathematically equal to rowsum(dO * O),
 * but independent of the bf16 rounding of the stored O: rowsum(dO * O) carries an error of about
 * 2^-9 * sum_d |dO_d O_d|, which reaches dQ and dK multiplied by scale * |sum_j P_ij K_j| and
 * dominates their error when softmax rows are sharply peaked (|O| ~ |V|).  Costs two extra
 * contractions and one exp2 per score, i.e. roughly one forward pass.  Use it in place of
 * nova_attn_bwd_preprocess when that accuracy matters; nova_attn_bwd accepts either Delta.
 *   Q, K, V, dO : in,  bf16 [B,H,T,D]
 *   LSE         : in,  fp32 [B,H,T] from nova_attn_fwd
 *   Delta       : out, fp32 [B,H,T]
 */
int nova_attn_bwd_preprocess_exact(const void* Q, const void* K, const void* V, const void* dO,
                                   const float* LSE, float* Delta, int B, int H, int T, int D,
                                   float scale, int causal, void* stream);

/*
 * Bytes of scratch nova_attn_bwd needs: an fp32 accumulator for dQ, [B,H,T,D] (rounded up to
 * 256 bytes).  Returns 0 if the shape is invalid.
 */
size_t nova_attn_bwd_workspace_bytes(int B, int H, int T, int D);

/*
 * Backward pass (paper Section 4.2, "The Backward Pass": dQ reduces over keys, dK and dV reduce over
 * queries, the probability matrix is recomputed from the cached log-sum-exp and never stored; the
 * causal loop bound is raised so tiles above the diagonal are never visited).
 *   Q, K, V, dO : in, bf16 [B,H,T,D]
 *   O           : in, bf16 [B,H,T,D]; accepted for symmetry and ignored (Delta already carries it)
 *   LSE, Delta  : in, fp32 [B,H,T] from nova_attn_fwd / nova_attn_bwd_preprocess
 *   dQ, dK, dV  : out, bf16 [B,H,T,D]; gradient of sum(O * dO) with respect to Q, K, V
 *   workspace   : device scratch of at least nova_attn_bwd_workspace_bytes(B,H,T,D) bytes, 16-byte
 *                 aligned; zeroed by the call itself on `stream`; contents afterwards unspecified.
 * dQ is accumulated in fp32 across key tiles with floating-point reduce-adds whose order is not fixed,
 * so its low-order bits may differ from run to run; dK and dV are deterministic.  A final pass scales
 * the accumulator, rounds it once to bf16 and writes dQ.
 */
int nova_attn_bwd(const void* Q, const void* K, const void* V, const void* O, const void* dO,
                  const float* LSE, const float* Delta, void* dQ, void* dK, void* dV,
                  int B, int H, int T, int D, float scale, int causal,
                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * The three steps nova_attn_bwd enqueues, selectable one by one so that each can be timed alone
 * (a measurement aid: the paper has no counterpart).  `steps` is a bit mask:
 *   NOVA_ATTN_BWD_STEP_ZERO     clear the fp32 dQ accumulator in `workspace`
 *   NOVA_ATTN_BWD_STEP_MAIN     the fused backward kernel: writes dK, dV, accumulates unscaled dQ
 *   NOVA_ATTN_BWD_STEP_CONVERT  dQ = bf16(scale * accumulator)
 * All three, in this order, are what nova_attn_bwd does; any other combination leaves sequencing to
 * the caller.  Arguments, validation and errors are those of nova_attn_bwd.
 */
#define NOVA_ATTN_BWD_STEP_ZERO 1
#define NOVA_ATTN_BWD_STEP_MAIN 2
#define NOVA_ATTN_BWD_STEP_CONVERT 4
int nova_attn_bwd_steps(const void* Q, const void* K, const void* V, const void* O, const void* dO,
                        const float* LSE, const float* Delta, void* dQ, void* dK, void* dV,
                        int B, int H, int T, int D, float scale, int causal,
                        void* workspace, size_t workspace_bytes, void* stream, int steps);

/*
 * Backward pass for callers that cannot allocate device memory (the paper has no counterpart).
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside another framework's fixed
 * memory plan, in a plugin that only ever sees its input and output buffers, or in a loop that must
 * not touch the allocator once it is running.  Such callers cannot provide the `workspace` of
 * nova_attn_bwd.  This variant takes the same inputs and outputs and keeps the fp32 dQ accumulator in
 * a fixed array inside the library instead.
 *
 *   - The array holds nova_attn_static_scratch_bytes() = 32 MiB, i.e. B*H*T*D <= 8 Mi elements (the
 *     GPT-2-small training shape B=8, H=12, T=1024, D=64 fits).  Larger problems are rejected with
 *     NOVA_ATTN_ERR_WORKSPACE before anything is launched; use nova_attn_bwd for those.
 *   - The array is part of the library image: a GPU holds the 32 MiB from the moment the library's
 *     device code is loaded on it until the process exits.  With the CUDA runtime's default lazy module
 *     loading that moment is the first call of this function on the device; with eager loading
 *     (CUDA_MODULE_LOADING=EAGER) it is the first use of the library.  A caller inside a fixed memory
 *     plan should therefore make one call at start-up, and must expect NOVA_ATTN_ERR_CUDA from it (code
 *     in nova_attn_last_cuda_error) if the 32 MiB no longer fit on the device.
 *   - The call allocates nothing: no cudaMalloc, no cudaFree, no allocating library routine.
 *   - The first call on a device looks up the array's device address (one runtime query, cached per
 *     device).  Make that first call before starting any stream capture.
 *   - All calls on a device share the one array.  Each call clears the part it uses before use, so
 *     what an earlier call left behind is harmless, but two calls whose GPU work overlaps (different
 *     streams, or different host threads) race on it and corrupt each other's dQ.  Serialise them.
 *   - Arguments, validation, results and error codes are otherwise those of nova_attn_bwd, checked in
 *     the same order: a NULL pointer, a bad shape, alignment or scale is reported as such even when the
 *     problem is also too large for the array.
 */
size_t nova_attn_static_scratch_bytes(void);
int nova_attn_bwd_static_scratch(const void* Q, const void* K, const void* V, const void* O,
                                 const void* dO, const float* LSE, const float* Delta,
                                 void* dQ, void* dK, void* dV, int B, int H, int T, int D,
                                 float scale, int causal, void* stream);

/*
 * Deterministic backward: the two-kernel form of the paper (Section 4.2, "The Backward Pass": one kernel
 * reduces dQ over keys, the other reduces dK and dV over queries; both rebuild the probability matrix from
 * the saved log-sum-exp).  Every output element is summed by one thread block in a fixed order, so dQ, dK
 * and dV are bitwise reproducible from run to run, and no workspace is needed.  The price: the score and
 * dP contractions are computed in both kernels (seven contractions for the five that are counted) and
 * the dQ kernel keeps one query tile in flight per SM, so it is slower than nova_attn_bwd; dK and dV are
 * bit-identical to nova_attn_bwd's, dQ differs from it in the last bits only (summation order).
 *   Q, K, V, dO : in,  bf16 [B,H,T,D]
 *   LSE, Delta  : in,  fp32 [B,H,T] from nova_attn_fwd / nova_attn_bwd_preprocess(_exact)
 *   dQ, dK, dV  : out, bf16 [B,H,T,D]
 * Validation and errors as for nova_attn_bwd (without the workspace).
 */
int nova_attn_bwd_deterministic(const void* Q, const void* K, const void* V, const void* dO,
                                const float* LSE, const float* Delta, void* dQ, void* dK, void* dV,
                                int B, int H, int T, int D, float scale, int causal, void* stream);

/*
 * Strided variants (paper Section 4.2: the per-head layout change around attention is expressed in the
 * access pattern, so the transposes between the fused projection output and the per-head tensors cost
 * nothing).  Each bf16 tensor is addressed as element (b, h, t, d) at
 *     base + b * batch + h * head + t * token + d          (strides in ELEMENTS, d contiguous),
 * so Q, K and V can be read straight out of a fused projection output [B, T, 3, H, D]
 * (Q: base + 0, K: base + H*D, V: base + 2*H*D, each with batch = T*3*H*D, head = D, token = 3*H*D) and
 * O, dQ, dK, dV written as [B, T, H, D] (batch = T*H*D, head = D, token = H*D), or any other layout with
 *   - every stride a multiple of 8 elements (16 bytes; NOVA_ATTN_ERR_ALIGNMENT otherwise),
 *   - token >= D, head >= 8, batch >= 8, every stride below 2^39 (NOVA_ATTN_ERR_SHAPE otherwise),
 *   - strides that the TMA descriptor encoder accepts once token / head / batch are sorted by stride (it
 *     rejects, with NOVA_ATTN_ERR_CUDA, layouts whose larger strides are not multiples it can express),
 *   - no two elements of an OUTPUT tensor at the same address, outputs not overlapping inputs.
 * LSE and Delta stay contiguous fp32 [B, H, T].  Everything else (shapes, validation, results, errors,
 * workspace) is as for nova_attn_fwd, nova_attn_bwd_preprocess and nova_attn_bwd; those three are the
 * special case batch = H*T*D, head = T*D, token = D.  nova_attn_bwd_strided takes no O (Delta carries it).
 */
typedef struct nova_attn_strides {
    long long batch, head, token;
} nova_attn_strides;

int nova_attn_fwd_strided(const void* Q, const void* K, const void* V, void* O, float* LSE,
                          int B, int H, int T, int D,
                          const nova_attn_strides* q_strides, const nova_attn_strides* k_strides,
                          const nova_attn_strides* v_strides, const nova_attn_strides* o_strides,
                          float scale, int causal, void* stream);
int nova_attn_bwd_preprocess_strided(const void* O, const void* dO, float* Delta, int B, int H, int T, int D,
                                     const nova_attn_strides* o_strides, const nova_attn_strides* do_strides,
                                     void* stream);
int nova_attn_bwd_strided(const void* Q, const void* K, const void* V, const void* dO,
                          const float* LSE, const float* Delta, void* dQ, void* dK, void* dV,
                          int B, int H, int T, int D,
                          const nova_attn_strides* q_strides, const nova_attn_strides* k_strides,
                          const nova_attn_strides* v_strides, const nova_attn_strides* do_strides,
                          const nova_attn_strides* dq_strides, const nova_attn_strides* dk_strides,
                          const nova_attn_strides* dv_strides,
                          float scale, int causal, void* workspace, size_t workspace_bytes, void* stream);

/* Static, never-freed description of a status code. */
const char* nova_attn_status_string(int status);

/* CUDA error code (cudaError_t or CUresult, as int) behind the calling thread's last
 * NOVA_ATTN_ERR_CUDA; 0 if none. */
int nova_attn_last_cuda_error(void);

/*
 * Test aid (the paper has no counterpart): lets a test make a bounded device-side wait run out without
 * hanging or faulting anything.  Every spin-wait in the kernels gives up after a cycle limit, the kernel
 * then drains its copies, frees its tensor memory and returns, and nova_attn_poll_device_status reports
 * NOVA_ATTN_ERR_TIMEOUT.  `limit_cycles` sets that limit for kernels launched afterwards by this process
 * (0 restores the default of 2^29 cycles, about a quarter of a second); it applies to nova_attn_fwd.
 * `inject` = 1 makes that kernel's loader leave out the request for its first K tile, so that the wait for
 * it expires; 0 is normal operation.  Returns NOVA_ATTN_ERR_SHAPE for a negative limit or an unknown
 * `inject`.  Not for production use: outputs of a call made with inject = 1 are invalid by construction.
 */
int nova_attn_test_configure_waits(long long limit_cycles, int inject);

/*
 * Host-side view of the backward kernel's work distribution (no GPU is touched): the work items of CTA
 * `cta` out of `n_ctas` for a problem of B*H = `BH` heads, `T` tokens, head dimension `D`, in the order the
 * CTA processes them.  An item is one 128-key tile of one head (paper Section 4.2: the backward pass loops
 * over key tiles and, for each, over the query tiles at or below the diagonal); the list is what decides
 * load balance and which heads' accumulators are in flight together.  Writes up to `capacity` pairs
 * (key tile, head index) into `items` (host, 2 * capacity ints; may be NULL when capacity is 0) and the
 * plan {heads per chunk, chunks, passes per full chunk, passes of the last chunk} into `plan4` (host, 4
 * ints, may be NULL).  Returns the number of items of that CTA (which may exceed `capacity`), or
 * NOVA_ATTN_ERR_SHAPE (negative, like every error code) for arguments out of range (BH, T < 1; D not 64 or 128; n_ctas < 1; cta outside
 * [0, n_ctas)).
 */
int nova_attn_bwd_work_list(int BH, long long T, int D, int causal, int n_ctas, int cta, int* items, int capacity,
                            int* plan4);

/*
 * Synchronises `stream`, then reads and clears the device status word of the current device.
 * Returns NOVA_ATTN_OK, NOVA_ATTN_ERR_TIMEOUT (a kernel gave up on a bounded wait; its outputs are
 * invalid) or NOVA_ATTN_ERR_CUDA.
 */
int nova_attn_poll_device_status(void* stream);

#ifdef __cplusplus
}
#endif
#endif /* NOVA_ATTN_H_ */
