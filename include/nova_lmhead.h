/*
 * libnova_attn - second workload: the fused language-model loss head (C ABI).
 *
 * Paper: Section 4.1, case study "Fusing a Reduction into a Contraction Epilogue", and Section 6.1, "Fused
 * Loss Head" (measured there on 8192 x 768 x 50304).  The projection onto the vocabulary and the softmax
 * cross-entropy statistics run as ONE contraction kernel: while an output tile is still in tensor memory its
 * epilogue reduces it to one partial (maximum, sum of exponentials) pair per row and per 128 vocabulary entries;
 * a small merge kernel then combines the partial pairs of a row, rescaling each sum by the exponential of the
 * difference of the maxima, into the row's log-sum-exp and loss.  The logits are written once (bf16, for the
 * backward pass, as in the paper) and never read back; pass NULL to leave them out altogether.
 *
 *   logits[i,n] = sum_k X[i,k] W[n,k]          fp32 accumulation of bf16 products
 *   lse[i]      = ln sum_n exp(logits[i,n])    natural log, from the fp32 accumulators (not the rounded logits)
 *   loss[i]     = lse[i] - logits[i, targets[i]]   if 0 <= targets[i] < N, else 0 (a row without a label)
 *
 * Conventions are those of nova_attn.h: device pointers, caller owns every buffer, work is only enqueued on
 * `stream` (a cudaStream_t passed as void*), nothing is allocated or synchronised, status codes are the
 * NOVA_ATTN_* values and nova_attn_status_string / nova_attn_poll_device_status apply.
 */
#ifndef NOVA_LMHEAD_H
#define NOVA_LMHEAD_H

#include <stddef.h>

#include "nova_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Bytes of workspace nova_lmhead_fwd needs: the partial pairs, ceil(N / 128) * M * 8 bytes (the layout of the
 * paper's "8192 x 786 partials", at this kernel's tile width), plus one fp32 per row for the target logit.
 * Returns 0 for arguments nova_lmhead_fwd would reject.
 */
size_t nova_lmhead_workspace_bytes(int M, int N, int K);

/*
 * X       bf16 [M, K]  hidden states, K contiguous                       (in)
 * W       bf16 [N, K]  vocabulary matrix, K contiguous                   (in)
 * targets int32 [M]    vocabulary index of each row's label; outside [0, N) = no label      (in)
 * logits  bf16 [M, N]  N contiguous; NULL = do not store the logits      (out)
 * lse     fp32 [M]     natural-log log-sum-exp of the row's logits       (out)
 * loss    fp32 [M]     cross-entropy of the row (0 for a row without a label)   (out)
 * workspace            at least nova_lmhead_workspace_bytes(M, N, K) bytes, 16-byte aligned; contents
 *                      need not be initialised and are overwritten
 *
 * Requirements: M, N, K >= 1; K and N multiples of 8 (rows of X, W and logits start on 16-byte boundaries);
 * X, W, logits and workspace 16-byte aligned, targets, lse and loss 4-byte aligned.  Errors (checked on the host before any launch): NOVA_ATTN_ERR_NULL,
 * NOVA_ATTN_ERR_SHAPE (non-positive or too large a dimension, K or N not a multiple of 8),
 * NOVA_ATTN_ERR_ALIGNMENT, NOVA_ATTN_ERR_WORKSPACE, NOVA_ATTN_ERR_UNSUPPORTED (device is not sm_100),
 * NOVA_ATTN_ERR_CUDA.  A device-side wait that runs out is reported by nova_attn_poll_device_status.
 */
int nova_lmhead_fwd(const void* X, const void* W, const int* targets, void* logits, float* lse, float* loss,
                    int M, int N, int K, void* workspace, size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* NOVA_LMHEAD_H */
