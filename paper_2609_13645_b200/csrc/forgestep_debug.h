/* Development entry points of libforgestep.so.  They are NOT part of the library's boundary (include/forgestep.h):
 * the switches are process-wide, not thread-safe, and exist for kernel benchmarks and ablations; the wait probe exists
 * so that a test can watch a bounded device-side wait run out without hanging anything. */
#ifndef FORGESTEP_DEBUG_H_
#define FORGESTEP_DEBUG_H_

#include <stdint.h>

#include "../../include/forgestep.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Force the GEMM tile width (128 or 256 columns); 0 = choose by tile count (default). */
void ft_debug_gemm_tile(int32_t bn);
/* 1 = CTA-pair (cta_group::2, 256 x 256 tile) GEMM kernel where it applies (default), 0 = single-CTA kernel only. */
void ft_debug_gemm_pairs(int32_t on);
/* 1 = balanced-K schedule where it applies and scratch is available (default), 0 = round-robin tiles. */
void ft_debug_gemm_balanced(int32_t on);
/* 1 = the two pairs of weight gradients of a layer (down + gate/up, output + qkv projection) run as one launch each
 * (default), 0 = one launch per weight gradient. */
void ft_debug_gemm_group(int32_t on);
/* 1 = plain bf16 outputs of the CTA-pair GEMM leave as TMA tensor stores (default), 0 = one row per thread with 32-byte
 * stores.  Both give the same bits. */
void ft_debug_gemm_tma_out(int32_t on);
/* 1 = the SwiGLU-backward epilogue of the CTA-pair GEMM moves gate / up and d_gate / d_up as TMA tiles through shared
 * memory (default), 0 = one row per thread with plain loads and stores.  Both give the same bits. */
void ft_debug_gemm_swiglu_tma(int32_t on);
/* 1 = kernels are launched with programmatic stream serialization (programmatic dependent launch: appendix "Optimization Catalog", "Cross-kernel scheduling"), the default; 0 = ordinary stream
 * order.  Graphs captured under one setting keep it. */
void ft_debug_pdl(int32_t on);

/* Largest bf16 logit-gradient buffer [max_batch * max_seq, vocab] a model created AFTERWARDS will carry (default 4 GiB):
 * within it the output head's two gradients are single contractions over all rows, above it they are formed per chunk
 * of rows with the weight gradient accumulating in memory.  0 forces the chunked form (tests cover both). */
void ft_debug_head_dz_limit(uint64_t bytes);

/* Enqueues, on the model's stream, a one-block kernel that waits on an mbarrier nobody ever arrives on, with the same
 * bounded wait the GEMM and attention kernels use but a limit of limit_cycles SM clocks (1 .. 20,000,000: at most about
 * 10 ms).  When the limit runs out the kernel records ERR_WAIT_TIMEOUT in the model's device status word and returns, so
 * the NEXT synchronising call of the model (ft_train_step with a loss pointer, ft_collect_step, ...) returns
 * FT_ETIMEOUT and clears the word; the context stays usable.  Nothing traps and nothing waits longer than the limit. */
ft_status ft_debug_wait_probe(ft_model* m, int64_t limit_cycles);

#ifdef __cplusplus
}
#endif
#endif /* FORGESTEP_DEBUG_H_ */
