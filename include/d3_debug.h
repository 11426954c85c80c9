/*
 * d3_debug.h -- measurement and test switches of the d3 library.
 *
 * Nothing here is part of the decoding path's contract (include/d3.h): these calls select
 * scheduling variants of the kernels for sweeps, force code paths that the default heuristics
 * would not take on small test shapes, and expose the give-up path of the bounded device-side
 * waits.  Results never change beyond the order of fp32 partial sums.  All settings are per
 * context and default to "let the library decide".
 */
#ifndef D3_DEBUG_H_
#define D3_DEBUG_H_

#include "d3.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Scheduling overrides of the tensor-core matmuls and of attention.  d3_tuning_defaults() fills in
 * the "library decides" value of every field; change the ones of interest and pass the struct to
 * d3_set_tuning().  INVALID_ARG for values outside the ranges given here. */
typedef struct d3_tuning {
  int32_t ring_kb;          /* shared-memory ring per CTA in KB, 0 = default (about 100 KB for matmuls of up
                               to 128 rows, 200 KB otherwise; the whole CTA of a chain launch, default 222); at most 224 */
  int32_t ctas_per_sm;      /* CTAs per SM the work is dealt to, 0 = default; at most 3 */
  int32_t producers;        /* copy-issuing warps (unit-range kernel) or issue pipelines (column strips):
                               0 = default, 1 or 2 */
  int32_t tile_columns;     /* output tile width of the unit-range kernel: 0 = by row count, 128 or 256 */
  int32_t attn_key_tiles;   /* attention: least number of 64-key tiles per key split, 0 = default (2); 1..7 */
  int32_t cluster_k_split;  /* skinny residual matmuls on K-splitting clusters: -1 = when it pays, 0 never */
  int32_t row_tile_pairs;   /* two 128-row tiles share each weight slab (129..511 rows): -1 = by shape, 0, 1 */
  int32_t round_robin;      /* wide matmuls deal whole tiles round-robin in a banded order: 1 (default), 0 */
  int32_t column_strips;    /* skinny matmuls as whole-K column strips: 0 = when it pays, 1 never,
                               2 with one CTA per SM, 3 wherever the shape allows */
  int32_t strip_stages;     /* explicit pipeline depth of the column-strip kernel, 0 = from ring_kb.  With two
                               issue pipelines every stage belongs to one pipeline, which takes an even
                               count: an odd one is refused (D3_ERR_UNSUPPORTED at the launch), not rounded */
  int32_t chain;            /* decode forwards of up to 64 rows run the matmuls between two attention kernels
                               as one persistent launch: -1 = when the shapes allow (default), 0 never */
  int32_t chain_clusters;   /* clusters of four CTAs the chain launches use: 0 = as many as are resident at once
                               (default); a smaller count is taken as given, a larger one is cut to that */
  int32_t chain_l2_ahead;   /* weight slabs the chain's L2 prefetch warp runs ahead of the ring: -1 = default
                               (0: no prefetch; measured neutral at 12 slabs and slower beyond), at most 256 */
  int32_t weights_as_rows;  /* matmuls of 129..256 rows with at most one 128-column tile per SM run with the weights as the
                               MMA's 128-row operand and a K-splitting cluster per tile: -1 = when the shape allows, 0 never */
  int32_t attention_tmem;   /* attention with both products on tcgen05 MMAs and the accumulators in tensor memory
                               (attn_tmem_kernel) instead of mma.sync (attn_tc_kernel): -1 = where measured faster
                               (default), 0 never, 1 wherever the shape allows (bf16, d_head 128), 64 or 128 = the same with
                               that many keys per tile (two CTAs per SM / one) instead of the launcher's choice, 2 = the persistent
                               form (one CTA per SM streams through its (sequence, kv head) pairs) wherever all packed rows
                               of a pair fit one 128-row tile, whatever the number of pairs */
  int32_t cta_pairs;        /* matmuls of more than 128 rows on tiled weights run 256 x 256 tiles on pairs of CTAs that share
                               one MMA (cta_group::2, gemm_pair_kernel): -1 = when the shape allows (default), 0 never */
} d3_tuning;
void d3_tuning_defaults(d3_tuning *t);
int d3_set_tuning(d3_ctx *ctx, const d3_tuning *t);

/* d3_generate runs a block's finalize forward together with the first denoise step of the next
 * block while the forward stays skinny (see d3_generate).  on = 0: every block is finalized in a
 * forward of its own; results are the same (bit for bit on the fp32 path). */
int d3_set_fused_finalize(d3_ctx *ctx, int on);

/* Give-up path of the bounded waits.  Every device-side wait of the kernels (mbarrier phases) ends
 * after a time limit, raises bit 0 of the device error word and lets its CTA leave in order (all
 * roles return, tensor memory is released); the next call that reads the error word returns
 * D3_ERR_DEVICE_TIMEOUT.  d3_debug_stall_probe exercises that path without any copy in flight: it
 * launches the unit-range matmul kernel on a context-owned 32 x 128 x 64 problem with the producer
 * warps told to issue no loads and a wait limit of limit_us microseconds (1..2000000), so the
 * MMA-issuing thread's first wait runs out, the epilogue warps see the CTA's abort flag, and the
 * kernel returns.  The call waits for the stream and returns D3_ERR_DEVICE_TIMEOUT when the error word
 * carries the time-out bit (the expected outcome), D3_OK if it does not.  d3_clear_error_word resets
 * the word so that the context can be used again. */
int d3_debug_stall_probe(d3_ctx *ctx, int32_t limit_us);
int d3_clear_error_word(d3_ctx *ctx);
/* The status a call returns for a device error word (host arithmetic only, no context):
 * D3_ERR_DEVICE_TIMEOUT when the time-out bit is set, D3_ERR_INVALID_ARG for any other bit, D3_OK for 0. */
int d3_status_of_error_word(uint32_t word);

#ifdef __cplusplus
}
#endif
#endif /* D3_DEBUG_H_ */
