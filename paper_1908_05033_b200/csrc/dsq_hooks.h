/*
 * dsq_hooks.h - process-wide tuning and test hooks of the tensor-core kernels.
 * Not part of the public interface (include/dsq.h): profiling tools and the
 * test-suite use them to force a tiling or a pipeline, or to make a bounded
 * wait run out.  Each hook sets one atomic integer that later dsq_conv2d /
 * dsq_gemm calls read; results never depend on the tuning hooks.
 */
#ifndef DSQ_HOOKS_H_
#define DSQ_HOOKS_H_

#ifdef __cplusplus
extern "C" {
#endif

/* Force the tile width along N (output channels): 32, 64, 128, 192 or 256;
 * 0 restores the automatic choice. */
int dsq_set_tile_n(int bn);

/* K steps (of 128 codes) per pipeline round: 1 or 2; 0 = automatic. */
int dsq_set_round_k_steps(int ks);

/* CTA pairs (clusters of two CTAs on one 256 x 256 tile, tcgen05
 * cta_group::2): 0 automatic, 1 never, 2 wherever the shapes allow. */
int dsq_set_cta_pairs(int mode);

/* Programmatic dependent launch of the tensor-core kernels (default 1): the
 * kernel's set-up may overlap the tail of the previous kernel of the stream;
 * it waits for that kernel (griddepcontrol.wait) before touching global
 * memory.  0 = plain launches. */
int dsq_set_dependent_launch(int on);

/* Limit of every device-side barrier wait in nanoseconds (default 2 s; 0
 * restores the default). */
int dsq_set_wait_limit_ns(long long ns);

/* 3x3 stride-1 convolutions on an expanded shared-memory window
 * (dsq_conv3.cu): 1 = where it is the faster kernel (default), 0 = never (the
 * im2col kernel takes them), 3 = wherever the geometry allows (transposed
 * tiles where those fit), 4 = as 3 but plain tiles only, 2 = as 4 with the row
 * phase of the window written into the A descriptor's base-offset field (a
 * probe of that field's meaning: the tensor core swizzles by absolute
 * shared-memory address, so this gives wrong numbers). */
int dsq_set_conv3_window(int mode);

/* Window kernel: 1 = weight tiles come by TMA from the blob's pre-expanded
 * int8 copy where it exists (default), 0 = always expand the packed rows in
 * the kernel. */
int dsq_set_conv3_expanded_weights(int on);

/* dsq_gemm with a workspace large enough for the expanded operands: 1 = take
 * the two-pass path where it is the faster one (default: M, N, K >= 1024 and
 * M N K >= 2^35), 0 = always the fused kernel, 2 = two passes whatever the
 * size (dsq_gemm_workspace_bytes answers accordingly). */
int dsq_set_gemm_two_pass(int on);

/* Test hook: in every later launch the thread that issues the TMA copies of
 * the packed B operand leaves out the copy of round `round` of its CTA
 * (0 = the first) and issues nothing after it; -1 switches the hook off.
 * The warps that wait for that copy then run into the wait limit: the kernel
 * records DSQ_ERR_TIMEOUT in the workspace, every role leaves its loop,
 * copies and MMAs already in flight are allowed to finish, tensor memory is
 * freed and the kernel returns.  Nothing faults and nothing waits longer
 * than the limit; the outputs of such a launch are undefined. */
int dsq_set_test_skip_b_round(int round);

#ifdef __cplusplus
}
#endif
#endif /* DSQ_HOOKS_H_ */
