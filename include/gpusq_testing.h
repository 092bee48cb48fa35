/*
 * gpusq -- hooks for the test suite.  NOT part of the library's interface: a
 * program that uses libgpusq.so has no reason to call these (the paper has no
 * counterpart).  They exist so that the parity tests can drive the GEMM
 * kernels through every tile height and through mixed tile heights on small
 * shapes, and so that the measurement script can time a few CTA pairs alone;
 * results never depend on them.
 *
 * All settings are process-wide atomics read by every later call of the
 * process, from any thread; they are meant to be set while no other thread is
 * issuing calls.
 */
#ifndef GPUSQ_TESTING_H
#define GPUSQ_TESTING_H

#ifdef __cplusplus
extern "C" {
#endif

/* Tokens per output tile: a multiple of 32 in [32, 224], all tiles of that
 * height; 0 restores the automatic choice (also of the mix below). */
int gpusq_set_block_tokens(int block_t);

/* Mixed heights: the first n_big token tiles block_t tokens high (block_t a
 * multiple of 32 in [64, 224]), the rest block_t - 32, as many as cover M. */
int gpusq_set_tile_mix(int block_t, int n_big);

/* Bound of the device-side waits of gpusq_quant_act's one-launch kernel, in
 * nanoseconds (default 2 s), and, with withhold_last_cta != 0, a planted
 * failure made on purpose in an allowed form: the last CTA never publishes its
 * maximum, so every CTA's bounded wait runs out, the kernel returns, and the
 * status word and the NaN scale described in gpusq.h can be observed.  Nothing
 * faults or hangs: the waits end at the bound. */
int gpusq_set_quant_act_wait(unsigned long long limit_ns, int withhold_last_cta);

/* The same for the GEMM kernels: bound of every device-side wait in microseconds
 * (default 2 s) and, with withhold_loads != 0, a planted failure in an allowed
 * form: the producers of the first CTA pair stop before the last k block of
 * their first tile, so the MMA issuer's bounded wait for that block runs out;
 * it raises the pair's abort flag, writes {GPUSQ_ERR_TIMEOUT, tile, role,
 * stage} to status_buf, every role of the pair leaves its loop, and the kernel
 * returns.  The other pairs finish their tiles.  Nothing faults or hangs. */
int gpusq_set_gemm_wait(unsigned limit_us, int withhold_loads);

/* Measurement hook: the GEMM launches use at most `clusters` CTA pairs (0 = as
 * many as the GPU holds, the default).  With the tokens cut in proportion,
 * every pair keeps its number of tiles, so the time per tile of one pair can
 * be read with little or no traffic from the other SMs (bench.py --tile-sweep). */
int gpusq_set_max_clusters(int clusters);

#ifdef __cplusplus
}
#endif
#endif /* GPUSQ_TESTING_H */
