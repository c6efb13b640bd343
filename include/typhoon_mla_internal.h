/*
 * typhoon_mla_internal.h -- measurement and test hooks of the MLA decode-attention library.
 *
 * Nothing here is needed to use the library (see typhoon_mla.h).  These entry points exist for
 * the test-suite and the benchmark: switches that select between implementations that compute the
 * same result, views into the prepared prefix, per-kernel timing, and a test kernel for the
 * bounded-wait mechanism.  The switches are process-wide atomics; every decode call reads them
 * once, at its start, and uses that snapshot for its plan and for all of its launches, so flipping
 * one from another thread cannot split a step between two settings.
 */
#ifndef TYPHOON_MLA_INTERNAL_H_
#define TYPHOON_MLA_INTERNAL_H_

#include "typhoon_mla.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Work decomposition the tcgen05 shared-prefix kernel (Algorithm 1 line 4) would use for a problem
 * size on a GPU with `num_sms` multiprocessors (0: 148, a B200): tokens per KV tile (64 for B <= 128,
 * else 128), number of contiguous tile ranges the H * n_tiles tiles are cut into, query-row groups
 * per range (CTAs = ranges * row_groups) and partial slots written per (request, head).  schedule:
 * 0 = the library's choice, 1 = every range inside one head ("column split"), 2 = ranges of equal
 * size over all heads ("stream-K").  Host, pure (a function of the sizes only, so the decomposition
 * and with it the summation order are reproducible).  INVALID_ARG for B < 1, L_s < 1, unsupported H
 * or schedule outside 0..2; no output is written then. */
int typhoon_mla_naive_plan(int32_t num_heads, int32_t B, int64_t L_s, int32_t schedule, int32_t num_sms,
                           int32_t* tile_tokens /* host */, int32_t* n_ranges /* host */,
                           int32_t* row_groups /* host */, int32_t* n_slots /* host */);

/* Read-only views of what the handle owns (for tests and accounting):
 * k_nope bf16 [H, Ls_padded/64, 2, 64, 64]; v_t bf16 [H, Ls_padded/64, 128, 64]. */
int typhoon_mla_shared_view(const typhoon_mla_shared_t* shared,
                            const void** k_nope, const void** v_t,
                            int64_t* Ls /* host */, int64_t* Ls_padded /* host */,
                            int64_t* owned_bytes /* host */);

/* Copy the expanded caches into caller buffers of H * Ls_padded * 128 bf16
 * elements each (device memory), on `stream`. */
int typhoon_mla_shared_export(const typhoon_mla_shared_t* shared, void* k_nope_dst, void* v_t_dst, void* stream);

/* A handle from typhoon_mla_prepare_shared_fp8: the E4M3 codes in logical order, K_nope as
 * uint8 [H, Ls_padded, 128] (token rows), V as uint8 [H, Ls_padded/64, 128, 64] (V^T in 64-token
 * blocks), and the scales as float [2][H] (K_nope, then V); device buffers, on `stream`.
 * INVALID_ARG for a 16-bit handle (and typhoon_mla_shared_export for an 8-bit one). */
int typhoon_mla_shared_export_fp8(const typhoon_mla_shared_t* shared, void* k_codes_dst, void* v_codes_dst,
                                  float* scales_dst, void* stream);

/* Which implementation of the tensor-core kernels runs: the tcgen05/TMEM/TMA kernels (default) or
 * the warp-MMA kernels kept as an on-GPU cross-check.  Affects later prepare_shared and decode calls. */
enum { TYPHOON_MLA_PATH_TCGEN05 = 0, TYPHOON_MLA_PATH_WARP_MMA = 1 };
int typhoon_mla_set_kernel_path(int32_t path);

/* In a hybrid step the absorb branch (Algorithm 1 lines 5-6) runs on a stream owned by the handle,
 * beside the naive kernel (line 4), and is joined before the projection (default).  0 keeps every
 * kernel on the caller's stream, one after the other. */
int typhoon_mla_set_overlap(int32_t enable);

/* The kernels of a step are launched with the programmatic-stream-serialization attribute (default):
 * a kernel may be scheduled while its predecessor in the stream is still running and waits, before its
 * first access to global memory, until that predecessor has completed.  0 gives ordinary stream-ordered
 * launches. */
int typhoon_mla_set_programmatic_launch(int32_t enable);

/* Work decomposition of the tcgen05 shared-prefix kernel (see typhoon_mla_naive_plan): 0 = the
 * library's choice (default), 1 = column split, 2 = stream-K. */
int typhoon_mla_set_naive_schedule(int32_t schedule);

/* Absorb-only steps attend the shared prefix with the batch-stacked kernel (default, tcgen05 path) or
 * feed it to the per-request suffix kernel as extra chunks (0). */
int typhoon_mla_set_stacked_absorb(int32_t enable);

/* Longest-first order used for ragged suffixes: perm[0..B) (device, int32) = request indices sorted
 * by descending seq_lens (device, int32), ties by ascending index.  B <= 4096. */
int typhoon_mla_order_by_length(const int32_t* seq_lens, int32_t B, int32_t* perm, void* stream);

/* Kernel kinds of the decode step, in launch order (Algorithm 1 lines 4-8). */
enum {
    TYPHOON_MLA_KERNEL_NAIVE_ATTN = 0,  /* line 4 */
    TYPHOON_MLA_KERNEL_Q_ABSORB = 1,    /* line 5 */
    TYPHOON_MLA_KERNEL_ABSORB_ATTN = 2, /* line 6 */
    TYPHOON_MLA_KERNEL_MERGE = 3,       /* merge of line 6's KV splits */
    TYPHOON_MLA_KERNEL_W_UV = 4,        /* line 7 */
    TYPHOON_MLA_KERNEL_COMBINE = 5,     /* line 8 */
    TYPHOON_MLA_NUM_KERNELS = 6
};

/*
 * Between profile_begin and profile_end every decode call of the process records a pair of CUDA
 * events around the launch of the chosen kernel kind, on the stream the kernel is launched on (up
 * to max_launches launches).  profile_end waits for the recorded events and returns the summed
 * device time in milliseconds and the number of launches timed.  Host, one profiling session at a
 * time, not to be used while other threads decode; begin allocates events, decode itself still
 * allocates nothing.
 */
int typhoon_mla_profile_begin(int32_t kernel_id, int32_t max_launches);
int typhoon_mla_profile_end(double* total_ms /* host */, int32_t* launches /* host */);

/* Number of kernels the last decode call of this thread launched. */
int typhoon_mla_last_launch_count(void);

/*
 * Exercises the bounded wait that every kernel of the library uses, without touching a production
 * kernel: a one-block kernel (no copies, no tensor memory) initialises a barrier on which nothing
 * ever arrives and waits on it with a deadline of `deadline_cycles` SM clocks (clamped to 1e3..1e8,
 * i.e. at most about 50 ms).  The wait runs out, the kernel ORs `code` (1..255) into the handle's
 * status word exactly as the production kernels do, and returns normally; the context stays usable.
 * Asynchronous on `stream`.
 */
int typhoon_mla_test_wait_expiry(const typhoon_mla_shared_t* shared, int64_t deadline_cycles, int32_t code, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TYPHOON_MLA_INTERNAL_H_ */
