/*
 * rs_profile.h -- instrumentation of librs.so for benchmarks: launch counting and per-kernel-class
 * device timing.  The paper reports whole-model throughput only (Sec. 4); nothing here has a
 * counterpart there, and no entry point of rs.h depends on it.
 */
#ifndef RS_PROFILE_H_
#define RS_PROFILE_H_

#include "rs.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Number of kernels the library has launched through this context so far. */
RS_API long long rs_launch_count(const rs_ctx* ctx);

/* While enabled, every launch through the context is bracketed by CUDA events on the launch
 * stream (up to 8192 launches between reads; later ones are not recorded).  rs_timing_read
 * synchronises `stream`, adds up the elapsed milliseconds and launch counts per class into the
 * two host arrays of RS_K_COUNT entries, and clears the record.  Errors: RS_ERR_INVALID_ARG on a
 * null argument, RS_ERR_CUDA when an event call fails. */
typedef enum {
    RS_K_LAYERNORM = 0, RS_K_GEMM = 1, RS_K_ATTN = 2, RS_K_SCORE = 3, RS_K_SELECT = 4, RS_K_GATHER = 5,
    RS_K_COUNT = 6
} rs_kernel_class;
RS_API rs_status rs_timing_enable(rs_ctx* ctx, int on);
RS_API rs_status rs_timing_read(rs_ctx* ctx, void* stream, double* ms /*host[RS_K_COUNT]*/,
                                long long* launches /*host[RS_K_COUNT]*/);

/* Tensor maps (the TMA descriptors of the tensor-core kernels) are encoded once per (pointer,
 * shape, box) and kept in a 128-slot cache of the context.  Hits and misses so far (host counters). */
RS_API rs_status rs_tmap_cache_stats(const rs_ctx* ctx, long long* hits /*host*/, long long* misses /*host*/);

/* Which of the two tensor-core attention kernels rs_attn_fwd picks for B samples, H heads and N tokens on a
 * GPU of sm_count SMs: 2 (two query tiles per thread block; also every N <= 128) or 3 (three).  Host
 * arithmetic only (the cost model of the choice); needs no context and no GPU. */
RS_API int rs_attn_kernel_choice(int sm_count, int B, int H, int N);

#ifdef __cplusplus
}
#endif
#endif /* RS_PROFILE_H_ */
