/*
 * bcjr_microbench -- measured pipe rates of the GPU, for the benchmark's roofline.
 *
 * Not a step of the paper's method (no passage to cite): the BCJR recursions of Eq. 5-7 are
 * bound by the special-function unit (one ex2 per state and step, one lg2 per group), the FP32
 * pipe and, in the two-CTA backward kernel, the exchange between the CTAs of a cluster; this call
 * measures those rates on the device at hand so that "fraction of peak" has a measured
 * denominator.
 */
#ifndef BCJR_MICROBENCH_H
#define BCJR_MICROBENCH_H

#include "bcjr_b200.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
    int32_t num_sms;
    int32_t pad;
    double sm_clock_mhz;              /* clock the register-only chains ran at (events vs. cycle counter) */
    double ex2_per_clk_sm;            /* ex2.approx results per clock per SM */
    double lg2_per_clk_sm;
    double fma_f32_per_clk_sm;        /* scalar fma.f32 thread-instructions per clock per SM */
    double fma_f32x2_per_clk_sm;      /* packed fma.f32x2 thread-instructions (pairs) per clock per SM */
    double ex2_gops;                  /* ex2 results per second over the whole GPU, 1e9/s */
    double fma_f32x2_gops;            /* packed pairs per second over the whole GPU, 1e9/s */
    double st_async_bytes_per_clk_sm; /* st.async.v4 to the peer CTA of a two-CTA cluster, both sending, landed */
    double cta_barrier_clk;           /* one named-barrier round of 512 threads, clocks */
    double mbarrier_round_clk;        /* one mbarrier round: an arrival per warp, 16 warps polling, clocks */
    double fma_f32x2_with_alu_per_clk_sm; /* packed pairs per clock per SM when every packed instruction has an integer
                                         instruction (the ALU pipe) beside it: equal to fma_f32x2_per_clk_sm if the two
                                         pipes overlap, two thirds of it if they take turns */
    double fma_f32x2_with_max_per_clk_sm; /* the same with a max.f32 (also the ALU pipe) beside every packed instruction */
    double fma_f32x2_with_ex2_per_clk_sm; /* the same with one ex2.approx (special-function unit) per four packed instructions */
    double fma_f32x2_with_f64_per_clk_sm; /* the same with one fma.f64 (fp64 pipe) per two packed instructions */
} bcjr_pipe_peaks;

/*
 * Runs the micro-benchmarks on CUDA device `device` (about 50 kernel launches of well under a
 * millisecond each on `cuda_stream`; synchronous; allocates and frees ~300 KB of device memory).
 *   out   host, filled on BCJR_OK
 * Errors: BCJR_EINVAL (out is NULL), BCJR_ECUDA / BCJR_ENOMEM (runtime failure), BCJR_ETIMEOUT (a
 * bounded device-side wait of the exchange or barrier kernels ran out; the figures are then void).
 */
bcjr_status bcjr_measure_pipe_peaks(int device, bcjr_pipe_peaks *out, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* BCJR_MICROBENCH_H */
