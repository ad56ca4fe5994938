// Sustained instruction-issue rates of the device, measured with three instruction streams.
//
// The plan search is bound by instruction issue (FP64 adds and compares, integer mask work,
// shared-memory broadcasts), not by memory, so the ceiling its throughput is compared with is
// the rate at which an SM actually issues such instructions.  Each kernel below keeps eight
// independent dependency chains per thread of one instruction kind and runs on four blocks of 256
// threads per SM (32 warps per SM, eight per scheduler), long enough to hide the pipe's latency.
// The count that is reported excludes the loop's own counter and branch (one of each per 128
// stream instructions).
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

namespace sailor {

constexpr int PEAK_THREADS = 256;
constexpr int PEAK_CHAINS = 8;
constexpr int PEAK_ROUNDS = 16;          // stream instructions per loop iteration = chains * rounds

enum PeakKind { PEAK_FFMA = 0, PEAK_IMAD = 1, PEAK_DADD = 2 };

template <int KIND>
__global__ void __launch_bounds__(PEAK_THREADS) issue_stream_kernel(uint32_t iters, float fa, float fb, uint32_t ia,
                                                                     uint32_t ib, double dc, double* sink) {
    const uint32_t tid = blockIdx.x * blockDim.x + threadIdx.x;
    if (KIND == PEAK_FFMA) {
        float x[PEAK_CHAINS];
#pragma unroll
        for (int j = 0; j < PEAK_CHAINS; ++j) x[j] = (float)(tid + j);
        for (uint32_t it = 0; it < iters; ++it) {
#pragma unroll
            for (int r = 0; r < PEAK_ROUNDS; ++r)
#pragma unroll
                for (int j = 0; j < PEAK_CHAINS; ++j) x[j] = __fmaf_rn(x[j], fa, fb);
        }
        float s = 0.f;
#pragma unroll
        for (int j = 0; j < PEAK_CHAINS; ++j) s += x[j];
        if (s == 12345.678f) sink[0] = s;                  // keeps the chains alive; practically never taken
    } else if (KIND == PEAK_IMAD) {
        uint32_t x[PEAK_CHAINS];
#pragma unroll
        for (int j = 0; j < PEAK_CHAINS; ++j) x[j] = tid + j;
        for (uint32_t it = 0; it < iters; ++it) {
#pragma unroll
            for (int r = 0; r < PEAK_ROUNDS; ++r)
#pragma unroll
                for (int j = 0; j < PEAK_CHAINS; ++j) x[j] = x[j] * ia + ib;
        }
        uint32_t s = 0;
#pragma unroll
        for (int j = 0; j < PEAK_CHAINS; ++j) s ^= x[j];
        if (s == 0x9e3779b9u && ia == 1u) sink[0] = (double)s;
    } else {
        double x[PEAK_CHAINS];
#pragma unroll
        for (int j = 0; j < PEAK_CHAINS; ++j) x[j] = (double)(tid + j);
        for (uint32_t it = 0; it < iters; ++it) {
#pragma unroll
            for (int r = 0; r < PEAK_ROUNDS; ++r)
#pragma unroll
                for (int j = 0; j < PEAK_CHAINS; ++j) x[j] = __dadd_rn(x[j], dc);
        }
        double s = 0.0;
#pragma unroll
        for (int j = 0; j < PEAK_CHAINS; ++j) s = __dadd_rn(s, x[j]);
        if (s == 12345.678) sink[0] = s;
    }
}

}  // namespace sailor
