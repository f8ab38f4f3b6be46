// Measured arithmetic ceilings of the device, for the roofline of the kernels that are not bound by memory
// (diagnostics: not part of the scoring path; see hann_probe_rates in include/hann.h).
//
//   * binary64 modular butterflies per second: the register-resident round of four stages the transform kernels run
//     (ArithF64::fwd on sixteen values per thread, twiddles in registers, one reduction per round), with no memory
//     traffic at all -- the rate no transform kernel can exceed;
//   * 32 x 32 -> 64-bit integer multiply-adds per second: eight accumulators per thread -- the rate that bounds the
//     multiply-accumulate's three such products per residue product.
#include "internal.h"
#include "nttcore.cuh"

namespace {

constexpr int kProbeThreads = 256;

__global__ void __launch_bounds__(kProbeThreads) k_probe_f64(double* out, int iters, const LimbConst* lt) {
    const ArithF64 ar(lt);
    double x[16];
#pragma unroll
    for (int e = 0; e < 16; e++) x[e] = (double)((threadIdx.x * 977 + e * 131 + blockIdx.x) % 1000003);
    // a twiddle pair that changes every round, so that nothing is hoisted out of the loop
    double w = 123456789012.0 + threadIdx.x;
    for (int it = 0; it < iters; it++) {
        const double2 tw = make_double2(w, w * ar.qinv);
#pragma unroll
        for (int s = 0; s < 4; s++) {
            const int span = 8 >> s;
#pragma unroll
            for (int e = 0; e < 16; e++)
                if (!(e & span)) ar.fwd(x[e], x[e + span], tw);
        }
#pragma unroll
        for (int e = 0; e < 16; e++) x[e] = ar.reduce(x[e]);
        w += 2.0;
    }
    double acc = 0;
#pragma unroll
    for (int e = 0; e < 16; e++) acc += x[e];
    out[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = acc;
}

// 32 x 32 -> 64-bit multiply-adds (mad.wide.u32), the instruction the multiply-accumulate kernels are made of
__global__ void __launch_bounds__(kProbeThreads) k_probe_imad(double* out, int iters) {
    unsigned long long acc[8];
#pragma unroll
    for (int k = 0; k < 8; k++) acc[k] = threadIdx.x + k;
    unsigned a = threadIdx.x * 2654435761u + 1u, b = blockIdx.x * 40503u + 3u;
    for (int i = 0; i < iters; i++) {
#pragma unroll
        for (int k = 0; k < 8; k++) acc[k] += (unsigned long long)(a ^ (unsigned)k) * (unsigned long long)b;
        a += 2;
        b = b * 3u + 1u;
    }
    unsigned long long t = 0;
#pragma unroll
    for (int k = 0; k < 8; k++) t += acc[k];
    out[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = (double)t;
}

}  // namespace

extern "C" int hann_probe_rates(hann_ctx* c, double* f64_butterflies_per_s, double* int32_madds_per_s) {
    if (!c) return HANN_EINVAL;
    if (!f64_butterflies_per_s || !int32_madds_per_s) {
        c->err = "hann_probe_rates: null pointer";
        return HANN_EINVAL;
    }
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess || cudaSetDevice(c->device) != cudaSuccess) {
        c->err = "hann_probe_rates: cannot select the context's device";
        return HANN_ECUDA;
    }
    int sms = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device);
    // whole waves: four rounds of as many CTAs as are resident at once
    int occ_f64 = 1, occ_imad = 1;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_f64, k_probe_f64, kProbeThreads, 0);
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_imad, k_probe_imad, kProbeThreads, 0);
    const int grid_f64 = sms * (occ_f64 > 0 ? occ_f64 : 1) * 4, grid_imad = sms * (occ_imad > 0 ? occ_imad : 1) * 4;
    const int grid = grid_f64 > grid_imad ? grid_f64 : grid_imad;
    double* out = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    int rc = HANN_OK;
    if (cudaMalloc(&out, (size_t)grid * kProbeThreads * 8) != cudaSuccess || cudaEventCreate(&e0) != cudaSuccess ||
        cudaEventCreate(&e1) != cudaSuccess) {
        cudaGetLastError();
        c->err = "hann_probe_rates: allocation failed";
        rc = HANN_ENOMEM;
    }
    const int it_f64 = 1500, it_imad = 10000;
    float ms_f64 = 0, ms_imad = 0;
    if (rc == HANN_OK) {
        // one untimed launch of each first (module load, clocks), then the timed ones
        for (int rep = 0; rep < 2; rep++) {
            cudaEventRecord(e0, c->stream);
            k_probe_f64<<<grid_f64, kProbeThreads, 0, c->stream>>>(out, it_f64, c->lt_dev);
            cudaEventRecord(e1, c->stream);
            if (cudaEventSynchronize(e1) != cudaSuccess) rc = HANN_ECUDA;
            cudaEventElapsedTime(&ms_f64, e0, e1);
            cudaEventRecord(e0, c->stream);
            k_probe_imad<<<grid_imad, kProbeThreads, 0, c->stream>>>(out, it_imad);
            cudaEventRecord(e1, c->stream);
            if (cudaEventSynchronize(e1) != cudaSuccess) rc = HANN_ECUDA;
            cudaEventElapsedTime(&ms_imad, e0, e1);
        }
        if (rc != HANN_OK || cudaGetLastError() != cudaSuccess) {
            c->err = "hann_probe_rates: a probe kernel failed";
            rc = HANN_ECUDA;
        }
    }
    if (rc == HANN_OK) {
        *f64_butterflies_per_s = (double)grid_f64 * kProbeThreads * it_f64 * 32.0 / (ms_f64 * 1e-3);   // 4 stages x 8 butterflies per round
        *int32_madds_per_s = (double)grid_imad * kProbeThreads * it_imad * 8.0 / (ms_imad * 1e-3);  // the ninth multiply of a round is not counted
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (out) cudaFree(out);
    cudaSetDevice(prev);
    return rc;
}
