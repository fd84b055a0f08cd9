// Error statistics of model outputs against an FP64 reference: the reduction behind the accuracy analysis of
// Section 6 (the deviations delta = D - D_real of Figure 3, their sign balance and size).  A grid-stride pass over
// the outputs, per-thread partial sums in FP64, warp shuffles, one atomic per warp and statistic.
#include <cuda_fp16.h>
#include "mmasim_internal.h"

namespace mmasim {
namespace {

constexpr int NSTAT = 8;

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ double warp_max(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}

template <bool ACC16>
__global__ void __launch_bounds__(256) stats_kernel(int64_t n, const void* D, const double* ref, double* stats) {
    double cnt = 0.0, sum = 0.0, sabs = 0.0, ssq = 0.0, nneg = 0.0, npos = 0.0, mx = 0.0, srel = 0.0;
    for (int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += int64_t(gridDim.x) * blockDim.x) {
        const double d = ACC16 ? double(__half2float(__ushort_as_half(static_cast<const unsigned short*>(D)[i])))
                               : double(__uint_as_float(static_cast<const uint32_t*>(D)[i]));
        const double r = ref[i];
        const double delta = d - r;
        if (!(fabs(delta) <= 1.7976931348623157e308)) continue;      // NaN or infinite on either side: not counted
        cnt += 1.0;
        sum += delta;
        sabs += fabs(delta);
        ssq += delta * delta;
        nneg += delta < 0.0 ? 1.0 : 0.0;
        npos += delta > 0.0 ? 1.0 : 0.0;
        mx = fmax(mx, fabs(delta));
        if (r != 0.0) srel += fabs(delta) / fabs(r);
    }
    const double v[NSTAT] = {warp_sum(cnt), warp_sum(sum), warp_sum(sabs), warp_sum(ssq), warp_sum(nneg), warp_sum(npos),
                             warp_max(mx), warp_sum(srel)};
    if ((threadIdx.x & 31) == 0) {
#pragma unroll
        for (int s = 0; s < NSTAT; ++s) {
            if (s == 6) atomicMax(reinterpret_cast<unsigned long long*>(stats + s), (unsigned long long)__double_as_longlong(v[s]));   // non-negative doubles order like their bit patterns
            else atomicAdd(stats + s, v[s]);
        }
    }
}

}  // namespace

int launch_error_stats(int acc, int64_t n, const void* D, const double* ref, double* stats, cudaStream_t stream) {
    if (acc != ACC_F32 && acc != ACC_F16) { set_error("mmasim_error_stats: the accumulator format must be FP32 or FP16"); return MMASIM_ERR_INVALID_ARG; }
    const int64_t want = (n + 255) / 256;
    const unsigned blocks = unsigned(want < 148 * 8 ? want : 148 * 8);
    if (acc == ACC_F16) stats_kernel<true><<<blocks, 256, 0, stream>>>(n, D, ref, stats);
    else stats_kernel<false><<<blocks, 256, 0, stream>>>(n, D, ref, stats);
    const cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) { set_error("mmasim_error_stats launch failed: %s", cudaGetErrorString(err)); return MMASIM_ERR_CUDA; }
    return MMASIM_OK;
}

}  // namespace mmasim
