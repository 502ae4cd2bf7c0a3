// Row-wise FP8 (E4M3) quantisation for the optional FP8 LM head (not part of the paper: the LM head is
// the largest weight stream of a draft step, and a draft head's precision affects only how many
// tokens the target accepts, never what it emits).  q[r, :] = e4m3(x[r, :] / scale[r]),
// scale[r] = max|x[r, :]| / 448 (1 for a zero row); round to nearest even, saturating.  Scale and
// quotient are formed with IEEE single-precision division, so the codes are reproducible.
#include <cuda_fp8.h>

#include "kernels.h"

namespace beagle {

namespace {

template <typename T>
__global__ void __launch_bounds__(256) quantize_rows_e4m3_kernel(const T* x, int cols, uint8_t* __restrict__ q,
                                                                float* __restrict__ scale) {
    constexpr int VN = VecOf<T>::N;
    const size_t row = blockIdx.x;
    const T* xr = x + row * cols;
    pdl_wait();
    pdl_launch_dependents();
    __shared__ float s_max[8];
    float m = 0.f;
    for (int i = threadIdx.x * VN; i < cols; i += 256 * VN) {          // cols is a multiple of 8
        float f[VN];
        unpack16<T>(ld_act16(xr + i), f);
#pragma unroll
        for (int k = 0; k < VN; ++k) m = fmaxf(m, fabsf(f[k]));
    }
    m = warp_max(m);
    if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = m;
    __syncthreads();
    float amax = s_max[0];
#pragma unroll
    for (int w = 1; w < 8; ++w) amax = fmaxf(amax, s_max[w]);
    const float sc = amax > 0.f ? __fdiv_rn(amax, 448.0f) : 1.0f;
    if (threadIdx.x == 0) scale[row] = sc;
    for (int i = threadIdx.x * VN; i < cols; i += 256 * VN) {
        float f[VN];
        unpack16<T>(ld_act16(xr + i), f);
        uint8_t o[VN];
#pragma unroll
        for (int k = 0; k < VN; ++k) o[k] = (uint8_t)__nv_cvt_float_to_fp8(__fdiv_rn(f[k], sc), __NV_SATFINITE, __NV_E4M3);
        if (VN == 8) *reinterpret_cast<uint2*>(q + row * cols + i) = *reinterpret_cast<const uint2*>(o);
        else *reinterpret_cast<uint32_t*>(q + row * cols + i) = *reinterpret_cast<const uint32_t*>(o);
    }
}

}  // namespace

int launch_quantize_rows_e4m3(int dtype, const void* x, long long rows, int cols, void* q, float* scale, cudaStream_t stream) {
    if (rows <= 0) return 0;
    if (cols % 8 || rows > 0x7fffffffll) return -1;
    if (dtype == 0) launch_pdl(quantize_rows_e4m3_kernel<float>, dim3((unsigned)rows), dim3(256), 0, stream, (const float*)x, cols, (uint8_t*)q, scale);
    else launch_pdl(quantize_rows_e4m3_kernel<bf16>, dim3((unsigned)rows), dim3(256), 0, stream, (const bf16*)x, cols, (uint8_t*)q, scale);
    return 1;
}

}  // namespace beagle
