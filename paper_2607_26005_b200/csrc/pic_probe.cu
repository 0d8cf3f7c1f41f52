// Two microbenchmarks that give the roofline its denominators on the machine at hand (measurement
// aids; they render nothing): a write-only stream with 128-bit stores, and a register-only FFMA loop.
#include <cuda_runtime.h>

#include <cstdio>

#include "../../include/pictura.h"

namespace pic {
void set_last_error(const char* msg);
}

namespace {

// Every thread writes 16-byte words a grid stride apart: the plain write-only stream the image
// store of the rasterizer competes with.
__global__ void __launch_bounds__(256) probe_fill_kernel(uint4* __restrict__ dst, size_t n_words) {
    const uint4 v = make_uint4(0x3c003c00u, 0x3c003c00u, 0x3c003c00u, 0x3c003c00u);
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n_words; i += (size_t)gridDim.x * blockDim.x) dst[i] = v;
}

// Eight independent chains of dependent fused multiply-adds per thread, registers only.
__global__ void __launch_bounds__(256) probe_ffma_kernel(float* __restrict__ out, int iters, float a, float b) {
    float x0 = threadIdx.x, x1 = x0 + 1.f, x2 = x0 + 2.f, x3 = x0 + 3.f, x4 = x0 + 4.f, x5 = x0 + 5.f, x6 = x0 + 6.f, x7 = x0 + 7.f;
#pragma unroll 4
    for (int i = 0; i < iters; ++i) {
        x0 = __fmaf_rn(x0, a, b); x1 = __fmaf_rn(x1, a, b); x2 = __fmaf_rn(x2, a, b); x3 = __fmaf_rn(x3, a, b);
        x4 = __fmaf_rn(x4, a, b); x5 = __fmaf_rn(x5, a, b); x6 = __fmaf_rn(x6, a, b); x7 = __fmaf_rn(x7, a, b);
    }
    out[blockIdx.x * (size_t)blockDim.x + threadIdx.x] = ((x0 + x1) + (x2 + x3)) + ((x4 + x5) + (x6 + x7));
}

pic_status fail(pic_status st, const char* what, cudaError_t ce) {
    char buf[256];
    snprintf(buf, sizeof(buf), "%s: %s", what, cudaGetErrorString(ce));
    pic::set_last_error(buf);
    return st;
}

}  // namespace

extern "C" pic_status pic_probe_fill(void* dst, uint64_t bytes, void* cuda_stream) {
    if (!dst || (reinterpret_cast<uintptr_t>(dst) & 15u) || (bytes & 15u)) {
        pic::set_last_error("pic_probe_fill: dst must be a 16-byte aligned device pointer and bytes a multiple of 16");
        return PIC_ERR_INVALID_ARG;
    }
    if (bytes == 0) return PIC_OK;
    int dev = 0, sms = 0;
    cudaError_t ce = cudaGetDevice(&dev);
    if (ce == cudaSuccess) ce = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (ce != cudaSuccess) return fail(PIC_ERR_CUDA, "pic_probe_fill", ce);
    probe_fill_kernel<<<(unsigned)(sms * 32), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(static_cast<uint4*>(dst), (size_t)(bytes / 16));
    ce = cudaGetLastError();
    return ce == cudaSuccess ? PIC_OK : fail(PIC_ERR_CUDA, "probe_fill_kernel", ce);
}

extern "C" pic_status pic_probe_ffma(float* out, uint64_t out_floats, int32_t iters, uint64_t* fma_count, void* cuda_stream) {
    if (!out || !fma_count || iters <= 0) {
        pic::set_last_error("pic_probe_ffma: out and fma_count are required, iters must be positive");
        return PIC_ERR_INVALID_ARG;
    }
    int dev = 0, sms = 0;
    cudaError_t ce = cudaGetDevice(&dev);
    if (ce == cudaSuccess) ce = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (ce != cudaSuccess) return fail(PIC_ERR_CUDA, "pic_probe_ffma", ce);
    const unsigned grid = (unsigned)(sms * 8);
    if (out_floats < (uint64_t)grid * 256u) {
        pic::set_last_error("pic_probe_ffma: out must hold 2048 floats per multiprocessor");
        return PIC_ERR_CAPACITY;
    }
    probe_ffma_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(out, iters, 0.999f, 0.001f);
    ce = cudaGetLastError();
    if (ce != cudaSuccess) return fail(PIC_ERR_CUDA, "probe_ffma_kernel", ce);
    *fma_count = (uint64_t)grid * 256u * 8u * (uint64_t)iters;
    return PIC_OK;
}
