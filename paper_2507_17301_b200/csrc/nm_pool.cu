// Max pooling over NHWC fp32 activations: the one layer between the stem and the first residual
// block of the ResNets measured in Sec. 4.5, so that a whole convolution backbone can be chained
// through this library.  Pure streaming work: one thread per (output pixel, 4 channels), 16-byte
// loads and stores, window positions outside the image ignored.
#include <cfloat>

#include "nm_internal.h"
#include "nm_ptx.cuh"

namespace {

__global__ void k_maxpool(const float4* __restrict__ x, int h, int w, int c4, int kh, int kw, int stride_h,
                          int stride_w, int pad_h, int pad_w, int ho, int wo, size_t total, float4* __restrict__ y)
{
    nmk::pdl_wait();   // x is usually the output of the kernel launched just before
    for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const int cq = static_cast<int>(i % c4);
        size_t pix = i / c4;
        const int ow = static_cast<int>(pix % wo);
        pix /= wo;
        const int oh = static_cast<int>(pix % ho);
        const size_t n = pix / ho;
        float4 m = make_float4(-FLT_MAX, -FLT_MAX, -FLT_MAX, -FLT_MAX);
        for (int i_h = 0; i_h < kh; ++i_h) {
            const int ih = oh * stride_h - pad_h + i_h;
            if (ih < 0 || ih >= h) continue;
            for (int i_w = 0; i_w < kw; ++i_w) {
                const int iw = ow * stride_w - pad_w + i_w;
                if (iw < 0 || iw >= w) continue;
                const float4 v = __ldg(x + ((n * h + ih) * w + iw) * c4 + cq);
                m.x = fmaxf(m.x, v.x); m.y = fmaxf(m.y, v.y); m.z = fmaxf(m.z, v.z); m.w = fmaxf(m.w, v.w);
            }
        }
        y[i] = m;
    }
}

// Self-test of the failure path the convolution kernels share: a wait on a barrier that nobody will
// ever complete runs out of its poll budget, the block reports through the status word exactly as
// the kernels do, and returns normally.
__global__ void k_wait_expiry(int* status, uint32_t polls)
{
    __shared__ uint64_t bar;
    const uint32_t b = nmk::smem_u32(&bar);
    if (threadIdx.x == 0) {
        nmk::mbar_init(b, 1);
        nmk::mbar_fence_init();
    }
    __syncthreads();
    const bool ok = nmk::mbar_wait_polls(b, 0, polls);
    if (!__syncthreads_and(ok ? 1 : 0) && threadIdx.x == 0) {
        atomicExch(status + 0, static_cast<int>(NM_ERR_TIMEOUT));
        atomicExch(status + 1, 99);   // where: the self-test
        atomicExch(status + 2, static_cast<int>(blockIdx.x));
    }
}

}  // namespace

extern "C" nm_status_t nm_selftest_wait_expiry(const nm_weights_t* w, void* cuda_stream)
{
    if (!w || w->magic != NM_MAGIC) return nmhost::fail(NM_ERR_INVALID_ARG, "nm_selftest_wait_expiry: bad weights handle");
    k_wait_expiry<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(w->status, 2000u);
    nmhost::count_launch(1);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return nmhost::fail(NM_ERR_CUDA, "nm_selftest_wait_expiry launch: %s", cudaGetErrorString(e));
    return NM_OK;
}

extern "C" nm_status_t nm_maxpool2d(const float* x, int batch, int h, int w, int c, int kh, int kw, int stride_h,
                                    int stride_w, int pad_h, int pad_w, float* y, void* cuda_stream)
{
    if (!x || !y) return nmhost::fail(NM_ERR_INVALID_ARG, "nm_maxpool2d: x or y is NULL");
    if (batch < 1 || h < 1 || w < 1 || c < 1 || kh < 1 || kw < 1 || stride_h < 1 || stride_w < 1 || pad_h < 0 || pad_w < 0)
        return nmhost::fail(NM_ERR_INVALID_ARG, "nm_maxpool2d: sizes must be positive, padding >= 0");
    if (pad_h >= kh || pad_w >= kw)
        return nmhost::fail(NM_ERR_INVALID_ARG, "nm_maxpool2d: padding must be smaller than the window (no empty windows)");
    if (c % 4 != 0) return nmhost::fail(NM_ERR_UNSUPPORTED, "nm_maxpool2d: c must be a multiple of 4");
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y)) & 15u)
        return nmhost::fail(NM_ERR_INVALID_ARG, "nm_maxpool2d: x and y must be 16-byte aligned");
    const long long eh = static_cast<long long>(h) + 2ll * pad_h - kh, ew = static_cast<long long>(w) + 2ll * pad_w - kw;
    if (eh < 0 || ew < 0) return nmhost::fail(NM_ERR_INVALID_ARG, "nm_maxpool2d: the window does not fit the padded image");
    const int ho = static_cast<int>(eh / stride_h) + 1, wo = static_cast<int>(ew / stride_w) + 1;
    const size_t total = static_cast<size_t>(batch) * ho * wo * (c / 4);
    size_t blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    cudaError_t e = nmhost::launch_pdl(k_maxpool, static_cast<unsigned>(blocks), 256u, 0, static_cast<cudaStream_t>(cuda_stream),
                                       reinterpret_cast<const float4*>(x), h, w, c / 4, kh, kw, stride_h, stride_w, pad_h,
                                       pad_w, ho, wo, total, reinterpret_cast<float4*>(y));
    nmhost::count_launch(1);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return nmhost::fail(NM_ERR_CUDA, "nm_maxpool2d launch: %s", cudaGetErrorString(e));
    return NM_OK;
}
