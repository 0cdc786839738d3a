// Variant 1: direct-gather sparse implicit GEMM (any shape).
//
// One CTA owns 128 output pixels and ONE pruning tile (tile_t output channels, which share a kept
// set).  For every chunk of 32 retained columns the four warps gather the activations
//     a[p][j] = x[n][oh*s - pad + kh_j*dil][ow*s - pad + kw_j*dil][c_j]      (zero outside the image)
// straight from NHWC global memory (lane = retained column j, so a warp reads one pixel's
// retained channels: neighbouring addresses), round them to TF32 and store them in the
// 128-byte-swizzled K-major layout tcgen05 reads; the matching [tile_t x 32] weight chunk is
// staged the same way.  One thread then issues four 128 x N x 8 TF32 MMAs that accumulate in
// tensor memory.  This is Algorithm 1 with the vector register replaced by a 128-pixel operand
// tile and the T accumulators by T TMEM columns; the gather is the fused im2col + packing of
// Sec. 3.2 without its buffer.  Epilogue: TMEM -> registers, + bias, ReLU, NHWC store.
//
// It is the fallback for shapes the slab kernel does not take (c_in not a multiple of 4, groups
// that straddle slabs) and the reference point the faster variant is measured against.
#include "nm_internal.h"
#include "nm_ptx.cuh"

namespace {

using namespace nmk;

constexpr int BM = 128;  // output pixels per CTA = MMA M
constexpr int A_BYTES = BM * NM_KCHUNK * 4;

__global__ void __launch_bounds__(128) k_conv_gather(const ConvParams p, const int umma_n, const int tmem_cols)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_bar;
    __shared__ uint32_t s_tmem;
    __shared__ int s_row_n[BM], s_row_ih0[BM], s_row_iw0[BM];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int r = blockIdx.y;  // pruning tile
    const long long pix0 = static_cast<long long>(blockIdx.x) * BM;

    const uint32_t a_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t b_base = a_base + A_BYTES;
    const uint32_t bar = smem_u32(&s_bar);

    // ---- set-up --------------------------------------------------------------------------------
    if (warp == 0) tmem_alloc(smem_u32(&s_tmem), tmem_cols);
    if (tid == 0) {
        mbar_init(bar, 1);
        mbar_fence_init();
    }
    {
        const long long pix = pix0 + tid;
        if (pix < p.pixels) {
            const int hw = p.ho * p.wo;
            const int n = static_cast<int>(pix / hw);
            const int rem = static_cast<int>(pix - static_cast<long long>(n) * hw);
            const int oh = rem / p.wo, ow = rem - oh * p.wo;
            s_row_n[tid] = n;
            s_row_ih0[tid] = oh * p.stride_h - p.pad_h;
            s_row_iw0[tid] = ow * p.stride_w - p.pad_w;
        } else {
            s_row_n[tid] = -1;
            s_row_ih0[tid] = 0;
            s_row_iw0[tid] = 0;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    const uint32_t idesc = umma_idesc_tf32(BM, umma_n);
    const uint64_t adesc0 = umma_desc_k_sw128(a_base, 1024);
    const uint64_t bdesc0 = umma_desc_k_sw128(b_base, 1024);

    const uint32_t* taps = p.taps + static_cast<size_t>(r) * p.kk_pad;
    const int row_base = warp * 32;
    uint32_t phase = 0;
    bool failed = false;

    // ---- main loop over chunks of 32 retained columns --------------------------------------------
    for (int c0 = 0; c0 < p.kk_pad; c0 += NM_KCHUNK) {
        // gather: lane = retained column c0 + lane
        const uint32_t tap = taps[c0 + lane];
        const bool tap_ok = tap != NM_TAP_PAD;
        const int dh = static_cast<int>(tap >> 24) * p.dil_h;
        const int dw = static_cast<int>((tap >> 16) & 0xFFu) * p.dil_w;
        const int c = static_cast<int>(tap & 0xFFFFu);
#pragma unroll 8
        for (int i = 0; i < 32; ++i) {
            const int row = row_base + i;
            const int n = s_row_n[row];
            const int ih = s_row_ih0[row] + dh, iw = s_row_iw0[row] + dw;
            float v = 0.f;
            if (tap_ok && n >= 0 && ih >= 0 && ih < p.h && iw >= 0 && iw < p.w)
                // self-checking build: the tap table may only name taps and channels of this layer
                NM_CHECKED(c < p.c_in && static_cast<int>(tap >> 24) < p.kh && static_cast<int>((tap >> 16) & 0xFFu) < p.kw && n < p.batch,
                           p.status, 101, tap)
                v = __ldg(p.x + ((static_cast<size_t>(n) * p.h + ih) * p.w + iw) * p.c_in + c);
            const uint32_t dst = a_base + row * 128 + ((((lane >> 2) ^ (row & 7))) << 4) + ((lane & 3) << 2);
            NM_CHECKED(dst >= a_base && dst + 4 <= a_base + A_BYTES, p.status, 102, dst - a_base)
            asm volatile("st.shared.f32 [%0], %1;" ::"r"(dst), "f"(to_tf32(v)) : "memory");
        }
        // weight chunk [umma_n rows x 32 columns]; rows past the tile or past c_out are zero
        for (int idx = tid; idx < umma_n * 8; idx += 128) {
            const int row = idx >> 3, ch = idx & 7;
            const int o = r * p.tile_t + row;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (row < p.tile_t && o < p.c_out)
                v = __ldg(reinterpret_cast<const float4*>(p.wt + static_cast<size_t>(o) * p.kk_pad + c0) + ch);
            const uint32_t dst = b_base + row * 128 + ((ch ^ (row & 7)) << 4);
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
                         : "memory");
        }
        fence_proxy_async();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
#pragma unroll
            for (int kq = 0; kq < NM_KCHUNK / 8; ++kq)
                umma_tf32_ss(tmem, adesc0 + 2 * kq, bdesc0 + 2 * kq, idesc, (c0 > 0 || kq > 0) ? 1u : 0u);
            umma_commit(bar);
        }
        const bool ok = mbar_wait(bar, phase);
        phase ^= 1;
        if (__syncthreads_or(ok ? 0 : 1)) {
            failed = true;
            break;
        }
    }

    // ---- epilogue ----------------------------------------------------------------------------------
    if (!failed) {
        tc_fence_after();
        const long long pix = pix0 + row_base + lane;
        float* yrow = p.y + static_cast<size_t>(pix < p.pixels ? pix : 0) * p.c_out;
        const int o_base = r * p.tile_t;
        const int n_valid = min(p.tile_t, p.c_out - o_base);
        const bool vec_ok = (p.c_out % 4 == 0) && (p.tile_t % 4 == 0);
        for (int col0 = 0; col0 < n_valid; col0 += 16) {
            uint32_t v[16];
            tmem_ld16(tmem + (static_cast<uint32_t>(row_base) << 16) + col0, v);
            tmem_ld_wait();
            if (pix < p.pixels) {
                if (vec_ok && col0 + 16 <= n_valid) {
#pragma unroll
                    for (int q = 0; q < 16; q += 4) {
                        float4 o4;
                        float* o = reinterpret_cast<float*>(&o4);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            float t = __uint_as_float(v[q + e]);
                            if (p.bias) t += __ldg(p.bias + o_base + col0 + q + e);
                            if (p.residual) t += __ldg(p.residual + (yrow - p.y) + o_base + col0 + q + e);
                            o[e] = p.relu ? fmaxf(t, 0.f) : t;
                        }
                        *reinterpret_cast<float4*>(yrow + o_base + col0 + q) = o4;
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < 16; ++q) {
                        if (col0 + q < n_valid) {
                            float t = __uint_as_float(v[q]);
                            if (p.bias) t += __ldg(p.bias + o_base + col0 + q);
                            if (p.residual) t += __ldg(p.residual + (yrow - p.y) + o_base + col0 + q);
                            yrow[o_base + col0 + q] = p.relu ? fmaxf(t, 0.f) : t;
                        }
                    }
                }
            }
        }
    } else if (tid == 0) {
        atomicExch(p.status + 0, static_cast<int>(NM_ERR_TIMEOUT));
        atomicExch(p.status + 1, 1);  // where: variant 1 main loop
        atomicExch(p.status + 2, static_cast<int>(blockIdx.x));
    }

    // ---- teardown ------------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, tmem_cols);
}

}  // namespace

namespace nmhost {

nm_status_t launch_conv_gather(const ConvParams& p, cudaStream_t st)
{
    const int umma_n = p.tile_t <= 16 ? 16 : ((p.tile_t + 15) / 16) * 16;
    if (umma_n > 256) return fail(NM_ERR_UNSUPPORTED, "nm_conv2d: tile_t %d exceeds 256", p.tile_t);
    int tmem_cols = 32;
    while (tmem_cols < umma_n) tmem_cols <<= 1;
    // shared memory: alignment slack + A tile + B tile; padded so that the CTAs resident on one
    // SM never ask for more than the 512 TMEM columns it has
    size_t smem = 1024 + A_BYTES + static_cast<size_t>(umma_n) * 128;
    const int max_ctas = 512 / tmem_cols;
    const size_t floor_bytes = (227 * 1024) / (max_ctas + 1) + 1;
    if (max_ctas < 16 && smem < floor_bytes) smem = floor_bytes;

    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(k_conv_gather, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(smem));
        if (e != cudaSuccess) return fail(NM_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    }
    const long long tiles_m = (p.pixels + BM - 1) / BM;
    if (tiles_m > 0x7FFFFFFFll) return fail(NM_ERR_UNSUPPORTED, "nm_conv2d: too many output pixels");
    const dim3 grid(static_cast<unsigned>(tiles_m), p.n_tiles);
    k_conv_gather<<<grid, 128, smem, st>>>(p, umma_n, tmem_cols);
    count_launch(1);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "nm_conv2d launch (variant 1): %s", cudaGetErrorString(e));
    return NM_OK;
}

}  // namespace nmhost
