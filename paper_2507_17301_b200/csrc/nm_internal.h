// Library-internal declarations shared by the host API and the kernel translation units.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/nm.h"

constexpr uint32_t NM_MAGIC = 0x4E4D5754u;  // "NMWT"
constexpr uint32_t NM_TAP_PAD = 0xFFFFFFFFu;  // tap-table entry of a padding column: gathers zero
constexpr int NM_KCHUNK = 32;               // kept columns per shared-memory operand chunk (128 B of TF32)

// Compressed weights of one layer.  `values` / `indices` are the canonical, exportable form;
// `wt` and `taps` are what the convolution kernels read.
struct nm_weights {
    uint32_t magic;
    int device;
    int c_out, kh, kw, c_in, k, kk, n_keep, m_group, tile_t, n_tiles;
    int kk_pad;          // kk rounded up to a multiple of NM_KCHUNK
    double l1_total, l1_kept;   // L1 mass of the dense weights / of the retained ones (l1_total < 0: not known)
    float* values;       // [c_out][kk]     exact fp32 copies of the retained weights
    uint16_t* indices;   // [n_tiles][kk]   retained column positions, ascending
    float* wt;           // [c_out][kk_pad] retained weights rounded to TF32 (nearest), zero padded
    uint32_t* taps;      // [n_tiles][kk_pad] kh << 24 | kw << 16 | c per retained column, NM_TAP_PAD in the padding
    int* status;         // device int[4]: [0] error code, [1] where, [2] block, [3] spare
    // Slab layout (variant 2); v2_ok = 0 when the N:M pattern does not fit it.
    // The reduction axis is cut into chunks of v2_g whole groups: v2_s = g * M source columns, of
    // which every tile keeps v2_kc = g * N (a multiple of 8, at most 32).
    int v2_ok, v2_g, v2_kc, v2_s, v2_chunks;
    float* wt2;          // [c_out][v2_chunks * 32] TF32 weights, chunk-major, first v2_kc of each 32 used
    uint8_t* rel2;       // [n_tiles][v2_chunks * 32] source column of each kept column, relative to its chunk
    // Expanded layout (variant 4): the pruned matrix back in dense shape, zeros in the pruned columns.
    float* splitk;       // scratch for split-K partial sums (variant 4), allocated by nm_autotune; may be NULL
    size_t splitk_bytes;
    float* wx;           // [ceil(k / 32)][wx_rows][32] TF32, rows swizzled (see k_expand); NULL when the shape rules the variant out
    int wx_rows;         // c_out rounded up to a multiple of 32 (the rows past c_out are zero)
    // Select layout (variant 8): chunks of sel_s source columns of which every tile keeps sel_kc; NULL when the
    // pattern or the shape rules the variant out.
    float* w3;           // [k / sel_s][c_out][32] TF32, rows swizzled (see k_build_w3)
    uint8_t* sel3;       // [k / sel_s][n_tiles][sel_mw bytes] select masks, 32-bit words (see k_build_sel3)
    int sel_s, sel_kc, sel_mw;
    // Plane layout (variant 9): per kernel row a [c_out][32] tile of (kw, c) slots; NULL when the shape rules it out.
    float* ws;           // [kh][c_out][32] TF32, rows swizzled (see k_build_ws)
};

// Geometry handed to the convolution kernels.
struct ConvParams {
    const float* x;
    const float* wt;
    const uint32_t* taps;
    const float* bias;
    const float* residual;   // shortcut input added before the activation: the output's shape, or NULL
    float* y;
    int* status;
    int batch, h, w, c_in, ho, wo, c_out;
    int stride_h, stride_w, pad_h, pad_w, dil_h, dil_w;
    int kh, kw;
    int kk, kk_pad, tile_t, n_tiles, relu;
    int n_keep, m_group;
    long long pixels;  // batch * ho * wo
    int k;
    // slab layout (variant 2)
    const float* wt2;
    const uint8_t* rel2;
    int v2_kc, v2_s, v2_chunks;
    // expanded layout (variant 4)
    const float* wx;
    int wx_rows;
    // split-K scratch of the handle (variant 4 with plan.split > 1, variant 8 with plan.ksplit > 1)
    float* splitk;
    size_t splitk_bytes;
    // select layout (variant 8)
    const float* w3;
    const uint8_t* sel3;
    int sel_s, sel_kc, sel_mw;
    // plane layout (variant 9)
    const float* ws;
};

#ifdef __CUDACC__
// Shortcut input of one output pixel from channel `channel` on, as float4s (NULL without a residual or past the end).
__device__ __forceinline__ const float4* nm_residual_row(const ConvParams& p, long long pixel, int channel)
{
    if (!p.residual || pixel >= p.pixels) return nullptr;
    return reinterpret_cast<const float4*>(p.residual + pixel * p.c_out + channel);
}
__device__ __forceinline__ void nm_add4(float4& a, const float4& b)
{
    a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
}
#endif

#ifdef __CUDACC__
// Self-checking build (-DNM_DEBUG_BOUNDS): the kernels that compute addresses from index data range-check
// every such address; a violation is recorded in the handle's status word (error code NM_ERR_INTERNAL, the
// site, the block, the offending value) and the access is skipped.  Nothing traps; nm_weights_check reports it.
#ifdef NM_DEBUG_BOUNDS
__device__ __forceinline__ void nm_debug_violation(int* status, int site, uint32_t value)
{
    if (atomicCAS(status + 0, 0, static_cast<int>(NM_ERR_INTERNAL)) == 0) {
        atomicExch(status + 1, site);
        atomicExch(status + 2, static_cast<int>(blockIdx.x));
        atomicExch(status + 3, static_cast<int>(value));
    }
}
#define NM_CHECKED(cond, status, site, value) \
    if (!(cond)) nm_debug_violation((status), (site), static_cast<uint32_t>(value)); else
#else
#define NM_CHECKED(cond, status, site, value)
#endif
#endif

namespace nmhost {
// Launches `kernel` so that it may begin while the previous kernel of the stream drains
// (programmatic dependent launch); the kernel orders itself with griddepcontrol.wait.
// NM_NO_PDL=1 in the environment falls back to a plain launch.
bool pdl_enabled();
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t st,
                       Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Raises a kernel's dynamic shared-memory limit on the current device, calling the runtime only when a launch
// needs more than the limit already in force (the call would otherwise sit between every two launches).
cudaError_t ensure_dynamic_smem(const void* kernel, size_t bytes);

// Sets the calling thread's error text and returns `s`.
nm_status_t fail(nm_status_t s, const char* fmt, ...);
void count_launch(int n = 1);

// nm_prune.cu
nm_status_t prune_on_device(const float* w_dense, nm_weights* h, cudaStream_t st);
nm_status_t build_from_compressed(const float* values, const uint16_t* indices, nm_weights* h, cudaStream_t st);

nm_status_t build_slab_layout(nm_weights* h, cudaStream_t st);
nm_status_t build_expanded_layout(nm_weights* h, cudaStream_t st);

// nm_conv_gather.cu — variant 1
nm_status_t launch_conv_gather(const ConvParams& p, cudaStream_t st);

// nm_conv_slab.cu — variant 2
bool slab_plan_ok(const ConvParams& p, const nm_plan_t* plan);
nm_status_t launch_conv_slab(const ConvParams& p, const nm_plan_t* plan, cudaStream_t st);

// nm_conv_expand.cu — variant 4
bool expand_plan_ok(const ConvParams& p, const nm_plan_t* plan);
size_t expand_splitk_bytes(const ConvParams& p, int splits);   // scratch a split-K plan of this layer needs
size_t expand_balanced_bytes(int bn);                          // scratch a balanced plan (split = -1) with this bn needs
nm_status_t launch_conv_expand(const ConvParams& p, const nm_plan_t* plan, cudaStream_t st);

// second pass of a plan that splits the reduction axis: y = act(sum of the `splits` partial sums
// [split][p_pad pixels][c_out] in p.splitk + bias + shortcut)
nm_status_t launch_splitk_reduce(const ConvParams& p, int splits, int p_pad, cudaStream_t st);

// nm_conv_rowrun.cu — variant 5
bool rowrun_plan_ok(const ConvParams& p, const nm_plan_t* plan);
nm_status_t launch_conv_rowrun(const ConvParams& p, const nm_plan_t* plan, cudaStream_t st);

// nm_conv_window.cu — variant 6
bool window_plan_ok(const ConvParams& p, const nm_plan_t* plan);
nm_status_t launch_conv_window(const ConvParams& p, const nm_plan_t* plan, cudaStream_t st);

// nm_conv_pair.cu — variant 7
bool pair_plan_ok(const ConvParams& p, const nm_plan_t* plan);
nm_status_t launch_conv_pair(const ConvParams& p, const nm_plan_t* plan, cudaStream_t st);

// nm_conv_stream.cu — variant 3
bool stream_plan_ok(const ConvParams& p, const nm_plan_t* plan);
nm_status_t launch_conv_stream(const ConvParams& p, const nm_plan_t* plan, cudaStream_t st);

// nm_conv_select.cu — variant 8
nm_status_t build_select_layout(nm_weights* h, cudaStream_t st);
bool select_plan_ok(const ConvParams& p, const nm_plan_t* plan);
size_t select_splitk_bytes(const ConvParams& p, int splits);
nm_status_t launch_conv_select(const ConvParams& p, const nm_plan_t* plan, cudaStream_t st);

// nm_conv_planes.cu — variant 9
nm_status_t build_planes_layout(nm_weights* h, cudaStream_t st);
bool planes_plan_ok(const ConvParams& p, const nm_plan_t* plan);
nm_status_t launch_conv_planes(const ConvParams& p, const nm_plan_t* plan, cudaStream_t st);
}  // namespace nmhost
