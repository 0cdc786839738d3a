// Variant 9: plane kernel — implicit GEMM for layers with at most four input channels and a horizontal
// stride of 1 or 2 (the 7x7 / 2, 3-channel stem of a ResNet), with NO patch matrix built anywhere:
// the tensor core reads the taps straight out of the input rows held in shared memory.
//
// A pixel's channels are padded to four floats (16 bytes), and the pixels of an input row (zero padding
// included) are stored de-interleaved by column parity when the stride is 2: plane q holds padded columns
// q, q + 2, ...  Then, for a fixed tap (kh, kw), the operand rows of CONSECUTIVE output pixels are
// consecutive 16-byte entries of one plane of one input row: eight of them are exactly one 8 x 16-byte
// core matrix of the tensor core's unswizzled K-major layout, the next eight output pixels the next 128
// bytes (stride between 8-row groups = 128 bytes), and the tap kw + 1 the same entries of the other plane
// (stride 2) or the next entry (stride 1): the stride between the two core matrices of a K = 8 MMA.  One
// tcgen05.mma of shape 128 x C_out x 8 therefore multiplies two taps x four channels of 128 output pixels
// of one output row, and the fused im2col + packing of Sec. 3.2 costs nothing but a descriptor.
//
//   loaders (8 warps)        copy the input rows of a band of R output rows from global memory into the
//                            planes: one thread per pixel, c_in loads and one 16-byte store; everything outside
//                            the image is written as zeros
//   MMA issuers (R threads)  one per output row of the band (its own accumulator columns): kh x ceil(kw / 2)
//                            MMAs against the weights, which stay in shared memory for the whole kernel
//                            (per kernel row a [C_out x 32] swizzled tile: kw padded to 8 taps, channels to 4,
//                            zeros in the padding and in pruned columns, so any N:M and tile width works)
//   epilogue (16 warps)      four per output row of the band (one per 32 accumulator lanes): TMEM -> registers,
//                            + bias (+ shortcut), ReLU, staged and stored with TMA; pixels past the end of the
//                            output row are clipped by the store's bounds check.  A 32 x 32 block takes a warp
//                            about 2 k cycles of latencies in series (TMEM load, staging, proxy fence, store),
//                            hence a warp per (row, lane quarter): the epilogue of an item is two blocks deep
// A work item is (image, band of R output rows); persistent CTAs, static schedule; accumulators and planes
// are double-buffered; every wait is bounded and reports through the handle's status word.
#include "nm_internal.h"
#include "nm_ptx.cuh"
#include "nm_tmap.cuh"

namespace {

using namespace nmk;

constexpr int BM = 128;
constexpr int MAX_R = 4;            // output rows per work item = MMA issuer threads
constexpr int LOAD_WARPS = 8;
constexpr int EPI_WARPS = 4 * MAX_R;
constexpr int THREADS = (4 + EPI_WARPS + LOAD_WARPS) * 32;   // warps 0-3 issuers, 4-19 epilogue, 20-27 loaders
constexpr int MAX_SLOTS = 3;
constexpr int STAGING_BYTES = EPI_WARPS * 4096;             // one 32 x 32 box per epilogue warp
constexpr int LOAD_UNROLL = 6;

struct PlaneCfg {
    int r;            // output rows per item
    int npair;        // MMAs per kernel row = ceil(kw / 2)
    int pe;           // 16-byte entries per plane
    int row_pitch;    // bytes per input row = planes * pe * 16
    int nrows;        // input rows per item = (r - 1) * stride_h + (kh - 1) * dil_h + 1
    int slot_bytes;   // nrows * row_pitch, plus slack for the rows past an output row's end
    int n_slots;
    int w_bytes;      // kh * c_out * 128
    int bands;        // ceil(ho / r)
    int acc_cols;     // r * c_out
    long long n_work; // batch * bands
};

__device__ __forceinline__ bool aborted(volatile int* flag) { return *flag != 0; }

template <int S>
__global__ void __launch_bounds__(THREADS, 1)
k_conv_planes(const ConvParams p, const PlaneCfg cfg, const __grid_constant__ CUtensorMap tm_y)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_wfull, s_pfull[MAX_SLOTS], s_pfree[MAX_SLOTS], s_accfull[2], s_accfree[2];
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t n_work = static_cast<uint32_t>(cfg.n_work);   // below 2^31: per-item arithmetic stays 32-bit
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t w_smem = base;
    const uint32_t staging = w_smem + ((cfg.w_bytes + 1023) / 1024) * 1024;
    const uint32_t planes = staging + STAGING_BYTES;
    volatile int* abort_flag = &s_abort;

    if (warp == 4) tmem_alloc(smem_u32(&s_tmem), 512);
    if (tid == 0) {
        mbar_init(smem_u32(&s_wfull), 1);
        for (int i = 0; i < MAX_SLOTS; ++i) {
            mbar_init(smem_u32(&s_pfull[i]), LOAD_WARPS);
            mbar_init(smem_u32(&s_pfree[i]), cfg.r);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&s_accfull[i]), cfg.r);
            mbar_init(smem_u32(&s_accfree[i]), EPI_WARPS);
        }
        mbar_fence_init();
        s_abort = 0;
        tma_prefetch_desc(&tm_y);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    pdl_launch_dependents();   // the next kernel may start its own set-up as SMs become free
    pdl_wait();                // from here on global memory written by the previous kernel is read

    if (warp < 4) {
        // =========================== MMA issuers ===========================
        if (lane == 0 && warp == 0) {
            mbar_arrive_expect_tx(smem_u32(&s_wfull), static_cast<uint32_t>(cfg.w_bytes));
            bulk_load_1d(w_smem, p.ws, static_cast<uint32_t>(cfg.w_bytes), smem_u32(&s_wfull));
        }
        if (lane == 0 && warp < cfg.r) {
            const int mi = warp;
            const uint32_t idesc = umma_idesc_tf32(BM, p.c_out);
            const uint32_t lbo = S == 2 ? static_cast<uint32_t>(cfg.pe) * 16u : 16u;
            const uint32_t pair_units = S == 2 ? 1u : 2u;   // 16-byte units from one pair of taps to the next
            const uint32_t w_row_units = static_cast<uint32_t>(p.c_out) * 8u;   // (c_out * 128 bytes) / 16
            const uint32_t a_row_units = static_cast<uint32_t>(p.dil_h * cfg.row_pitch) >> 4;
            RingPos rp;
            uint32_t ab = 0, acc_par = 0;
            bool acc_wrapped = false;
            if (!mbar_wait(smem_u32(&s_wfull), 0)) *abort_flag = 9;
            const uint64_t b0 = umma_desc_k_sw128(w_smem, 1024);
            for (uint32_t work = blockIdx.x; work < n_work && !aborted(abort_flag); work += gridDim.x) {
                if (acc_wrapped && !mbar_wait_lone(smem_u32(&s_accfree[ab]), acc_par ^ 1u)) { *abort_flag = 5; break; }
                if (!mbar_wait_lone(smem_u32(&s_pfull[rp.s]), rp.parity)) { *abort_flag = 6; break; }
                tc_fence_after();
                const uint32_t acc = tmem + ab * cfg.acc_cols + mi * p.c_out;
                uint64_t a_row = umma_desc_k_plain(planes + rp.s * cfg.slot_bytes + mi * p.stride_h * cfg.row_pitch, lbo, 128);
                uint64_t b_row = b0;
                for (int khi = 0; khi < p.kh; ++khi) {
                    for (int j = 0; j < cfg.npair; ++j)
                        umma_tf32_ss(acc, a_row + j * pair_units, b_row + 2 * j, idesc, (khi > 0 || j > 0) ? 1u : 0u);
                    a_row += a_row_units;
                    b_row += w_row_units;
                }
                umma_commit(smem_u32(&s_pfree[rp.s]));
                umma_commit(smem_u32(&s_accfull[ab]));
                rp.advance(cfg.n_slots);
                if (ab == 1) { acc_par ^= 1u; acc_wrapped = true; }
                ab ^= 1u;
            }
        }
    } else if (warp < 4 + EPI_WARPS) {
        // =========================== epilogue ===========================
        const int q = warp & 3, mi = (warp - 4) >> 2;   // TMEM lane quarter, output row of the band
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t box = staging + (warp - 4) * 4096;
        const uint32_t stage_row = box + lane * 128;
        const uint32_t rx = static_cast<uint32_t>(lane & 7);
        const int n_blk = p.c_out / 32;
        const bool has_row = mi < cfg.r;
        uint32_t nb = 0, ti = 0;
        // the bias of a block is held one value per lane and fetched a block ahead (it is the same for every item)
        float bias_next = has_row ? bias_lane_load(p.bias, 0, p.c_out, lane) : 0.f;
        for (uint32_t work = blockIdx.x; work < n_work; work += gridDim.x, ++ti) {
            const int ab = static_cast<int>(ti & 1u);
            const bool ok = aborted(abort_flag) || mbar_wait(smem_u32(&s_accfull[ab]), (ti >> 1) & 1u);
            if (!__all_sync(0xFFFFFFFFu, ok)) *abort_flag = 8;
            if (__any_sync(0xFFFFFFFFu, aborted(abort_flag))) break;
            tc_fence_after();
            const int n = static_cast<int>(work / static_cast<uint32_t>(cfg.bands));
            const int oh = static_cast<int>(work - static_cast<uint32_t>(n) * static_cast<uint32_t>(cfg.bands)) * cfg.r + mi;
            const bool row_ok = has_row && oh < p.ho;
            const bool box_ok = row_ok && q * 32 < p.wo;
            const long long box_pixel = (static_cast<long long>(n) * p.ho + oh) * p.wo + q * 32;
            const int box_rows = p.wo - q * 32 < 32 ? p.wo - q * 32 : 32;
            for (int blk = 0; has_row && blk < n_blk; ++blk, ++nb) {
                uint32_t v[32];
                tmem_ld32(tmem + lane_addr + ab * cfg.acc_cols + mi * p.c_out + blk * 32, v);
                const float bias_cur = bias_next;
                bias_next = bias_lane_load(p.bias, blk + 1 < n_blk ? (blk + 1) * 32 : 0, p.c_out, lane);
                if (lane == 0 && nb >= 1) tma_store_wait_read();   // the store that last read the box is done with it
                __syncwarp();
                tmem_ld_wait();
                if (blk == n_blk - 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&s_accfree[ab]));
                }
                const int relu_now = p.residual ? 0 : p.relu;   // with a shortcut input the activation follows the addition
#pragma unroll
                for (int qq = 0; qq < 8; ++qq) {
                    float o[4];
                    const float4 bv = bias_quad(bias_cur, qq);
                    o[0] = __uint_as_float(v[qq * 4 + 0]) + bv.x;
                    o[1] = __uint_as_float(v[qq * 4 + 1]) + bv.y;
                    o[2] = __uint_as_float(v[qq * 4 + 2]) + bv.z;
                    o[3] = __uint_as_float(v[qq * 4 + 3]) + bv.w;
                    if (relu_now) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) o[e] = fmaxf(o[e], 0.f);
                    }
                    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(stage_row + ((qq ^ rx) << 4)), "f"(o[0]),
                                 "f"(o[1]), "f"(o[2]), "f"(o[3])
                                 : "memory");
                }
                if (p.residual && box_ok) {
                    __syncwarp();
                    add_residual_box(box, p.residual + box_pixel * p.c_out + blk * 32, p.c_out, box_rows, p.relu, lane);
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                    // output seen as (channel, ow, n * ho + oh): pixels past the row's end are clipped
                    if (box_ok) tma_store_3d(&tm_y, box, blk * 32, q * 32, n * p.ho + oh);
                    tma_store_commit();
                }
            }
            if (!has_row) {   // a band of fewer rows than warps: nothing to read
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&s_accfree[ab]));
            }
        }
        if (lane == 0) tma_store_wait_read();   // shared memory must outlive the stores' reads; the writes complete with the grid
    } else {
        // =========================== loaders ===========================
        // One thread per padded pixel: entry (row j, padded column pp) of the band goes to plane pp % S,
        // entry pp / S.  Consecutive threads take consecutive pixels, so global loads coalesce.
        const int lt = tid - (4 + EPI_WARPS) * 32;
        const int row_px = S * cfg.pe;                 // padded pixels per row as laid out
        const int total = cfg.nrows * row_px;
        RingPos rp;
        for (uint32_t work = blockIdx.x; work < n_work && !aborted(abort_flag); work += gridDim.x) {
            const bool ok = !rp.wrapped || mbar_wait_lone(smem_u32(&s_pfree[rp.s]), rp.parity ^ 1u);
            if (!__all_sync(0xFFFFFFFFu, ok)) *abort_flag = 2;
            if (__any_sync(0xFFFFFFFFu, aborted(abort_flag))) break;
            const int n = static_cast<int>(work / static_cast<uint32_t>(cfg.bands));
            const int oh0 = static_cast<int>(work - static_cast<uint32_t>(n) * static_cast<uint32_t>(cfg.bands)) * cfg.r;
            const int ih0 = oh0 * p.stride_h - p.pad_h;
            const float* img = p.x + static_cast<size_t>(n) * p.h * p.w * p.c_in;
            const uint32_t slot = planes + rp.s * cfg.slot_bytes;
            int j = lt / row_px, pp = lt - j * row_px;      // this thread's first pixel
            const int dj = (LOAD_WARPS * 32) / row_px, dpp = (LOAD_WARPS * 32) - dj * row_px;
            for (int f = lt; f < total; f += LOAD_WARPS * 32 * LOAD_UNROLL) {
                float4 v[LOAD_UNROLL];
                uint32_t dst[LOAD_UNROLL];
#pragma unroll
                for (int u = 0; u < LOAD_UNROLL; ++u) {
                    v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                    const int ih = ih0 + j, iw = pp - p.pad_w;
                    const bool live = f + u * LOAD_WARPS * 32 < total;
                    dst[u] = live ? slot + j * cfg.row_pitch + ((pp % S) * cfg.pe + pp / S) * 16 : 0u;
                    if (live && ih >= 0 && ih < p.h && iw >= 0 && iw < p.w) {
                        const float* src = img + (static_cast<size_t>(ih) * p.w + iw) * p.c_in;
                        if (p.c_in == 4) {
                            v[u] = __ldg(reinterpret_cast<const float4*>(src));
                        } else {
                            v[u].x = __ldg(src);
                            if (p.c_in > 1) v[u].y = __ldg(src + 1);
                            if (p.c_in > 2) v[u].z = __ldg(src + 2);
                        }
                    }
                    pp += dpp; j += dj;
                    if (pp >= row_px) { pp -= row_px; ++j; }
                }
#pragma unroll
                for (int u = 0; u < LOAD_UNROLL; ++u)
                    if (dst[u])
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst[u]), "f"(v[u].x), "f"(v[u].y), "f"(v[u].z),
                                     "f"(v[u].w)
                                     : "memory");
            }
            fence_proxy_async();   // the tensor core reads these bytes through the async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_pfull[rp.s]));
            rp.advance(cfg.n_slots);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && s_abort != 0) {
        (void)mbar_wait(smem_u32(&s_wfull), 0);   // the weight copy may still be in flight
        atomicExch(p.status + 0, static_cast<int>(NM_ERR_TIMEOUT));
        atomicExch(p.status + 1, 90 + s_abort);
        atomicExch(p.status + 2, static_cast<int>(blockIdx.x));
    }
    if (warp == 4) tmem_dealloc(tmem, 512);
}

int sm_count()
{
    static int n = 0;
    if (n == 0) {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
            n = v;
        else
            n = 148;
    }
    return n;
}

bool make_cfg(const ConvParams& p, const nm_plan_t* plan, PlaneCfg* cfg, size_t* smem_out)
{
    if (!p.ws || !nmtm::available()) return false;
    if (p.c_in > 4 || p.kw > 8 || p.dil_w != 1 || (p.stride_w != 1 && p.stride_w != 2)) return false;
    if (p.wo > BM || p.c_out % 32 != 0 || p.c_out > 256) return false;
    if (static_cast<long long>(p.batch) * p.h * p.w * p.c_in >= (1ll << 31)) return false;
    if (p.c_in == 4 && (reinterpret_cast<uintptr_t>(p.x) & 15u) != 0) return false;
    const int s = p.stride_w;
    int r = 256 / p.c_out;                      // two accumulator sets of r * c_out columns in 512
    if (r > MAX_R) r = MAX_R;
    if (plan && plan->split > 0 && plan->split < r) r = plan->split;
    if (r > p.ho) r = p.ho;
    if (r < 1) return false;
    cfg->r = r;
    cfg->npair = (p.kw + 1) / 2;
    // padded columns a valid output pixel can touch: 0 .. s * (wo - 1) + 2 * npair - 1; laid out in whole planes
    const int cols = s * (p.wo - 1) + 2 * cfg->npair;
    const int padded = p.w + 2 * p.pad_w;
    int pe = ((cols > padded ? cols : padded) + s - 1) / s;
    pe = (pe + 1) & ~1;
    cfg->pe = pe;
    cfg->row_pitch = s * pe * 16;
    cfg->nrows = (r - 1) * p.stride_h + (p.kh - 1) * p.dil_h + 1;
    // rows 8 * ceil(wo / 8) .. 127 of an MMA read past the entries a row has: up to 128 + npair entries from
    // the row's first one; the slack keeps those reads inside the slot (their products are never stored)
    cfg->slot_bytes = ((cfg->nrows * cfg->row_pitch + (BM + 2 * cfg->npair) * 16 + 127) / 128) * 128;
    cfg->w_bytes = p.kh * p.c_out * 128;
    cfg->bands = (p.ho + r - 1) / r;
    cfg->acc_cols = r * p.c_out;
    cfg->n_work = static_cast<long long>(p.batch) * cfg->bands;
    if (cfg->n_work >= (1ll << 31) || static_cast<long long>(p.batch) * p.ho >= (1ll << 31)) return false;
    if (cfg->w_bytes >= (1 << 20)) return false;   // one copy, one mbarrier phase
    const size_t fixed = 1024 + static_cast<size_t>((cfg->w_bytes + 1023) / 1024) * 1024 + STAGING_BYTES;
    const size_t budget = 227 * 1024 - 1024;       // static shared memory: barriers and flags
    int n_slots = plan && plan->stages > 0 ? plan->stages : MAX_SLOTS;
    if (n_slots > MAX_SLOTS) return false;
    while (n_slots > 2 && !(plan && plan->stages > 0) && fixed + static_cast<size_t>(n_slots) * cfg->slot_bytes > budget) --n_slots;
    if (n_slots < 2 || fixed + static_cast<size_t>(n_slots) * cfg->slot_bytes > budget) return false;
    cfg->n_slots = n_slots;
    const size_t smem = fixed + static_cast<size_t>(n_slots) * cfg->slot_bytes;
    *smem_out = smem < 120 * 1024 ? 120 * 1024 : smem;   // one CTA per SM: it owns all of tensor memory
    return true;
}

// Output seen as (c_out, wo, batch * ho) with a 32-channel x 32-pixel x 1-row box.
bool encode_y_rows(const ConvParams& p, CUtensorMap* tm)
{
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(p.c_out), static_cast<cuuint64_t>(p.wo),
                                static_cast<cuuint64_t>(p.batch) * p.ho};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(p.c_out) * 4, static_cast<cuuint64_t>(p.wo) * p.c_out * 4};
    const cuuint32_t box[3] = {32, 32, 1};
    const cuuint32_t es[3] = {1, 1, 1};
    return nmtm::encoders().tiled(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, p.y, dims, strides, box, es,
                                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The handle's weights for this kernel: ws[kh][c_out][32] TF32; a row holds the taps of one kernel row as
// (kw, c) with c padded to 4 and kw to 8, its 16-byte pieces (one tap each) XOR-ed with (o % 8) (128-byte
// swizzle); zeros in the padding and in pruned columns.
__global__ void k_build_ws(const float* __restrict__ values, const uint16_t* __restrict__ indices, int c_out, int kk,
                           int tile_t, int kw, int c_in, float* __restrict__ ws)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int o = blockIdx.y;
    if (j >= kk) return;
    const int k = indices[static_cast<size_t>(o / tile_t) * kk + j];
    const int run = kw * c_in;
    const int khi = k / run, r = k - khi * run;
    const int kwi = r / c_in, c = r - kwi * c_in;
    ws[(static_cast<size_t>(khi) * c_out + o) * 32 + ((kwi ^ (o & 7)) << 2) + c] = to_tf32(values[static_cast<size_t>(o) * kk + j]);
}

}  // namespace

namespace nmhost {

nm_status_t build_planes_layout(nm_weights* h, cudaStream_t st)
{
    h->ws = nullptr;
    if (h->c_in > 4 || h->kw > 8 || h->c_out % 32 != 0 || h->c_out > 256 || h->kk == 0 || h->kh * h->c_out * 128 >= (1 << 20))
        return NM_OK;
    const size_t bytes = static_cast<size_t>(h->kh) * h->c_out * 32 * sizeof(float);
    if (cudaMalloc(&h->ws, bytes) != cudaSuccess) {
        (void)cudaGetLastError();
        h->ws = nullptr;
        return fail(NM_ERR_ALLOC, "cannot allocate the plane-kernel weights (%zu bytes)", bytes);
    }
    cudaError_t e = cudaMemsetAsync(h->ws, 0, bytes, st);
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "plane layout memset: %s", cudaGetErrorString(e));
    const dim3 grid((h->kk + 127) / 128, h->c_out);
    k_build_ws<<<grid, 128, 0, st>>>(h->values, h->indices, h->c_out, h->kk, h->tile_t, h->kw, h->c_in, h->ws);
    count_launch(1);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "plane layout kernel: %s", cudaGetErrorString(e));
    return NM_OK;
}

bool planes_plan_ok(const ConvParams& p, const nm_plan_t* plan)
{
    PlaneCfg cfg;
    size_t smem;
    return make_cfg(p, plan, &cfg, &smem);
}

nm_status_t launch_conv_planes(const ConvParams& p, const nm_plan_t* plan, cudaStream_t st)
{
    PlaneCfg cfg;
    size_t smem = 0;
    if (!make_cfg(p, plan, &cfg, &smem))
        return fail(NM_ERR_UNSUPPORTED, "nm_conv2d: the plane kernel does not take this layer / plan");
    alignas(64) CUtensorMap tm_y;
    if (!encode_y_rows(p, &tm_y)) return fail(NM_ERR_CUDA, "nm_conv2d: tensor-map encoding failed (variant 9)");
    auto kernel = p.stride_w == 2 ? k_conv_planes<2> : k_conv_planes<1>;
    cudaError_t e = nmhost::ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), smem);
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "cudaFuncSetAttribute (variant 9): %s", cudaGetErrorString(e));
    const long long grid = cfg.n_work < sm_count() ? cfg.n_work : sm_count();
    e = nmhost::launch_pdl(kernel, static_cast<unsigned>(grid), THREADS, smem, st, p, cfg, tm_y);
    nmhost::count_launch(1);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "nm_conv2d launch (variant 9): %s", cudaGetErrorString(e));
    return NM_OK;
}

}  // namespace nmhost
