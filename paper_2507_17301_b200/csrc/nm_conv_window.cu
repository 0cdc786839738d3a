// Variant 6: window kernel — stride-1 convolutions with a spatial kernel (3x3 and the like) as an
// implicit GEMM whose taps are SHIFTED VIEWS of one input patch held in shared memory.
//
// The im2col form re-reads every input element once per tap (nine 128-byte rows per pixel and
// 32-channel block through the TMA unit).  Here one tiled TMA load brings, per 32-channel block,
// the patch [R + (kh-1)*dil rows x Wp = W + 2*pad columns] once, zero-filled outside the image,
// in the 128-byte-swizzled layout: one 128-byte row per patch pixel.  Output positions are
// numbered along the PADDED width (position = row * Wp + column), so the A operand of tap (i, j)
// for 128 consecutive positions is simply the 128 patch rows that start (i*dil_h*Wp + j*dil_w)
// rows further down: the same shared-memory bytes, another descriptor start address.  Positions
// whose column falls in the padding produce junk rows that are never stored.
//
//   patch producer (1 thread)   one 4-D tiled TMA load per 32-channel block and work item
//   weight producer (1 thread)  one contiguous bulk copy per (32-channel block, tap): the
//                               expanded, pre-swizzled weights [BN x 32] (zeros = pruned columns)
//   MMA issuers (1 thread per   per block and tap four 128 x BN x 8 TF32 tcgen05.mma
//   M-tile)
//   epilogue (4 warps)          TMEM -> registers, + bias, ReLU, 16-byte stores straight to NHWC (each
//                               thread owns one position = 128 contiguous bytes per 32-channel block;
//                               no staging buffer, so shared memory goes to patches and weights)
// A work item is (image, block of R output rows, BN channels) with R * Wp <= 128 * MT positions
// (MT = 1..4 M-tiles sharing patch and weights, each with its own issuer thread and accumulator).
// Persistent CTAs, static schedule, bounded waits.
#include "nm_internal.h"
#include "nm_ptx.cuh"
#include "nm_tmap.cuh"

namespace {

using namespace nmk;

constexpr int BM = 128;
constexpr int MAX_MT = 4;
constexpr int THREADS = 384;   // warps: 0 patch producer, 1 weight producer, 2-5 MMA issuers, 6 TMEM, 8-11 epilogue
constexpr int MAX_P = 4;    // patch ring slots
constexpr int MAX_W = 12;   // weight ring slots

struct WinCfg {
    int bn, n_slices;
    int mt;            // M-tiles per item (1 .. 4)
    int n_acc;         // accumulator sets in tensor memory: 2 when 2 * mt * bn <= 512, else 1
    int r_rows;        // output rows per item
    int wp;            // padded width = positions per output row
    int pr;            // patch rows = r_rows + (kh - 1) * dil_h
    int patch_bytes;   // TMA box bytes = pr * wp * 128
    int pslot_bytes;   // patch slot incl. overrun rows, multiple of 1024
    int n_p, n_w;      // ring depths
    int n_kb;          // c_in / 32
    int row_blocks;    // ceil(ho / r_rows)
    long long n_work;
};

__device__ __forceinline__ bool aborted(volatile int* flag) { return *flag != 0; }

__device__ __forceinline__ void tma_load_tiled_4d(uint32_t dst, const void* tmap, uint32_t bar, int c, int w, int h, int n)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(tmap), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n)
        : "memory");
}
// K-major, 128-byte-swizzled operand whose first row may sit on any 128-byte boundary of a
// 1024-byte-aligned buffer: the tensor core derives the swizzle phase of a row from its
// shared-memory address (as the TMA unit did when it wrote the row), so a view shifted by whole
// rows needs nothing but another start address (checked bit for bit by the integer-valued tests).
__device__ __forceinline__ uint64_t desc_rows(uint32_t addr) { return umma_desc_k_sw128(addr, 1024); }

struct ItemPos {
    int slice, n, oh0;
};
__device__ __forceinline__ ItemPos item_of(uint32_t work, const WinCfg& cfg)
{
    ItemPos it;
    it.slice = static_cast<int>(work % static_cast<uint32_t>(cfg.n_slices));
    const uint32_t rest = work / static_cast<uint32_t>(cfg.n_slices);
    const int rb = static_cast<int>(rest % static_cast<uint32_t>(cfg.row_blocks));
    it.n = static_cast<int>(rest / static_cast<uint32_t>(cfg.row_blocks));
    it.oh0 = rb * cfg.r_rows;
    return it;
}

__global__ void __launch_bounds__(THREADS, 1)
k_conv_window(const ConvParams p, const WinCfg cfg, const __grid_constant__ CUtensorMap tm_x)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_pfull[MAX_P], s_pfree[MAX_P], s_wfull[MAX_W], s_wfree[MAX_W], s_accfull[2], s_accfree[2];
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t n_work = static_cast<uint32_t>(cfg.n_work);   // below 2^31: per-item arithmetic stays 32-bit
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t p_ring = base;
    const uint32_t w_ring = p_ring + cfg.n_p * cfg.pslot_bytes;
    const uint32_t w_bytes = static_cast<uint32_t>(cfg.bn) * 128u;
    const uint32_t wslot_bytes = (w_bytes + 1023u) & ~1023u;
    const int n_taps = p.kh * p.kw;
    const int acc_cols = cfg.mt * cfg.bn;
    volatile int* abort_flag = &s_abort;

    if (warp == 6) tmem_alloc(smem_u32(&s_tmem), 512);
    if (tid == 0) {
        for (int i = 0; i < MAX_P; ++i) { mbar_init(smem_u32(&s_pfull[i]), 1); mbar_init(smem_u32(&s_pfree[i]), cfg.mt); }
        for (int i = 0; i < MAX_W; ++i) { mbar_init(smem_u32(&s_wfull[i]), 1); mbar_init(smem_u32(&s_wfree[i]), cfg.mt); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&s_accfull[i]), cfg.mt); mbar_init(smem_u32(&s_accfree[i]), 4); }
        mbar_fence_init();
        s_abort = 0;
        tma_prefetch_desc(&tm_x);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    pdl_launch_dependents();
    pdl_wait();

    if (warp == 0) {
        // =========================== patch producer ===========================
        if (lane == 0) {
            RingPos rp;
            int issued = 0;
            for (uint32_t work = blockIdx.x; work < n_work && !aborted(abort_flag); work += gridDim.x) {
                const ItemPos it = item_of(work, cfg);
                for (int kb = 0; kb < cfg.n_kb; ++kb) {
                    if (rp.wrapped && !mbar_wait_lone(smem_u32(&s_pfree[rp.s]), rp.parity ^ 1u)) *abort_flag = 2;
                    if (aborted(abort_flag)) break;
                    const uint32_t bar = smem_u32(&s_pfull[rp.s]);
                    mbar_arrive_expect_tx(bar, static_cast<uint32_t>(cfg.patch_bytes));
                    tma_load_tiled_4d(p_ring + rp.s * cfg.pslot_bytes, &tm_x, bar, kb * 32, -p.pad_w, it.oh0 - p.pad_h, it.n);
                    rp.advance(cfg.n_p);
                    ++issued;
                }
            }
            if (aborted(abort_flag)) {
                for (int back = 0; back < cfg.n_p && back < issued; ++back) {
                    if (rp.s == 0) { rp.s = cfg.n_p; rp.parity ^= 1u; }
                    --rp.s;
                    (void)mbar_wait(smem_u32(&s_pfull[rp.s]), rp.parity);
                }
            }
        }
    } else if (warp == 1) {
        // =========================== weight producer ===========================
        if (lane == 0) {
            RingPos rw;
            int issued = 0;
            const size_t blk_floats = static_cast<size_t>(p.c_out) * 32;
            for (uint32_t work = blockIdx.x; work < n_work && !aborted(abort_flag); work += gridDim.x) {
                const ItemPos it = item_of(work, cfg);
                const float* w0 = p.wx + static_cast<size_t>(it.slice) * cfg.bn * 32;
                for (int kb = 0; kb < cfg.n_kb && !aborted(abort_flag); ++kb) {
                    const float* wsrc = w0 + static_cast<size_t>(kb) * blk_floats;   // tap 0 of this channel block
                    for (int t = 0; t < n_taps; ++t) {
                        if (rw.wrapped && !mbar_wait_lone(smem_u32(&s_wfree[rw.s]), rw.parity ^ 1u)) *abort_flag = 9;
                        if (aborted(abort_flag)) break;
                        const uint32_t bar = smem_u32(&s_wfull[rw.s]);
                        mbar_arrive_expect_tx(bar, w_bytes);
                        bulk_load_1d(w_ring + rw.s * wslot_bytes, wsrc, w_bytes, bar);
                        wsrc += static_cast<size_t>(cfg.n_kb) * blk_floats;          // same channels, next tap
                        rw.advance(cfg.n_w);
                        ++issued;
                    }
                }
            }
            if (aborted(abort_flag)) {
                for (int back = 0; back < cfg.n_w && back < issued; ++back) {
                    if (rw.s == 0) { rw.s = cfg.n_w; rw.parity ^= 1u; }
                    --rw.s;
                    (void)mbar_wait(smem_u32(&s_wfull[rw.s]), rw.parity);
                }
            }
        }
    } else if (warp >= 2 && warp < 2 + cfg.mt) {
        // =========================== MMA issuers ===========================
        // One thread per M-tile: a single thread cannot issue small MMAs as fast as the tensor core
        // retires them, and the M-tiles have separate accumulators, so each gets its own issuer.
        // Ring slots and accumulator hand-offs count one commit per issuer.
        if (lane == 0) {
            const int mi = warp - 2;
            const uint32_t idesc = umma_idesc_tf32(BM, cfg.bn);
            // one tap to the right = dil_w patch rows of 128 bytes; after the last tap of a kernel row,
            // back to the first column and dil_h patch lines (Wp rows each) down
            const uint32_t dw_units = static_cast<uint32_t>(p.dil_w) * 8u;
            const uint32_t dh_units = static_cast<uint32_t>(p.dil_h * cfg.wp - p.kw * p.dil_w) * 8u;
            RingPos rp, rw;
            uint32_t ab = 0, acc_par = 0;
            bool acc_wrapped = false;
            for (uint32_t work = blockIdx.x; work < n_work && !aborted(abort_flag); work += gridDim.x) {
                if (acc_wrapped && !mbar_wait_lone(smem_u32(&s_accfree[ab]), acc_par ^ 1u)) { *abort_flag = 5; break; }
                tc_fence_after();
                const uint32_t acc = tmem + ab * acc_cols + mi * cfg.bn;
                for (int kb = 0; kb < cfg.n_kb && !aborted(abort_flag); ++kb) {
                    if (!mbar_wait_lone(smem_u32(&s_pfull[rp.s]), rp.parity)) { *abort_flag = 6; break; }
                    // descriptors are built once per patch / weight slot and advanced by adding 16-byte units:
                    // this thread's instruction stream is the issue rate of the whole CTA
                    const uint64_t a_patch = desc_rows(p_ring + rp.s * cfg.pslot_bytes + mi * (BM * 128));
                    uint32_t row_units = 0;          // (tap row offset * 128 bytes) / 16
                    int tj = 0;
                    for (int t = 0; t < n_taps; ++t) {
                        if (!mbar_wait_lone(smem_u32(&s_wfull[rw.s]), rw.parity)) { *abort_flag = 7; break; }
                        tc_fence_after();
                        const uint64_t b_desc = umma_desc_k_sw128(w_ring + rw.s * wslot_bytes, 1024);
                        const uint64_t a_desc = a_patch + row_units;
                        umma_tf32_ss(acc, a_desc, b_desc, idesc, (kb > 0 || t > 0) ? 1u : 0u);
                        umma_tf32_ss(acc, a_desc + 2, b_desc + 2, idesc, 1u);
                        umma_tf32_ss(acc, a_desc + 4, b_desc + 4, idesc, 1u);
                        umma_tf32_ss(acc, a_desc + 6, b_desc + 6, idesc, 1u);
                        umma_commit(smem_u32(&s_wfree[rw.s]));
                        rw.advance(cfg.n_w);
                        row_units += dw_units;
                        if (++tj == p.kw) { tj = 0; row_units += dh_units; }
                    }
                    if (aborted(abort_flag)) break;
                    umma_commit(smem_u32(&s_pfree[rp.s]));
                    rp.advance(cfg.n_p);
                }
                if (aborted(abort_flag)) break;
                umma_commit(smem_u32(&s_accfull[ab]));
                if (cfg.n_acc == 2) {
                    if (ab == 1) { acc_par ^= 1u; acc_wrapped = true; }
                    ab ^= 1u;
                } else {
                    acc_par ^= 1u;
                    acc_wrapped = true;
                }
            }
        }
    } else if (warp >= 8) {
        // =========================== epilogue ===========================
        const int q = warp & 3;
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const int n_blk = cfg.bn / 32;
        uint32_t ti = 0;
        for (uint32_t work = blockIdx.x; work < n_work; work += gridDim.x, ++ti) {
            const ItemPos it = item_of(work, cfg);
            const int ab = cfg.n_acc == 2 ? static_cast<int>(ti & 1u) : 0;
            const bool ok = aborted(abort_flag) ||
                            mbar_wait(smem_u32(&s_accfull[ab]), (cfg.n_acc == 2 ? (ti >> 1) : ti) & 1u);
            if (!__all_sync(0xFFFFFFFFu, ok)) *abort_flag = 8;
            if (__any_sync(0xFFFFFFFFu, aborted(abort_flag))) break;
            tc_fence_after();
            const int o0 = it.slice * cfg.bn;
            for (int m = 0; m < cfg.mt; ++m) {
                // this thread's position: row of the block and column along the padded width
                const int pos = m * BM + q * 32 + lane;
                const int r = pos / cfg.wp, ow = pos - r * cfg.wp;
                const bool valid = r < cfg.r_rows && ow < p.wo && it.oh0 + r < p.ho;
                float* yrow = p.y + ((static_cast<size_t>(it.n) * p.ho + (valid ? it.oh0 + r : 0)) * p.wo + (valid ? ow : 0)) * p.c_out + o0;
                for (int blk = 0; blk < n_blk; ++blk) {
                    uint32_t v[32];
                    tmem_ld32(tmem + lane_addr + ab * acc_cols + m * cfg.bn + blk * 32, v);
                    tmem_ld_wait();
                    if (m == cfg.mt - 1 && blk == n_blk - 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&s_accfree[ab]));
                    }
                    if (valid) {
#pragma unroll
                        for (int qq = 0; qq < 8; ++qq) {
                            float4 o;
                            float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (p.bias) bv = __ldg(reinterpret_cast<const float4*>(p.bias + o0 + blk * 32) + qq);
                            if (p.residual)
                                nm_add4(bv, __ldg(reinterpret_cast<const float4*>(p.residual + (yrow - p.y) + blk * 32 + qq * 4)));
                            o.x = __uint_as_float(v[qq * 4 + 0]) + bv.x;
                            o.y = __uint_as_float(v[qq * 4 + 1]) + bv.y;
                            o.z = __uint_as_float(v[qq * 4 + 2]) + bv.z;
                            o.w = __uint_as_float(v[qq * 4 + 3]) + bv.w;
                            if (p.relu) {
                                o.x = fmaxf(o.x, 0.f); o.y = fmaxf(o.y, 0.f); o.z = fmaxf(o.z, 0.f); o.w = fmaxf(o.w, 0.f);
                            }
                            *reinterpret_cast<float4*>(yrow + blk * 32 + qq * 4) = o;
                        }
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && s_abort != 0) {
        atomicExch(p.status + 0, static_cast<int>(NM_ERR_TIMEOUT));
        atomicExch(p.status + 1, 60 + s_abort);
        atomicExch(p.status + 2, static_cast<int>(blockIdx.x));
    }
    if (warp == 6) tmem_dealloc(tmem, 512);
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

bool make_cfg(const ConvParams& p, const nm_plan_t* plan, WinCfg* cfg, size_t* smem_out)
{
    if (!p.wx || !nmtm::available()) return false;
    if (p.stride_h != 1 || p.stride_w != 1 || p.kh * p.kw < 2) return false;
    if (p.c_in % 32 != 0 || p.c_out % 32 != 0) return false;
    if (p.pad_w > 127 || p.pad_h > 127) return false;
    const int wp = p.w + 2 * p.pad_w;
    if (wp - p.dil_w * (p.kw - 1) != p.wo || p.wo > 256) return false;
    int mt = plan && plan->split > 0 ? plan->split : 2;
    if (mt * BM < wp) mt = (wp + BM - 1) / BM;          // one output row must fit the item
    if (mt < 1 || mt > MAX_MT) return false;
    int r_rows = (BM * mt) / wp;
    if (r_rows > p.ho) r_rows = p.ho;
    const int pr = r_rows + (p.kh - 1) * p.dil_h;
    if (pr > 256 || wp > 256) return false;
    int bn = 0;
    if (plan && plan->bn > 0) {
        bn = plan->bn;
    } else {
        for (int cand : {256, 128, 64, 32, 96, 160, 192, 224})
            if (cand <= p.c_out && p.c_out % cand == 0 && mt * cand <= 512) { bn = cand; break; }
    }
    if (bn < 32 || bn > 256 || bn % 32 != 0 || p.c_out % bn != 0 || mt * bn > 512) return false;
    cfg->n_acc = 2 * mt * bn <= 512 ? 2 : 1;
    cfg->bn = bn;
    cfg->n_slices = p.c_out / bn;
    cfg->mt = mt;
    cfg->r_rows = r_rows;
    cfg->wp = wp;
    cfg->pr = pr;
    cfg->patch_bytes = pr * wp * 128;
    if (cfg->patch_bytes >= (1 << 20)) return false;
    // rows the last M-tile's furthest tap can touch: junk positions read past the patch proper
    int rows = BM * mt + (p.kh - 1) * p.dil_h * wp + (p.kw - 1) * p.dil_w;
    if (rows < pr * wp) rows = pr * wp;
    cfg->pslot_bytes = ((rows * 128 + 1023) / 1024) * 1024;
    cfg->n_kb = p.c_in / 32;
    cfg->row_blocks = (p.ho + r_rows - 1) / r_rows;
    cfg->n_work = static_cast<long long>(p.batch) * cfg->row_blocks * cfg->n_slices;
    if (cfg->n_work >= (1ll << 31)) return false;
    const int wslot = ((bn * 128 + 1023) / 1024) * 1024;
    const int budget = 227 * 1024 - 2048;
    int n_p = 2, n_w = plan && plan->stages > 0 ? plan->stages : MAX_W;
    if (n_w > MAX_W || n_w < 2) return false;
    while (n_w > 3 && n_p * cfg->pslot_bytes + n_w * wslot > budget) --n_w;
    if (n_p * cfg->pslot_bytes + n_w * wslot > budget) return false;
    while (n_p < MAX_P && (n_p + 1) * cfg->pslot_bytes + n_w * wslot <= budget) ++n_p;
    cfg->n_p = n_p;
    cfg->n_w = n_w;
    size_t smem = 1024 + static_cast<size_t>(n_p) * cfg->pslot_bytes + static_cast<size_t>(n_w) * wslot;
    *smem_out = smem < 120 * 1024 ? 120 * 1024 : smem;
    return true;
}

// Activations as a tiled map (C, W, H, N) with a 32-channel x Wp x PR x 1 box: rows and columns
// outside the image (the padding) are filled with zeros by the load.
bool encode_x_patch(const ConvParams& p, const WinCfg& cfg, CUtensorMap* tm)
{
    const cuuint64_t dims[4] = {static_cast<cuuint64_t>(p.c_in), static_cast<cuuint64_t>(p.w), static_cast<cuuint64_t>(p.h),
                                static_cast<cuuint64_t>(p.batch)};
    const cuuint64_t strides[3] = {static_cast<cuuint64_t>(p.c_in) * 4, static_cast<cuuint64_t>(p.w) * p.c_in * 4,
                                   static_cast<cuuint64_t>(p.h) * p.w * p.c_in * 4};
    const cuuint32_t box[4] = {32, static_cast<cuuint32_t>(cfg.wp), static_cast<cuuint32_t>(cfg.pr), 1};
    const cuuint32_t es[4] = {1, 1, 1, 1};
    return nmtm::encoders().tiled(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(p.x), dims, strides, box, es,
                                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

namespace nmhost {

bool window_plan_ok(const ConvParams& p, const nm_plan_t* plan)
{
    WinCfg cfg;
    size_t smem;
    return make_cfg(p, plan, &cfg, &smem);
}

nm_status_t launch_conv_window(const ConvParams& p, const nm_plan_t* plan, cudaStream_t st)
{
    WinCfg cfg;
    size_t smem = 0;
    if (!make_cfg(p, plan, &cfg, &smem))
        return fail(NM_ERR_UNSUPPORTED, "nm_conv2d: the window kernel does not take this layer / plan");
    alignas(64) CUtensorMap tm_x;
    if (!encode_x_patch(p, cfg, &tm_x))
        return fail(NM_ERR_CUDA, "nm_conv2d: tensor-map encoding failed (variant 6)");
    cudaError_t e = nmhost::ensure_dynamic_smem(reinterpret_cast<const void*>(k_conv_window), smem);
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "cudaFuncSetAttribute (variant 6): %s", cudaGetErrorString(e));
    const long long grid = cfg.n_work < sm_count() ? cfg.n_work : sm_count();
    e = launch_pdl(k_conv_window, static_cast<unsigned>(grid), THREADS, smem, st, p, cfg, tm_x);
    count_launch(1);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "nm_conv2d launch (variant 6): %s", cudaGetErrorString(e));
    return NM_OK;
}

}  // namespace nmhost
