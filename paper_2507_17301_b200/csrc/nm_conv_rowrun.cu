// Variant 5: row-run kernel — implicit GEMM for layers with few input channels (the 7x7, 3-channel
// stem of a ResNet), where a 32-channel slab does not exist and TMA's im2col mode cannot be used
// (a pixel's channels are fewer than 16 bytes).
//
// With NHWC activations and dil_w = 1, the (kw, c) part of a patch row is ONE contiguous run of
// kw * c_in floats of the input row.  One work item is one output row (at most 128 pixels):
//   producer (1 thread)    bulk-copies the kh input rows the item needs into shared memory: with
//                          dil_h = 1 they are adjacent in memory, so ONE copy brings them all (rows
//                          outside the image are simply not copied);
//   builders (2 x 8 warps)    lay the patch matrix [128 pixels x K] down in 32-column sub-tiles in the
//                          K-major, 128-byte-swizzled layout the tensor core reads: lane = column,
//                          so a warp reads 32 consecutive floats of a run and writes one 128-byte
//                          row, both free of bank conflicts.  Padding is resolved per column with a
//                          precomputed range of valid output pixels (outside it, past the end of
//                          the output row and for kernel rows outside the image the builders write
//                          zeros).  This is the fused im2col + packing of
//                          Sec. 3.2 done in shared memory; nothing of it reaches global memory;
//   MMA issuer (1 thread)  four 128 x C_out x 8 TF32 tcgen05.mma per sub-tile against the weights,
//                          which stay resident in shared memory for the whole kernel (expanded
//                          layout: pruned columns are zeros, so any N:M and any tile width works;
//                          the stem itself is unpruned);
//   epilogue (4 warps)     TMEM -> registers, + bias, ReLU, staged and stored with TMA; pixels past
//                          the end of the output row are clipped by the store's bounds check.
// Every wait is bounded and reports through the handle's status word.
#include "nm_internal.h"
#include "nm_ptx.cuh"
#include "nm_tmap.cuh"

namespace {

using namespace nmk;

constexpr int BM = 128;
constexpr int SUB_BYTES = BM * 128;
constexpr int A_RING = 4;
constexpr int MAX_SETS = 4;   // row sets in flight: the copy of item i + n_sets - 1 is issued while item i is built
constexpr int NB_GROUPS = 2;                  // builder groups of 8 warps taking alternate sub-tiles
constexpr int THREADS = (8 + 8 * NB_GROUPS) * 32;
constexpr int STAGING_BYTES = 4 * 2 * 4096;
constexpr int MAX_KB = 16;   // sub-tiles of 32 columns: K <= 512

struct RowCfg {
    int nkb;          // ceil(K / 32)
    int run;          // kw * c_in: contiguous floats per kernel row
    int pitch;        // floats per row buffer = w * c_in
    int row_bytes;    // w * c_in * 4
    int bn;           // = c_out
    int w_bytes;      // nkb * bn * 128
    int rowset_bytes; // kh * pitch * 4
    int n_sets;       // row sets in the ring (2 .. MAX_SETS)
    long long n_work; // batch * ho
};

__device__ __forceinline__ bool aborted(volatile int* flag) { return *flag != 0; }

__global__ void __launch_bounds__(THREADS, 1)
k_conv_rowrun(const ConvParams p, const RowCfg cfg, const __grid_constant__ CUtensorMap tm_y)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_wfull, s_rfull[MAX_SETS], s_rfree[MAX_SETS], s_afull[A_RING], s_afree[A_RING], s_accfull[2], s_accfree[2];
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort;
    __shared__ int s_koff[MAX_KB * 32];   // per column: kernel row << 24 | float offset inside the row set; -1 = padding
    __shared__ uint32_t s_range[MAX_KB * 32];   // per column: first valid output pixel << 16 | number of valid ones

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t n_work = static_cast<uint32_t>(cfg.n_work);   // below 2^31: per-item arithmetic stays 32-bit
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t w_smem = base;
    const uint32_t a_ring = w_smem + ((cfg.w_bytes + 1023) / 1024) * 1024;
    const uint32_t staging = a_ring + A_RING * SUB_BYTES;
    const uint32_t rowbuf = staging + STAGING_BYTES;                 // two row sets, then 16 bytes of zeros
    const uint32_t zero_row = rowbuf + cfg.n_sets * cfg.rowset_bytes;
    volatile int* abort_flag = &s_abort;

    if (warp == 2) tmem_alloc(smem_u32(&s_tmem), 512);
    if (tid == 0) {
        mbar_init(smem_u32(&s_wfull), 1);
        for (int i = 0; i < MAX_SETS; ++i) {
            mbar_init(smem_u32(&s_rfull[i]), 1);
            mbar_init(smem_u32(&s_rfree[i]), 8 * NB_GROUPS);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&s_accfull[i]), 1);
            mbar_init(smem_u32(&s_accfree[i]), 4);
        }
        for (int i = 0; i < A_RING; ++i) {
            mbar_init(smem_u32(&s_afull[i]), 8);
            mbar_init(smem_u32(&s_afree[i]), 1);
        }
        mbar_fence_init();
        s_abort = 0;
        tma_prefetch_desc(&tm_y);
    }
    // per-column tables, and the word of zeros every invalid element is read from
    {
        if (tid < 4) asm volatile("st.shared.u32 [%0], %1;" ::"r"(zero_row + tid * 4), "r"(0u) : "memory");
        for (int i = tid; i < cfg.nkb * 32; i += THREADS) {
            const int khi = i / cfg.run;
            const int kr = i - khi * cfg.run;          // position inside the run: kw * c_in + c
            const int kwi = (kr / p.c_in) * p.dil_w;   // (dil_w = 1)
            s_koff[i] = i < p.k ? ((khi << 24) | (khi * cfg.pitch + kr)) : -1;
            // output pixels ow with 0 <= ow * stride_w - pad_w + kwi < w, clipped to the output row
            int lo = p.pad_w - kwi;
            lo = lo > 0 ? (lo + p.stride_w - 1) / p.stride_w : 0;
            int hi = p.w + p.pad_w - 1 - kwi;
            hi = hi >= 0 ? hi / p.stride_w : -1;
            if (hi > p.wo - 1) hi = p.wo - 1;
            const int cnt = hi >= lo ? hi - lo + 1 : 0;
            s_range[i] = (static_cast<uint32_t>(lo) << 16) | static_cast<uint32_t>(cnt);
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    pdl_launch_dependents();   // the next kernel may start its own set-up as SMs become free
    pdl_wait();                // from here on global memory written by the previous kernel is read

    if (warp == 0) {
        // =========================== producer ===========================
        if (lane == 0) {
            mbar_arrive_expect_tx(smem_u32(&s_wfull), static_cast<uint32_t>(cfg.w_bytes));
            bulk_load_1d(w_smem, p.wx, static_cast<uint32_t>(cfg.w_bytes), smem_u32(&s_wfull));
            RingPos rs;
            int issued = 0;
            for (uint32_t work = blockIdx.x; work < n_work && !aborted(abort_flag); work += gridDim.x) {
                const int n = static_cast<int>(work / static_cast<uint32_t>(p.ho)), oh = static_cast<int>(work - static_cast<uint32_t>(n) * static_cast<uint32_t>(p.ho));
                if (rs.wrapped && !mbar_wait_lone(smem_u32(&s_rfree[rs.s]), rs.parity ^ 1u)) { *abort_flag = 2; break; }
                const int ih0 = oh * p.stride_h - p.pad_h;
                const uint32_t bar = smem_u32(&s_rfull[rs.s]);
                const uint32_t dst0 = rowbuf + rs.s * cfg.rowset_bytes;
                const float* img = p.x + static_cast<size_t>(n) * p.h * p.w * p.c_in;
                if (p.dil_h == 1) {
                    // the kernel rows are adjacent input rows: one copy of the ones inside the image
                    const int first = ih0 > 0 ? ih0 : 0;
                    const int last = ih0 + p.kh - 1 < p.h - 1 ? ih0 + p.kh - 1 : p.h - 1;
                    const int cnt = last >= first ? last - first + 1 : 0;
                    mbar_arrive_expect_tx(bar, static_cast<uint32_t>(cnt) * cfg.row_bytes);
                    if (cnt > 0)
                        bulk_load_1d(dst0 + (first - ih0) * cfg.row_bytes, img + static_cast<size_t>(first) * p.w * p.c_in,
                                     static_cast<uint32_t>(cnt) * cfg.row_bytes, bar);
                } else {
                    int valid = 0;
                    for (int r = 0; r < p.kh; ++r) {
                        const int ih = ih0 + r * p.dil_h;
                        valid += (ih >= 0 && ih < p.h) ? 1 : 0;
                    }
                    mbar_arrive_expect_tx(bar, static_cast<uint32_t>(valid) * cfg.row_bytes);
                    for (int r = 0; r < p.kh; ++r) {
                        const int ih = ih0 + r * p.dil_h;
                        if (ih >= 0 && ih < p.h)
                            bulk_load_1d(dst0 + r * cfg.row_bytes, img + static_cast<size_t>(ih) * p.w * p.c_in,
                                         static_cast<uint32_t>(cfg.row_bytes), bar);
                    }
                }
                ++issued;
                rs.advance(cfg.n_sets);
            }
            if (aborted(abort_flag)) {
                (void)mbar_wait(smem_u32(&s_wfull), 0);
                for (int back = 0; back < cfg.n_sets && back < issued; ++back) {
                    if (rs.s == 0) { rs.s = cfg.n_sets; rs.parity ^= 1u; }
                    --rs.s;
                    (void)mbar_wait(smem_u32(&s_rfull[rs.s]), rs.parity);
                }
            }
        }
    } else if (warp == 1) {
        // =========================== MMA issuer ===========================
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_tf32(BM, cfg.bn);
            if (!mbar_wait(smem_u32(&s_wfull), 0)) *abort_flag = 9;
            RingPos rp;
            uint32_t ab = 0, acc_par = 0;
            bool acc_wrapped = false;
            for (uint32_t work = blockIdx.x; work < n_work && !aborted(abort_flag); work += gridDim.x) {
                if (acc_wrapped && !mbar_wait_lone(smem_u32(&s_accfree[ab]), acc_par ^ 1u)) { *abort_flag = 5; break; }
                tc_fence_after();
                const uint32_t acc = tmem + ab * cfg.bn;
                for (int j = 0; j < cfg.nkb; ++j) {
                    if (!mbar_wait_lone(smem_u32(&s_afull[rp.s]), rp.parity)) { *abort_flag = 6; break; }
                    tc_fence_after();
                    const uint64_t adesc = umma_desc_k_sw128(a_ring + rp.s * SUB_BYTES, 1024);
                    const uint64_t bdesc = umma_desc_k_sw128(w_smem + j * cfg.bn * 128, 1024);
#pragma unroll
                    for (int kq = 0; kq < 4; ++kq)
                        umma_tf32_ss(acc, adesc + 2 * kq, bdesc + 2 * kq, idesc, (j > 0 || kq > 0) ? 1u : 0u);
                    umma_commit(smem_u32(&s_afree[rp.s]));
                    rp.advance(A_RING);
                }
                if (aborted(abort_flag)) break;
                umma_commit(smem_u32(&s_accfull[ab]));
                if (ab == 1) { acc_par ^= 1u; acc_wrapped = true; }
                ab ^= 1u;
            }
        }
    } else if (warp >= 4 && warp < 8) {
        // =========================== epilogue ===========================
        const int q = warp & 3;
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t my_staging = staging + q * 2 * 4096;
        const uint32_t rx = static_cast<uint32_t>(lane & 7);
        const int n_blk = cfg.bn / 32;
        uint32_t nb = 0, ti = 0;
        for (uint32_t work = blockIdx.x; work < n_work; work += gridDim.x, ++ti) {
            const int ab = static_cast<int>(ti & 1u);
            const bool ok = aborted(abort_flag) || mbar_wait(smem_u32(&s_accfull[ab]), (ti >> 1) & 1u);
            if (!__all_sync(0xFFFFFFFFu, ok)) *abort_flag = 8;
            if (__any_sync(0xFFFFFFFFu, aborted(abort_flag))) break;
            tc_fence_after();
            for (int blk = 0; blk < n_blk; ++blk, ++nb) {
                uint32_t v[32];
                tmem_ld32(tmem + lane_addr + ab * cfg.bn + blk * 32, v);
                tmem_ld_wait();
                if (blk == n_blk - 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&s_accfree[ab]));
                }
                const uint32_t box = my_staging + (nb & 1u) * 4096;
                if (lane == 0 && nb >= 2) tma_store_wait_read_n<1>();
                __syncwarp();
                const uint32_t stage_row = box + lane * 128;
                // pixel of this thread: output row `work`, column q * 32 + lane (past the row's end: none)
                const float4* rrow = nm_residual_row(
                    p, q * 32 + lane < p.wo ? static_cast<long long>(work) * p.wo + q * 32 + lane : p.pixels, blk * 32);
#pragma unroll
                for (int qq = 0; qq < 8; ++qq) {
                    float o[4];
                    float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (p.bias) bv = __ldg(reinterpret_cast<const float4*>(p.bias + blk * 32) + qq);
                    if (rrow) nm_add4(bv, __ldg(rrow + qq));
                    o[0] = __uint_as_float(v[qq * 4 + 0]) + bv.x;
                    o[1] = __uint_as_float(v[qq * 4 + 1]) + bv.y;
                    o[2] = __uint_as_float(v[qq * 4 + 2]) + bv.z;
                    o[3] = __uint_as_float(v[qq * 4 + 3]) + bv.w;
                    if (p.relu) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) o[e] = fmaxf(o[e], 0.f);
                    }
                    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(stage_row + ((qq ^ rx) << 4)), "f"(o[0]),
                                 "f"(o[1]), "f"(o[2]), "f"(o[3])
                                 : "memory");
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                    // output seen as (channel, ow, n * ho + oh): pixels past the row's end are clipped
                    if (q * 32 < p.wo) tma_store_3d(&tm_y, box, blk * 32, q * 32, static_cast<int>(work));
                    tma_store_commit();
                }
            }
        }
        if (lane == 0) tma_store_wait_read();   // shared memory must outlive the stores' reads; the writes complete with the grid
    } else if (warp >= 8) {
        // =========================== builders ===========================
        // Two groups of eight warps build alternate sub-tiles, so that one group's barrier waits and
        // arrivals overlap the other's loads and stores.  Inside a group warp bw takes rows bw, bw + 8, ...
        const int bw = (warp - 8) & 7;
        const int grp = (warp - 8) >> 3;
        uint32_t turn = 0;   // parity of the running sub-tile count: whose sub-tile the next one is
        RingPos rp;
        RingPos rs;
        for (uint32_t work = blockIdx.x; work < n_work && !aborted(abort_flag); work += gridDim.x) {
            const int n = static_cast<int>(work / static_cast<uint32_t>(p.ho)), oh = static_cast<int>(work - static_cast<uint32_t>(n) * static_cast<uint32_t>(p.ho));
            const int ih0 = oh * p.stride_h - p.pad_h;
            bool ok = mbar_wait_lone(smem_u32(&s_rfull[rs.s]), rs.parity);
            if (!__all_sync(0xFFFFFFFFu, ok)) *abort_flag = 3;
            if (__any_sync(0xFFFFFFFFu, aborted(abort_flag))) break;
            const uint32_t rows = rowbuf + rs.s * cfg.rowset_bytes;
            for (int j = 0; j < cfg.nkb; ++j, turn ^= 1u) {
                if (turn != static_cast<uint32_t>(grp)) {   // the other group's sub-tile
                    rp.advance(A_RING);
                    continue;
                }
                ok = !rp.wrapped || mbar_wait_lone(smem_u32(&s_afree[rp.s]), rp.parity ^ 1u);
                if (!__all_sync(0xFFFFFFFFu, ok)) *abort_flag = 4;
                if (__any_sync(0xFFFFFFFFu, aborted(abort_flag))) break;
                const int ko = s_koff[j * 32 + lane];
                const uint32_t rng = s_range[j * 32 + lane];
                const int lo = static_cast<int>(rng >> 16);
                uint32_t cnt = 0;                  // valid output pixels of this column: lo .. lo + cnt - 1
                uint32_t src = zero_row;
                if (ko >= 0) {
                    const int khi = ko >> 24;
                    const int ih = ih0 + khi * p.dil_h;
                    if (ih >= 0 && ih < p.h) cnt = rng & 0xFFFFu;
                    // element of output pixel 0 (before the row's start for padded columns: never read there)
                    src = rows + ((ko & 0xFFFFFF) - p.pad_w * p.c_in) * 4;
                }
                const int step8 = p.stride_w * p.c_in * 4 * 8;   // bytes between pixels ow and ow + 8
                // rows bw, bw + 8, ...: (row % 8) is the same for all of them, so is the swizzle term
                uint32_t dst = a_ring + rp.s * SUB_BYTES + ((lane & 3) << 2) + bw * 128 +
                               ((static_cast<uint32_t>(lane >> 2) ^ static_cast<uint32_t>(bw)) << 4);
                src += bw * (step8 >> 3);
                uint32_t v[BM / 8];
                // Rows 16 .. 95 lie inside every column's range of valid pixels on all but the border items
                // (then for the whole warp): they are copied without the per-row test.
                const bool inner = __all_sync(0xFFFFFFFFu, lo <= 16 && static_cast<uint32_t>(96 - lo) <= cnt);
                if (inner) {
#pragma unroll
                    for (int i = 0; i < BM / 8; ++i) {
                        if (i >= 2 && i < 12) {
                            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v[i]) : "r"(src));
                        } else {
                            const bool valid = static_cast<uint32_t>(bw + i * 8 - lo) < cnt;
                            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v[i]) : "r"(valid ? src : zero_row));
                        }
                        src += step8;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < BM / 8; ++i) {
                        const bool valid = static_cast<uint32_t>(bw + i * 8 - lo) < cnt;
                        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v[i]) : "r"(valid ? src : zero_row));
                        src += step8;
                    }
                }
#pragma unroll
                for (int i = 0; i < BM / 8; ++i) {
                    asm volatile("st.shared.u32 [%0], %1;" ::"r"(dst), "r"(v[i]) : "memory");
                    dst += 8 * 128;
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&s_afull[rp.s]));
                rp.advance(A_RING);
            }
            if (aborted(abort_flag)) break;
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_rfree[rs.s]));
            rs.advance(cfg.n_sets);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && s_abort != 0) {
        atomicExch(p.status + 0, static_cast<int>(NM_ERR_TIMEOUT));
        atomicExch(p.status + 1, 50 + s_abort);
        atomicExch(p.status + 2, static_cast<int>(blockIdx.x));
    }
    if (warp == 2) tmem_dealloc(tmem, 512);
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

bool make_cfg(const ConvParams& p, RowCfg* cfg, size_t* smem_out)
{
    if (!p.wx || !nmtm::available()) return false;
    if (p.dil_w != 1 || p.wo > BM) return false;
    if (p.c_out % 32 != 0 || p.c_out > 256) return false;
    if ((static_cast<long long>(p.w) * p.c_in * 4) % 16 != 0) return false;   // bulk copies move whole 16-byte pieces
    if (static_cast<long long>(p.batch) * p.h * p.w * p.c_in >= (1ll << 31)) return false;
    cfg->nkb = (p.k + 31) / 32;
    if (cfg->nkb > MAX_KB) return false;
    cfg->run = p.kw * p.c_in;
    cfg->pitch = p.w * p.c_in;
    if (static_cast<long long>(p.kh) * p.w * p.c_in * 4 >= (1 << 20)) return false;   // one copy, one mbarrier phase
    if (p.wo > 0xFFFF) return false;
    cfg->row_bytes = p.w * p.c_in * 4;
    cfg->bn = p.c_out;
    cfg->w_bytes = cfg->nkb * cfg->bn * 128;
    cfg->rowset_bytes = p.kh * cfg->pitch * 4;
    cfg->n_work = static_cast<long long>(p.batch) * p.ho;
    if (static_cast<long long>(p.batch) * p.ho >= (1ll << 31)) return false;
    const size_t fixed = 1024 + static_cast<size_t>((cfg->w_bytes + 1023) / 1024) * 1024 + A_RING * SUB_BYTES + STAGING_BYTES + 16;
    cfg->n_sets = MAX_SETS;
    while (cfg->n_sets > 2 && fixed + static_cast<size_t>(cfg->n_sets) * cfg->rowset_bytes > 227 * 1024 - 4096) --cfg->n_sets;
    const size_t smem = fixed + static_cast<size_t>(cfg->n_sets) * cfg->rowset_bytes;
    if (smem > 227 * 1024 - 4096) return false;
    *smem_out = smem < 120 * 1024 ? 120 * 1024 : smem;
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

}  // namespace

namespace nmhost {

bool rowrun_plan_ok(const ConvParams& p, const nm_plan_t* /*plan*/)
{
    RowCfg cfg;
    size_t smem;
    return make_cfg(p, &cfg, &smem);
}

nm_status_t launch_conv_rowrun(const ConvParams& p, const nm_plan_t* /*plan*/, cudaStream_t st)
{
    RowCfg cfg;
    size_t smem = 0;
    if (!make_cfg(p, &cfg, &smem))
        return fail(NM_ERR_UNSUPPORTED, "nm_conv2d: the row-run kernel does not take this layer");
    alignas(64) CUtensorMap tm_y;
    if (!encode_y_rows(p, &tm_y)) return fail(NM_ERR_CUDA, "nm_conv2d: tensor-map encoding failed (variant 5)");
    cudaError_t e = nmhost::ensure_dynamic_smem(reinterpret_cast<const void*>(k_conv_rowrun), smem);
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "cudaFuncSetAttribute (variant 5): %s", cudaGetErrorString(e));
    const long long grid = cfg.n_work < sm_count() ? cfg.n_work : sm_count();
    e = nmhost::launch_pdl(k_conv_rowrun, static_cast<unsigned>(grid), THREADS, smem, st, p, cfg, tm_y);
    nmhost::count_launch(1);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "nm_conv2d launch (variant 5): %s", cudaGetErrorString(e));
    return NM_OK;
}

}  // namespace nmhost
