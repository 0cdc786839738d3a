// Variant 7: pair kernel — the expanded-operand implicit GEMM run by PAIRS of CTAs (thread-block
// clusters of two, tcgen05 cta_group::2).
//
// With one CTA per work item the expanded-operand kernel is bound by shared-memory bandwidth on
// reduction-heavy layers: per 32-column stage a CTA writes 16 KB of activations and 32 KB of
// weights (256 channels) and its four MMAs read 48 KB, 96 KB for 512 tensor-pipe cycles.  A pair
// MMA of shape 256 x BN x 8 spans two SMs: each CTA supplies its own 128 pixels of A and only
// HALF of the BN weight rows (the hardware exchanges the halves), so per stage and CTA 32 KB are
// written and 32 KB read.  The accumulator rows of a CTA's pixels stay in its own tensor memory,
// so the epilogue is the single-CTA one.
//
//   producer (1 thread per CTA)   TMA im2col load of the CTA's slab + one bulk copy of its half of
//                                 the weight block per stage (local barrier)
//   relay (1 thread, second CTA)  forwards "stage landed" to the first CTA's barrier
//   MMA issuer (1 thread, first   four 256 x BN x 8 TF32 pair MMAs per stage; commits are multicast
//   CTA)                          to both CTAs' "stage free" / "accumulator full" barriers
//   epilogue (8 warps per CTA)    TMEM -> registers, + bias (+ shortcut), ReLU, swizzled staging,
//                                 TMA store; releases the accumulator on the first CTA's barrier
// A work item is (two consecutive blocks of 128 pixels, BN channels); pairs walk the items in a
// static persistent schedule.  Every mbarrier wait is bounded; the two cluster-wide barriers at
// start and end are reached by all threads unconditionally.
#include "nm_internal.h"
#include "nm_ptx.cuh"
#include "nm_tmap.cuh"

namespace {

using namespace nmk;

constexpr int BM = 128;
constexpr int SUB_BYTES = BM * 128;
constexpr int NSTAGE_MAX = 10;
constexpr int THREADS = 384;    // 4 service warps + 8 epilogue warps
constexpr int BOX_BYTES = 4096;

struct PairCfg {
    int bn;           // output channels per work item (N of the pair MMA)
    int half_rows;    // weight rows each CTA holds: bn / 2
    int n_slices;
    int stages;
    int b_bytes;      // weight bytes per stage and CTA
    int stage_bytes;
    int n_sub;        // stages per work item: (K / 32) / kblk
    int kblk;         // 32-column blocks per stage (1 or 2): one barrier round trip covers kblk * 4 MMAs
    int sub_bytes;    // bytes of one 32-column block in a stage: activations + this CTA's weight rows
    int boxes;        // output staging boxes per epilogue warp
    long long n_work; // pair items
};

__device__ __forceinline__ bool aborted(volatile int* flag) { return *flag != 0; }

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
k_conv_pair(const ConvParams p, const PairCfg cfg, const __grid_constant__ CUtensorMap tm_x,
            const __grid_constant__ CUtensorMap tm_y)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_full[NSTAGE_MAX], s_free[NSTAGE_MAX], s_accfull[2], s_accfree[2];
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();                  // 0: issues the MMAs
    const uint32_t pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const uint32_t n_work = static_cast<uint32_t>(cfg.n_work);
    const int NS = cfg.stages, n_sub = cfg.n_sub;
    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t staging = ring + NS * cfg.stage_bytes;
    volatile int* abort_flag = &s_abort;

    if (warp == 2) tmem_alloc_pair(smem_u32(&s_tmem), 512);
    if (tid == 0) {
        for (int i = 0; i < NSTAGE_MAX; ++i) {
            // first CTA: its producer's expect-tx arrival + the relay's; second CTA: its producer's
            mbar_init(smem_u32(&s_full[i]), rank == 0 ? 2 : 1);
            mbar_init(smem_u32(&s_free[i]), 1);   // multicast MMA commit
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&s_accfull[i]), 1);    // multicast MMA commit
            mbar_init(smem_u32(&s_accfree[i]), 16);   // the epilogue warps of both CTAs (used in the first CTA)
        }
        mbar_fence_init();
        s_abort = 0;
        tma_prefetch_desc(&tm_x);
        tma_prefetch_desc(&tm_y);
    }
    tc_fence_before();
    cluster_sync_all();   // barriers of both CTAs are initialised before either CTA signals the other
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    pdl_launch_dependents();
    pdl_wait();

    if (warp == 0) {
        // =========================== producer (both CTAs) ===========================
        if (lane == 0) {
            int issued = 0;
            const int hw = p.ho * p.wo;
            const uint32_t w_bytes = static_cast<uint32_t>(cfg.half_rows) * 128u;
            const uint32_t tx = static_cast<uint32_t>(cfg.kblk) * (SUB_BYTES + w_bytes);
            const size_t w_step = static_cast<size_t>(p.c_out) * 32;
            RingPos rp;
            for (uint32_t work = pair; work < n_work && !aborted(abort_flag); work += n_pairs) {
                const int slice = static_cast<int>(work % static_cast<uint32_t>(cfg.n_slices));
                const uint32_t pix0 = ((work / static_cast<uint32_t>(cfg.n_slices)) * 2u + rank) * BM;
                const int n0 = static_cast<int>(pix0 / static_cast<uint32_t>(hw));
                const int rem = static_cast<int>(pix0 - static_cast<uint32_t>(n0) * static_cast<uint32_t>(hw));
                const int oh0 = rem / p.wo, ow0 = rem - oh0 * p.wo;
                const int w0 = ow0 * p.stride_w - p.pad_w, h0 = oh0 * p.stride_h - p.pad_h;
                const float* wsrc = p.wx + (static_cast<size_t>(slice) * cfg.bn + rank * cfg.half_rows) * 32;
                int ch = 0, tw = 0, off_w = 0, off_h = 0;
                for (int c = 0; c < n_sub; ++c) {
                    if (rp.wrapped && !mbar_wait_lone(smem_u32(&s_free[rp.s]), rp.parity ^ 1u)) *abort_flag = 2;
                    if (aborted(abort_flag)) break;
                    uint32_t a_smem = ring + rp.s * cfg.stage_bytes;
                    const uint32_t bar = smem_u32(&s_full[rp.s]);
                    mbar_arrive_expect_tx(bar, tx);
                    for (int j = 0; j < cfg.kblk; ++j) {
                        tma_load_im2col_4d(a_smem, &tm_x, bar, ch, w0, h0, n0, static_cast<uint16_t>(off_w),
                                           static_cast<uint16_t>(off_h));
                        bulk_load_1d(a_smem + SUB_BYTES, wsrc, w_bytes, bar);
                        a_smem += cfg.sub_bytes;
                        wsrc += w_step;
                        ch += 32;
                        if (ch >= p.c_in) {
                            ch = 0;
                            off_w += p.dil_w;
                            if (++tw == p.kw) { tw = 0; off_w = 0; off_h += p.dil_h; }
                        }
                    }
                    rp.advance(NS);
                    ++issued;
                }
            }
            // Walk back over the stages still in use.  On the normal path: wait until the pair MMAs
            // have released them, so that no multicast arrival is still on its way to this CTA when
            // it leaves.  After an abort: let the loads in flight land.
            const bool bad = aborted(abort_flag);
            for (int back = 0; back < NS && back < issued; ++back) {
                if (rp.s == 0) { rp.s = NS; rp.parity ^= 1u; }
                --rp.s;
                if (bad) (void)mbar_wait(smem_u32(&s_full[rp.s]), rp.parity);
                else if (!mbar_wait(smem_u32(&s_free[rp.s]), rp.parity)) { *abort_flag = 3; break; }
            }
        }
    } else if (warp == 1 && rank == 1) {
        // =========================== relay (second CTA) ===========================
        if (lane == 0) {
            RingPos rp;
            for (uint32_t work = pair; work < n_work && !aborted(abort_flag); work += n_pairs) {
                for (int c = 0; c < n_sub; ++c) {
                    if (!mbar_wait_lone(smem_u32(&s_full[rp.s]), rp.parity)) { *abort_flag = 4; break; }
                    mbar_arrive_cluster_relaxed(mapa_shared(smem_u32(&s_full[rp.s]), 0));
                    rp.advance(NS);
                }
            }
        }
    } else if (warp == 1) {
        // =========================== MMA issuer (first CTA) ===========================
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_tf32(2 * BM, cfg.bn);
            RingPos rp;
            uint32_t ab = 0, acc_par = 0;
            bool acc_wrapped = false;
            for (uint32_t work = pair; work < n_work && !aborted(abort_flag); work += n_pairs) {
                if (acc_wrapped && !mbar_wait_cluster(smem_u32(&s_accfree[ab]), acc_par ^ 1u)) {
                    *abort_flag = 5;
                    break;
                }
                tc_fence_after();
                const uint32_t acc = tmem + ab * cfg.bn;
                for (int c = 0; c < n_sub; ++c) {
                    if (!mbar_wait_lone(smem_u32(&s_full[rp.s]), rp.parity)) { *abort_flag = 6; break; }
                    tc_fence_after();
                    const uint32_t a_smem = ring + rp.s * cfg.stage_bytes;
                    uint64_t adesc = umma_desc_k_sw128(a_smem, 1024);
                    uint64_t bdesc = umma_desc_k_sw128(a_smem + SUB_BYTES, 1024);
                    for (int j = 0; j < cfg.kblk; ++j) {
#pragma unroll
                        for (int kq = 0; kq < 4; ++kq)
                            umma_tf32_ss_pair(acc, adesc + 2 * kq, bdesc + 2 * kq, idesc, (c > 0 || j > 0 || kq > 0) ? 1u : 0u);
                        adesc += cfg.sub_bytes >> 4;   // the next 32-column block of the stage (start address in 16-byte units)
                        bdesc += cfg.sub_bytes >> 4;
                    }
                    umma_commit_pair(smem_u32(&s_free[rp.s]));
                    rp.advance(NS);
                }
                if (aborted(abort_flag)) break;
                umma_commit_pair(smem_u32(&s_accfull[ab]));
                if (ab == 1) { acc_par ^= 1u; acc_wrapped = true; }
                ab ^= 1u;
            }
        }
    } else if (warp >= 4) {
        // =========================== epilogue (both CTAs) ===========================
        const int q = warp & 3;
        const int half = (warp - 4) >> 2;
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t my_staging = staging + (warp - 4) * cfg.boxes * BOX_BYTES;
        const uint32_t box_toggle = cfg.boxes == 2 ? 1u : 0u;
        const uint32_t rx = static_cast<uint32_t>(lane & 7);
        const int n_blk = cfg.bn / 32;
        uint32_t nb = 0, ti = 0;
        for (uint32_t work = pair; work < n_work; work += n_pairs, ++ti) {
            const int slice = static_cast<int>(work % static_cast<uint32_t>(cfg.n_slices));
            const uint32_t pix0 = ((work / static_cast<uint32_t>(cfg.n_slices)) * 2u + rank) * BM;
            const int ab = static_cast<int>(ti & 1u);
            const long long box_pix = static_cast<long long>(pix0) + q * 32;
            const bool res_pass = p.residual != nullptr && box_pix < p.pixels;
            const int res_rows = p.pixels - box_pix < 32 ? static_cast<int>(p.pixels - box_pix) : 32;
            const float* res_base = res_pass ? p.residual + box_pix * p.c_out + slice * cfg.bn : nullptr;
            float4 rv[8];
            if (res_pass && half < n_blk) load_residual_box(rv, res_base + half * 32, p.c_out, res_rows, lane);
            const int o0 = slice * cfg.bn;
            float bias_next = half < n_blk ? bias_lane_load(p.bias, o0 + half * 32, p.c_out, lane) : 0.f;   // first block's bias
            const bool ok = aborted(abort_flag) || mbar_wait(smem_u32(&s_accfull[ab]), (ti >> 1) & 1u);
            if (!__all_sync(0xFFFFFFFFu, ok)) *abort_flag = 8;
            if (__any_sync(0xFFFFFFFFu, aborted(abort_flag))) break;
            tc_fence_after();
            const uint32_t accfree_remote = mapa_shared(smem_u32(&s_accfree[ab]), 0);
            for (int blk = half; blk < n_blk; blk += 2, ++nb) {
                uint32_t v[32];
                tmem_ld32(tmem + lane_addr + ab * cfg.bn + blk * 32, v);
                tmem_ld_wait();
                if (blk + 2 >= n_blk) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(accfree_remote);
                }
                const uint32_t box = my_staging + (nb & box_toggle) * BOX_BYTES;
                if (lane == 0) {
                    if (cfg.boxes == 2) { if (nb >= 2) tma_store_wait_read_n<1>(); }
                    else if (nb >= 1) tma_store_wait_read_n<0>();
                }
                __syncwarp();
                const uint32_t stage_row = box + lane * 128;
                const int relu_now = res_pass ? 0 : p.relu;
                const float bias_cur = bias_next;
                if (blk + 2 < n_blk) bias_next = bias_lane_load(p.bias, o0 + (blk + 2) * 32, p.c_out, lane);   // a block ahead
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
                if (res_pass) {
                    __syncwarp();
                    apply_residual_box(box, rv, p.relu, lane);
                    if (blk + 2 < n_blk) load_residual_box(rv, res_base + (blk + 2) * 32, p.c_out, res_rows, lane);
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                    if (pix0 + q * 32 < p.pixels) tma_store_2d(&tm_y, box, o0 + blk * 32, static_cast<int>(pix0) + q * 32);
                    tma_store_commit();
                }
            }
        }
        if (lane == 0) tma_store_wait_read();
    }

    tc_fence_before();
    cluster_sync_all();   // neither CTA leaves (or frees tensor memory) while the other may still signal it
    if (tid == 0 && s_abort != 0) {
        atomicExch(p.status + 0, static_cast<int>(NM_ERR_TIMEOUT));
        atomicExch(p.status + 1, 70 + s_abort);
        atomicExch(p.status + 2, static_cast<int>(blockIdx.x));
    }
    if (warp == 2) tmem_dealloc_pair(tmem, 512);
}

bool make_cfg(const ConvParams& p, const nm_plan_t* plan, PairCfg* cfg)
{
    if (!p.wx || !nmtm::available()) return false;
    if (p.c_in % 32 != 0 || p.c_out % 32 != 0) return false;
    if (!nmtm::im2col_geometry_ok(p)) return false;
    if (static_cast<long long>(p.batch) * p.h * p.w * p.c_in * 4 < 131072) return false;
    if (p.pixels >= (1ll << 31) - 2 * BM) return false;
    int bn = plan && plan->bn > 0 ? plan->bn : (p.c_out % 256 == 0 ? 256 : 128);
    if ((bn != 128 && bn != 256) || p.c_out % bn != 0) return false;
    if (plan && plan->split != 0) return false;   // no split of the reduction axis in this kernel
    cfg->bn = bn;
    cfg->half_rows = bn / 2;
    cfg->n_slices = p.c_out / bn;
    cfg->b_bytes = cfg->half_rows * 128;         // 8 or 16 KB: keeps every stage 1024-byte aligned
    cfg->sub_bytes = SUB_BYTES + cfg->b_bytes;
    // two 32-column blocks per stage (the default where K / 32 is even) halve the per-stage costs of
    // the lone threads: waits, commits, the relay's arrival
    cfg->kblk = plan && plan->kblk > 0 ? plan->kblk : ((p.k / 32) % 2 == 0 ? 2 : 1);
    if (cfg->kblk > 2 || (p.k / 32) % cfg->kblk != 0) return false;
    cfg->stage_bytes = cfg->kblk * cfg->sub_bytes;
    cfg->n_sub = (p.k / 32) / cfg->kblk;
    cfg->boxes = p.k / 32 <= 8 ? 2 : 1;
    const int budget = 227 * 1024 - 1024 - 8 * cfg->boxes * BOX_BYTES - 1024;
    int stages = plan && plan->stages > 0 ? plan->stages : NSTAGE_MAX;
    if (stages > NSTAGE_MAX || stages < 2) return false;
    if (plan && plan->stages > 0) {
        if (stages * cfg->stage_bytes > budget) return false;
    } else {
        while (stages > 2 && stages * cfg->stage_bytes > budget) --stages;
        if (stages * cfg->stage_bytes > budget) return false;
    }
    cfg->stages = stages;
    const long long pix_blocks = (p.pixels + BM - 1) / BM;
    cfg->n_work = ((pix_blocks + 1) / 2) * cfg->n_slices;
    if (cfg->n_work >= (1ll << 30)) return false;
    return true;
}

size_t smem_bytes(const PairCfg& cfg)
{
    size_t smem = 1024 + static_cast<size_t>(cfg.stages) * cfg.stage_bytes + 8 * cfg.boxes * BOX_BYTES;
    return smem < 120 * 1024 ? 120 * 1024 : smem;   // one CTA per SM: the pair owns all 512 TMEM columns of both
}

// Pairs of SMs that can hold one cluster each at the same time (per device; 0 = clusters unavailable).
int max_pairs(size_t smem)
{
    static int cached[64];
    static bool known[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (!known[dev]) {
        cudaLaunchConfig_t lc = {};
        lc.gridDim = dim3(2);
        lc.blockDim = dim3(THREADS);
        lc.dynamicSmemBytes = smem;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        lc.attrs = attr;
        lc.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, k_conv_pair, &lc) != cudaSuccess) {
            (void)cudaGetLastError();
            n = 0;
        }
        cached[dev] = n;
        known[dev] = true;
    }
    return cached[dev];
}

}  // namespace

namespace nmhost {

bool pair_plan_ok(const ConvParams& p, const nm_plan_t* plan)
{
    PairCfg cfg;
    return make_cfg(p, plan, &cfg);
}

nm_status_t launch_conv_pair(const ConvParams& p, const nm_plan_t* plan, cudaStream_t st)
{
    PairCfg cfg;
    if (!make_cfg(p, plan, &cfg))
        return fail(NM_ERR_UNSUPPORTED, "nm_conv2d: the pair kernel does not take this layer / plan");
    alignas(64) CUtensorMap tm_x, tm_y;
    if (!nmtm::encode_x_im2col(p, BM, &tm_x) || !nmtm::encode_y_tiled(p, &tm_y))
        return fail(NM_ERR_CUDA, "nm_conv2d: tensor-map encoding failed (variant 7)");
    const size_t smem = smem_bytes(cfg);
    cudaError_t e = nmhost::ensure_dynamic_smem(reinterpret_cast<const void*>(k_conv_pair), smem);
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "cudaFuncSetAttribute (variant 7): %s", cudaGetErrorString(e));
    const int pairs_max = max_pairs(smem);   // every configuration takes a whole SM, so the first answer holds for all
    if (pairs_max < 1) return fail(NM_ERR_UNSUPPORTED, "nm_conv2d: this device runs no clusters of two CTAs (variant 7)");
    const long long pairs = cfg.n_work < pairs_max ? cfg.n_work : pairs_max;
    e = nmhost::launch_pdl(k_conv_pair, static_cast<unsigned>(2 * pairs), THREADS, smem, st, p, cfg, tm_x, tm_y);
    nmhost::count_launch(1);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "nm_conv2d launch (variant 7): %s", cudaGetErrorString(e));
    return NM_OK;
}

}  // namespace nmhost
