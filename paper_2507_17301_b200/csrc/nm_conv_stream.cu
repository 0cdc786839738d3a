// Variant 3: stream kernel — persistent, warp-specialised sparse implicit GEMM.
//
// One CTA per SM walks a static list of work items (128 output pixels x BN output channels,
// BN = G pruning tiles).  The reduction axis is cut into chunks of whole N:M groups: S source
// columns (32 or 64) of which every tile keeps KC.  Roles, all connected by mbarriers:
//
//   producer (1 thread)     TMA: im2col-mode loads bring the DENSE activation slab
//                           [128 pixels x S columns] (stride, dilation, tap offset and zero
//                           padding done by the hardware), a tiled load brings the weight chunk
//                           [BN x KC] (K-major, 128-byte swizzle), a bulk copy brings each tile's
//                           kept-column offsets.  Ring of 3-6 stages keeps HBM requests in flight.
//   compactors (8 warps)    thread = pixel row = TMEM lane, two warps per lane quadrant (one per
//                           half of the chunk).  Each reads its row's share of the slab ONCE with
//                           conflict-free 16-byte loads (one load = one group of 4 source columns)
//                           and, for every tile of the CTA, selects that tile's kept columns
//                           in registers (warp-uniform selectors), rounds them to TF32 and writes
//                           them into the tile's operand columns in tensor memory: the fused
//                           im2col + packing of Sec. 3.2 restricted to the surviving columns.
//   MMA issuer (1 thread)   D[128 x T] += A[tmem] * W[smem]^T, KC/8 tcgen05.mma per tile and chunk
//                           (Algorithm 1: the T accumulators are T TMEM columns).
//   epilogue (4 warps)      TMEM -> registers, + bias, ReLU, staged through shared memory in the
//                           swizzled layout and written to NHWC with TMA stores.  With two
//                           accumulator buffers it overlaps the next item's main loop.
//
// Every wait is bounded; on expiry the CTA raises an abort flag, every role drains to the common
// exit, the producer waits (bounded) for loads still in flight, TMEM is released, and the host
// learns of it through the status word.
#include "nm_internal.h"
#include "nm_ptx.cuh"
#include "nm_tmap.cuh"

namespace {

using namespace nmk;

constexpr int BM = 128;
constexpr int SUB_BYTES = BM * 128;   // one 32-column slab sub-tile
constexpr int NSTAGE_MAX = 6;
constexpr int A_COL0 = 256;           // TMEM: accumulators in columns [0, 256), operand sets above
constexpr int THREADS = 512;
constexpr int STAGING_BYTES = 4 * 2 * 4096;  // per epilogue warp two 32 x 32 output boxes

struct StreamCfg {
    int g;            // pruning tiles per CTA
    int bn;           // output channels per CTA = g * tile_t
    int n_slices;     // work items along the channel axis
    int n_acc;        // accumulator buffers: 2 when bn <= 128
    int stages;
    int b_bytes;      // weight bytes per stage
    int stage_bytes;
    int set_cols;     // TMEM columns of one operand set = g * 32
    long long n_work;
};

__device__ __forceinline__ bool aborted(volatile int* flag) { return *flag != 0; }

__device__ __forceinline__ float4 lds128(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// One of the MG floats of a group (MG / 4 consecutive 16-byte pieces) by a warp-uniform offset.
template <int MG>
__device__ __forceinline__ float pick(const float4* L, uint32_t r);
template <>
__device__ __forceinline__ float pick<4>(const float4* L, uint32_t r)
{
    const float lo = (r & 1u) ? L[0].y : L[0].x;
    const float hi = (r & 1u) ? L[0].w : L[0].z;
    return (r & 2u) ? hi : lo;
}
template <>
__device__ __forceinline__ float pick<8>(const float4* L, uint32_t r)
{
    const float a = pick<4>(L, r), b = pick<4>(L + 1, r);
    return (r & 4u) ? b : a;
}

// Round-to-nearest (ties away) onto the TF32 grid: the tensor core reads the upper 19 bits.
__device__ __forceinline__ uint32_t round_tf32_bits(float f) { return __float_as_uint(f) + 0x1000u; }

template <int N>
__device__ __forceinline__ void tmem_st_n(uint32_t taddr, const uint32_t* v)
{
    if constexpr (N == 16) {
        tmem_st16(taddr, v);
    } else if constexpr (N == 12) {
        tmem_st8(taddr, v);
        tmem_st4(taddr + 8, v + 8);
    } else if constexpr (N == 8) {
        tmem_st8(taddr, v);
    } else {
        static_assert(N == 4, "unsupported operand width");
        tmem_st4(taddr, v);
    }
}

// NK kept columns in every group of MG source columns; NK == MG == 4 stands for "all kept".
template <int NK, int MG>
struct Pattern {
    static constexpr bool DENSE = NK == MG;
    static constexpr int S = (DENSE || (MG == 4 && NK == 3)) ? 32 : 64;  // source columns per chunk
    static constexpr int GROUPS = S / MG;
    static constexpr int KC = GROUPS * NK;   // kept columns per chunk and tile
    static constexpr int SEGS = S / 32;
    static constexpr int GW = GROUPS / 2;    // groups per compactor half
    static constexpr int KW = GW * NK;       // kept columns per compactor half
    static constexpr int LW = S / 8;         // 16-byte loads per compactor thread and chunk
};

template <int NK, int MG>
__global__ void __launch_bounds__(THREADS, 1)
k_conv_stream(const ConvParams p, const StreamCfg cfg, const __grid_constant__ CUtensorMap tm_x,
              const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_y)
{
    using P = Pattern<NK, MG>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_full[NSTAGE_MAX], s_free[NSTAGE_MAX], s_aready[2], s_afree[2], s_accfull[2], s_accfree[2];
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t n_work = static_cast<uint32_t>(cfg.n_work);   // below 2^31: per-item arithmetic stays 32-bit
    const int NS = cfg.stages, n_chunks = p.v2_chunks, g = cfg.g, T = p.tile_t;
    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t staging = ring + NS * cfg.stage_bytes;
    volatile int* abort_flag = &s_abort;

    // ---- set-up ----------------------------------------------------------------------------------
    if (warp == 2) tmem_alloc(smem_u32(&s_tmem), 512);
    if (tid == 0) {
        for (int i = 0; i < NSTAGE_MAX; ++i) {
            mbar_init(smem_u32(&s_full[i]), 1);       // producer's expect-tx arrival
            mbar_init(smem_u32(&s_free[i]), 8 + 1);   // compactor warps + MMA commit
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&s_aready[i]), 8);     // compactor warps
            mbar_init(smem_u32(&s_afree[i]), 1);      // MMA commit
            mbar_init(smem_u32(&s_accfull[i]), 1);    // MMA commit
            mbar_init(smem_u32(&s_accfree[i]), 4);    // epilogue warps
        }
        mbar_fence_init();
        s_abort = 0;
        tma_prefetch_desc(&tm_x);
        tma_prefetch_desc(&tm_w);
        tma_prefetch_desc(&tm_y);
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
            const int hw = p.ho * p.wo;
            const size_t rpitch = static_cast<size_t>(n_chunks) * 32;
            const uint32_t tx_fixed = static_cast<uint32_t>(cfg.bn) * 128u + static_cast<uint32_t>(g) * 32u;
            RingPos rp;
            int issued = 0;
            for (uint32_t work = blockIdx.x; work < n_work && !aborted(abort_flag); work += gridDim.x) {
                const int slice = static_cast<int>(work % static_cast<uint32_t>(cfg.n_slices));
                const uint32_t pix0 = (work / static_cast<uint32_t>(cfg.n_slices)) * BM;
                const int n0 = static_cast<int>(pix0 / static_cast<uint32_t>(hw));
                const int rem = static_cast<int>(pix0 - static_cast<uint32_t>(n0) * static_cast<uint32_t>(hw));
                const int oh0 = rem / p.wo, ow0 = rem - oh0 * p.wo;
                const int w0 = ow0 * p.stride_w - p.pad_w, h0 = oh0 * p.stride_h - p.pad_h;
                const uint8_t* rsrc = p.rel2 + static_cast<size_t>(slice * g) * rpitch;
                int ch = 0, off_w = 0, off_h = 0, tw = 0, k0 = 0;   // position of the next 32-column sub-tile
                for (int c = 0; c < n_chunks; ++c) {
                    if (rp.wrapped && !mbar_wait_lone(smem_u32(&s_free[rp.s]), rp.parity ^ 1u)) *abort_flag = 2;
                    if (aborted(abort_flag)) break;
                    const uint32_t b_smem = ring + rp.s * cfg.stage_bytes;
                    const uint32_t slab = b_smem + cfg.b_bytes;
                    const uint32_t relbuf = slab + P::SEGS * SUB_BYTES;
                    const uint32_t bar = smem_u32(&s_full[rp.s]);
                    const int live = (P::SEGS == 2 && k0 + 32 >= p.k) ? 1 : P::SEGS;
                    mbar_arrive_expect_tx(bar, static_cast<uint32_t>(live) * SUB_BYTES + tx_fixed);
                    for (int seg = 0; seg < P::SEGS; ++seg) {
                        if (seg < live)
                            tma_load_im2col_4d(slab + seg * SUB_BYTES, &tm_x, bar, ch, w0, h0, n0,
                                               static_cast<uint16_t>(off_w), static_cast<uint16_t>(off_h));
                        k0 += 32;
                        ch += 32;
                        if (ch >= p.c_in) {
                            ch = 0;
                            off_w += p.dil_w;
                            if (++tw == p.kw) { tw = 0; off_w = 0; off_h += p.dil_h; }
                        }
                    }
                    tma_load_2d(b_smem, &tm_w, bar, c * 32, slice * cfg.bn);
                    for (int t = 0; t < g; ++t) bulk_load_1d(relbuf + t * 32, rsrc + t * rpitch + c * 32, 32u, bar);
                    rp.advance(NS);
                    ++issued;
                }
            }
            if (aborted(abort_flag)) {
                // loads already issued still target this CTA's shared memory: let them land
                for (int back = 0; back < NS && back < issued; ++back) {
                    if (rp.s == 0) { rp.s = NS; rp.parity ^= 1u; }
                    --rp.s;
                    (void)mbar_wait(smem_u32(&s_full[rp.s]), rp.parity);
                }
            }
        }
    } else if (warp == 1) {
        // =========================== MMA issuer ===========================
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_tf32(BM, T);
            RingPos rp;
            uint32_t set = 0, set_par = 0;          // operand set of this chunk, parity of its current use
            uint32_t ab = 0, acc_par = 0;           // accumulator buffer of this item, parity of its current use
            bool acc_wrapped = false;
            for (uint32_t work = blockIdx.x; work < n_work && !aborted(abort_flag); work += gridDim.x) {
                if (acc_wrapped && !mbar_wait_lone(smem_u32(&s_accfree[ab]), acc_par ^ 1u)) {
                    *abort_flag = 5;
                    break;
                }
                tc_fence_after();
                const uint32_t acc = tmem + ab * cfg.bn;
                for (int c = 0; c < n_chunks; ++c) {
                    if (!mbar_wait_lone(smem_u32(&s_full[rp.s]), rp.parity)) { *abort_flag = 6; break; }
                    if (!mbar_wait_lone(smem_u32(&s_aready[set]), set_par)) { *abort_flag = 7; break; }
                    if (aborted(abort_flag)) break;
                    tc_fence_after();
                    const uint32_t b_smem = ring + rp.s * cfg.stage_bytes;
                    const uint32_t a_set = tmem + A_COL0 + set * cfg.set_cols;
                    for (int t = 0; t < g; ++t) {
                        const uint64_t bdesc = umma_desc_k_sw128(b_smem + t * T * 128, 1024);
#pragma unroll
                        for (int kq = 0; kq < P::KC / 8; ++kq)
                            umma_tf32_ts(acc + t * T, a_set + t * 32 + kq * 8, bdesc + 2 * kq, idesc,
                                         (c > 0 || kq > 0) ? 1u : 0u);
                    }
                    umma_commit(smem_u32(&s_afree[set]));
                    umma_commit(smem_u32(&s_free[rp.s]));
                    rp.advance(NS);
                    if (set == 1) set_par ^= 1u;
                    set ^= 1u;
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
    } else if (warp >= 4 && warp < 8) {
        // =========================== epilogue ===========================
        const int q = warp & 3;
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t my_staging = staging + q * 2 * 4096;
        const uint32_t rx = static_cast<uint32_t>(lane & 7);
        const int n_blk = cfg.bn / 32;
        uint32_t ti = 0;
        uint32_t nb = 0;  // staging boxes this warp has filled so far
        for (uint32_t work = blockIdx.x; work < n_work; work += gridDim.x, ++ti) {
            const int slice = static_cast<int>(work % static_cast<uint32_t>(cfg.n_slices));
            const uint32_t pix0 = (work / static_cast<uint32_t>(cfg.n_slices)) * BM;
            const int ab = cfg.n_acc == 2 ? static_cast<int>(ti & 1u) : 0;
            const bool ok = aborted(abort_flag) ||
                            mbar_wait(smem_u32(&s_accfull[ab]), (cfg.n_acc == 2 ? (ti >> 1) : ti) & 1u);
            if (!__all_sync(0xFFFFFFFFu, ok)) *abort_flag = 8;
            if (__any_sync(0xFFFFFFFFu, aborted(abort_flag))) break;
            tc_fence_after();
            const int o0 = slice * cfg.bn;
            for (int blk = 0; blk < n_blk; ++blk, ++nb) {
                uint32_t v[32];
                tmem_ld32(tmem + lane_addr + ab * cfg.bn + blk * 32, v);
                tmem_ld_wait();
                if (blk == n_blk - 1) {
                    // the accumulator buffer may be overwritten from here on
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&s_accfree[ab]));
                }
                const uint32_t box = my_staging + (nb & 1u) * 4096;
                if (lane == 0 && nb >= 2) tma_store_wait_read_n<1>();  // the box's previous store has read it
                __syncwarp();
                const uint32_t stage_row = box + lane * 128;
                // with a shortcut input the activation waits for the second pass below
                const long long box_pix = static_cast<long long>(pix0) + q * 32;
                const bool res_pass = p.residual != nullptr && box_pix < p.pixels;
                const int relu_now = res_pass ? 0 : p.relu;
#pragma unroll
                for (int qq = 0; qq < 8; ++qq) {
                    float o[4];
                    float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (p.bias) bv = __ldg(reinterpret_cast<const float4*>(p.bias + o0 + blk * 32) + qq);
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
                    const long long left = p.pixels - box_pix;
                    add_residual_box(box, p.residual + box_pix * p.c_out + o0 + blk * 32, p.c_out,
                                     left < 32 ? static_cast<int>(left) : 32, p.relu, lane);
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                    if (pix0 + q * 32 < p.pixels)
                        tma_store_2d(&tm_y, box, o0 + blk * 32, static_cast<int>(pix0) + q * 32);
                    tma_store_commit();
                }
            }
        }
        if (lane == 0) tma_store_wait_read();   // shared memory must outlive the stores' reads; the writes complete with the grid
    } else if (warp >= 8) {
        // =========================== compactors ===========================
        const int wg = (warp - 8) >> 2;   // which half of the chunk
        const int q = warp & 3;           // TMEM lane quadrant
        const int row = q * 32 + lane;
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t rx = static_cast<uint32_t>(row & 7);
        constexpr int CI0_STEP = P::LW;   // first 16-byte piece of half `wg`
        RingPos rp;
        uint32_t set = 0, set_par = 0;
        bool set_wrapped = false;
        for (uint32_t work = blockIdx.x; work < n_work && !aborted(abort_flag); work += gridDim.x) {
            for (int c = 0; c < n_chunks; ++c) {
                const int s = rp.s;
                bool ok = mbar_wait_lone(smem_u32(&s_full[s]), rp.parity);
                if (!__all_sync(0xFFFFFFFFu, ok)) *abort_flag = 3;
                ok = !set_wrapped || mbar_wait_lone(smem_u32(&s_afree[set]), set_par ^ 1u);
                if (!__all_sync(0xFFFFFFFFu, ok)) *abort_flag = 4;
                if (__any_sync(0xFFFFFFFFu, aborted(abort_flag))) break;
                tc_fence_after();
                const uint32_t slab = ring + s * cfg.stage_bytes + cfg.b_bytes;
                const uint32_t relbuf = slab + P::SEGS * SUB_BYTES;
                const int ci0 = wg * CI0_STEP;
                const bool live = c * P::S + (ci0 >> 3) * 32 < p.k;   // this half's sub-tile was loaded
                float4 L[P::LW];
#pragma unroll
                for (int i = 0; i < P::LW; ++i) {
                    const int ci = ci0 + i;
                    L[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                    // self-checking build: the row's pieces lie inside this stage's slab
                    NM_CHECKED((ci >> 3) < P::SEGS && slab + (ci >> 3) * SUB_BYTES + row * 128 + 128 <= relbuf, p.status, 301, ci)
                    if (live) L[i] = lds128(slab + (ci >> 3) * SUB_BYTES + row * 128 + ((static_cast<uint32_t>(ci & 7) ^ rx) << 4));
                }
                const uint32_t a_set = tmem + lane_addr + A_COL0 + set * cfg.set_cols + wg * P::KW;
                for (int t = 0; t < g; ++t) {
                    uint32_t sel[P::KW / 4];
                    if constexpr (!P::DENSE) {
#pragma unroll
                        for (int i = 0; i < P::KW / 4; ++i) sel[i] = lds32(relbuf + t * 32 + wg * P::KW + 4 * i);
                    }
                    uint32_t v[P::KW];
#pragma unroll
                    for (int j = 0; j < P::KW; ++j) {
                        float f;
                        if constexpr (P::DENSE) {
                            const float4& l4 = L[j >> 2];
                            f = (j & 3) == 0 ? l4.x : (j & 3) == 1 ? l4.y : (j & 3) == 2 ? l4.z : l4.w;
                        } else {
                            const uint32_t r = (sel[j >> 2] >> (8 * (j & 3))) & static_cast<uint32_t>(MG - 1);
                            f = 0.f;
                            // self-checking build: a kept-column offset, taken whole, lies inside the chunk's source columns
                            NM_CHECKED(((sel[j >> 2] >> (8 * (j & 3))) & 0xFFu) < static_cast<uint32_t>(P::S), p.status, 302, sel[j >> 2])
                            f = pick<MG>(&L[(j / NK) * (MG / 4)], r);
                        }
                        v[j] = round_tf32_bits(f);   // a half that was not loaded holds zeros: 0x1000 is below TF32's last bit
                    }
                    tmem_st_n<P::KW>(a_set + t * 32, v);
                }
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(smem_u32(&s_aready[set]));
                    mbar_arrive(smem_u32(&s_free[s]));
                }
                rp.advance(NS);
                if (set == 1) { set_par ^= 1u; set_wrapped = true; }
                set ^= 1u;
            }
        }
    }

    // ---- common exit ---------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (tid == 0 && s_abort != 0) {
        atomicExch(p.status + 0, static_cast<int>(NM_ERR_TIMEOUT));
        atomicExch(p.status + 1, 30 + s_abort);
        atomicExch(p.status + 2, static_cast<int>(blockIdx.x));
    }
    if (warp == 2) tmem_dealloc(tmem, 512);
}

// ---- launch configuration --------------------------------------------------------------------------

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

// 0 = pattern not covered, otherwise NK * 16 + MG of the kernel instance.
int pattern_code(const ConvParams& p)
{
    if (p.n_keep == p.m_group) return 4 * 16 + 4;
    if (p.m_group == 4 && p.n_keep >= 1 && p.n_keep <= 3) return p.n_keep * 16 + 4;
    if (p.m_group == 8 && (p.n_keep == 1 || p.n_keep == 2 || p.n_keep == 4)) return p.n_keep * 16 + 8;
    return 0;
}

template <int NK, int MG>
bool layout_matches(const ConvParams& p)
{
    return p.v2_s == Pattern<NK, MG>::S && p.v2_kc == Pattern<NK, MG>::KC;
}

bool make_cfg(const ConvParams& p, const nm_plan_t* plan, StreamCfg* cfg)
{
    if (!p.wt2 || !p.rel2 || !nmtm::available()) return false;
    const int code = pattern_code(p);
    if (code == 0) return false;
    bool layout_ok = false;
    switch (code) {
        case 1 * 16 + 4: layout_ok = layout_matches<1, 4>(p); break;
        case 2 * 16 + 4: layout_ok = layout_matches<2, 4>(p); break;
        case 3 * 16 + 4: layout_ok = layout_matches<3, 4>(p); break;
        case 4 * 16 + 4: layout_ok = layout_matches<4, 4>(p); break;
        case 1 * 16 + 8: layout_ok = layout_matches<1, 8>(p); break;
        case 2 * 16 + 8: layout_ok = layout_matches<2, 8>(p); break;
        case 4 * 16 + 8: layout_ok = layout_matches<4, 8>(p); break;
    }
    if (!layout_ok) return false;
    const int T = p.tile_t;
    if (p.c_in % 32 != 0 || T % 16 != 0 || T > 256 || p.c_out % T != 0) return false;
    if (!nmtm::im2col_geometry_ok(p)) return false;
    // im2col maps of very small tensors are left to the other kernels
    if (static_cast<long long>(p.batch) * p.h * p.w * p.c_in * 4 < 131072) return false;
    if (p.pixels >= (1ll << 31) - BM) return false;
    int g;
    if (plan && plan->bn > 0) {
        if (plan->bn % T != 0) return false;
        g = plan->bn / T;
    } else {
        g = 1;
        for (int cand = 4; cand >= 1; --cand)
            if (cand * T <= 128 && p.n_tiles % cand == 0 && (cand * T) % 32 == 0) { g = cand; break; }
    }
    if (g < 1 || g > 4 || g * T > 256 || p.n_tiles % g != 0 || (g * T) % 32 != 0) return false;
    cfg->g = g;
    cfg->bn = g * T;
    cfg->n_slices = p.n_tiles / g;
    cfg->n_acc = cfg->bn <= 128 ? 2 : 1;
    cfg->set_cols = g * 32;
    cfg->b_bytes = ((cfg->bn * 128 + 1023) / 1024) * 1024;   // whole swizzle atoms
    cfg->stage_bytes = cfg->b_bytes + (p.v2_s / 32) * SUB_BYTES + 1024;  // offsets area padded to keep stages aligned
    const int budget = 227 * 1024 - 1024 - STAGING_BYTES - 1024;         // alignment slack, staging, static shared
    int stages = plan && plan->stages > 0 ? plan->stages : NSTAGE_MAX;
    if (stages > NSTAGE_MAX) return false;
    if (plan && plan->stages > 0) {
        if (stages * cfg->stage_bytes > budget) return false;
    } else {
        while (stages > 2 && stages * cfg->stage_bytes > budget) --stages;
        if (stages * cfg->stage_bytes > budget) return false;
    }
    cfg->stages = stages;
    const long long pix_blocks = (p.pixels + BM - 1) / BM;
    cfg->n_work = pix_blocks * cfg->n_slices;
    if (cfg->n_work >= (1ll << 31)) return false;
    return true;
}

template <int NK, int MG>
nm_status_t launch(const ConvParams& p, const StreamCfg& cfg, cudaStream_t st)
{
    alignas(64) CUtensorMap tm_x, tm_w, tm_y;
    if (!nmtm::encode_x_im2col(p, BM, &tm_x) || !nmtm::encode_w_tiled(p, cfg.bn, &tm_w) ||
        !nmtm::encode_y_tiled(p, &tm_y))
        return nmhost::fail(NM_ERR_CUDA, "nm_conv2d: tensor-map encoding failed (variant 3)");
    size_t smem = 1024 + static_cast<size_t>(cfg.stages) * cfg.stage_bytes + STAGING_BYTES;
    if (smem < 120 * 1024) smem = 120 * 1024;   // one CTA per SM: it owns all 512 TMEM columns
    cudaError_t e = nmhost::ensure_dynamic_smem(reinterpret_cast<const void*>(k_conv_stream<NK, MG>), smem);
    if (e != cudaSuccess) return nmhost::fail(NM_ERR_CUDA, "cudaFuncSetAttribute (variant 3): %s", cudaGetErrorString(e));
    const long long grid = cfg.n_work < sm_count() ? cfg.n_work : sm_count();
    e = nmhost::launch_pdl(k_conv_stream<NK, MG>, static_cast<unsigned>(grid), THREADS, smem, st, p, cfg, tm_x, tm_w, tm_y);
    nmhost::count_launch(1);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return nmhost::fail(NM_ERR_CUDA, "nm_conv2d launch (variant 3): %s", cudaGetErrorString(e));
    return NM_OK;
}

}  // namespace

namespace nmhost {

bool stream_plan_ok(const ConvParams& p, const nm_plan_t* plan)
{
    StreamCfg cfg;
    return make_cfg(p, plan, &cfg);
}

nm_status_t launch_conv_stream(const ConvParams& p, const nm_plan_t* plan, cudaStream_t st)
{
    StreamCfg cfg;
    if (!make_cfg(p, plan, &cfg))
        return fail(NM_ERR_UNSUPPORTED, "nm_conv2d: the stream kernel does not take this layer / plan");
    switch (pattern_code(p)) {
        case 1 * 16 + 4: return launch<1, 4>(p, cfg, st);
        case 2 * 16 + 4: return launch<2, 4>(p, cfg, st);
        case 3 * 16 + 4: return launch<3, 4>(p, cfg, st);
        case 4 * 16 + 4: return launch<4, 4>(p, cfg, st);
        case 1 * 16 + 8: return launch<1, 8>(p, cfg, st);
        case 2 * 16 + 8: return launch<2, 8>(p, cfg, st);
        case 4 * 16 + 8: return launch<4, 8>(p, cfg, st);
    }
    return fail(NM_ERR_UNSUPPORTED, "nm_conv2d: N:M pattern not covered by the stream kernel");
}

}  // namespace nmhost
