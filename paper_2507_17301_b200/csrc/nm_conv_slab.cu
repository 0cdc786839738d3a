// Variant 2: slab kernel — warp-specialised sparse implicit GEMM with the gathered operand in
// tensor memory.
//
// One CTA owns 128 output pixels and as many pruning tiles as fit 128 accumulator columns; two
// CTAs fit on an SM, so one CTA's epilogue overlaps the other's main loop.  The reduction axis
// is cut into chunks of G whole N:M groups (S = G*M source columns, of which every tile keeps
// KC = G*N).  Per chunk:
//   producer      brings the DENSE activation slab [128 pixels x S columns] into shared memory
//                 once, as 32-column sub-tiles in the 128-byte-swizzled layout, plus the weight
//                 chunk [channels x KC] (same layout, K-major).  Fast path: one thread issues
//                 TMA loads — im2col mode for the activations (the hardware walks the 128 output
//                 pixels, applies stride / dilation / the tap offset and zero-fills the padding),
//                 tiled mode for the weights.  General path (c_in % 32 != 0, tile_t % 8 != 0 or a
//                 tensor under 128 KiB): four warps of 4-byte cp.async with the same layout.
//   compactors    (4 warps, thread = pixel = TMEM lane) pick each tile's KC kept columns out of
//                 the slab by index (warp-uniform offsets), round to TF32 and write them to a
//                 TMEM operand buffer with tcgen05.st: the fused im2col + packing of Sec. 3.2
//                 restricted to the surviving columns, TMEM standing in for the packed strip;
//   MMA issuer    (1 thread) D[128 x T] += A[tmem] * W_chunk[smem]^T, KC/8 tcgen05.mma per tile:
//                 Algorithm 1's T accumulator registers are T TMEM columns.
// Epilogue (the compactor warps): TMEM -> registers, + bias, ReLU, NHWC store.
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, reports through the
// status word and drains to the common exit where TMEM is released.
#include "nm_internal.h"
#include "nm_ptx.cuh"
#include "nm_tmap.cuh"

namespace {

using namespace nmk;

constexpr int BM = 128;
constexpr int MAX_BN_COLS = 128;   // accumulator columns per CTA
constexpr int NA = 4;              // TMEM operand buffers of 32 columns
constexpr int TMEM_COLS = 256;     // 128 accumulator + 4 x 32 operand columns
constexpr int NSTAGE_MAX = 4;
constexpr int SUB_BYTES = BM * 128;  // one 32-column slab sub-tile

struct SlabCfg {
    int g_tiles;      // pruning tiles per CTA
    int umma_n;       // accumulator columns per tile (tile_t rounded up to 16)
    int n_slices;     // CTAs along the channel axis
    int stages;
    int segs;         // 32-column sub-tiles per slab chunk
    int b_rows;       // weight rows staged per chunk
    int b_tile_rows;  // row distance between two tiles' weights in shared memory
    int b_bytes, stage_bytes;
    int use_tma;
    int tma_store;    // epilogue through shared memory + TMA store
};

__device__ __forceinline__ bool aborted(volatile int* flag) { return *flag != 0; }

template <int KC, bool TMA>
__global__ void __launch_bounds__(288, 2)
k_conv_slab(const ConvParams p, const SlabCfg cfg, const __grid_constant__ CUtensorMap tm_x,
            const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_y)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_full[NSTAGE_MAX], s_free[NSTAGE_MAX], s_aready[NA], s_afree[NA], s_dready;
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort;
    __shared__ int s_rowoff[BM];
    __shared__ unsigned long long s_rowmask[BM];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slice = blockIdx.x % cfg.n_slices;
    const long long pix0 = static_cast<long long>(blockIdx.x / cfg.n_slices) * BM;
    const int tile0 = slice * cfg.g_tiles;
    const int g_here = min(cfg.g_tiles, p.n_tiles - tile0);
    const int S = p.v2_s, n_chunks = p.v2_chunks, NS = cfg.stages;

    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;  // stage: [weight tile][slab sub-tiles]
    volatile int* abort_flag = &s_abort;

    // ---- set-up ----------------------------------------------------------------------------------
    if (warp == 8) tmem_alloc(smem_u32(&s_tmem), TMEM_COLS);
    if (tid == 0) {
        for (int i = 0; i < NSTAGE_MAX; ++i) {
            mbar_init(smem_u32(&s_full[i]), TMA ? 1 : 128);  // TMA issuer, or the producer threads
            mbar_init(smem_u32(&s_free[i]), 128 + 1);        // compactor threads + MMA commit
        }
        for (int i = 0; i < NA; ++i) {
            mbar_init(smem_u32(&s_aready[i]), 128);          // compactor threads
            mbar_init(smem_u32(&s_afree[i]), 1);             // MMA commit
        }
        mbar_init(smem_u32(&s_dready), 1);
        mbar_fence_init();
        s_abort = 0;
        if (TMA) {
            tma_prefetch_desc(&tm_x);
            tma_prefetch_desc(&tm_w);
        }
    }
    if (!TMA && tid < BM) {
        const long long pix = pix0 + tid;
        int off = 0;
        unsigned long long mask = 0;
        if (pix < p.pixels) {
            const int hw = p.ho * p.wo;
            const int n = static_cast<int>(pix / hw);
            const int rem = static_cast<int>(pix - static_cast<long long>(n) * hw);
            const int oh = rem / p.wo, ow = rem - oh * p.wo;
            const int ih0 = oh * p.stride_h - p.pad_h, iw0 = ow * p.stride_w - p.pad_w;
            off = ((n * p.h + ih0) * p.w + iw0) * p.c_in;
            for (int t = 0; t < p.kh * p.kw; ++t) {
                const int ih = ih0 + (t / p.kw) * p.dil_h, iw = iw0 + (t % p.kw) * p.dil_w;
                if (ih >= 0 && ih < p.h && iw >= 0 && iw < p.w) mask |= 1ull << t;
            }
        }
        s_rowoff[tid] = off;
        s_rowmask[tid] = mask;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;

    if (warp >= 4 && warp < 8) {
        if (TMA) {
            // =========================== TMA producer (one thread) ===========================
            if (tid == 128) {
                const int hw = p.ho * p.wo;
                const int n0 = static_cast<int>(pix0 / hw);
                const int rem = static_cast<int>(pix0 - static_cast<long long>(n0) * hw);
                const int oh0 = rem / p.wo, ow0 = rem - oh0 * p.wo;
                const int w0 = ow0 * p.stride_w - p.pad_w, h0 = oh0 * p.stride_h - p.pad_h;
                const uint32_t b_box_bytes = static_cast<uint32_t>(cfg.b_rows) * 128u;
                for (int c = 0; c < n_chunks; ++c) {
                    const int s = c % NS;
                    if (c >= NS && !mbar_wait(smem_u32(&s_free[s]), ((c / NS) - 1) & 1)) *abort_flag = 2;
                    if (aborted(abort_flag)) break;
                    const uint32_t b_smem = ring + s * cfg.stage_bytes;
                    const uint32_t slab = b_smem + cfg.b_bytes;
                    const uint32_t bar = smem_u32(&s_full[s]);
                    int live = 0;
                    for (int seg = 0; seg < cfg.segs; ++seg) live += (c * S + seg * 32 < p.k) ? 1 : 0;
                    mbar_arrive_expect_tx(bar, static_cast<uint32_t>(live) * SUB_BYTES + b_box_bytes);
                    for (int seg = 0; seg < cfg.segs; ++seg) {
                        const int k0 = c * S + seg * 32;
                        if (k0 >= p.k) break;
                        const int tap = k0 / p.c_in, cc = k0 - tap * p.c_in;
                        tma_load_im2col_4d(slab + seg * SUB_BYTES, &tm_x, bar, cc, w0, h0, n0,
                                           static_cast<uint16_t>((tap % p.kw) * p.dil_w),
                                           static_cast<uint16_t>((tap / p.kw) * p.dil_h));
                    }
                    tma_load_2d(b_smem, &tm_w, bar, c * 32, tile0 * p.tile_t);
                }
            }
        } else {
            // =========================== cp.async producers (4 warps) ===========================
            const int pw = warp - 4, ptid = tid - 128;
            constexpr int QPR = KC / 4;  // 16-byte pieces per weight row
            const size_t wpitch = static_cast<size_t>(n_chunks) * 32;
            for (int c = 0; c < n_chunks; ++c) {
                const int s = c % NS;
                if (c >= NS && !mbar_wait(smem_u32(&s_free[s]), ((c / NS) - 1) & 1)) *abort_flag = 2;
                if (aborted(abort_flag)) break;
                const uint32_t b_smem = ring + s * cfg.stage_bytes;
                const uint32_t slab = b_smem + cfg.b_bytes;
                // activation slab: lane = source column, this warp's 32 pixels one after another
                for (int seg = 0; seg < cfg.segs; ++seg) {
                    const int colc = seg * 32 + lane;            // column inside the chunk
                    const int k = c * S + colc;                  // flattened (kh, kw, c) column
                    const bool col_ok = colc < S && k < p.k;
                    const int tap = col_ok ? k / p.c_in : 0;
                    const int cc = col_ok ? k - tap * p.c_in : 0;
                    const int delta = ((tap / p.kw) * p.dil_h * p.w + (tap % p.kw) * p.dil_w) * p.c_in + cc;
                    const uint32_t dst0 = slab + seg * SUB_BYTES + ((lane & 3) << 2);
#pragma unroll 4
                    for (int i = 0; i < 32; ++i) {
                        const int row = pw * 32 + i;
                        const bool ok = col_ok && ((s_rowmask[row] >> tap) & 1ull);
                        const float* src = ok ? p.x + (s_rowoff[row] + delta) : p.x;
                        cp_async4(dst0 + row * 128 + (((lane >> 2) ^ (row & 7)) << 4), src, ok ? 4u : 0u);
                    }
                }
                // weight chunk: rows = the CTA's channels (tile-major, umma_n rows per tile)
                for (int piece = ptid; piece < cfg.b_rows * QPR; piece += 128) {
                    const int row = piece / QPR, q = piece - row * QPR;
                    const int t = row / cfg.umma_n, rr = row - t * cfg.umma_n;
                    const int o = (tile0 + t) * p.tile_t + rr;
                    const bool ok = t < g_here && rr < p.tile_t && o < p.c_out;
                    const float* src = ok ? p.wt2 + static_cast<size_t>(o) * wpitch + c * 32 + q * 4 : p.wt2;
                    cp_async16(b_smem + row * 128 + ((q ^ (row & 7)) << 4), src, ok ? 16u : 0u);
                }
                cp_async_commit();
                // signal the previous chunk once its copies have landed (one group stays in flight)
                if (c > 0) {
                    cp_async_wait<1>();
                    fence_proxy_async();
                    mbar_arrive(smem_u32(&s_full[(c - 1) % NS]));
                }
            }
            cp_async_wait<0>();
            fence_proxy_async();
            if (!aborted(abort_flag)) mbar_arrive(smem_u32(&s_full[(n_chunks - 1) % NS]));
        }
    } else if (warp < 4) {
        // =========================== compactors, then epilogue ===========================
        const int row = tid;  // TMEM lane = pixel row
        const uint32_t lane_addr = static_cast<uint32_t>(warp * 32) << 16;
        const uint32_t rx4 = static_cast<uint32_t>(row & 7) << 4;
        const size_t rpitch = static_cast<size_t>(n_chunks) * 32;
        int use = 0;  // running count of operand-buffer uses
        for (int c = 0; c < n_chunks && !aborted(abort_flag); ++c) {
            const int s = c % NS;
            const uint32_t slab_row = ring + s * cfg.stage_bytes + cfg.b_bytes + row * 128;
            for (int t = 0; t < g_here; ++t, ++use) {
                // kept-column offsets of this (tile, chunk): warp-uniform, fetched before the waits
                uint32_t relw[KC / 4];
                const uint32_t* rp = reinterpret_cast<const uint32_t*>(p.rel2 + static_cast<size_t>(tile0 + t) * rpitch + c * 32);
#pragma unroll
                for (int q = 0; q < KC / 4; ++q) relw[q] = __ldg(rp + q);
                // (the votes keep the warp together for the .sync.aligned TMEM stores that follow)
                bool ok = t != 0 || mbar_wait(smem_u32(&s_full[s]), (c / NS) & 1);
                if (!__all_sync(0xFFFFFFFFu, ok)) { *abort_flag = 3; break; }
                const int buf = use % NA;
                ok = use < NA || mbar_wait(smem_u32(&s_afree[buf]), ((use / NA) - 1) & 1);
                if (!__all_sync(0xFFFFFFFFu, ok)) { *abort_flag = 4; break; }
                tc_fence_after();
                uint32_t v[KC];
#pragma unroll
                for (int j = 0; j < KC; ++j) {
                    const uint32_t rel = (relw[j >> 2] >> ((j & 3) * 8)) & 0xFFu;
                    // sub-tile (rel / 32), 16-byte piece ((rel / 4) % 8) ^ (row % 8), word rel % 4
                    const uint32_t u = ((rel & 31u) << 2) + ((rel >> 5) * SUB_BYTES);
                    float f = 0.f;
                    // self-checking build: a kept-column offset must lie inside the chunk's source columns
                    NM_CHECKED(rel < static_cast<uint32_t>(p.v2_s), p.status, 201, rel)
                    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(f) : "r"(slab_row + (u ^ rx4)));
                    v[j] = __float_as_uint(to_tf32(f));
                }
                const uint32_t a_addr = tmem + lane_addr + MAX_BN_COLS + buf * 32;
#pragma unroll
                for (int q = 0; q < KC / 8; ++q) tmem_st8(a_addr + q * 8, v + q * 8);
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(smem_u32(&s_aready[buf]));
            }
            if (aborted(abort_flag)) break;
            mbar_arrive(smem_u32(&s_free[s]));  // this thread is done reading the slab of stage s
        }
        // ---- epilogue ----
        {
            const bool ok = aborted(abort_flag) || mbar_wait(smem_u32(&s_dready), 0);
            if (!__all_sync(0xFFFFFFFFu, ok)) *abort_flag = 5;
        }
        if (cfg.tma_store) {
            // coalesced path: 32-column blocks staged in the (now idle) ring in the swizzled layout
            // a tiled TMA store expects, one 32 x 32 box per warp and block
            if (!__any_sync(0xFFFFFFFFu, aborted(abort_flag))) {
                tc_fence_after();
                const int bn_cols = g_here * p.tile_t;          // contiguous: tile_t is a multiple of 16 here
                const int o0 = tile0 * p.tile_t;
                for (int blk = 0; blk * 32 < bn_cols; ++blk) {
                    uint32_t v[32];
                    tmem_ld32(tmem + lane_addr + blk * 32, v);
                    tmem_ld_wait();
                    const uint32_t stage_row = ring + blk * SUB_BYTES + row * 128;
                    const float4* rrow = nm_residual_row(p, pix0 + row, o0 + blk * 32);
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        float o[4];
                        float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (p.bias) bv = __ldg(reinterpret_cast<const float4*>(p.bias + o0 + blk * 32) + q);
                        if (rrow) nm_add4(bv, __ldg(rrow + q));
                        o[0] = __uint_as_float(v[q * 4 + 0]) + bv.x;
                        o[1] = __uint_as_float(v[q * 4 + 1]) + bv.y;
                        o[2] = __uint_as_float(v[q * 4 + 2]) + bv.z;
                        o[3] = __uint_as_float(v[q * 4 + 3]) + bv.w;
                        if (p.relu) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) o[e] = fmaxf(o[e], 0.f);
                        }
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(stage_row + ((q ^ (row & 7)) << 4)),
                                     "f"(o[0]), "f"(o[1]), "f"(o[2]), "f"(o[3])
                                     : "memory");
                    }
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0 && pix0 + warp * 32 < p.pixels)
                        tma_store_2d(&tm_y, ring + blk * SUB_BYTES + warp * 32 * 128, o0 + blk * 32,
                                     static_cast<int>(pix0) + warp * 32);
                }
                if (lane == 0) {
                    tma_store_commit();
                    tma_store_wait_read();  // shared memory must outlive the stores' reads
                }
            }
        } else if (!__any_sync(0xFFFFFFFFu, aborted(abort_flag))) {
            tc_fence_after();
            const long long pix = pix0 + row;
            float* yrow = p.y + static_cast<size_t>(pix < p.pixels ? pix : 0) * p.c_out;
            const bool vec_ok = (p.c_out % 4 == 0) && (p.tile_t % 4 == 0);
            for (int t = 0; t < g_here; ++t) {
                const int o_base = (tile0 + t) * p.tile_t;
                const int n_valid = min(p.tile_t, p.c_out - o_base);
                for (int col0 = 0; col0 < n_valid; col0 += 16) {
                    uint32_t v[16];
                    tmem_ld16(tmem + lane_addr + t * cfg.umma_n + col0, v);
                    tmem_ld_wait();
                    if (pix < p.pixels) {
                        if (vec_ok && col0 + 16 <= n_valid) {
#pragma unroll
                            for (int q = 0; q < 16; q += 4) {
                                float4 o4;
                                float* o = reinterpret_cast<float*>(&o4);
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    float tt = __uint_as_float(v[q + e]);
                                    if (p.bias) tt += __ldg(p.bias + o_base + col0 + q + e);
                                    if (p.residual) tt += __ldg(p.residual + (yrow - p.y) + o_base + col0 + q + e);
                                    o[e] = p.relu ? fmaxf(tt, 0.f) : tt;
                                }
                                *reinterpret_cast<float4*>(yrow + o_base + col0 + q) = o4;
                            }
                        } else {
#pragma unroll
                            for (int q = 0; q < 16; ++q) {
                                if (col0 + q < n_valid) {
                                    float tt = __uint_as_float(v[q]);
                                    if (p.bias) tt += __ldg(p.bias + o_base + col0 + q);
                                    if (p.residual) tt += __ldg(p.residual + (yrow - p.y) + o_base + col0 + q);
                                    yrow[o_base + col0 + q] = p.relu ? fmaxf(tt, 0.f) : tt;
                                }
                            }
                        }
                    }
                }
            }
        }
    } else if (tid == 256) {
        // =========================== MMA issuer ===========================
        const uint32_t idesc = umma_idesc_tf32(BM, cfg.umma_n);
        int use = 0;
        for (int c = 0; c < n_chunks && !aborted(abort_flag); ++c) {
            const int s = c % NS;
            if (!mbar_wait(smem_u32(&s_full[s]), (c / NS) & 1)) { *abort_flag = 6; break; }
            const uint32_t b_smem = ring + s * cfg.stage_bytes;
            for (int t = 0; t < g_here; ++t, ++use) {
                const int buf = use % NA;
                if (!mbar_wait(smem_u32(&s_aready[buf]), (use / NA) & 1)) { *abort_flag = 7; break; }
                tc_fence_after();
                const uint64_t bdesc = umma_desc_k_sw128(b_smem + t * cfg.b_tile_rows * 128, 1024);
                const uint32_t a_addr = tmem + MAX_BN_COLS + buf * 32;
#pragma unroll
                for (int kq = 0; kq < KC / 8; ++kq)
                    umma_tf32_ts(tmem + t * cfg.umma_n, a_addr + kq * 8, bdesc + 2 * kq, idesc, (c > 0 || kq > 0) ? 1u : 0u);
                umma_commit(smem_u32(&s_afree[buf]));
            }
            if (aborted(abort_flag)) break;
            umma_commit(smem_u32(&s_free[s]));  // weight chunk of stage s consumed
        }
        if (!aborted(abort_flag)) umma_commit(smem_u32(&s_dready));
    }

    // ---- common exit ---------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (tid == 0 && s_abort != 0) {
        atomicExch(p.status + 0, static_cast<int>(NM_ERR_TIMEOUT));
        atomicExch(p.status + 1, 20 + s_abort);
        atomicExch(p.status + 2, static_cast<int>(blockIdx.x));
    }
    if (warp == 8) tmem_dealloc(tmem, TMEM_COLS);
}

// ---- launch configuration --------------------------------------------------------------------------
bool tma_admissible(const ConvParams& p)
{
    if (p.c_in % 32 != 0 || p.tile_t % 8 != 0) return false;
    // im2col maps of very small tensors are not used: the cp.async path takes them
    if (static_cast<long long>(p.batch) * p.h * p.w * p.c_in * 4 < 131072) return false;
    return nmtm::im2col_geometry_ok(p) && nmtm::available();
}

bool make_cfg(const ConvParams& p, const nm_plan_t* plan, SlabCfg* cfg)
{
    if (!p.wt2 || !p.rel2) return false;
    if (p.kh * p.kw > 64) return false;                                   // tap-validity mask is 64 bits
    if (static_cast<long long>(p.batch) * p.h * p.w * p.c_in >= (1ll << 31)) return false;  // 32-bit element offsets
    const int umma_n = p.tile_t <= 16 ? 16 : ((p.tile_t + 15) / 16) * 16;
    if (umma_n > MAX_BN_COLS) return false;
    int g = MAX_BN_COLS / umma_n;
    if (plan && plan->bn > 0) {
        if (plan->bn % p.tile_t != 0) return false;
        g = plan->bn / p.tile_t;
        if (g < 1 || g * umma_n > MAX_BN_COLS) return false;
    }
    g = g < p.n_tiles ? g : p.n_tiles;
    cfg->use_tma = tma_admissible(p) && !(plan && plan->split == 1) ? 1 : 0;  // split = 1 forces the cp.async producer
    cfg->g_tiles = g;
    cfg->umma_n = umma_n;
    cfg->n_slices = (p.n_tiles + g - 1) / g;
    cfg->segs = (p.v2_s + 31) / 32;
    cfg->b_tile_rows = cfg->use_tma ? p.tile_t : umma_n;
    cfg->b_rows = g * cfg->b_tile_rows;
    // room for the MMA of the last tile to read umma_n rows; whole 1024-byte swizzle atoms
    cfg->b_bytes = ((((g - 1) * cfg->b_tile_rows + umma_n) * 128 + 1023) / 1024) * 1024;
    cfg->stage_bytes = cfg->segs * SUB_BYTES + cfg->b_bytes;
    const int budget = 110 * 1024;                  // two CTAs per SM
    int stages = plan && plan->stages > 0 ? plan->stages : 3;
    if (stages > NSTAGE_MAX) return false;
    while (stages > 1 && stages * cfg->stage_bytes + 1024 > budget && !(plan && plan->stages > 0)) --stages;
    if (stages * cfg->stage_bytes + 1024 > 225 * 1024) return false;
    cfg->stages = stages;
    // TMA-store epilogue: channel blocks of 32 must tile the CTA's channel range exactly, the
    // staging blocks must fit the ring, and the pixel count must fit the map's 32-bit coordinate
    const int bn_cols = g * p.tile_t;
    cfg->tma_store = nmtm::available() && p.tile_t % 16 == 0 && bn_cols % 32 == 0 && p.c_out % 4 == 0 &&
                     (bn_cols / 32) * SUB_BYTES <= stages * cfg->stage_bytes && p.pixels < (1ll << 31) &&
                     p.n_tiles % g == 0 && p.c_out % p.tile_t == 0 && !(plan && plan->split == 2);
    return true;
}

template <int KC, bool TMA>
nm_status_t launch(const ConvParams& p, const SlabCfg& cfg, cudaStream_t st)
{
    alignas(64) CUtensorMap tm_x, tm_w, tm_y;
    memset(&tm_x, 0, sizeof(tm_x));
    memset(&tm_w, 0, sizeof(tm_w));
    memset(&tm_y, 0, sizeof(tm_y));
    if (TMA && (!nmtm::encode_x_im2col(p, BM, &tm_x) || !nmtm::encode_w_tiled(p, cfg.b_rows, &tm_w)))
        return nmhost::fail(NM_ERR_CUDA, "nm_conv2d: tensor-map encoding failed");
    if (cfg.tma_store && !nmtm::encode_y_tiled(p, &tm_y))
        return nmhost::fail(NM_ERR_CUDA, "nm_conv2d: output tensor-map encoding failed");
    size_t smem = static_cast<size_t>(cfg.stages) * cfg.stage_bytes + 1024;
    if (smem < 78 * 1024) smem = 78 * 1024;  // never more than two CTAs (2 x 256 TMEM columns) per SM
    cudaError_t e = nmhost::ensure_dynamic_smem(reinterpret_cast<const void*>(k_conv_slab<KC, TMA>), smem);
    if (e != cudaSuccess) return nmhost::fail(NM_ERR_CUDA, "cudaFuncSetAttribute (variant 2): %s", cudaGetErrorString(e));
    const long long tiles_m = (p.pixels + BM - 1) / BM;
    const long long blocks = tiles_m * cfg.n_slices;
    if (blocks > 0x7FFFFFFFll) return nmhost::fail(NM_ERR_UNSUPPORTED, "nm_conv2d: too many output tiles");
    k_conv_slab<KC, TMA><<<static_cast<unsigned>(blocks), 288, smem, st>>>(p, cfg, tm_x, tm_w, tm_y);
    nmhost::count_launch(1);
    e = cudaGetLastError();
    if (e != cudaSuccess) return nmhost::fail(NM_ERR_CUDA, "nm_conv2d launch (variant 2): %s", cudaGetErrorString(e));
    return NM_OK;
}

template <int KC>
nm_status_t launch_kc(const ConvParams& p, const SlabCfg& cfg, cudaStream_t st)
{
    return cfg.use_tma ? launch<KC, true>(p, cfg, st) : launch<KC, false>(p, cfg, st);
}

}  // namespace

namespace nmhost {

bool slab_plan_ok(const ConvParams& p, const nm_plan_t* plan)
{
    SlabCfg cfg;
    return make_cfg(p, plan, &cfg);
}

nm_status_t launch_conv_slab(const ConvParams& p, const nm_plan_t* plan, cudaStream_t st)
{
    SlabCfg cfg;
    if (!make_cfg(p, plan, &cfg)) return fail(NM_ERR_UNSUPPORTED, "nm_conv2d: the slab kernel does not take this layer / plan");
    switch (p.v2_kc) {
        case 8: return launch_kc<8>(p, cfg, st);
        case 16: return launch_kc<16>(p, cfg, st);
        case 24: return launch_kc<24>(p, cfg, st);
        case 32: return launch_kc<32>(p, cfg, st);
    }
    return fail(NM_ERR_UNSUPPORTED, "nm_conv2d: unsupported kept-columns-per-chunk %d", p.v2_kc);
}

}  // namespace nmhost
