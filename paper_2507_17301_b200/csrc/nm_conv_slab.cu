// Variant 2: slab kernel — warp-specialised sparse implicit GEMM with the gathered operand in
// tensor memory.
//
// One CTA owns 128 output pixels and up to NM_SLAB_MAX_TILES pruning tiles (<= 128 output
// channels); two CTAs fit on an SM, so one CTA's epilogue overlaps the other's main loop.
// The reduction axis is cut into chunks of G whole N:M groups (S = G*M source columns, of which
// every tile keeps KC = G*N).  Per chunk:
//   producers (4 warps)   cp.async the DENSE activation slab [128 pixels x S columns] once
//                         (zero-filled outside the image; row pitch S+1 words so that a column can
//                         be read by 32 pixels without bank conflicts) and the weight chunk
//                         [channels x KC] in the 128-byte-swizzled K-major layout;
//   compactors (4 warps)  thread = pixel; for each tile pick its KC kept columns out of the slab
//                         by index (warp-uniform offsets), round to TF32 and write them to a TMEM
//                         operand buffer with tcgen05.st  -> this is the fused im2col + packing
//                         of Sec. 3.2 restricted to the surviving columns, with TMEM in the role
//                         of the packed strip;
//   MMA issuer (1 thread) D[128 x T] += A[tmem] * W_chunk[smem]^T, KC/8 tcgen05.mma per tile:
//                         Algorithm 1's T accumulators are T TMEM columns.
// Epilogue (the compactor warps): TMEM -> registers, + bias, ReLU, NHWC store.
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, reports through the
// status word and drains to the common exit where TMEM is released.
#include "nm_internal.h"
#include "nm_ptx.cuh"

namespace {

using namespace nmk;

constexpr int BM = 128;
constexpr int MAX_BN_COLS = 128;   // accumulator columns per CTA
constexpr int NA = 4;              // TMEM operand buffers of 32 columns
constexpr int TMEM_COLS = 256;     // 128 accumulator + 4 x 32 operand columns
constexpr int NSTAGE_MAX = 4;

struct SlabCfg {
    int g_tiles;      // pruning tiles per CTA
    int umma_n;       // accumulator columns per tile (tile_t rounded up to 16)
    int n_slices;     // CTAs along the channel axis
    int stages;
    int slab_pitch;   // words per slab row (S + 1, odd)
    int slab_bytes, b_bytes, stage_bytes;
};

__device__ __forceinline__ bool aborted(volatile int* flag) { return *flag != 0; }

template <int KC>
__global__ void __launch_bounds__(288, 2) k_conv_slab(const ConvParams p, const SlabCfg cfg)
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

    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;  // stage: [B tile (1024-aligned)][slab]
    volatile int* abort_flag = &s_abort;

    // ---- set-up ----------------------------------------------------------------------------------
    if (warp == 8) tmem_alloc(smem_u32(&s_tmem), TMEM_COLS);
    if (tid == 0) {
        for (int i = 0; i < NSTAGE_MAX; ++i) {
            mbar_init(smem_u32(&s_full[i]), 128);       // producer threads
            mbar_init(smem_u32(&s_free[i]), 128 + 1);   // compactor threads + MMA commit
        }
        for (int i = 0; i < NA; ++i) {
            mbar_init(smem_u32(&s_aready[i]), 128);     // compactor threads
            mbar_init(smem_u32(&s_afree[i]), 1);        // MMA commit
        }
        mbar_init(smem_u32(&s_dready), 1);
        mbar_fence_init();
        s_abort = 0;
    }
    if (tid < BM) {
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
        // =========================== producers ===========================
        const int pw = warp - 4, ptid = tid - 128;
        const int segs = (S + 31) / 32;
        const int b_rows = cfg.g_tiles * cfg.umma_n;
        constexpr int QPR = KC / 4;  // 16-byte pieces per weight row
        const size_t wpitch = static_cast<size_t>(n_chunks) * 32;
        for (int c = 0; c < n_chunks; ++c) {
            const int s = c % NS;
            if (c >= NS) {
                if (!mbar_wait(smem_u32(&s_free[s]), ((c / NS) - 1) & 1)) { *abort_flag = 2; }
            }
            if (aborted(abort_flag)) break;
            const uint32_t b_smem = ring + s * cfg.stage_bytes;
            const uint32_t slab = b_smem + cfg.b_bytes;
            // activation slab: lane = source column, this warp's 32 pixels one after another
            for (int seg = 0; seg < segs; ++seg) {
                const int colc = seg * 32 + lane;            // column inside the chunk
                const int k = c * S + colc;                  // flattened (kh, kw, c) column
                const bool col_ok = colc < S && k < p.k;
                const int tap = col_ok ? k / p.c_in : 0;
                const int cc = col_ok ? k - tap * p.c_in : 0;
                const int delta = ((tap / p.kw) * p.dil_h * p.w + (tap % p.kw) * p.dil_w) * p.c_in + cc;
                const uint32_t dst0 = slab + static_cast<uint32_t>(colc) * 4u;
                if (colc < S) {
#pragma unroll 4
                    for (int i = 0; i < 32; ++i) {
                        const int row = pw * 32 + i;
                        const bool ok = col_ok && ((s_rowmask[row] >> tap) & 1ull);
                        const float* src = ok ? p.x + (s_rowoff[row] + delta) : p.x;
                        cp_async4(dst0 + static_cast<uint32_t>(row * cfg.slab_pitch) * 4u, src, ok ? 4u : 0u);
                    }
                }
            }
            // weight chunk: rows = the CTA's channels (tile-major, umma_n rows per tile)
            for (int piece = ptid; piece < b_rows * QPR; piece += 128) {
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
    } else if (warp < 4) {
        // =========================== compactors, then epilogue ===========================
        const int row = tid;  // TMEM lane = pixel row
        const uint32_t lane_addr = static_cast<uint32_t>(warp * 32) << 16;
        const size_t rpitch = static_cast<size_t>(n_chunks) * 32;
        int use = 0;  // running count of operand-buffer uses
        for (int c = 0; c < n_chunks && !aborted(abort_flag); ++c) {
            const int s = c % NS;
            const uint32_t slab_row = ring + s * cfg.stage_bytes + cfg.b_bytes + static_cast<uint32_t>(row * cfg.slab_pitch) * 4u;
            for (int t = 0; t < g_here; ++t, ++use) {
                // kept-column offsets of this (tile, chunk): warp-uniform, fetched before the waits
                uint32_t relw[KC / 4];
                const uint32_t* rp = reinterpret_cast<const uint32_t*>(p.rel2 + static_cast<size_t>(tile0 + t) * rpitch + c * 32);
#pragma unroll
                for (int q = 0; q < KC / 4; ++q) relw[q] = __ldg(rp + q);
                // (the vote keeps the warp together for the .sync.aligned TMEM stores that follow)
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
                    float f;
                    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(f) : "r"(slab_row + rel * 4u));
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
        if (!__any_sync(0xFFFFFFFFu, aborted(abort_flag))) {
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
                const uint64_t bdesc = umma_desc_k_sw128(b_smem + t * cfg.umma_n * 128, 1024);
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
    cfg->g_tiles = g;
    cfg->umma_n = umma_n;
    cfg->n_slices = (p.n_tiles + g - 1) / g;
    cfg->slab_pitch = p.v2_s + 1 + (p.v2_s % 2);  // odd number of words
    cfg->slab_bytes = ((BM * cfg->slab_pitch * 4 + 1023) / 1024) * 1024;
    cfg->b_bytes = g * umma_n * 128;                // multiple of 2048
    cfg->stage_bytes = cfg->slab_bytes + cfg->b_bytes;
    const int budget = 110 * 1024;                  // two CTAs per SM
    int stages = plan && plan->stages > 0 ? plan->stages : 3;
    if (stages > NSTAGE_MAX) return false;
    while (stages > 1 && stages * cfg->stage_bytes + 1024 > budget && !(plan && plan->stages > 0)) --stages;
    if (stages * cfg->stage_bytes + 1024 > 225 * 1024) return false;
    cfg->stages = stages;
    return true;
}

template <int KC>
nm_status_t launch(const ConvParams& p, const SlabCfg& cfg, cudaStream_t st)
{
    size_t smem = static_cast<size_t>(cfg.stages) * cfg.stage_bytes + 1024;
    if (smem < 78 * 1024) smem = 78 * 1024;  // never more than two CTAs (2 x 256 TMEM columns) per SM
    cudaError_t e = cudaFuncSetAttribute(k_conv_slab<KC>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return nmhost::fail(NM_ERR_CUDA, "cudaFuncSetAttribute (variant 2): %s", cudaGetErrorString(e));
    const long long tiles_m = (p.pixels + BM - 1) / BM;
    const long long blocks = tiles_m * cfg.n_slices;
    if (blocks > 0x7FFFFFFFll) return nmhost::fail(NM_ERR_UNSUPPORTED, "nm_conv2d: too many output tiles");
    k_conv_slab<KC><<<static_cast<unsigned>(blocks), 288, smem, st>>>(p, cfg);
    nmhost::count_launch(1);
    e = cudaGetLastError();
    if (e != cudaSuccess) return nmhost::fail(NM_ERR_CUDA, "nm_conv2d launch (variant 2): %s", cudaGetErrorString(e));
    return NM_OK;
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
        case 8: return launch<8>(p, cfg, st);
        case 16: return launch<16>(p, cfg, st);
        case 24: return launch<24>(p, cfg, st);
        case 32: return launch<32>(p, cfg, st);
    }
    return fail(NM_ERR_UNSUPPORTED, "nm_conv2d: unsupported kept-columns-per-chunk %d", p.v2_kc);
}

}  // namespace nmhost
