// Variant 8: select kernel — persistent, warp-specialised sparse implicit GEMM that contracts over
// the RETAINED columns only (Algorithm 1) and pays for the fused im2col + packing pass of Sec. 3.2
// with two bitwise selects per retained element and tile.
//
// One CTA per SM walks a static list of work items: 128 output pixels x BN output channels
// (BN = G pruning tiles of T channels), optionally one of several ranges of the reduction axis.
// The reduction axis is cut into chunks of whole N:M groups: S source columns (32 or 64) of one
// kernel tap, of which every tile keeps KC.  Roles, connected by mbarriers (every wait bounded):
//
//   activation producer   TMA brings the DENSE activations of a chunk into shared memory, one
//   (1 thread)            128-byte row per pixel and 32-channel block (128-byte swizzle), in one of
//                         two forms.  "im2col": one im2col-mode load per chunk and 32-channel block
//                         (stride, dilation, tap offset and zero padding done by the hardware).
//                         "patch" (stride 1, output size = input size): the pixels of a block and
//                         their halo are CONSECUTIVE rows of the [pixels][channels] view of the input,
//                         so one plain 2-D load per 32-channel block brings everything all kh*kw taps
//                         need; a tap is the same rows shifted by a constant, and a thread whose tap
//                         falls outside the image reads a row of zeros instead.  A 3x3 layer so moves
//                         a ninth of the im2col form's bytes through the TMA unit.
//   weight producer       one bulk copy per chunk brings the G tiles' retained weights [G*T x KC]
//   (1 thread)            (stored as the swizzled shared-memory image), another their select masks.
//   compactors (2 teams   thread = pixel row = TMEM lane, one warp per lane quadrant and team; the teams take
//   of 4 warps)           alternate chunks, so that the barrier round trips and load latencies of one chunk
//                         overlap the selects of the other.  A thread reads its row of the chunk ONCE with
//                         conflict-free 16-byte loads (half a chunk at a time) and, for every tile of the
//                         item, picks that tile's retained columns out of its registers: the j-th retained
//                         column of a group of M lies at one of the positions j .. j + (M - N), so it is a
//                         chain of M - N bitwise selects (lop3) under warp-uniform masks precomputed at
//                         pruning time.  The result goes to the tile's operand columns in tensor memory
//                         (tcgen05.st).
//   MMA issuers           D[128 x n] += A[tmem] * W[smem]^T, KC / 8 tcgen05.mma per chunk and unit, a unit
//   (up to 4 threads)     being n = BN / 4 accumulator columns of one tile (the T accumulators of Algorithm 1
//                         are T TMEM columns).  A lone thread issues an MMA every ~125 cycles whatever its
//                         size, a 128 x 64 x 8 MMA runs in 35: the units of an item are dealt to up to four
//                         issuer threads, each with accumulator columns of its own.
//   epilogue (8 warps)    TMEM -> registers, + bias, (+ shortcut), ReLU, staged through shared memory
//                         and written to NHWC with TMA stores; with two accumulator buffers it
//                         overlaps the next item's main loop.
//
// Activations are fed to the tensor core as they are (it reads the upper 19 bits: truncation to
// TF32); weights were rounded to nearest at pruning time.
#include "nm_internal.h"
#include "nm_ptx.cuh"
#include "nm_tmap.cuh"

namespace {

using namespace nmk;

constexpr int BM = 128;
constexpr int THREADS = 576;   // warps: 0 activation producer, 1 weight producer, 2 3 16 17 MMA issuers, 4-7 epilogue, 8-15 compactors
constexpr int THREADS_EPI8 = 704;   // ... and four more epilogue warps, 18-21 (the registers per thread then drop from 96 to 80)
constexpr int MAX_P = 4;       // activation ring slots
constexpr int MAX_W = 8;       // weight ring slots
constexpr int MAX_SETS = 4;    // operand sets in tensor memory
constexpr int MAX_ISS = 4;
constexpr int MAX_TAPS = 32;
constexpr int A_COL0 = 256;    // TMEM: accumulators in columns [0, 256), operand sets above
constexpr int STAGING_BYTES = 4 * 2 * 4096;   // two boxes per epilogue warp (twice that with eight epilogue warps)

struct SelCfg {
    int g, bn, n_slices, n_acc, n_iss;
    int mma_n, n_units; // accumulator columns per MMA and MMA units per work item (bn = n_units * mma_n)
    int patch;          // 1 = patch loads, 0 = im2col loads
    int taps;           // chunks per activation stage: kh * kw (patch) or 1 (im2col)
    int n_cb;           // chunks per tap = c_in / S
    int prow;           // rows of one 32-channel sub-tile of an activation stage
    int lo;             // patch: first patch row relative to the block's first pixel (<= 0)
    int seg_bytes;      // prow * 128
    int p_bytes;        // activation stage = SEGS sub-tiles
    int w_bytes;        // g * T * 128
    int m_bytes;        // g * mask words * 4
    int wstage_bytes;   // w_bytes + m_bytes rounded up to 1024
    int n_p, n_w, n_sets, kcp, set_cols;
    int ksplit, p_pad;
    int epi8;           // eight epilogue warps instead of four
    int alias_staging;  // 1: the output staging boxes lie over the start of the activation ring (one work item per CTA)
    int boxes;          // staging boxes (32 pixels x 32 channels) per epilogue warp: 2, or one per channel block when aliased
    int n_act;          // activation stages per work item
    long long n_work;
};

__device__ __forceinline__ bool aborted(volatile int* flag) { return *flag != 0; }

// Bounded wait that also gives up once another role has raised the abort flag (looked at every 64 polls, off
// the path of a wait that is already satisfied).
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int* flag)
{
    if (mbar_test_wait(bar, parity)) return true;
    for (uint32_t i = 0; i < kWaitPolls; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 63u) == 63u && *flag != 0) return false;
    }
    return false;
}

// Four consecutive 32-bit words of shared memory into dst[0..3].
__device__ __forceinline__ void lds128(uint32_t addr, uint32_t* dst)
{
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(dst[0]), "=r"(dst[1]), "=r"(dst[2]), "=r"(dst[3]) : "r"(addr));
}
// m ? a : b, bit by bit (m is all ones or all zeros)
__device__ __forceinline__ uint32_t bsel(uint32_t m, uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xCA;" : "=r"(d) : "r"(m), "r"(a), "r"(b));
    return d;
}

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

// NK kept columns in every group of MG source columns.
template <int NK, int MG>
struct Pattern {
    static constexpr int D = MG - NK;                        // selects per retained column
    static constexpr int S = (MG == 4 && NK == 3) ? 32 : 64; // source columns per chunk
    static constexpr int SEGS = S / 32;
    static constexpr int GROUPS = S / MG;
    static constexpr int KC = GROUPS * NK;                   // kept columns per chunk and tile
    static constexpr int GW = GROUPS / 2;                    // groups per compactor half
    static constexpr int KW = GW * NK;                       // kept columns per compactor half
    static constexpr int LW = S / 8;                         // 16-byte pieces of a row per compactor half
    static constexpr int MW = GROUPS * NK * D;               // select masks (32-bit words) per tile and chunk
    static constexpr int HW = MW / 2;                        // ... per half of the chunk (a multiple of 4 for every pattern)
    static constexpr int MWP = MW * 4;                       // bytes a tile's masks of one chunk occupy
};

struct Item {
    int split, slice;
    uint32_t pix0;
};
__device__ __forceinline__ Item item_of(uint32_t work, const SelCfg& cfg)
{
    Item it;
    it.split = static_cast<int>(work % static_cast<uint32_t>(cfg.ksplit));
    const uint32_t rest = work / static_cast<uint32_t>(cfg.ksplit);
    it.slice = static_cast<int>(rest % static_cast<uint32_t>(cfg.n_slices));
    it.pix0 = (rest / static_cast<uint32_t>(cfg.n_slices)) * BM;
    return it;
}

template <int NK, int MG, int EPI8>
__global__ void __launch_bounds__(EPI8 ? THREADS_EPI8 : THREADS, 1)
k_conv_select(const ConvParams p, const SelCfg cfg, const __grid_constant__ CUtensorMap tm_x,
              const __grid_constant__ CUtensorMap tm_y)
{
    using P = Pattern<NK, MG>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_pfull[MAX_P], s_pfree[MAX_P], s_wfull[MAX_W], s_wfree[MAX_W], s_aready[MAX_SETS], s_accfull[2],
        s_accfree[2];
    __shared__ __align__(1024) float s_zero[8 * 32];   // eight rows of zeros, one per swizzle phase (an out-of-image tap reads
                                                          // the row of its own phase: no bank conflict with its neighbours)
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t n_work = static_cast<uint32_t>(cfg.n_work);   // below 2^31: per-item arithmetic stays 32-bit
    const int T = p.tile_t, g = cfg.g;
    const uint32_t p_ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t w_ring = p_ring + cfg.n_p * cfg.p_bytes;
    const uint32_t ring_end = w_ring + cfg.n_w * cfg.wstage_bytes;
    // with one work item per CTA the epilogue starts when every load has been consumed: its staging boxes reuse the ring
    const uint32_t staging = cfg.alias_staging ? p_ring : ring_end;
    const int n_chunks_item = cfg.n_act * cfg.taps;
    volatile int* abort_flag = &s_abort;

    // ---- set-up ----------------------------------------------------------------------------------
    if (warp == 2) tmem_alloc(smem_u32(&s_tmem), 512);
    if (tid == 0) {
        for (int i = 0; i < MAX_P; ++i) {
            mbar_init(smem_u32(&s_pfull[i]), 1);              // producer's expect-tx arrival
            mbar_init(smem_u32(&s_pfree[i]), cfg.taps > 1 ? 8 : 4);   // compactor warps that read the stage
        }
        for (int i = 0; i < MAX_W; ++i) {
            mbar_init(smem_u32(&s_wfull[i]), 1);
            // one compactor team (it has read the masks) + one MMA commit per issuer (the weights and the operand set
            // have been read): the weight producer waits on it before refilling the slot, a compactor team before it
            // overwrites the operand set that chunk used
            mbar_init(smem_u32(&s_wfree[i]), 4 + cfg.n_iss);
        }
        for (int i = 0; i < MAX_SETS; ++i) {
            mbar_init(smem_u32(&s_aready[i]), 4);             // one compactor team: operand set written AND weights landed
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&s_accfull[i]), cfg.n_iss);
            mbar_init(smem_u32(&s_accfree[i]), EPI8 ? 8 : 4);  // epilogue warps
        }
        mbar_fence_init();
        s_abort = 0;
        tma_prefetch_desc(&tm_x);
        tma_prefetch_desc(&tm_y);
    }
    if (tid < 8 * 32) s_zero[tid] = 0.f;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    pdl_launch_dependents();   // the next kernel may start its own set-up as SMs become free
    pdl_wait();                // from here on global memory written by the previous kernel is read

    if (warp == 0) {
        // =========================== activation producer ===========================
        if (lane == 0) {
            const int hw = p.ho * p.wo;
            RingPos rp;
            int issued = 0;
            for (uint32_t work = blockIdx.x; work < n_work && !aborted(abort_flag); work += gridDim.x) {
                const Item it = item_of(work, cfg);
                const int n0 = static_cast<int>(it.pix0 / static_cast<uint32_t>(hw));
                const int rem = static_cast<int>(it.pix0 - static_cast<uint32_t>(n0) * static_cast<uint32_t>(hw));
                const int oh0 = rem / p.wo, ow0 = rem - oh0 * p.wo;
                const int w0 = ow0 * p.stride_w - p.pad_w, h0 = oh0 * p.stride_h - p.pad_h;
                // first activation stage of this item's range of the reduction axis
                int a = it.split * cfg.n_act;
                int tap = 0, cb = a;                       // im2col: stage a = chunk a = (tap, cb)
                if (!cfg.patch) { tap = a / cfg.n_cb; cb = a - tap * cfg.n_cb; }
                int ti = tap / p.kw, tj = tap - ti * p.kw;
                if (cfg.patch) {
                    // the item's activations, all channel blocks: out of HBM now, not one ring slot at a time
                    for (int s = cfg.n_p; s < cfg.n_act; ++s)
                        for (int seg = 0; seg < P::SEGS; ++seg)
                            l2_prefetch_tile_2d(&tm_x, ((a + s) * P::SEGS + seg) * 32, static_cast<int>(it.pix0) + cfg.lo);
                }
                for (int s = 0; s < cfg.n_act; ++s) {
                    if (rp.wrapped && !mbar_wait_lone(smem_u32(&s_pfree[rp.s]), rp.parity ^ 1u)) *abort_flag = 2;
                    if (aborted(abort_flag)) break;
                    const uint32_t dst = p_ring + rp.s * cfg.p_bytes;
                    const uint32_t bar = smem_u32(&s_pfull[rp.s]);
                    mbar_arrive_expect_tx(bar, static_cast<uint32_t>(P::SEGS) * cfg.seg_bytes);
#pragma unroll
                    for (int seg = 0; seg < P::SEGS; ++seg) {
                        const int ch = (cb * P::SEGS + seg) * 32;
                        if (cfg.patch)
                            tma_load_2d(dst + seg * cfg.seg_bytes, &tm_x, bar, ch, static_cast<int>(it.pix0) + cfg.lo);
                        else
                            tma_load_im2col_4d(dst + seg * cfg.seg_bytes, &tm_x, bar, ch, w0, h0, n0,
                                               static_cast<uint16_t>(tj * p.dil_w), static_cast<uint16_t>(ti * p.dil_h));
                    }
                    if (++cb == cfg.n_cb && !cfg.patch) {
                        cb = 0;
                        if (++tj == p.kw) { tj = 0; ++ti; }
                    }
                    rp.advance(cfg.n_p);
                    ++issued;
                }
            }
            if (aborted(abort_flag)) {
                // loads already issued still target this CTA's shared memory: let them land
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
            const size_t chunk_floats = static_cast<size_t>(p.c_out) * 32;
            const size_t chunk_mbytes = static_cast<size_t>(p.n_tiles) * P::MWP;
            const uint32_t tx = static_cast<uint32_t>(cfg.w_bytes + cfg.m_bytes);
            for (uint32_t work = blockIdx.x; work < n_work && !aborted(abort_flag); work += gridDim.x) {
                const Item it = item_of(work, cfg);
                const float* wsl = p.w3 + static_cast<size_t>(it.slice) * cfg.bn * 32;
                const uint8_t* msl = p.sel3 + static_cast<size_t>(it.slice) * g * P::MWP;
                const int a0 = it.split * cfg.n_act;
                for (int s = 0; s < cfg.n_act && !aborted(abort_flag); ++s) {
                    // patch: stage = channel block a0 + s, its chunks are (tap, block) for every tap; im2col: chunk a0 + s
                    int c = a0 + s;
                    for (int t = 0; t < cfg.taps; ++t, c += cfg.n_cb) {
                        if (rw.wrapped && !mbar_wait_lone(smem_u32(&s_wfree[rw.s]), rw.parity ^ 1u)) *abort_flag = 9;
                        if (aborted(abort_flag)) break;
                        const uint32_t dst = w_ring + rw.s * cfg.wstage_bytes;
                        const uint32_t bar = smem_u32(&s_wfull[rw.s]);
                        mbar_arrive_expect_tx(bar, tx);
                        bulk_load_1d(dst, wsl + static_cast<size_t>(c) * chunk_floats, static_cast<uint32_t>(cfg.w_bytes), bar);
                        if (P::MW > 0)
                            bulk_load_1d(dst + cfg.w_bytes, msl + static_cast<size_t>(c) * chunk_mbytes,
                                         static_cast<uint32_t>(cfg.m_bytes), bar);
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
    } else if (warp == 2 || warp == 3 || warp == 16 || warp == 17) {
        // =========================== MMA issuers ===========================
        const int iss = warp < 4 ? warp - 2 : warp - 14;
        if (lane == 0 && iss < cfg.n_iss) {
            const uint32_t idesc = umma_idesc_tf32(BM, cfg.mma_n);
            const int units_per_tile = T / cfg.mma_n;
            RingPos rw;
            uint32_t set = 0, set_par = 0;
            uint32_t ab = 0, acc_par = 0;
            bool acc_wrapped = false;
            // A chunk is ready when its compactor team has arrived: the team waits for the chunk's weights (they
            // come with its masks) before it starts, so this one barrier stands for both.  One commit per chunk
            // releases the weight slot and, through the same barrier, the operand set.
            for (uint32_t work = blockIdx.x; work < n_work && !aborted(abort_flag); work += gridDim.x) {
                if (acc_wrapped && !wait_or_abort(smem_u32(&s_accfree[ab]), acc_par ^ 1u, abort_flag)) {
                    *abort_flag = 5;
                    break;
                }
                tc_fence_after();
                const uint32_t acc = tmem + ab * cfg.bn;
                for (int c = 0; c < n_chunks_item; ++c) {
                    if (!wait_or_abort(smem_u32(&s_aready[set]), set_par, abort_flag)) { *abort_flag = 7; break; }
                    tc_fence_after();
                    const uint32_t b_smem = w_ring + rw.s * cfg.wstage_bytes;
                    const uint32_t a_set = tmem + A_COL0 + set * cfg.set_cols;
                    for (int u = iss; u < cfg.n_units; u += cfg.n_iss) {
                        const uint64_t bdesc = umma_desc_k_sw128(b_smem + u * cfg.mma_n * 128, 1024);
                        const uint32_t a_tile = a_set + (u / units_per_tile) * cfg.kcp;
#pragma unroll
                        for (int kq = 0; kq < P::KC / 8; ++kq)
                            NM_CHECKED(((acc - tmem) & 0xFFFFu) + (u + 1) * cfg.mma_n <= 256u && ((a_tile - tmem) & 0xFFFFu) + kq * 8 + 8 <= 512u &&
                                           b_smem + (u + 1) * cfg.mma_n * 128 <= ring_end && b_smem >= w_ring,
                                       p.status, 801, u * 1000 + kq)
                            umma_tf32_ts(acc + u * cfg.mma_n, a_tile + kq * 8, bdesc + 2 * kq, idesc, (c > 0 || kq > 0) ? 1u : 0u);
                    }
                    umma_commit(smem_u32(&s_wfree[rw.s]));
                    rw.advance(cfg.n_w);
                    if (++set == static_cast<uint32_t>(cfg.n_sets)) { set = 0; set_par ^= 1u; }
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
    } else if ((warp >= 4 && warp < 8) || (EPI8 && warp >= 18)) {
        // =========================== epilogue ===========================
        // With eight epilogue warps two warps per 32 accumulator lanes take alternate 32-channel blocks: a block costs
        // a warp about a thousand cycles of latencies in series (TMEM load, staging, proxy fence, store), so the warps,
        // not their instructions, set the pace of an item's epilogue.  It pays where an item has few chunks (pointwise
        // layers with many output channels); elsewhere the compactors need the registers the extra warps take.
        const int q = warp & 3;
        constexpr int ESTEP = EPI8 ? 2 : 1;
        const int half = warp >= 18 ? 1 : 0;
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t my_staging = staging + (half * 4 + q) * cfg.boxes * 4096;
        const uint32_t rx = static_cast<uint32_t>(lane & 7);
        const int n_blk = cfg.bn / 32;
        uint32_t ti = 0;
        uint32_t nb = 0;  // staging boxes this warp has filled so far
        for (uint32_t work = blockIdx.x; work < n_work; work += gridDim.x, ++ti) {
            const Item it = item_of(work, cfg);
            const int ab = cfg.n_acc == 2 ? static_cast<int>(ti & 1u) : 0;
            const bool ok = aborted(abort_flag) ||
                            mbar_wait(smem_u32(&s_accfull[ab]), (cfg.n_acc == 2 ? (ti >> 1) : ti) & 1u);
            if (!__all_sync(0xFFFFFFFFu, ok)) *abort_flag = 8;
            if (__any_sync(0xFFFFFFFFu, aborted(abort_flag))) break;
            tc_fence_after();
            const int o0 = it.slice * cfg.bn;
            // a split of the reduction axis stores raw partial sums [split][pixel][channel] (bias, shortcut and
            // activation are switched off by the launcher and applied by the reduction pass)
            const long long box_pix = static_cast<long long>(it.pix0) + q * 32;
            const int store_row = it.split * cfg.p_pad + static_cast<int>(it.pix0) + q * 32;
            const bool in_range = cfg.ksplit > 1 || box_pix < p.pixels;
            if (EPI8 && half >= n_blk) {   // a single channel block: the second warp of the quarter only releases the buffer
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&s_accfree[ab]));
            }
            for (int blk = half; blk < n_blk; blk += ESTEP, ++nb) {
                const float bias_l = bias_lane_load(p.bias, o0 + blk * 32, p.c_out, lane);
                uint32_t v[32];
                tmem_ld32(tmem + lane_addr + ab * cfg.bn + blk * 32, v);
                tmem_ld_wait();
                if (blk + ESTEP >= n_blk) {
                    // the accumulator buffer may be overwritten from here on
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&s_accfree[ab]));
                }
                // two boxes: the box's previous store (two blocks ago) has read it; a box per block: nothing to wait for
                const uint32_t box = my_staging + (cfg.boxes == 2 ? (nb & 1u) : static_cast<uint32_t>(blk / ESTEP)) * 4096;
                if (cfg.boxes == 2 && lane == 0 && nb >= 2) tma_store_wait_read_n<1>();
                __syncwarp();
                const uint32_t stage_row = box + lane * 128;
                const bool res_pass = p.residual != nullptr && box_pix < p.pixels;
                const int relu_now = res_pass ? 0 : p.relu;   // with a shortcut input the activation waits for the second pass
#pragma unroll
                for (int qq = 0; qq < 8; ++qq) {
                    const float4 bv = bias_quad(bias_l, qq);
                    float o[4];
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
                    if (in_range) tma_store_2d(&tm_y, box, o0 + blk * 32, store_row);
                    tma_store_commit();
                }
            }
        }
        if (lane == 0) tma_store_wait_read();   // shared memory must outlive the stores' reads; the writes complete with the grid
    } else if (warp >= 8 && warp < 16) {
        // =========================== compactors ===========================
        const uint32_t team = static_cast<uint32_t>(warp - 8) >> 2;   // chunks cg = team (mod 2) are this warp's
        const int q = warp & 3;                                       // TMEM lane quadrant
        const int row = q * 32 + lane;
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t zero_row = smem_u32(s_zero);
        const int hw = p.ho * p.wo;
        RingPos rp, rw, rold;              // rold: weight slot of the chunk n_sets chunks back
        uint32_t set = 0, set_par = 0;
        uint32_t cg = 0;                   // chunks of this CTA so far (all items)
        bool pre_w = false, pre_a = false; // barriers of this team's next chunk found complete ahead of time
        for (uint32_t work = blockIdx.x; work < n_work && !aborted(abort_flag); work += gridDim.x) {
            const Item it = item_of(work, cfg);
            uint32_t vbits = 0xFFFFFFFFu;   // taps of this thread's pixel that lie inside the image
            if (cfg.patch) {
                vbits = 0;
                const long long pix = static_cast<long long>(it.pix0) + row;
                if (pix < p.pixels) {
                    const uint32_t pu = static_cast<uint32_t>(pix);
                    const int rem = static_cast<int>(pu % static_cast<uint32_t>(hw));
                    const int oh = rem / p.wo, ow = rem - oh * p.wo;
                    int t = 0;
                    for (int i = 0; i < p.kh; ++i) {
                        const int ih = oh + i * p.dil_h - p.pad_h;
                        for (int j = 0; j < p.kw; ++j, ++t) {
                            const int iw = ow + j * p.dil_w - p.pad_w;
                            if (ih >= 0 && ih < p.h && iw >= 0 && iw < p.w) vbits |= 1u << t;
                        }
                    }
                }
            }
            bool failed = false;
            for (int s = 0; s < cfg.n_act && !failed; ++s) {
                const uint32_t act = p_ring + rp.s * cfg.p_bytes;
                const uint32_t pfull = smem_u32(&s_pfull[rp.s]), pfree = smem_u32(&s_pfree[rp.s]);
                const uint32_t ppar = rp.parity;
                rp.advance(cfg.n_p);
                bool stage_seen = false;
                // patch form: rows between the first patch row and this pixel's source row of tap (ti, tj)
                int shift_row = cfg.patch ? -p.pad_h * p.w - p.pad_w - cfg.lo : 0, shift = shift_row;
                int tj = 0;
                for (int t = 0; t < cfg.taps; ++t, ++cg) {
                    const uint32_t my_shift = static_cast<uint32_t>(shift);
                    shift += p.dil_w;
                    if (++tj == p.kw) { tj = 0; shift_row += p.dil_h * p.w; shift = shift_row; }
                    const uint32_t wst = w_ring + rw.s * cfg.wstage_bytes;
                    const uint32_t wfull = smem_u32(&s_wfull[rw.s]), wfree = smem_u32(&s_wfree[rw.s]), wpar = rw.parity;
                    const uint32_t aready = smem_u32(&s_aready[set]);
                    const uint32_t a_set = tmem + lane_addr + A_COL0 + set * cfg.set_cols;
                    // the operand set was last used by chunk cg - n_sets: its MMAs are done when its weight slot is free
                    const bool set_reused = cg >= static_cast<uint32_t>(cfg.n_sets);
                    const uint32_t afree = smem_u32(&s_wfree[rold.s]), apar = rold.parity;
                    if (set_reused) rold.advance(cfg.n_w);
                    rw.advance(cfg.n_w);
                    if (++set == static_cast<uint32_t>(cfg.n_sets)) { set = 0; set_par ^= 1u; }
                    if ((cg & 1u) != team) continue;
                    bool ok = stage_seen || wait_or_abort(pfull, ppar, abort_flag);
                    stage_seen = true;
                    ok = ok && (pre_w || wait_or_abort(wfull, wpar, abort_flag));
                    ok = ok && (!set_reused || pre_a || wait_or_abort(afree, apar, abort_flag));
                    if (!__all_sync(0xFFFFFFFFu, ok)) { *abort_flag = 3; failed = true; break; }
                    tc_fence_after();
                    // address of this thread's row with the swizzle phase folded in: piece i lies at a0 ^ (i << 4)
                    const uint32_t pr = static_cast<uint32_t>(row) + (cfg.patch ? my_shift : 0u);
                    const bool live_row = !cfg.patch || ((vbits >> t) & 1u);
                    const uint32_t a0 = (live_row ? act + pr * 128u : zero_row + (pr & 7u) * 128u) + ((pr & 7u) << 4);
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        // S = 64: half h is 32-channel sub-tile h; S = 32: half h is the 16-byte pieces 4 h .. 4 h + 3 of the
                        // one sub-tile (a piece index enters the address XOR-ed with the row's swizzle phase)
                        const uint32_t ah = P::SEGS == 1 ? a0 ^ (static_cast<uint32_t>(half) << 6)
                                            : live_row   ? a0 + static_cast<uint32_t>(half) * cfg.seg_bytes
                                                         : a0;
                        uint32_t x[P::LW * 4];   // this half's S / 2 source columns of the row
#pragma unroll
                        for (int i = 0; i < P::LW; ++i) {
                            x[4 * i] = x[4 * i + 1] = x[4 * i + 2] = x[4 * i + 3] = 0u;
                            NM_CHECKED((ah >= p_ring && ah + 128u <= w_ring + 128u && (ah & 15u) == 0u) || (ah & ~1023u) == zero_row, p.status, 802, ah)
                            lds128(ah ^ (static_cast<uint32_t>(i) << 4), x + 4 * i);
                        }
                        if (half == 1) {
                            // the barriers of this team's next chunk, looked up while the loads are in flight
                            RingPos nw = rw, no = rold;
                            nw.advance(cfg.n_w);
                            if (cg + 1 >= static_cast<uint32_t>(cfg.n_sets)) no.advance(cfg.n_w);
                            pre_w = mbar_test_wait(smem_u32(&s_wfull[nw.s]), nw.parity);
                            pre_a = mbar_test_wait(smem_u32(&s_wfree[no.s]), no.parity);
                        }
                        const uint32_t mbase = wst + cfg.w_bytes + half * (P::HW * 4);
                        for (int tile = 0; tile < g; ++tile) {
                            // this half's select masks of the tile: full-width words (a byte per mask widened by a byte
                            // permute moves less through shared memory but doubles the work of the ALU pipe, which
                            // executes logic operations at half rate and is the busier of the two with several tiles)
                            uint32_t M[P::HW];
#pragma unroll
                            for (int i = 0; i < P::HW / 4; ++i) {
                                M[4 * i] = M[4 * i + 1] = M[4 * i + 2] = M[4 * i + 3] = 0u;
                                NM_CHECKED(mbase + tile * P::MWP + i * 16 + 16 <= ring_end && mbase >= w_ring && (mbase & 15u) == 0u, p.status, 803, mbase)
                                lds128(mbase + tile * P::MWP + i * 16, M + 4 * i);
                            }
                            uint32_t v[P::KW];
#pragma unroll
                            for (int gi = 0; gi < P::GW; ++gi) {
#pragma unroll
                                for (int j = 0; j < NK; ++j) {
                                    uint32_t r = x[gi * MG + j + P::D];
#pragma unroll
                                    for (int i = P::D - 1; i >= 0; --i) r = bsel(M[(gi * NK + j) * P::D + i], x[gi * MG + j + i], r);
                                    v[gi * NK + j] = r;
                                }
                            }
                            NM_CHECKED(((a_set - tmem) & 0xFFFFu) + tile * cfg.kcp + half * P::KW + P::KW <= 512u &&
                                           ((a_set - tmem) & 0xFFFFu) >= static_cast<uint32_t>(A_COL0) && ((a_set - tmem) >> 16) == static_cast<uint32_t>(q * 32),
                                       p.status, 804, a_set - tmem)
                            tmem_st_n<P::KW>(a_set + tile * cfg.kcp + half * P::KW, v);
                        }
                    }
                    tmem_st_wait();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(aready);
                        mbar_arrive(wfree);
                        if (t + 2 >= cfg.taps) mbar_arrive(pfree);   // this team's last chunk of the stage
                    }
                }
            }
            if (failed) break;
        }
    }

    // ---- common exit ---------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (tid == 0 && s_abort != 0) {
        atomicExch(p.status + 0, static_cast<int>(NM_ERR_TIMEOUT));
        atomicExch(p.status + 1, 80 + s_abort);
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
    if (p.m_group == 4 && p.n_keep >= 1 && p.n_keep <= 3) return p.n_keep * 16 + 4;
    if (p.m_group == 8 && (p.n_keep == 1 || p.n_keep == 2 || p.n_keep == 4)) return p.n_keep * 16 + 8;
    return 0;
}

template <int NK, int MG>
void pattern_dims(int* s, int* kc, int* mw)
{
    *s = Pattern<NK, MG>::S;
    *kc = Pattern<NK, MG>::KC;
    *mw = Pattern<NK, MG>::MWP;
}

bool dims_of(int code, int* s, int* kc, int* mw)
{
    switch (code) {
        case 1 * 16 + 4: pattern_dims<1, 4>(s, kc, mw); return true;
        case 2 * 16 + 4: pattern_dims<2, 4>(s, kc, mw); return true;
        case 3 * 16 + 4: pattern_dims<3, 4>(s, kc, mw); return true;
        case 1 * 16 + 8: pattern_dims<1, 8>(s, kc, mw); return true;
        case 2 * 16 + 8: pattern_dims<2, 8>(s, kc, mw); return true;
        case 4 * 16 + 8: pattern_dims<4, 8>(s, kc, mw); return true;
    }
    return false;
}

bool make_cfg(const ConvParams& p, const nm_plan_t* plan, SelCfg* cfg)
{
    if (!p.w3 || !p.sel3 || !nmtm::available()) return false;
    int S = 0, KC = 0, MW = 0;
    if (!dims_of(pattern_code(p), &S, &KC, &MW)) return false;
    if (p.sel_s != S || p.sel_kc != KC || p.sel_mw != MW) return false;   // the handle's layout is this kernel's
    const int T = p.tile_t;
    if (p.c_in % S != 0 || T % 16 != 0 || T > 256 || p.c_out % T != 0) return false;
    if (static_cast<long long>(p.batch) * p.h * p.w * p.c_in * 4 < 131072) return false;   // tensor maps of tiny inputs: other kernels
    if (p.pixels >= (1ll << 31) - BM) return false;
    const int taps = p.kh * p.kw;
    // activation loads: the patch form needs stride 1, an output of the input's size, and a halo that fits a TMA box
    const int lo = -(p.pad_h * p.w + p.pad_w);
    const int hi = ((p.kh - 1) * p.dil_h - p.pad_h) * p.w + (p.kw - 1) * p.dil_w - p.pad_w;
    const bool patch_ok = p.stride_h == 1 && p.stride_w == 1 && p.ho == p.h && p.wo == p.w && taps <= MAX_TAPS && hi >= 0 &&
                          BM + hi - lo <= 256 && static_cast<long long>(p.batch) * p.h * p.w < (1ll << 31);
    int loads = plan ? plan->loads : 0;
    if (loads == 0) loads = (patch_ok && taps > 1) ? 2 : 1;
    if (loads == 2 && !patch_ok) return false;
    if (loads == 1 && !nmtm::im2col_geometry_ok(p)) return false;
    if (loads != 1 && loads != 2) return false;
    cfg->patch = loads == 2;
    cfg->taps = cfg->patch ? taps : 1;
    cfg->n_cb = p.c_in / S;
    cfg->lo = cfg->patch ? lo : 0;
    cfg->prow = cfg->patch ? ((BM + hi - lo + 7) / 8) * 8 : BM;
    cfg->seg_bytes = cfg->prow * 128;
    cfg->p_bytes = (S / 32) * cfg->seg_bytes;
    int g;
    if (plan && plan->bn > 0) {
        if (plan->bn % T != 0) return false;
        g = plan->bn / T;
    } else {
        g = 1;
        for (int cand = 4; cand >= 1; --cand)
            if (cand * T <= 256 && p.n_tiles % cand == 0 && (cand * T) % 32 == 0) { g = cand; break; }
    }
    if (g < 1 || g > 4 || g * T > 256 || p.n_tiles % g != 0 || (g * T) % 32 != 0) return false;
    cfg->g = g;
    cfg->bn = g * T;
    cfg->n_slices = p.n_tiles / g;
    cfg->n_acc = cfg->bn <= 128 ? 2 : 1;
    // MMA units: the item's accumulator columns cut into up to four pieces, none across two tiles
    // (as many units as issuer threads asked for: a plan with fewer issuers gets wider MMAs)
    const int want = plan && plan->issuers > 0 ? plan->issuers : MAX_ISS;
    if (want > MAX_ISS) return false;
    int sub = 1;
    while (g * sub < want && sub < 4) sub *= 2;
    while (sub > 1 && (T % sub != 0 || (T / sub) % 16 != 0)) sub /= 2;
    cfg->mma_n = T / sub;
    cfg->n_units = g * sub;
    int n_iss = want < cfg->n_units ? want : cfg->n_units;
    if (plan && plan->issuers > cfg->n_units) return false;
    cfg->n_iss = n_iss;
    cfg->kcp = KC <= 8 ? 8 : KC <= 16 ? 16 : 32;
    cfg->set_cols = g * cfg->kcp;
    cfg->n_sets = 256 / cfg->set_cols >= MAX_SETS ? MAX_SETS : 2;   // 2 or 4: the two compactor teams alternate sets
    cfg->w_bytes = cfg->bn * 128;
    cfg->m_bytes = g * MW;
    cfg->wstage_bytes = ((cfg->w_bytes + cfg->m_bytes + 1023) / 1024) * 1024;
    // split of the reduction axis: whole activation stages per range
    const int ksplit = plan && plan->ksplit > 1 ? plan->ksplit : 1;
    const int n_act_total = cfg->patch ? cfg->n_cb : cfg->n_cb * taps;
    if (ksplit > 8 || n_act_total % ksplit != 0) return false;
    cfg->ksplit = ksplit;
    cfg->n_act = n_act_total / ksplit;
    cfg->p_pad = static_cast<int>(((p.pixels + BM - 1) / BM) * BM);
    if (ksplit > 1 && (!p.splitk || p.c_out % 4 != 0 ||
                       p.splitk_bytes < static_cast<size_t>(ksplit) * cfg->p_pad * p.c_out * sizeof(float) ||
                       static_cast<long long>(ksplit) * cfg->p_pad >= (1ll << 31)))
        return false;   // the partial-sum scratch is reserved by nm_autotune / nm_weights_reserve
    // Shared memory: the activation ring, the rest to the weight ring.  The two compactor teams take alternate
    // chunks and wait on a barrier by phase parity, so a team must meet EVERY use of a ring slot it waits on, or a
    // wait for use k + 2 would pass on the completion of use k: the weight ring has an even number of slots (a slot
    // always holds chunks of one parity, i.e. of one team), and so has the activation ring when a stage is one chunk
    // (with several chunks per stage both teams read every stage).
    const long long pix_blocks = (p.pixels + BM - 1) / BM;
    cfg->n_work = pix_blocks * cfg->n_slices * ksplit;
    if (cfg->n_work >= (1ll << 31)) return false;
    cfg->alias_staging = cfg->n_work <= sm_count();
    // epilogue warps: plan.split = 1 four, 2 eight, 0 eight where an item has few chunks and several channel blocks
    if (plan && (plan->split < 0 || plan->split > 2)) return false;
    cfg->epi8 = plan && plan->split > 0 ? plan->split == 2 : (cfg->n_act * cfg->taps <= 4 && cfg->bn >= 64);
    const int staging_bytes = cfg->epi8 ? 2 * STAGING_BYTES : STAGING_BYTES;
    // alignment slack, static shared, and the output staging unless it can lie over the ring
    const int budget = 227 * 1024 - 1024 - 4096 - (cfg->alias_staging ? 0 : staging_bytes);   // static: barriers, 1 KB of zero rows and their alignment
    const bool paired = cfg->taps == 1;
    int n_p = 2;
    if (plan && plan->stages > 0) n_p = plan->stages;
    if (n_p < 1 || n_p > MAX_P || (paired && n_p % 2 != 0)) return false;
    if (!(plan && plan->stages > 0)) {
        if (paired && 4 * cfg->p_bytes + 4 * cfg->wstage_bytes <= budget) n_p = 4;
        while (n_p > (paired ? 2 : 1) && n_p * cfg->p_bytes + 2 * cfg->wstage_bytes > budget) n_p -= paired ? 2 : 1;
    }
    int n_w = (budget - n_p * cfg->p_bytes) / cfg->wstage_bytes;
    if (n_w > MAX_W) n_w = MAX_W;
    n_w &= ~1;
    if (n_w < 2) return false;
    cfg->n_p = n_p;
    cfg->n_w = n_w;
    // a set is released through the weight slot of the chunk that used it: the slot must not come round again sooner
    if (cfg->n_sets > n_w) cfg->n_sets = n_w >= 4 ? 4 : 2;
    cfg->boxes = 2;
    if (cfg->alias_staging) {
        // one work item per CTA: the rings are idle when the epilogue runs, every channel block gets a box of its own
        const int ring_bytes = n_p * cfg->p_bytes + n_w * cfg->wstage_bytes;
        const int warps = cfg->epi8 ? 8 : 4, per_warp = (cfg->bn / 32 + (cfg->epi8 ? 1 : 0)) / (cfg->epi8 ? 2 : 1);
        if (per_warp >= 2 && ring_bytes >= warps * per_warp * 4096) cfg->boxes = per_warp;   // a box per block the warp handles
        else if (ring_bytes < staging_bytes) cfg->alias_staging = 0;
    }
    return true;
}

// The input as a plain 2-D tensor [batch * h * w pixels][c_in] with a box of 32 channels x `rows` pixels.
bool encode_x_rows(const ConvParams& p, int rows, CUtensorMap* tm)
{
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(p.c_in), static_cast<cuuint64_t>(p.batch) * p.h * p.w};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(p.c_in) * 4};
    const cuuint32_t box[2] = {32, static_cast<cuuint32_t>(rows)};
    const cuuint32_t es[2] = {1, 1};
    return nmtm::encoders().tiled(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(p.x), dims, strides, box, es,
                                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int NK, int MG>
nm_status_t launch(const ConvParams& p, const SelCfg& cfg, cudaStream_t st)
{
    ConvParams q = p;
    if (cfg.ksplit > 1) {
        q.y = p.splitk;
        q.pixels = static_cast<long long>(cfg.ksplit) * cfg.p_pad;   // rows of the store map
        q.bias = nullptr;
        q.residual = nullptr;
        q.relu = 0;
    }
    alignas(64) CUtensorMap tm_x, tm_y;
    const bool ok_x = cfg.patch ? encode_x_rows(p, cfg.prow, &tm_x) : nmtm::encode_x_im2col(p, BM, &tm_x);
    if (!ok_x || !nmtm::encode_y_tiled(q, &tm_y))
        return nmhost::fail(NM_ERR_CUDA, "nm_conv2d: tensor-map encoding failed (variant 8)");
    q.pixels = p.pixels;
    size_t smem = 1024 + static_cast<size_t>(cfg.n_p) * cfg.p_bytes + static_cast<size_t>(cfg.n_w) * cfg.wstage_bytes +
                  (cfg.alias_staging ? 0 : (cfg.epi8 ? 2 : 1) * STAGING_BYTES);
    if (smem < 120 * 1024) smem = 120 * 1024;   // one CTA per SM: it owns all 512 TMEM columns
    const auto kernel = cfg.epi8 ? k_conv_select<NK, MG, 1> : k_conv_select<NK, MG, 0>;
    cudaError_t e = nmhost::ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), smem);
    if (e != cudaSuccess) return nmhost::fail(NM_ERR_CUDA, "cudaFuncSetAttribute (variant 8): %s", cudaGetErrorString(e));
    const long long grid = cfg.n_work < sm_count() ? cfg.n_work : sm_count();
    e = nmhost::launch_pdl(kernel, static_cast<unsigned>(grid), cfg.epi8 ? THREADS_EPI8 : THREADS, smem, st, q, cfg, tm_x, tm_y);
    nmhost::count_launch(1);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return nmhost::fail(NM_ERR_CUDA, "nm_conv2d launch (variant 8): %s", cudaGetErrorString(e));
    if (cfg.ksplit > 1) return nmhost::launch_splitk_reduce(p, cfg.ksplit, cfg.p_pad, st);
    return NM_OK;
}

// ---- the handle's copy of the compressed form for this kernel -------------------------------------------
// Retained weights per chunk as the shared-memory image the tensor core reads: w3[chunk][o][32] TF32, of a row's
// 32 slots the first KC used, the row's 16-byte pieces XOR-ed with (o % 8) (128-byte swizzle), so that the
// rows of any run of tiles are one contiguous bulk copy.
__global__ void k_build_w3(const float* __restrict__ values, const uint16_t* __restrict__ indices, int c_out, int kk,
                           int tile_t, int s_cols, int kc, float* __restrict__ w3)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int o = blockIdx.y;
    if (j >= kk) return;
    const int col = indices[static_cast<size_t>(o / tile_t) * kk + j];
    const int chunk = col / s_cols;
    const int jj = j - chunk * kc;   // every group is full: a chunk holds exactly kc retained columns
    w3[(static_cast<size_t>(chunk) * c_out + o) * 32 + ((((jj >> 2) ^ (o & 7)) << 2) | (jj & 3))] =
        nmk::to_tf32(values[static_cast<size_t>(o) * kk + j]);
}

// Select masks: for retained column j (the jn-th of its group, at position pos in the group) the D = M - N words
// m[i] = all ones iff pos == jn + i, i < D (all zero: the column is the last candidate, jn + D); `mw` bytes per tile and chunk.
__global__ void k_build_sel3(const uint16_t* __restrict__ indices, int n_tiles, int kk, int n_keep, int m_group,
                             int s_cols, int kc, int mw, uint8_t* __restrict__ sel3)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int r = blockIdx.y;
    if (j >= kk) return;
    const int d = m_group - n_keep;
    const int col = indices[static_cast<size_t>(r) * kk + j];
    const int chunk = col / s_cols;
    const int jj = j - chunk * kc;           // slot within the chunk = group-in-chunk * N + jn
    const int jn = jj % n_keep;
    const int pos = col % m_group;
    uint32_t* m = reinterpret_cast<uint32_t*>(sel3 + (static_cast<size_t>(chunk) * n_tiles + r) * mw) + static_cast<size_t>(jj) * d;
    for (int i = 0; i < d; ++i) m[i] = (pos == jn + i) ? 0xFFFFFFFFu : 0u;
}

}  // namespace

namespace nmhost {

nm_status_t build_select_layout(nm_weights* h, cudaStream_t st)
{
    h->w3 = nullptr;
    h->sel3 = nullptr;
    h->sel_s = h->sel_kc = h->sel_mw = 0;
    ConvParams probe = {};
    probe.n_keep = h->n_keep;
    probe.m_group = h->m_group;
    int S = 0, KC = 0, MW = 0;
    if (!dims_of(pattern_code(probe), &S, &KC, &MW)) return NM_OK;
    if (h->kk == 0 || h->k % h->m_group != 0 || h->c_in % S != 0 || h->tile_t % 16 != 0 || h->c_out % h->tile_t != 0)
        return NM_OK;
    const int chunks = h->k / S;
    const size_t wbytes = static_cast<size_t>(chunks) * h->c_out * 32 * sizeof(float);
    const size_t mbytes = static_cast<size_t>(chunks) * h->n_tiles * MW;
    if (cudaMalloc(&h->w3, wbytes) != cudaSuccess || cudaMalloc(&h->sel3, mbytes) != cudaSuccess) {
        (void)cudaGetLastError();
        cudaFree(h->w3);
        h->w3 = nullptr;
        h->sel3 = nullptr;
        return fail(NM_ERR_ALLOC, "cannot allocate the select-kernel weights");
    }
    cudaError_t e = cudaMemsetAsync(h->w3, 0, wbytes, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->sel3, 0, mbytes, st);   // the padding bytes of a tile's masks
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "select layout memset: %s", cudaGetErrorString(e));
    const dim3 gw((h->kk + 127) / 128, h->c_out), gm((h->kk + 127) / 128, h->n_tiles);
    k_build_w3<<<gw, 128, 0, st>>>(h->values, h->indices, h->c_out, h->kk, h->tile_t, S, KC, h->w3);
    k_build_sel3<<<gm, 128, 0, st>>>(h->indices, h->n_tiles, h->kk, h->n_keep, h->m_group, S, KC, MW, h->sel3);
    count_launch(2);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "select layout kernels: %s", cudaGetErrorString(e));
    h->sel_s = S;
    h->sel_kc = KC;
    h->sel_mw = MW;
    return NM_OK;
}

bool select_plan_ok(const ConvParams& p, const nm_plan_t* plan)
{
    SelCfg cfg;
    return make_cfg(p, plan, &cfg);
}

size_t select_splitk_bytes(const ConvParams& p, int splits)
{
    const size_t p_pad = static_cast<size_t>((p.pixels + BM - 1) / BM) * BM;
    return static_cast<size_t>(splits) * p_pad * p.c_out * sizeof(float);
}

nm_status_t launch_conv_select(const ConvParams& p, const nm_plan_t* plan, cudaStream_t st)
{
    SelCfg cfg;
    if (!make_cfg(p, plan, &cfg))
        return fail(NM_ERR_UNSUPPORTED, "nm_conv2d: the select kernel does not take this layer / plan%s",
                    plan && plan->ksplit > 1 ? " (a split plan needs scratch: nm_weights_reserve)" : "");
    switch (pattern_code(p)) {
        case 1 * 16 + 4: return launch<1, 4>(p, cfg, st);
        case 2 * 16 + 4: return launch<2, 4>(p, cfg, st);
        case 3 * 16 + 4: return launch<3, 4>(p, cfg, st);
        case 1 * 16 + 8: return launch<1, 8>(p, cfg, st);
        case 2 * 16 + 8: return launch<2, 8>(p, cfg, st);
        case 4 * 16 + 8: return launch<4, 8>(p, cfg, st);
    }
    return fail(NM_ERR_UNSUPPORTED, "nm_conv2d: N:M pattern not covered by the select kernel");
}

}  // namespace nmhost
