// Variant 4: expanded-operand kernel — persistent implicit GEMM that feeds the tensor core the
// DENSE activation slab straight from shared memory and lets zero weights stand for the pruned
// columns.
//
// Nothing is compacted: the slab [128 pixels x 32 source columns] that TMA's im2col mode lays
// down in the 128-byte-swizzled K-major layout IS the A operand, and the B operand is the pruned
// weight matrix re-expanded to its dense [channels x K] shape (TF32, zeros in the pruned
// columns, built once per handle).  The tensor core therefore spends M/N times the kept FLOPs,
// but no thread ever touches an activation.  It moves the same HBM bytes as the gathering
// kernels (with N:M groups along the channel axis every 16-byte vector holds survivors, so a
// gather cannot skip input bytes either), which makes it the right choice wherever the layer is
// bound by HBM and the tensor pipe has slack; the auto-tuner decides per layer by measurement.
// The pruning tile width plays no role here, so any tile_t is accepted.
//
//   producer (1 thread)   TMA im2col load of the slab + one contiguous bulk copy of the weight block
//                         (stored pre-swizzled, so it costs no per-row TMA requests) per stage; a
//                         weight slice of at most 128 KB is instead fetched once and stays resident
//                         (the grid is then a multiple of the slice count, so a CTA keeps its slice)
//   MMA issuer (1 thread) four 128 x BN x 8 TF32 tcgen05.mma (SS) per stage into one of two
//                         accumulator buffers in tensor memory
//   epilogue (8 warps)    TMEM -> registers, + bias, ReLU, swizzled staging, TMA store to NHWC;
//                         overlaps the next work item's main loop
// Work items (128 pixels x BN channels) are walked in a static persistent schedule; every wait is
// bounded and reports through the handle's status word.
//
// Balanced mode (plan.split = -1), for layers with fewer work items than would keep every SM busy:
// the (item, stage) pairs of the whole layer are laid end to end and cut into one contiguous,
// equally long range per CTA, so an item may be shared by two or more CTAs.  A CTA whose range
// begins inside an item handles that part FIRST, stores the raw partial accumulator to its own
// slot of the handle's scratch and raises a per-warp flag; the CTA whose range holds the item's
// first stage handles it LAST, waits (bounded) for the flags of the others, adds their partial sums
// to its accumulator, lowers the flags again (every flag has exactly one reader, so the scratch is
// back in its cleared state when the launch ends and a recorded launch can be replayed) and runs
// the normal epilogue.  Ranges are handed out from the end of the
// layer to CTA 0 upwards, so a CTA only ever waits for CTAs with a lower index, whose first action
// is the store it waits for.
#include "nm_internal.h"
#include "nm_ptx.cuh"
#include "nm_tmap.cuh"

namespace {

using namespace nmk;

constexpr int BM = 128;
constexpr int SUB_BYTES = BM * 128;
constexpr int NSTAGE_MAX = 10;
constexpr int WRES_MAX = 128 * 1024;            // largest weight slice kept resident
constexpr int THREADS = 384;                   // 4 service warps + 8 epilogue warps
constexpr int BOX_BYTES = 4096;                // one 32-pixel x 32-channel output box

struct ExpandCfg {
    int bn;           // output channels per work item
    int n_slices;
    int stages;
    int b_bytes;      // weight bytes per stage (bn rows of 128 bytes)
    int stage_bytes;
    int w_res;        // 1: this CTA's weight slice stays resident in shared memory (it is loaded once)
    int wres_bytes;   // bytes of the resident slice: all 32-column blocks of bn rows
    int n_sub;        // pipeline stages one work item reduces over: (K / 32) / ksplit / kblk
    int kblk;         // 32-column blocks per stage (1 or 2): one barrier round trip then covers kblk * 4 MMAs
    int n_iss;        // MMA issuer threads (1 or 2): two take alternate pipeline stages of an item, each into an accumulator of its own
    int n_acc;        // accumulator buffers (of n_iss accumulators each) in tensor memory: 2 when they fit, else 1
    int sub_bytes;    // bytes of one 32-column block inside a stage: activations (+ streamed weights)
    int ksplit;       // K splits (1 = none): a work item covers one of them and stores raw partial sums
    int p_pad;        // pixel blocks * 128: rows of one split in the partial-sum scratch
    int boxes;        // output staging boxes per epilogue warp: 2 for short reductions, 1 when the ring needs the room
    int balanced;     // 1: contiguous (item, stage) ranges per CTA, partial sums through per-CTA scratch slots
    long long n_work;
};

__device__ __forceinline__ bool aborted(volatile int* flag) { return *flag != 0; }

// One piece of work of a CTA: stages [sb, se) of work item `work`.
struct Seg {
    uint32_t work;
    int sb, se;
};
// Walks a CTA's pieces: whole items `first, first + stride, ...` in the static schedule, or the
// contiguous range of (item, stage) units of balanced mode.
template <bool BAL>
struct SegIter {
    uint32_t cur, end, stride;
    int stages;
    __device__ __forceinline__ bool next(Seg& g)
    {
        if (cur >= end) return false;
        if (!BAL) {
            g.work = cur; g.sb = 0; g.se = stages;
            cur += stride;
            return true;
        }
        g.work = cur / static_cast<uint32_t>(stages);
        g.sb = static_cast<int>(cur - g.work * static_cast<uint32_t>(stages));
        const uint32_t left = end - cur, room = static_cast<uint32_t>(stages - g.sb);
        const int len = static_cast<int>(left < room ? left : room);
        g.se = g.sb + len;
        cur += static_cast<uint32_t>(len);
        return true;
    }
};
// First (item, stage) unit of the range at position j of `n` equal ranges over `units`.
__device__ __forceinline__ uint32_t range_begin(uint32_t j, uint32_t n, uint32_t units)
{
    return static_cast<uint32_t>(static_cast<unsigned long long>(j) * units / n);
}
template <bool BAL>
__device__ __forceinline__ SegIter<BAL> make_iter(const ExpandCfg& cfg)
{
    SegIter<BAL> it;
    it.stages = cfg.n_sub;
    if (!BAL) {
        it.cur = blockIdx.x; it.end = static_cast<uint32_t>(cfg.n_work); it.stride = gridDim.x;
    } else {
        // ranges are handed out from the end of the layer: CTA b takes position gridDim.x - 1 - b
        const uint32_t units = static_cast<uint32_t>(cfg.n_work) * static_cast<uint32_t>(cfg.n_sub);
        const uint32_t j = gridDim.x - 1u - blockIdx.x;
        it.cur = range_begin(j, gridDim.x, units);
        it.end = range_begin(j + 1u, gridDim.x, units);
        it.stride = 0;
    }
    return it;
}
__device__ __forceinline__ uint32_t ld_acquire_gpu(const uint32_t* ptr)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_gpu(uint32_t* ptr, uint32_t v)
{
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(ptr), "r"(v) : "memory");
}

// KBLK: 32-column blocks per pipeline stage; BAL: balanced mode.  Compile-time, so that the lone producer and
// issuer threads of the common configuration (1, false) run exactly the instructions they need.
template <int KBLK, bool BAL>
__global__ void __launch_bounds__(THREADS, 1)
k_conv_expand(const ConvParams p, const ExpandCfg cfg, const __grid_constant__ CUtensorMap tm_x,
              const __grid_constant__ CUtensorMap tm_y)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_full[NSTAGE_MAX], s_free[NSTAGE_MAX], s_accfull[2], s_accfree[2], s_wres;
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int NS = cfg.stages, n_sub = cfg.n_sub;
    const uint32_t wres = (smem_u32(smem_raw) + 1023u) & ~1023u;   // resident weight slice (may be empty)
    const uint32_t ring = wres + cfg.wres_bytes;
    const uint32_t staging = ring + NS * cfg.stage_bytes;
    volatile int* abort_flag = &s_abort;

    if (warp == 2) tmem_alloc(smem_u32(&s_tmem), 512);
    if (tid == 0) {
        for (int i = 0; i < NSTAGE_MAX; ++i) {
            mbar_init(smem_u32(&s_full[i]), 1);   // producer's expect-tx arrival
            mbar_init(smem_u32(&s_free[i]), 1);   // the commit of the issuer that read the stage
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&s_accfull[i]), cfg.n_iss);   // MMA commits
            mbar_init(smem_u32(&s_accfree[i]), 8);   // epilogue warps
        }
        mbar_init(smem_u32(&s_wres), 1);
        mbar_fence_init();
        s_abort = 0;
        tma_prefetch_desc(&tm_x);
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
            int issued = 0;
            const int hw = p.ho * p.wo;
            const uint32_t tx = static_cast<uint32_t>(KBLK) * (SUB_BYTES + (cfg.w_res ? 0u : static_cast<uint32_t>(cfg.bn) * 128u));
            const int n_blk32 = n_sub * KBLK;   // 32-column blocks per work item
            if (cfg.w_res) {
                // the grid is a multiple of the slice count, so every work item of this CTA has the
                // same channel slice: its weights are fetched once
                const int slice = static_cast<int>(blockIdx.x % static_cast<uint32_t>(cfg.n_slices));
                mbar_arrive_expect_tx(smem_u32(&s_wres), static_cast<uint32_t>(n_blk32) * static_cast<uint32_t>(cfg.bn) * 128u);
                for (int c = 0; c < n_blk32; ++c)
                    bulk_load_1d(wres + c * cfg.b_bytes, p.wx + (static_cast<size_t>(c) * p.wx_rows + slice * cfg.bn) * 32,
                                 static_cast<uint32_t>(cfg.bn) * 128u, smem_u32(&s_wres));
            }
            const uint32_t w_bytes = static_cast<uint32_t>(cfg.bn) * 128u;
            const size_t w_step = static_cast<size_t>(p.wx_rows) * 32;   // floats between two 32-column blocks
            RingPos rp;
            SegIter<BAL> it = make_iter<BAL>(cfg);
            Seg seg;
            while (!aborted(abort_flag) && it.next(seg)) {
                // The item's coordinates, with the divisions the common cases do not need left out: this thread
                // issues the kernel's first load only after them.
                const uint32_t work = seg.work;
                uint32_t slice = 0, rest = work, ks = 0;
                if (cfg.n_slices > 1) {
                    rest = work / static_cast<uint32_t>(cfg.n_slices);
                    slice = work - rest * static_cast<uint32_t>(cfg.n_slices);
                }
                if (cfg.ksplit > 1) {
                    const uint32_t pb = rest / static_cast<uint32_t>(cfg.ksplit);
                    ks = rest - pb * static_cast<uint32_t>(cfg.ksplit);
                    rest = pb;
                }
                const uint32_t pix0 = rest * BM;
                const int n0 = static_cast<int>(pix0 / static_cast<uint32_t>(hw));
                const int rem = static_cast<int>(pix0 - static_cast<uint32_t>(n0) * static_cast<uint32_t>(hw));
                const int oh0 = rem / p.wo, ow0 = rem - oh0 * p.wo;
                const int w0 = ow0 * p.stride_w - p.pad_w, h0 = oh0 * p.stride_h - p.pad_h;
                // first 32-column block of this item's share of the reduction axis
                const int c0 = static_cast<int>(ks) * n_blk32 + seg.sb * KBLK;
                const float* wsrc = p.wx + static_cast<size_t>(slice) * cfg.bn * 32 + static_cast<size_t>(c0) * w_step;
                int ch = 0, tw = 0, off_w = 0, off_h = 0;
                if (c0 != 0) {
                    const int tap0 = (c0 * 32) / p.c_in, th = tap0 / p.kw;
                    ch = c0 * 32 - tap0 * p.c_in;
                    tw = tap0 - th * p.kw;
                    off_w = tw * p.dil_w;
                    off_h = th * p.dil_h;
                }
                for (int c = seg.sb; c < seg.se; ++c) {
                    if (rp.wrapped && !mbar_wait_lone(smem_u32(&s_free[rp.s]), rp.parity ^ 1u)) *abort_flag = 2;
                    if (aborted(abort_flag)) break;
                    uint32_t a_smem = ring + rp.s * cfg.stage_bytes;
                    const uint32_t bar = smem_u32(&s_full[rp.s]);
                    mbar_arrive_expect_tx(bar, tx);
#pragma unroll
                    for (int j = 0; j < KBLK; ++j) {
                        tma_load_im2col_4d(a_smem, &tm_x, bar, ch, w0, h0, n0, static_cast<uint16_t>(off_w),
                                           static_cast<uint16_t>(off_h));
                        if (!cfg.w_res) bulk_load_1d(a_smem + SUB_BYTES, wsrc, w_bytes, bar);
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
            if (aborted(abort_flag)) {
                // loads already issued still target this CTA's shared memory: let them land
                if (cfg.w_res) (void)mbar_wait(smem_u32(&s_wres), 0);
                for (int back = 0; back < NS && back < issued; ++back) {
                    if (rp.s == 0) { rp.s = NS; rp.parity ^= 1u; }
                    --rp.s;
                    (void)mbar_wait(smem_u32(&s_full[rp.s]), rp.parity);
                }
            }
        }
    } else if (warp == 1 || warp == 3) {
        // =========================== MMA issuers ===========================
        // A thread issues a tcgen05.mma about every 124 cycles whatever its width, and a barrier test and a commit per
        // stage on top of that, while the tensor core completes a 128 x 256 x 8 MMA in 128 cycles and narrower ones
        // sooner: one thread cannot keep it busy.  A plan may therefore have two issuer threads that take ALTERNATE
        // stages of a work item, each accumulating into columns of its own (the epilogue adds the two): the reduction
        // axis is split, not the channels, so both issue full-width MMAs.  A ring slot is released by the one commit of
        // the thread that read it.  Ownership goes by SLOT (even slots the first thread, odd slots the second; the ring
        // then has an even number of slots): a wait by phase parity is only right for a waiter that has seen every
        // earlier use of the slot, and with ownership by position inside the item a thread would skip uses of a slot
        // at the seams between items (found as a fault on the GPU, reproduced and fixed in a CPU model of the protocol).
        const int iss = warp >> 1;
        if (lane == 0 && iss < cfg.n_iss) {
            const uint32_t idesc = umma_idesc_tf32(BM, cfg.bn);
            const bool shared_k = cfg.n_iss == 2;
            if (cfg.w_res && !mbar_wait(smem_u32(&s_wres), 0)) *abort_flag = 9;
            RingPos rp;
            uint32_t ab = 0, acc_par = 0;   // accumulator buffer of this item, parity of its current use
            bool acc_wrapped = false;
            SegIter<BAL> it = make_iter<BAL>(cfg);
            Seg seg;
            while (!aborted(abort_flag) && it.next(seg)) {
                if (acc_wrapped && !mbar_wait_lone(smem_u32(&s_accfree[ab]), acc_par ^ 1u)) {
                    *abort_flag = 5;
                    break;
                }
                tc_fence_after();
                const uint32_t acc = tmem + (ab * cfg.n_iss + iss) * cfg.bn;
                uint32_t started = 0;   // 0 until this thread's first MMA of the item, which overwrites the accumulator
                for (int c = seg.sb; c < seg.se; ++c) {
                    if (shared_k && (rp.s & 1) != iss) {   // the other thread's slot
                        rp.advance(NS);
                        continue;
                    }
                    if (!mbar_wait_lone(smem_u32(&s_full[rp.s]), rp.parity)) { *abort_flag = 6; break; }
                    tc_fence_after();
                    const uint32_t a_smem = ring + rp.s * cfg.stage_bytes;
                    uint64_t adesc = umma_desc_k_sw128(a_smem, 1024);
                    uint64_t bdesc = umma_desc_k_sw128(cfg.w_res ? wres + c * KBLK * cfg.b_bytes : a_smem + SUB_BYTES, 1024);
                    const uint32_t b_step = KBLK > 1 ? static_cast<uint32_t>(cfg.w_res ? cfg.b_bytes : cfg.sub_bytes) >> 4 : 0u;
#pragma unroll
                    for (int j = 0; j < KBLK; ++j) {
#pragma unroll
                        for (int kq = 0; kq < 4; ++kq)
                            umma_tf32_ss(acc, adesc + 2 * kq, bdesc + 2 * kq, idesc, (j > 0 || kq > 0) ? 1u : started);
                        if (j + 1 < KBLK) {
                            adesc += static_cast<uint32_t>(cfg.sub_bytes) >> 4;   // next 32-column block (start address field, 16-byte units)
                            bdesc += b_step;
                        }
                    }
                    started = 1u;
                    umma_commit(smem_u32(&s_free[rp.s]));
                    rp.advance(NS);
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
    } else if (warp >= 4) {
        // =========================== epilogue ===========================
        const int q = warp & 3;            // TMEM lane quadrant
        const int half = (warp - 4) >> 2;  // which channel blocks of 32: blk = 2 * i + half
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t my_staging = staging + (warp - 4) * cfg.boxes * BOX_BYTES;
        const uint32_t box_toggle = cfg.boxes == 2 ? 1u : 0u;
        const uint32_t rx = static_cast<uint32_t>(lane & 7);
        const int n_blk = cfg.bn / 32;
        uint32_t nb = 0, ti = 0;
        uint32_t stage_count = 0;   // stages of all earlier pieces of this CTA
        // balanced mode: this CTA's partial-sum slot (128 rows x bn) and its warps' flags, in the handle's scratch
        const uint32_t units = static_cast<uint32_t>(cfg.n_work) * static_cast<uint32_t>(cfg.n_sub);
        const size_t slot_floats = static_cast<size_t>(BM) * cfg.bn;
        // scratch layout: eight flag words per CTA first, then the slots
        uint32_t* const flags = reinterpret_cast<uint32_t*>(p.splitk);
        float* const slots = p.splitk + static_cast<size_t>(gridDim.x) * 8;
        const int my_row = q * 32 + lane;
        SegIter<BAL> it = make_iter<BAL>(cfg);
        Seg seg;
        for (; it.next(seg); ++ti) {
            const uint32_t work = seg.work;
            const bool publish = BAL && seg.sb > 0;                   // a later part of an item: store raw sums
            const bool finish = BAL && seg.sb == 0 && seg.se < n_sub;  // the first part: add the others' sums
            const int slice = static_cast<int>(work % static_cast<uint32_t>(cfg.n_slices));
            const uint32_t rest = work / static_cast<uint32_t>(cfg.n_slices);
            const int ks = static_cast<int>(rest % static_cast<uint32_t>(cfg.ksplit));
            const uint32_t pix0 = (rest / static_cast<uint32_t>(cfg.ksplit)) * BM;
            const int ab = cfg.n_acc == 2 ? static_cast<int>(ti & 1u) : 0;
            // two issuers: stages went to them by ring slot, i.e. by the parity of the running stage count; a piece of
            // one stage is in the accumulator of that stage's owner, a longer one in both
            const uint32_t piece_first = stage_count;
            stage_count += static_cast<uint32_t>(seg.se - seg.sb);
            const bool two_acc = cfg.n_iss == 2 && seg.se - seg.sb >= 2;
            const uint32_t acc_first = (cfg.n_iss == 2 && seg.se - seg.sb == 1) ? (piece_first & 1u) : 0u;
            // the shortcut input does not depend on the accumulator: its first box is requested before the
            // wait for the main loop, every later box while the one before it is being stored
            const long long box_pix = static_cast<long long>(pix0) + q * 32;
            const bool res_pass = p.residual != nullptr && box_pix < p.pixels && !publish;
            const int res_rows = p.pixels - box_pix < 32 ? static_cast<int>(p.pixels - box_pix) : 32;
            const float* res_base = res_pass ? p.residual + box_pix * p.c_out + slice * cfg.bn : nullptr;
            float4 rv[8];
            const int cols_left = p.c_out - slice * cfg.bn;   // channels of this slice that exist (may end inside a box)
            const int o0 = slice * cfg.bn;
            float bias_next = half < n_blk ? bias_lane_load(p.bias, o0 + half * 32, p.c_out, lane) : 0.f;   // first block's bias
            if (res_pass && half < n_blk) load_residual_box(rv, res_base + half * 32, p.c_out, res_rows, lane, cols_left - half * 32);
            // positions (of the equal ranges) that hold the rest of this item: first_pos + 1 .. last_pos.  Their
            // partial sums were stored long ago (they are those CTAs' first piece of work), so the flags are
            // checked and, where no shortcut input occupies the registers, the first counterpart's sums of
            // this warp's first block are requested BEFORE the wait for this CTA's own accumulator.
            uint32_t first_pos = 0, last_pos = 0;
            bool ahead = false;
            if (finish) {
                first_pos = gridDim.x - 1u - blockIdx.x;
                const uint32_t u_last = (work + 1u) * static_cast<uint32_t>(n_sub) - 1u;
                last_pos = static_cast<uint32_t>(static_cast<unsigned long long>(u_last) * gridDim.x / units);
                while (last_pos + 1u < gridDim.x && range_begin(last_pos + 1u, gridDim.x, units) <= u_last) ++last_pos;
                while (last_pos > first_pos && range_begin(last_pos, gridDim.x, units) > u_last) --last_pos;
                // each of this warp's counterparts has stored its rows and raised its flag (bounded wait)
                for (uint32_t pos = first_pos + 1u; pos <= last_pos; ++pos) {
                    const uint32_t* f = flags + (gridDim.x - 1u - pos) * 8u + (warp - 4);
                    bool seen = false;
                    for (uint32_t poll = 0; poll < kWaitPolls && !seen; ++poll) seen = ld_acquire_gpu(f) == 1u;
                    if (!seen) *abort_flag = 10;
                }
                if (!res_pass && half < n_blk && !aborted(abort_flag)) {
                    const float4* src = reinterpret_cast<const float4*>(slots + slot_floats * (gridDim.x - 2u - first_pos)) +
                                        static_cast<size_t>(half) * 8 * BM + my_row;
#pragma unroll
                    for (int qq = 0; qq < 8; ++qq) rv[qq] = __ldcg(src + qq * BM);
                    ahead = true;
                }
            }
            const bool ok = aborted(abort_flag) || mbar_wait(smem_u32(&s_accfull[ab]), (cfg.n_acc == 2 ? (ti >> 1) : ti) & 1u);
            if (!__all_sync(0xFFFFFFFFu, ok)) *abort_flag = 8;
            if (__any_sync(0xFFFFFFFFu, aborted(abort_flag))) break;
            tc_fence_after();
            for (int blk = half; blk < n_blk; blk += 2, ++nb) {
                uint32_t v[32];
                tmem_ld32(tmem + lane_addr + (ab * cfg.n_iss + acc_first) * cfg.bn + blk * 32, v);
                if (two_acc) {
                    uint32_t v2[32];
                    tmem_ld32(tmem + lane_addr + (ab * cfg.n_iss + 1) * cfg.bn + blk * 32, v2);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) + __uint_as_float(v2[e]));
                } else {
                    tmem_ld_wait();
                }
                if (blk + 2 >= n_blk) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&s_accfree[ab]));
                }
                if (publish) {
                    // raw partial sums of this thread's row; the slot is laid out [channel quad][row], so the 32
                    // lanes of a warp (32 consecutive rows) write 512 contiguous bytes per instruction
                    float4* dst = reinterpret_cast<float4*>(slots + slot_floats * blockIdx.x) +
                                  static_cast<size_t>(blk) * 8 * BM + my_row;
#pragma unroll
                    for (int qq = 0; qq < 8; ++qq)
                        __stcg(dst + qq * BM, make_float4(__uint_as_float(v[qq * 4 + 0]), __uint_as_float(v[qq * 4 + 1]),
                                                     __uint_as_float(v[qq * 4 + 2]), __uint_as_float(v[qq * 4 + 3])));
                    --nb;   // no staging box used
                    continue;
                }
                if (finish) {
                    uint32_t pos_from = first_pos + 1u;
                    if (ahead) {
#pragma unroll
                        for (int qq = 0; qq < 8; ++qq) {
                            v[qq * 4 + 0] = __float_as_uint(__uint_as_float(v[qq * 4 + 0]) + rv[qq].x);
                            v[qq * 4 + 1] = __float_as_uint(__uint_as_float(v[qq * 4 + 1]) + rv[qq].y);
                            v[qq * 4 + 2] = __float_as_uint(__uint_as_float(v[qq * 4 + 2]) + rv[qq].z);
                            v[qq * 4 + 3] = __float_as_uint(__uint_as_float(v[qq * 4 + 3]) + rv[qq].w);
                        }
                        if (blk + 2 < n_blk) {   // a block ahead
                            const float4* nxt = reinterpret_cast<const float4*>(slots + slot_floats * (gridDim.x - 2u - first_pos)) +
                                                static_cast<size_t>(blk + 2) * 8 * BM + my_row;
#pragma unroll
                            for (int qq = 0; qq < 8; ++qq) rv[qq] = __ldcg(nxt + qq * BM);
                        }
                        ++pos_from;
                    }
                    for (uint32_t pos = pos_from; pos <= last_pos; ++pos) {
                        const float4* src = reinterpret_cast<const float4*>(slots + slot_floats * (gridDim.x - 1u - pos)) +
                                            static_cast<size_t>(blk) * 8 * BM + my_row;
                        float4 t4[8];
#pragma unroll
                        for (int qq = 0; qq < 8; ++qq) t4[qq] = __ldcg(src + qq * BM);
#pragma unroll
                        for (int qq = 0; qq < 8; ++qq) {
                            const float4 t = t4[qq];
                            v[qq * 4 + 0] = __float_as_uint(__uint_as_float(v[qq * 4 + 0]) + t.x);
                            v[qq * 4 + 1] = __float_as_uint(__uint_as_float(v[qq * 4 + 1]) + t.y);
                            v[qq * 4 + 2] = __float_as_uint(__uint_as_float(v[qq * 4 + 2]) + t.z);
                            v[qq * 4 + 3] = __float_as_uint(__uint_as_float(v[qq * 4 + 3]) + t.w);
                        }
                    }
                }
                const uint32_t box = my_staging + (nb & box_toggle) * BOX_BYTES;
                if (lane == 0) {
                    // the store that last read this box must be done with it
                    if (cfg.boxes == 2) { if (nb >= 2) tma_store_wait_read_n<1>(); }
                    else if (nb >= 1) tma_store_wait_read_n<0>();
                }
                __syncwarp();
                const uint32_t stage_row = box + lane * 128;
                // with a shortcut input the activation waits for the second pass below
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
                    if (blk + 2 < n_blk)
                        load_residual_box(rv, res_base + (blk + 2) * 32, p.c_out, res_rows, lane, cols_left - (blk + 2) * 32);
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                    if (pix0 + q * 32 < p.pixels)
                        tma_store_2d(&tm_y, box, o0 + blk * 32, ks * cfg.p_pad + static_cast<int>(pix0) + q * 32);
                    tma_store_commit();
                }
            }
            if (n_blk == 1 && half == 1) {
                // a single channel block: the second warp of the quadrant only releases the buffer
                if (lane == 0) mbar_arrive(smem_u32(&s_accfree[ab]));
            }
            if (publish) {
                // every lane's stores are ordered before the flag the reading warp acquires
                __threadfence();
                __syncwarp();
                if (lane == 0) st_release_gpu(flags + blockIdx.x * 8u + (warp - 4), 1u);
            }
            if (finish) {
                // this warp was the only reader of its counterparts' flags and has consumed their sums
                __syncwarp();
                if (lane == 0)
                    for (uint32_t pos = first_pos + 1u; pos <= last_pos; ++pos)
                        flags[(gridDim.x - 1u - pos) * 8u + (warp - 4)] = 0u;
            }
        }
        if (lane == 0) tma_store_wait_read();   // shared memory must outlive the stores' reads; the writes complete with the grid
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && s_abort != 0) {
        atomicExch(p.status + 0, static_cast<int>(NM_ERR_TIMEOUT));
        atomicExch(p.status + 1, 40 + s_abort);
        atomicExch(p.status + 2, static_cast<int>(blockIdx.x));
    }
    if (warp == 2) tmem_dealloc(tmem, 512);
}

// Second pass of a split-K plan: y[p][c] = act(sum over splits of partial[s][p][c] + bias[c] + residual[p][c]).
__global__ void k_splitk_reduce(const float4* __restrict__ part, int splits, size_t split_stride4, size_t n4, int c_out4,
                                const float4* __restrict__ bias, const float4* __restrict__ residual, int relu,
                                float4* __restrict__ y)
{
    nmk::pdl_wait();   // the partial sums come from the kernel launched just before
    for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < n4;
         i += static_cast<size_t>(gridDim.x) * blockDim.x) {
        float4 a = part[i];
        for (int s = 1; s < splits; ++s) {
            const float4 b = part[i + s * split_stride4];
            a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
        }
        if (bias) {
            const float4 b = __ldg(bias + (i % c_out4));
            a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
        }
        if (residual) {
            const float4 b = __ldg(residual + i);
            a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
        }
        if (relu) { a.x = fmaxf(a.x, 0.f); a.y = fmaxf(a.y, 0.f); a.z = fmaxf(a.z, 0.f); a.w = fmaxf(a.w, 0.f); }
        y[i] = a;
    }
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

bool make_cfg(const ConvParams& p, const nm_plan_t* plan, ExpandCfg* cfg)
{
    if (!p.wx || !nmtm::available()) return false;
    // whole 32-channel input blocks, or a pointwise layer whose last block the TMA unit fills up with zeros;
    // output channels in whole float4s (the expanded weights are padded to 32-row blocks)
    const bool pointwise = p.kh == 1 && p.kw == 1;
    if (p.c_in % 32 != 0 && !(pointwise && p.c_in % 4 == 0)) return false;
    if (p.c_out % 4 != 0 || p.wx_rows < p.c_out || p.wx_rows % 32 != 0) return false;
    if (!nmtm::im2col_geometry_ok(p)) return false;
    if (static_cast<long long>(p.batch) * p.h * p.w * p.c_in * 4 < 131072) return false;
    if (p.pixels >= (1ll << 31) - BM) return false;
    int bn = 0;
    if (plan && plan->bn > 0) {
        bn = plan->bn;
    } else {
        for (int cand : {128, 256, 64, 96, 32, 160, 192, 224})
            if (cand <= p.wx_rows && p.wx_rows % cand == 0) { bn = cand; break; }
    }
    if (bn < 32 || bn > 256 || bn % 32 != 0 || p.wx_rows % bn != 0) return false;
    cfg->bn = bn;
    cfg->n_slices = p.wx_rows / bn;
    cfg->b_bytes = ((bn * 128 + 1023) / 1024) * 1024;
    const int splits = plan && plan->split > 1 ? plan->split : 1;
    const bool balanced = plan && plan->split == -1;
    const int k_blocks = (p.k + 31) / 32;   // the last block of a pointwise layer may be partly zero fill
    if (splits > 8 || k_blocks % splits != 0) return false;
    cfg->ksplit = splits;
    const int blk32 = k_blocks / splits;   // 32-column blocks per work item
    const int kblk = plan && plan->kblk > 0 ? plan->kblk : 1;
    if (kblk > 2 || blk32 % kblk != 0) return false;
    cfg->kblk = kblk;
    cfg->n_sub = blk32 / kblk;
    // one issuer thread unless the plan asks for two (alternate stages, an accumulator each; one accumulator buffer
    // instead of two when both pairs do not fit the 512 columns)
    const int n_iss = plan && plan->issuers > 0 ? plan->issuers : 1;
    if (n_iss < 1 || n_iss > 2) return false;
    cfg->n_iss = n_iss;
    cfg->n_acc = 2 * n_iss * bn <= 512 ? 2 : 1;
    cfg->p_pad = static_cast<int>(((p.pixels + BM - 1) / BM) * BM);
    if (splits > 1 && (!p.splitk || p.splitk_bytes < static_cast<size_t>(splits) * cfg->p_pad * p.c_out * sizeof(float) ||
                       static_cast<long long>(splits) * cfg->p_pad >= (1ll << 31)))
        return false;   // the partial-sum scratch is reserved by nm_autotune
    cfg->boxes = blk32 <= 8 ? 2 : 1;   // long reductions: the epilogue is rare, the ring needs the bytes
    // A weight slice that fits stays resident (plan.split == 1 asks for streaming instead): the ring
    // then holds activations only and is deeper.  Needs one fixed slice per CTA, i.e. a grid that is a
    // multiple of the slice count.
    cfg->wres_bytes = 0;
    cfg->w_res = 0;
    if (splits == 1 && !balanced && !(plan && plan->split == 1) && blk32 * cfg->b_bytes <= WRES_MAX && cfg->n_slices <= sm_count()) {
        cfg->w_res = 1;
        cfg->wres_bytes = blk32 * cfg->b_bytes;
        if (cfg->wres_bytes > 64 * 1024) cfg->boxes = 1;   // a large slice: give the output staging's room to the ring
    }
    cfg->sub_bytes = SUB_BYTES + (cfg->w_res ? 0 : cfg->b_bytes);
    cfg->stage_bytes = kblk * cfg->sub_bytes;
    const int budget = 227 * 1024 - 1024 - 8 * cfg->boxes * BOX_BYTES - 1024 - cfg->wres_bytes;
    int stages = plan && plan->stages > 0 ? plan->stages : NSTAGE_MAX;
    if (stages > NSTAGE_MAX) return false;
    if (plan && plan->stages > 0) {
        if (stages * cfg->stage_bytes > budget) return false;
        if (n_iss == 2 && stages % 2 != 0) return false;   // two issuers own alternate ring slots
    } else {
        while (stages > 2 && stages * cfg->stage_bytes > budget) --stages;
        if (n_iss == 2) stages &= ~1;
        if (stages * cfg->stage_bytes > budget) return false;
    }
    cfg->stages = stages;
    cfg->n_work = ((p.pixels + BM - 1) / BM) * cfg->n_slices * splits;
    if (cfg->n_work >= (1ll << 31)) return false;
    cfg->balanced = 0;
    if (balanced) {
        // one range per SM; needs at least one (item, stage) unit per CTA and the per-CTA slots + flags in the scratch
        const long long units = cfg->n_work * cfg->n_sub;
        if (units < sm_count() || units >= (1ll << 31)) return false;
        if (!p.splitk || p.splitk_bytes < nmhost::expand_balanced_bytes(bn)) return false;
        cfg->balanced = 1;
    }
    return true;
}

}  // namespace

namespace nmhost {

size_t expand_balanced_bytes(int bn)
{
    // per SM: a slot of 128 rows x bn partial sums, and eight flag words (one per epilogue warp)
    return static_cast<size_t>(sm_count()) * (static_cast<size_t>(BM) * bn * sizeof(float) + 8 * sizeof(uint32_t));
}

bool expand_plan_ok(const ConvParams& p, const nm_plan_t* plan)
{
    ExpandCfg cfg;
    return make_cfg(p, plan, &cfg);
}

nm_status_t launch_conv_expand(const ConvParams& p, const nm_plan_t* plan, cudaStream_t st)
{
    ExpandCfg cfg;
    if (!make_cfg(p, plan, &cfg))
        return fail(NM_ERR_UNSUPPORTED, "nm_conv2d: the expanded-operand kernel does not take this layer / plan%s",
                    plan && (plan->split > 1 || plan->split == -1) ? " (a split or balanced plan needs scratch: nm_weights_reserve)" : "");
    // a split-K plan stores raw partial sums [split][pixel][channel] in the handle's scratch; bias and
    // activation are applied by the reduction pass
    ConvParams q = p;
    if (cfg.ksplit > 1) {
        q.y = p.splitk;
        q.pixels = static_cast<long long>(cfg.ksplit) * cfg.p_pad;   // rows of the store map
        q.bias = nullptr;
        q.residual = nullptr;
        q.relu = 0;
    }
    alignas(64) CUtensorMap tm_x, tm_y;
    if (!nmtm::encode_x_im2col(p, BM, &tm_x) || !nmtm::encode_y_tiled(q, &tm_y))
        return fail(NM_ERR_CUDA, "nm_conv2d: tensor-map encoding failed (variant 4)");
    q.pixels = p.pixels;
    size_t smem = 1024 + cfg.wres_bytes + static_cast<size_t>(cfg.stages) * cfg.stage_bytes + 8 * cfg.boxes * BOX_BYTES;
    if (smem < 120 * 1024) smem = 120 * 1024;   // one CTA per SM: it owns all 512 TMEM columns
    using Kernel = void (*)(const ConvParams, const ExpandCfg, const CUtensorMap, const CUtensorMap);
    const Kernel kernel = cfg.balanced ? (cfg.kblk == 2 ? k_conv_expand<2, true> : k_conv_expand<1, true>)
                                       : (cfg.kblk == 2 ? k_conv_expand<2, false> : k_conv_expand<1, false>);
    cudaError_t e = nmhost::ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), smem);
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "cudaFuncSetAttribute (variant 4): %s", cudaGetErrorString(e));
    long long grid = cfg.n_work < sm_count() ? cfg.n_work : sm_count();
    if (cfg.balanced) grid = sm_count();
    if (cfg.w_res) grid = (grid / cfg.n_slices) * cfg.n_slices;   // n_work is a multiple of n_slices, so grid >= n_slices
    e = nmhost::launch_pdl(kernel, static_cast<unsigned>(grid), THREADS, smem, st, q, cfg, tm_x, tm_y);
    nmhost::count_launch(1);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "nm_conv2d launch (variant 4): %s", cudaGetErrorString(e));
    if (cfg.ksplit > 1) return launch_splitk_reduce(p, cfg.ksplit, cfg.p_pad, st);
    return NM_OK;
}

nm_status_t launch_splitk_reduce(const ConvParams& p, int splits, int p_pad, cudaStream_t st)
{
    const size_t n4 = static_cast<size_t>(p.pixels) * p.c_out / 4;
    const size_t stride4 = static_cast<size_t>(p_pad) * p.c_out / 4;
    size_t blocks = (n4 + 255) / 256;
    if (blocks > static_cast<size_t>(sm_count()) * 8) blocks = static_cast<size_t>(sm_count()) * 8;
    cudaError_t e = nmhost::launch_pdl(k_splitk_reduce, static_cast<unsigned>(blocks), 256u, 0, st,
                                       reinterpret_cast<const float4*>(p.splitk), splits, stride4, n4, p.c_out / 4,
                                       reinterpret_cast<const float4*>(p.bias), reinterpret_cast<const float4*>(p.residual),
                                       p.relu, reinterpret_cast<float4*>(p.y));
    nmhost::count_launch(1);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "nm_conv2d launch (split-K reduction): %s", cudaGetErrorString(e));
    return NM_OK;
}

size_t expand_splitk_bytes(const ConvParams& p, int splits)
{
    const size_t p_pad = static_cast<size_t>((p.pixels + BM - 1) / BM) * BM;
    return static_cast<size_t>(splits) * p_pad * p.c_out * sizeof(float);
}

}  // namespace nmhost
