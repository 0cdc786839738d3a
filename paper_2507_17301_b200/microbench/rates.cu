// Hardware rates that shaped the convolution kernels, measured in isolation on one GPU (every SM runs the same loop):
//
//   select   a compactor's inner loop: 128 pixel rows x 64 source columns read from a 128-byte-swizzled slab with
//            16-byte loads, the 2:4 retained columns of `g` tiles picked with bitwise selects, results stored to tensor
//            memory.  Modes: copy (no selection: the cost of reading the slab), word masks (one 32-bit mask per select,
//            loaded from shared memory), byte masks (one byte per select, widened with a byte permute).
//   mma      TF32 tcgen05.mma of shape 128 x N x 8 issued back to back by 1, 2 or 4 threads (each with accumulator
//            columns of its own), A from tensor memory (TS) or from shared memory (SS).
//   intake   bytes per cycle an SM takes in from L2: bulk copies of 32 KB, tiled TMA loads of 128 rows x 128 bytes (swizzled), or
//            one of each per stage, four stages in flight, every SM reading its own 1 MB window of a buffer that fits the L2.
//   cp       tcgen05.cp of an operand tile from shared to tensor memory: layout check, issue rate, and the rate of
//            the pattern "four copies, four TS MMAs" per 32-column block from one and from two threads.
//
// Prints cycles per unit of work from clock64 and from CUDA events.  Nothing here is used by the library.
#include <cstdio>
#include <cstdlib>
#include <cuda_runtime.h>

#include "../csrc/nm_ptx.cuh"
#include "../csrc/nm_tmap.cuh"
using namespace nmk;

#define CK(x)                                                                                  \
    do {                                                                                       \
        cudaError_t e = (x);                                                                   \
        if (e != cudaSuccess) {                                                                \
            std::printf("CUDA error %s at line %d\n", cudaGetErrorString(e), __LINE__);        \
            std::exit(1);                                                                      \
        }                                                                                      \
    } while (0)

__device__ __forceinline__ void lds128(uint32_t a, uint32_t* d)
{
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]) : "r"(a));
}
__device__ __forceinline__ uint32_t bsel(uint32_t m, uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xCA;" : "=r"(d) : "r"(m), "r"(a), "r"(b));
    return d;
}
template <int K>
__device__ __forceinline__ uint32_t mask_of_byte(uint32_t w)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %1, %2;" : "=r"(d) : "r"(w), "n"(0x8888 | (0x1111 * K)));
    return d;
}

// MODE 0: copy, 1: word masks, 2: byte masks.  `warps` compactor warps (8 or 16), two per TMEM lane quadrant and half.
template <int MODE>
__global__ void __launch_bounds__(512, 1) k_select(int iters, int g, int warps, long long* cycles)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t s_tmem;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t slab = base, masks = base + 32768;   // 2 x 16 KB slab, then g x 2 halves x 128 bytes of masks
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    for (int i = tid; i < 8192 + 1024; i += blockDim.x) reinterpret_cast<uint32_t*>(smem_raw)[i] = (i * 2654435761u) >> 3;
    if (warp == 0) tmem_alloc(smem_u32(&s_tmem), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    const long long t0 = clock64();
    if (warp < warps) {
        const int q = warp & 3, half = (warp >> 2) & 1, row = q * 32 + lane;
        const uint32_t rx = row & 7, lane_addr = static_cast<uint32_t>(q * 32) << 16;
        for (int it = 0; it < iters; ++it) {
            uint32_t x[32];
#pragma unroll
            for (int i = 0; i < 8; ++i) lds128(slab + half * 16384 + row * 128 + ((static_cast<uint32_t>(i) ^ rx) << 4), x + 4 * i);
            for (int t = 0; t < g; ++t) {
                uint32_t v[16];
                const uint32_t mb = masks + (t * 2 + half) * 128;
                if (MODE == 1) {
                    uint32_t m[32];
#pragma unroll
                    for (int i = 0; i < 8; ++i) lds128(mb + 16 * i, m + 4 * i);
#pragma unroll
                    for (int gi = 0; gi < 8; ++gi) {
                        v[2 * gi] = bsel(m[4 * gi], x[4 * gi], bsel(m[4 * gi + 1], x[4 * gi + 1], x[4 * gi + 2]));
                        v[2 * gi + 1] = bsel(m[4 * gi + 2], x[4 * gi + 1], bsel(m[4 * gi + 3], x[4 * gi + 2], x[4 * gi + 3]));
                    }
                } else if (MODE == 2) {
                    uint32_t m[8];
                    lds128(mb, m);
                    lds128(mb + 16, m + 4);
#pragma unroll
                    for (int gi = 0; gi < 8; ++gi) {
                        v[2 * gi] = bsel(mask_of_byte<0>(m[gi]), x[4 * gi], bsel(mask_of_byte<1>(m[gi]), x[4 * gi + 1], x[4 * gi + 2]));
                        v[2 * gi + 1] =
                            bsel(mask_of_byte<2>(m[gi]), x[4 * gi + 1], bsel(mask_of_byte<3>(m[gi]), x[4 * gi + 2], x[4 * gi + 3]));
                    }
                } else {
#pragma unroll
                    for (int gi = 0; gi < 8; ++gi) { v[2 * gi] = x[4 * gi]; v[2 * gi + 1] = x[4 * gi + 1]; }
                }
                tmem_st16(tmem + lane_addr + 256 + ((it & 1) * 4 + t) * 32 + half * 16, v);
            }
            tmem_st_wait();
        }
    }
    __syncthreads();
    if (tid == 0) cycles[blockIdx.x] = clock64() - t0;
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

// `issuers` threads (lane 0 of warps 0 ..) each issue `count` MMAs 128 x n x 8 into accumulator columns of their own.
__global__ void __launch_bounds__(256, 1) k_mma(int count, int n, int issuers, int ss, long long* cycles)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t s_tmem;
    __shared__ uint64_t s_done[4];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    for (int i = tid; i < 16384; i += blockDim.x) reinterpret_cast<uint32_t*>(smem_raw)[i] = 0;
    if (warp == 7) tmem_alloc(smem_u32(&s_tmem), 512);
    if (tid == 0) {
        for (int i = 0; i < 4; ++i) mbar_init(smem_u32(&s_done[i]), 1);
        mbar_fence_init();
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    const long long t0 = clock64();
    if (warp < issuers && lane == 0) {
        const uint32_t idesc = umma_idesc_tf32(128, n);
        // operand layouts: 128-byte-swizzled K-major rows, or unswizzled K-major core matrices (8 rows x 16 bytes = 128
        // contiguous bytes; 128 bytes between 8-row groups; A: 1856 bytes between the two core matrices along K, as in the
        // plane kernel; B: n * 16 bytes, i.e. a [K / 4][n][16 bytes] image)
        const uint64_t a_sw = umma_desc_k_sw128(base + 32768, 1024), a_pl = umma_desc_k_plain(base + 32768, 1856, 128);
        const uint64_t b_sw = umma_desc_k_sw128(base, 1024), b_pl = umma_desc_k_plain(base, n * 16, 128);
        const uint32_t b_step = static_cast<uint32_t>(2 * n);   // two core-matrix columns of B, in 16-byte units
        const uint32_t acc = tmem + warp * (256 / issuers);   // 256 / issuers >= n
        // B unswizzled inside the 1 KB atoms of the swizzled layout ([8 rows][128 bytes] stored as [8 K pieces][8 rows][16 bytes]):
        // 128 bytes between core matrices along K, 1024 between 8-row groups; a run of rows stays one contiguous copy
        const uint64_t b_at = umma_desc_k_plain(base, 128, 1024);
        const bool a_plain = (ss & 2) != 0, b_plain = (ss & 4) != 0, b_atom = (ss & 8) != 0;
        for (int i = 0; i < count; ++i) {
            const uint64_t bd = b_atom ? b_at + 16 * (i & 3) : b_plain ? b_pl + (i & 3) * b_step : b_sw + 2 * (i & 3);
            if (ss & 1) umma_tf32_ss(acc, a_plain ? a_pl + (i & 3) : a_sw + 2 * (i & 3), bd, idesc, 1u);
            else umma_tf32_ts(acc, tmem + 256 + (i & 7) * 8, bd, idesc, 1u);
        }
        umma_commit(smem_u32(&s_done[warp]));
        if (!mbar_wait(smem_u32(&s_done[warp]), 0)) std::printf("wait expired\n");
    }
    __syncthreads();
    if (tid == 0) cycles[blockIdx.x] = clock64() - t0;
    tc_fence_before();
    __syncthreads();
    if (warp == 7) tmem_dealloc(tmem, 512);
}


// MODE 0: layout check (a swizzled 128 x 32 tile with element (row, col) = row * 32 + col is copied with four
// tcgen05.cp and read back; prints the number of mismatches).  MODE 1: `count` copies back to back from one thread.
// MODE 2: per 32-column block four copies then four 128 x n x 8 TS MMAs on the copied columns, one thread.
// MODE 3: the same with the copies issued by a second thread (hand-over through mbarriers, four operand slots).
__global__ void __launch_bounds__(256, 1) k_cp(int mode, int count, int n, long long* cycles, int* mismatches)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t s_tmem;
    __shared__ uint64_t s_done[2], s_ready[4], s_free[4];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // B region (32 KB of zeros) at base, A tile at base + 32768: row r = 128 bytes, 16-byte pieces XOR-ed with r % 8
    for (int i = tid; i < 8192; i += blockDim.x) reinterpret_cast<uint32_t*>(smem_raw + (base - smem_u32(smem_raw)))[i] = 0;
    for (int i = tid; i < 128 * 32; i += blockDim.x) {
        const int r = i >> 5, c = i & 31;
        const uint32_t off = 32768u + r * 128u + ((static_cast<uint32_t>(c >> 2) ^ static_cast<uint32_t>(r & 7)) << 4) + (c & 3) * 4u;
        *reinterpret_cast<float*>(smem_raw + (base - smem_u32(smem_raw)) + off) = static_cast<float>(i);
    }
    if (warp == 7) tmem_alloc(smem_u32(&s_tmem), 512);
    if (tid == 0) {
        for (int i = 0; i < 2; ++i) mbar_init(smem_u32(&s_done[i]), 1);
        for (int i = 0; i < 4; ++i) { mbar_init(smem_u32(&s_ready[i]), 1); mbar_init(smem_u32(&s_free[i]), 1); }
        mbar_fence_init();
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    const uint64_t a_sw = umma_desc_k_sw128(base + 32768, 1024), b_sw = umma_desc_k_sw128(base, 1024);
    const uint32_t idesc = umma_idesc_tf32(128, n);
    const long long t0 = clock64();
    if (mode == 0) {
        if (tid == 0) {
            for (int kq = 0; kq < 4; ++kq) tmem_cp_128x256b(tmem + 256 + kq * 8, a_sw + 2 * kq);
            umma_commit(smem_u32(&s_done[0]));
        }
        if (!mbar_wait(smem_u32(&s_done[0]), 0) && lane == 0) std::printf("wait expired\n");
        tc_fence_after();
        if (warp < 4) {
            uint32_t v[32];
            tmem_ld32(tmem + (static_cast<uint32_t>(warp * 32) << 16) + 256, v);
            tmem_ld_wait();
            int bad = 0;
            for (int c = 0; c < 32; ++c) bad += __uint_as_float(v[c]) != static_cast<float>((warp * 32 + lane) * 32 + c);
            if (bad && blockIdx.x == 0) atomicAdd(mismatches, bad);
        }
    } else if (mode == 1) {
        if (tid == 0) {
            for (int i = 0; i < count; ++i) tmem_cp_128x256b(tmem + 256 + (i & 15) * 8, a_sw + 2 * (i & 3));
            umma_commit(smem_u32(&s_done[0]));
            if (!mbar_wait(smem_u32(&s_done[0]), 0)) std::printf("wait expired\n");
        }
    } else if (mode == 2) {
        if (tid == 0) {
            for (int i = 0; i < count; ++i) {
                const uint32_t slot = tmem + 256 + (i & 3) * 32;
                for (int kq = 0; kq < 4; ++kq) tmem_cp_128x256b(slot + kq * 8, a_sw + 2 * kq);
                for (int kq = 0; kq < 4; ++kq) umma_tf32_ts(tmem, slot + kq * 8, b_sw + 2 * kq, idesc, 1u);
            }
            umma_commit(smem_u32(&s_done[0]));
            if (!mbar_wait(smem_u32(&s_done[0]), 0)) std::printf("wait expired\n");
        }
    } else {
        if (warp == 0 && lane == 0) {          // copier
            for (int i = 0; i < count; ++i) {
                const int sl = i & 3;
                if (i >= 4 && !mbar_wait(smem_u32(&s_free[sl]), ((i >> 2) - 1) & 1)) { std::printf("copier wait expired\n"); break; }
                tc_fence_after();
                for (int kq = 0; kq < 4; ++kq) tmem_cp_128x256b(tmem + 256 + sl * 32 + kq * 8, a_sw + 2 * kq);
                umma_commit(smem_u32(&s_ready[sl]));
            }
        } else if (warp == 1 && lane == 0) {   // MMA issuer
            for (int i = 0; i < count; ++i) {
                const int sl = i & 3;
                if (!mbar_wait(smem_u32(&s_ready[sl]), (i >> 2) & 1)) { std::printf("issuer wait expired\n"); break; }
                tc_fence_after();
                for (int kq = 0; kq < 4; ++kq) umma_tf32_ts(tmem, tmem + 256 + sl * 32 + kq * 8, b_sw + 2 * kq, idesc, 1u);
                umma_commit(smem_u32(&s_free[sl]));
            }
            umma_commit(smem_u32(&s_done[0]));
            if (!mbar_wait(smem_u32(&s_done[0]), 0)) std::printf("wait expired\n");
        }
    }
    __syncthreads();
    if (tid == 0) cycles[blockIdx.x] = clock64() - t0;
    tc_fence_before();
    __syncthreads();
    if (warp == 7) tmem_dealloc(tmem, 512);
}

// The main loop of a pipelined kernel without its loads: one thread issues `group` SS MMAs 128 x 256 x 8 per ring stage
// (four stages of 48 KB: 16 KB of A, 32 KB of B), then a tcgen05.commit to the stage's barrier; with `wait` it first tests
// another stage's barrier (non-blocking), as an issuer does before it reads a stage.
__global__ void __launch_bounds__(256, 1) k_mma_loop(int stages_total, int group, int wait, long long* cycles)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t s_tmem;
    __shared__ uint64_t s_done, s_ring[4];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int tid = threadIdx.x, warp = tid >> 5;
    for (int i = tid; i < 4 * 12288; i += blockDim.x) reinterpret_cast<uint32_t*>(smem_raw)[i] = 0;
    if (warp == 7) tmem_alloc(smem_u32(&s_tmem), 512);
    if (tid == 0) {
        mbar_init(smem_u32(&s_done), 1);
        for (int i = 0; i < 4; ++i) mbar_init(smem_u32(&s_ring[i]), 1);
        mbar_fence_init();
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    const long long t0 = clock64();
    if (tid == 0) {
        const uint32_t idesc = umma_idesc_tf32(128, 256);
        uint32_t sink = 0;
        // wait = 2: the commits of two stages are issued together after the second stage's MMAs
        for (int st = 0; st < stages_total; ++st) {
            const uint32_t stage = base + (st & 3) * 49152;
            if (wait) sink += mbar_test_wait(smem_u32(&s_ring[(st + 2) & 3]), (st >> 2) & 1) ? 1u : 0u;
            const uint64_t adesc = umma_desc_k_sw128(stage, 1024), bdesc = umma_desc_k_sw128(stage + 16384, 1024);
            for (int i = 0; i < group; ++i) umma_tf32_ss(tmem, adesc + 2 * (i & 3), bdesc + 2 * (i & 3), idesc, 1u);
            if (wait != 2) {
                umma_commit(smem_u32(&s_ring[st & 3]));
            } else if (st & 1) {
                umma_commit(smem_u32(&s_ring[(st - 1) & 3]));
                umma_commit(smem_u32(&s_ring[st & 3]));
            }
        }
        umma_commit(smem_u32(&s_done));
        if (!mbar_wait(smem_u32(&s_done), 0)) std::printf("wait expired\n");
        if (sink == 0xFFFFFFFFu) std::printf("%u\n", sink);
    }
    __syncthreads();
    if (tid == 0) cycles[blockIdx.x] = clock64() - t0;
    tc_fence_before();
    __syncthreads();
    if (warp == 7) tmem_dealloc(tmem, 512);
}

// One buffer pair read over and over: does the placement of the two operands in shared memory matter?  A (16 KB) at
// `a_off`, B (32 KB) at `b_off` from a 1024-byte-aligned base; `group` MMAs cycle over the four K-steps of the tile.
__global__ void __launch_bounds__(256, 1) k_mma_place(int count, uint32_t a_off, uint32_t b_off, int ksteps, long long* cycles)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t s_tmem;
    __shared__ uint64_t s_done;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int tid = threadIdx.x, warp = tid >> 5;
    for (int i = tid; i < 49152; i += blockDim.x) reinterpret_cast<uint32_t*>(smem_raw)[i] = 0;
    if (warp == 7) tmem_alloc(smem_u32(&s_tmem), 512);
    if (tid == 0) { mbar_init(smem_u32(&s_done), 1); mbar_fence_init(); }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    const long long t0 = clock64();
    if (tid == 0) {
        const uint32_t idesc = umma_idesc_tf32(128, 256);
        const uint64_t adesc = umma_desc_k_sw128(base + a_off, 1024), bdesc = umma_desc_k_sw128(base + b_off, 1024);
        for (int i = 0; i < count; ++i) {
            const int kq = ksteps == 4 ? (i & 3) : 0;
            umma_tf32_ss(tmem, adesc + 2 * kq, bdesc + 2 * kq, idesc, 1u);
        }
        umma_commit(smem_u32(&s_done));
        if (!mbar_wait(smem_u32(&s_done), 0)) std::printf("wait expired\n");
    }
    __syncthreads();
    if (tid == 0) cycles[blockIdx.x] = clock64() - t0;
    tc_fence_before();
    __syncthreads();
    if (warp == 7) tmem_dealloc(tmem, 512);
}

// MODE 0: one 32 KB bulk copy per stage; 1: one tiled TMA load of 128 rows x 128 bytes (16 KB) per stage; 2: both (48 KB, the
// expanded-operand kernel's stage).  One thread keeps four stages in flight; nothing consumes the data.
__global__ void __launch_bounds__(128, 1) k_intake(int mode, int stages_total, const float* src, const __grid_constant__ CUtensorMap tm,
                                                  long long* cycles)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_full[4];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    if (threadIdx.x == 0) {
        for (int i = 0; i < 4; ++i) mbar_init(smem_u32(&s_full[i]), 1);
        mbar_fence_init();
    }
    __syncthreads();
    const long long t0 = clock64();
    if (threadIdx.x == 0) {
        const uint32_t tx = mode == 0 ? 32768u : mode == 1 ? 16384u : 49152u;
        const float* mine = src + static_cast<size_t>(blockIdx.x) * 262144;       // 1 MB window per SM
        for (int st = 0; st < stages_total + 4; ++st) {
            const int sl = st & 3;
            if (st >= 4 && !mbar_wait(smem_u32(&s_full[sl]), ((st >> 2) - 1) & 1)) { std::printf("wait expired\n"); break; }
            if (st < stages_total) {
                const uint32_t dst = base + sl * 49152, bar = smem_u32(&s_full[sl]);
                mbar_arrive_expect_tx(bar, tx);
                const int piece = st & 7;                                        // 8 pieces of 64 KB: 512 KB per SM, 74 MB in all (fits the L2)
                if (mode != 1) bulk_load_1d(dst + 16384, mine + piece * 16384, 32768, bar);
                if (mode != 0) tma_load_2d(dst, &tm, bar, (st & 7) * 32, static_cast<int>(blockIdx.x) * 1024 + (piece & 7) * 128);
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) cycles[blockIdx.x] = clock64() - t0;
}

template <typename F>
float best_ms(F f)
{
    cudaEvent_t a, b;
    CK(cudaEventCreate(&a));
    CK(cudaEventCreate(&b));
    f();
    CK(cudaDeviceSynchronize());
    float best = 1e9f;
    for (int i = 0; i < 3; ++i) {
        CK(cudaEventRecord(a));
        f();
        CK(cudaEventRecord(b));
        CK(cudaEventSynchronize(b));
        float ms;
        CK(cudaEventElapsedTime(&ms, a, b));
        best = ms < best ? ms : best;
    }
    return best;
}

int main()
{
    int sms = 0;
    CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0));
    long long* cyc;
    CK(cudaMalloc(&cyc, sms * sizeof(long long)));
    const size_t smem = 100 * 1024;
    CK(cudaFuncSetAttribute(k_select<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    CK(cudaFuncSetAttribute(k_select<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    CK(cudaFuncSetAttribute(k_select<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    CK(cudaFuncSetAttribute(k_mma, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    long long h = 0;
    const char* mode_name[3] = {"copy", "word masks", "byte masks"};
    const int iters = 4000;
    for (int warps : {8, 16}) {
        for (int g : {1, 2, 4}) {
            for (int mode = 0; mode < 3; ++mode) {
                auto run = [&] {
                    if (mode == 0) k_select<0><<<sms, 512, smem>>>(iters, g, warps, cyc);
                    if (mode == 1) k_select<1><<<sms, 512, smem>>>(iters, g, warps, cyc);
                    if (mode == 2) k_select<2><<<sms, 512, smem>>>(iters, g, warps, cyc);
                };
                const float ms = best_ms(run);
                CK(cudaMemcpy(&h, cyc, sizeof(h), cudaMemcpyDeviceToHost));
                const double chunks = static_cast<double>(iters) * (warps / 8);
                std::printf("select  %-10s tiles=%d warps=%2d : %6.0f cycles per chunk of 128 rows x 64 source columns (%.1f ns)\n",
                            mode_name[mode], g, warps, static_cast<double>(h) / chunks, ms * 1e6 / chunks);
            }
        }
    }
    const char* names[12] = {"TS", "SS", "", "SS plain A", "TS plain B", "SS plain B", "", "SS plain A, B",
                             "TS atom B", "SS atom B", "", "SS plain A, atom B"};
    for (int ss : {0, 4, 8, 1, 3, 5, 7, 9, 11}) {   // bit 0: A from shared memory, bit 1: A unswizzled, bit 2: B unswizzled
        for (int n : {64, 128, 256}) {
            for (int issuers : {1, 2, 4}) {
                if (256 / issuers < n) continue;
                const int count = 8192;
                const float ms = best_ms([&] { k_mma<<<sms, 256, smem>>>(count, n, issuers, ss, cyc); });
                CK(cudaMemcpy(&h, cyc, sizeof(h), cudaMemcpyDeviceToHost));
                const double total = static_cast<double>(count) * issuers;
                std::printf("mma     %s N=%3d issuers=%d : %6.1f cycles per MMA, %6.1f ns, %5.0f TFLOP/s over %d SMs\n", names[ss], n,
                            issuers, static_cast<double>(h) / total, ms * 1e6 / total,
                            sms * total * 128.0 * n * 8 * 2 / (ms * 1e-3) / 1e12, sms);
            }
        }
    }
    {
        const size_t big = 200 * 1024;
        CK(cudaFuncSetAttribute(k_mma_loop, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(big)));
        for (int group : {4, 8, 16}) {
            for (int wait : {0, 1, 2}) {
                const int total = 8192 / group;
                const float ms = best_ms([&] { k_mma_loop<<<sms, 256, big>>>(total, group, wait, cyc); });
                CK(cudaMemcpy(&h, cyc, sizeof(h), cudaMemcpyDeviceToHost));
                std::printf("loop    SS N=256, %2d MMAs per stage, commit per stage%s : %6.1f cycles per MMA (%.1f ns)\n", group,
                            wait == 2 ? ", barrier test before, commits in pairs" : wait ? ", barrier test before" : "", static_cast<double>(h) / 8192, ms * 1e6 / 8192);
            }
        }
    }
    {
        const size_t big = 200 * 1024;
        CK(cudaFuncSetAttribute(k_mma_place, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(big)));
        const uint32_t offs[][2] = {{32768, 0}, {0, 16384}, {0, 32768}, {49152, 65536}, {0, 49152}, {1024, 32768}, {0, 98304}, {131072, 0}};
        for (const auto& o : offs) {
            for (int ksteps : {4, 1}) {
                const float ms = best_ms([&] { k_mma_place<<<sms, 256, big>>>(8192, o[0], o[1], ksteps, cyc); });
                CK(cudaMemcpy(&h, cyc, sizeof(h), cudaMemcpyDeviceToHost));
                std::printf("place   SS N=256, A at %6u, B at %6u, %s : %6.1f cycles per MMA (%.1f ns)\n", o[0], o[1],
                            ksteps == 4 ? "four K-steps in turn" : "one K-step repeated ", static_cast<double>(h) / 8192, ms * 1e6 / 8192);
            }
        }
    }
    if (nmtm::available()) {
        // a [148 * 1024 rows][256 floats] buffer, of which every SM re-reads 512 KB of its own 1 MB (74 MB in all: L2 hits)
        const size_t rows = static_cast<size_t>(sms) * 1024, cols = 256;
        float* buf;
        CK(cudaMalloc(&buf, rows * cols * sizeof(float)));
        CK(cudaMemset(buf, 0, rows * cols * sizeof(float)));
        alignas(64) CUtensorMap tm;
        const cuuint64_t dims[2] = {cols, rows};
        const cuuint64_t strides[1] = {cols * sizeof(float)};
        const cuuint32_t box[2] = {32, 128}, es[2] = {1, 1};
        if (nmtm::encoders().tiled(&tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, buf, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS) {
            const size_t big = 200 * 1024;
            CK(cudaFuncSetAttribute(k_intake, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(big)));
            const char* what[3] = {"32 KB bulk copy per stage        ", "16 KB tiled load per stage       ", "bulk copy + tiled load (48 KB)   "};
            const double bytes[3] = {32768, 16384, 49152};
            for (int mode = 0; mode < 3; ++mode) {
                const int total = 2048;
                const float ms = best_ms([&] { k_intake<<<sms, 128, big>>>(mode, total, buf, tm, cyc); });
                CK(cudaMemcpy(&h, cyc, sizeof(h), cudaMemcpyDeviceToHost));
                std::printf("intake  %s: %6.1f cycles per stage, %5.1f bytes per cycle and SM, %5.2f TB/s over %d SMs\n", what[mode],
                            static_cast<double>(h) / total, bytes[mode] * total / static_cast<double>(h),
                            sms * bytes[mode] * total / (ms * 1e-3) / 1e12, sms);
            }
        }
        CK(cudaFree(buf));
    }
    {
        CK(cudaFuncSetAttribute(k_cp, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
        int* bad;
        CK(cudaMalloc(&bad, sizeof(int)));
        CK(cudaMemset(bad, 0, sizeof(int)));
        k_cp<<<sms, 256, smem>>>(0, 0, 256, cyc, bad);
        CK(cudaDeviceSynchronize());
        int hb = -1;
        CK(cudaMemcpy(&hb, bad, sizeof(int), cudaMemcpyDeviceToHost));
        std::printf("cp      layout check: %d mismatching elements of 4096 (row -> lane, 8 consecutive floats -> 8 columns)\n", hb);
        const int count = 4096;
        float ms = best_ms([&] { k_cp<<<sms, 256, smem>>>(1, count, 256, cyc, bad); });
        CK(cudaMemcpy(&h, cyc, sizeof(h), cudaMemcpyDeviceToHost));
        std::printf("cp      128x256b copies back to back, one thread : %6.1f cycles per copy (%.1f ns)\n", static_cast<double>(h) / count, ms * 1e6 / count);
        for (int mode : {2, 3}) {
            for (int n : {128, 256}) {
                ms = best_ms([&] { k_cp<<<sms, 256, smem>>>(mode, count, n, cyc, bad); });
                CK(cudaMemcpy(&h, cyc, sizeof(h), cudaMemcpyDeviceToHost));
                std::printf("cp+mma  4 copies + 4 TS MMAs N=%3d per 32-column block, %s : %6.1f cycles per block, %5.0f TFLOP/s over %d SMs\n", n,
                            mode == 2 ? "one thread " : "two threads", static_cast<double>(h) / count,
                            sms * static_cast<double>(count) * 4 * 128.0 * n * 8 * 2 / (ms * 1e-3) / 1e12, sms);
            }
        }
        CK(cudaFree(bad));
    }
    CK(cudaFree(cyc));
    return 0;
}
