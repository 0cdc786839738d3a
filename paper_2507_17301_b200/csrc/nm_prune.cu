// Column-wise N:M pruning at tile level (Sec. 3.1) on the device, and construction of the
// kernel-side copies of the compressed form (Sec. 2.1; inputs W and Idx of Algorithm 1).
//
// Four small kernels, all one thread per (tile, column) or (row, retained column):
//   score    s[r][k]   = sum over the tile's rows of |w[o][k]|, fp64, ascending row order; a sum that
//            is NaN (a NaN weight) counts as +infinity, so that the order below is total
//   select   keep[r][k] = 1 iff fewer than N columns of k's group beat it, where column i beats
//            column k when s[i] > s[k], or s[i] == s[k] and i < k (lower column wins ties)
//   compact  position of each kept column = N * group + number of kept columns before it in its
//            group; writes the index array and the decoded (kh, kw, c) tap table
//   gather   values[o][j] = w[o][idx[j]] (bit copy) and the TF32-rounded, zero-padded copy
// The selection rule is the closed form of "pick the largest N times": both orderings are the
// sort by (score descending, column ascending), so the result is unique and bit-reproducible as
// long as the fp64 sums are formed in the same order everywhere.
#include <cstdio>

#include "nm_internal.h"
#include "nm_ptx.cuh"

namespace {

__global__ void k_score(const float* __restrict__ w, int c_out, int k, int tile_t, double* __restrict__ score)
{
    const int col = blockIdx.x * blockDim.x + threadIdx.x;
    const int r = blockIdx.y;
    if (col >= k) return;
    const int row0 = r * tile_t;
    const int row1 = min(row0 + tile_t, c_out);
    double s = 0.0;
    for (int o = row0; o < row1; ++o) s += fabs(static_cast<double>(w[static_cast<size_t>(o) * k + col]));
    // NaN compares false with everything: such a column would neither beat nor be beaten, and its
    // group would keep more than N columns.  It ranks as +infinity instead (ties by column).
    score[static_cast<size_t>(r) * k + col] = (s == s) ? s : static_cast<double>(INFINITY);
}

__global__ void k_select(const double* __restrict__ score, int k, int n_keep, int m_group,
                         uint8_t* __restrict__ keep)
{
    const int col = blockIdx.x * blockDim.x + threadIdx.x;
    const int r = blockIdx.y;
    if (col >= k) return;
    const double* s = score + static_cast<size_t>(r) * k;
    const int g0 = (col / m_group) * m_group;
    const int g1 = min(g0 + m_group, k);
    const double mine = s[col];
    int beaten_by = 0;
    for (int i = g0; i < g1; ++i) {
        const double si = s[i];
        beaten_by += (si > mine) || (si == mine && i < col);
    }
    keep[static_cast<size_t>(r) * k + col] = beaten_by < n_keep ? 1 : 0;
}

// L1 mass of all columns and of the retained ones: mass[0] += score, mass[1] += score * keep.
__global__ void k_mass(const double* __restrict__ score, const uint8_t* __restrict__ keep, size_t cells,
                       double* __restrict__ mass)
{
    double all = 0.0, kept = 0.0;
    for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < cells;
         i += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const double s = score[i];
        all += s;
        if (keep[i]) kept += s;
    }
    for (int d = 16; d > 0; d >>= 1) {
        all += __shfl_down_sync(0xFFFFFFFFu, all, d);
        kept += __shfl_down_sync(0xFFFFFFFFu, kept, d);
    }
    if ((threadIdx.x & 31) == 0) {
        atomicAdd(mass + 0, all);
        atomicAdd(mass + 1, kept);
    }
}

__global__ void k_compact(const uint8_t* __restrict__ keep, int k, int kk, int kk_pad, int n_keep, int m_group,
                          int c_in, int kw, uint16_t* __restrict__ indices, uint32_t* __restrict__ taps)
{
    const int col = blockIdx.x * blockDim.x + threadIdx.x;
    const int r = blockIdx.y;
    if (col >= k) return;
    const uint8_t* kp = keep + static_cast<size_t>(r) * k;
    if (!kp[col]) return;
    const int g = col / m_group;
    int pos = g * n_keep;  // every earlier group is a full one and kept exactly n_keep
    for (int i = g * m_group; i < col; ++i) pos += kp[i];
    // a group never holds more than N kept columns (the order of the scores is total); the bound
    // makes sure that no input whatsoever can place a column outside its group's slots
    if (pos >= min(kk, (g + 1) * n_keep)) return;
    indices[static_cast<size_t>(r) * kk + pos] = static_cast<uint16_t>(col);
    const int c = col % c_in, tap = col / c_in;
    taps[static_cast<size_t>(r) * kk_pad + pos] =
        (static_cast<uint32_t>(tap / kw) << 24) | (static_cast<uint32_t>(tap % kw) << 16) | static_cast<uint32_t>(c);
}

// From indices alone (import path): tap table.
__global__ void k_taps_from_indices(const uint16_t* __restrict__ indices, int kk, int kk_pad, int c_in, int kw,
                                    uint32_t* __restrict__ taps)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int r = blockIdx.y;
    if (j >= kk) return;
    const int col = indices[static_cast<size_t>(r) * kk + j];
    const int c = col % c_in, tap = col / c_in;
    taps[static_cast<size_t>(r) * kk_pad + j] =
        (static_cast<uint32_t>(tap / kw) << 24) | (static_cast<uint32_t>(tap % kw) << 16) | static_cast<uint32_t>(c);
}

__global__ void k_gather_values(const float* __restrict__ w, const uint16_t* __restrict__ indices, int k, int kk,
                                int kk_pad, int tile_t, float* __restrict__ values, float* __restrict__ wt)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int o = blockIdx.y;
    if (j >= kk_pad) return;
    float v = 0.f;
    if (j < kk) {
        v = w[static_cast<size_t>(o) * k + indices[static_cast<size_t>(o / tile_t) * kk + j]];
        values[static_cast<size_t>(o) * kk + j] = v;
    }
    wt[static_cast<size_t>(o) * kk_pad + j] = nmk::to_tf32(v);
}

// Import path: values already compacted.
__global__ void k_round_values(const float* __restrict__ values, int kk, int kk_pad, float* __restrict__ wt)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int o = blockIdx.y;
    if (j >= kk_pad) return;
    const float v = j < kk ? values[static_cast<size_t>(o) * kk + j] : 0.f;
    wt[static_cast<size_t>(o) * kk_pad + j] = nmk::to_tf32(v);
}

// Slab layout: kept column j of a tile lies in chunk k_j / S at position j - chunk * KC (every
// group before the last is full, so a chunk of G groups holds exactly KC = G * N kept columns).
__global__ void k_build_slab(const float* __restrict__ values, const uint16_t* __restrict__ indices, int kk,
                             int tile_t, int s_cols, int kc, int chunks, float* __restrict__ wt2,
                             uint8_t* __restrict__ rel2)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int o = blockIdx.y;
    if (j >= kk) return;
    const int r = o / tile_t;
    const int col = indices[static_cast<size_t>(r) * kk + j];
    const int chunk = col / s_cols;
    const int jj = j - chunk * kc;
    const size_t pitch = static_cast<size_t>(chunks) * 32;
    wt2[static_cast<size_t>(o) * pitch + chunk * 32 + jj] = nmk::to_tf32(values[static_cast<size_t>(o) * kk + j]);
    if (o == r * tile_t) rel2[static_cast<size_t>(r) * pitch + chunk * 32 + jj] = static_cast<uint8_t>(col - chunk * s_cols);
}

// Expanded layout: element (o, k) = TF32(values[o][j]) where k = indices[o / T][j], zero elsewhere,
// stored as the shared-memory image the tensor core reads: blocks of 32 columns, inside a block
// one 128-byte row per output channel whose 16-byte pieces are XOR-ed with (o % 8) (the 128-byte
// swizzle), so that any run of channels starting at a multiple of 8 is one contiguous bulk copy.
__global__ void k_expand(const float* __restrict__ values, const uint16_t* __restrict__ indices, int rows, int kk,
                         int tile_t, float* __restrict__ wx)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int o = blockIdx.y;
    if (j >= kk) return;
    const int col = indices[static_cast<size_t>(o / tile_t) * kk + j];
    const int blk = col >> 5, kc = col & 31;
    wx[(static_cast<size_t>(blk) * rows + o) * 32 + ((((kc >> 2) ^ (o & 7)) << 2) | (kc & 3))] =
        nmk::to_tf32(values[static_cast<size_t>(o) * kk + j]);
}

// Import path: every index row must be strictly ascending and below k, and hold the N:M structure
// the kernels rely on: retained column j lies in group j / N (a tail group of m' < M columns keeps
// min(N, m'), which the same quotient covers).
__global__ void k_check_indices(const uint16_t* __restrict__ indices, int kk, int k, int n_keep, int m_group,
                                int* __restrict__ bad)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int r = blockIdx.y;
    if (j >= kk) return;
    const int v = indices[static_cast<size_t>(r) * kk + j];
    if (v >= k || (j > 0 && indices[static_cast<size_t>(r) * kk + j - 1] >= v) || v / m_group != j / n_keep)
        atomicExch(bad, 1);
}

#define NM_CUDA_TRY(call)                                                                                   \
    do {                                                                                                    \
        cudaError_t e__ = (call);                                                                           \
        if (e__ != cudaSuccess) {                                                                           \
            st_out = nmhost::fail(NM_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e__));            \
            goto done;                                                                                      \
        }                                                                                                   \
    } while (0)

}  // namespace

namespace nmhost {

nm_status_t prune_on_device(const float* w_dense, nm_weights* h, cudaStream_t st)
{
    nm_status_t st_out = NM_OK;
    double* score = nullptr;
    double* mass = nullptr;
    uint8_t* keep = nullptr;
    const size_t cells = static_cast<size_t>(h->n_tiles) * h->k;
    const dim3 blk(128);
    const dim3 grid_cols((h->k + 127) / 128, h->n_tiles);
    const dim3 grid_vals((h->kk_pad + 127) / 128, h->c_out);

    if (cudaMalloc(&score, cells * sizeof(double)) != cudaSuccess || cudaMalloc(&keep, cells) != cudaSuccess) {
        (void)cudaGetLastError();
        st_out = fail(NM_ERR_ALLOC, "nm_prune: cannot allocate %zu bytes of scratch", cells * 9);
        goto done;
    }
    NM_CUDA_TRY(cudaMemsetAsync(h->taps, 0xFF, static_cast<size_t>(h->n_tiles) * h->kk_pad * sizeof(uint32_t), st));
    k_score<<<grid_cols, blk, 0, st>>>(w_dense, h->c_out, h->k, h->tile_t, score);
    k_select<<<grid_cols, blk, 0, st>>>(score, h->k, h->n_keep, h->m_group, keep);
    k_compact<<<grid_cols, blk, 0, st>>>(keep, h->k, h->kk, h->kk_pad, h->n_keep, h->m_group, h->c_in, h->kw,
                                         h->indices, h->taps);
    k_gather_values<<<grid_vals, blk, 0, st>>>(w_dense, h->indices, h->k, h->kk, h->kk_pad, h->tile_t, h->values,
                                               h->wt);
    count_launch(4);
    NM_CUDA_TRY(cudaGetLastError());
    {
        // retained share of the L1 mass (the accuracy proxy reported next to a tile width)
        double host_mass[2] = {0.0, 0.0};
        NM_CUDA_TRY(cudaMalloc(&mass, 2 * sizeof(double)));
        NM_CUDA_TRY(cudaMemsetAsync(mass, 0, 2 * sizeof(double), st));
        size_t blocks = (cells + 255) / 256;
        if (blocks > 1024) blocks = 1024;
        k_mass<<<static_cast<unsigned>(blocks), 256, 0, st>>>(score, keep, cells, mass);
        count_launch(1);
        NM_CUDA_TRY(cudaGetLastError());
        NM_CUDA_TRY(cudaMemcpyAsync(host_mass, mass, sizeof(host_mass), cudaMemcpyDeviceToHost, st));
        NM_CUDA_TRY(cudaStreamSynchronize(st));  // also: the scratch is freed below
        h->l1_total = host_mass[0];
        h->l1_kept = host_mass[1];
    }
done:
    cudaFree(score);
    cudaFree(keep);
    cudaFree(mass);
    return st_out;
}

nm_status_t build_slab_layout(nm_weights* h, cudaStream_t st)
{
    h->v2_ok = 0;
    // keep-all is the 1:1 pattern; otherwise the chunk is the largest whole number of groups
    // whose kept columns number a multiple of 8 up to 32 and whose source columns number <= 64
    const int n = h->n_keep == h->m_group ? 1 : h->n_keep;
    const int m = h->n_keep == h->m_group ? 1 : h->m_group;
    int g = 0;
    for (int cand = 32 / n; cand >= 1; --cand)
        if ((cand * n) % 8 == 0 && cand * m <= 64) { g = cand; break; }
    if (g == 0 || h->kk == 0) return NM_OK;
    h->v2_g = g; h->v2_kc = g * n; h->v2_s = g * m;
    h->v2_chunks = (h->k + h->v2_s - 1) / h->v2_s;
    const size_t pitch = static_cast<size_t>(h->v2_chunks) * 32;
    if (cudaMalloc(&h->wt2, static_cast<size_t>(h->c_out) * pitch * sizeof(float)) != cudaSuccess ||
        cudaMalloc(&h->rel2, static_cast<size_t>(h->n_tiles) * pitch) != cudaSuccess) {
        (void)cudaGetLastError();
        return fail(NM_ERR_ALLOC, "cannot allocate the slab-layout weights");
    }
    cudaError_t e = cudaMemsetAsync(h->wt2, 0, static_cast<size_t>(h->c_out) * pitch * sizeof(float), st);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->rel2, 0, static_cast<size_t>(h->n_tiles) * pitch, st);
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "slab layout memset: %s", cudaGetErrorString(e));
    const dim3 grid((h->kk + 127) / 128, h->c_out);
    k_build_slab<<<grid, 128, 0, st>>>(h->values, h->indices, h->kk, h->tile_t, h->v2_s, h->v2_kc, h->v2_chunks,
                                       h->wt2, h->rel2);
    count_launch(1);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "slab layout kernel: %s", cudaGetErrorString(e));
    h->v2_ok = 1;
    return NM_OK;
}

nm_status_t build_expanded_layout(nm_weights* h, cudaStream_t st)
{
    h->wx = nullptr;
    h->wx_rows = 0;
    // only shapes the kernels that read it take: output channels in whole float4s (rows are padded with
    // zeros to blocks of 32), and either whole 32-column slabs (expanded-operand kernel) or a short
    // reduction axis (row-run kernel, pointwise layers)
    if (h->c_out % 4 != 0 || h->kk == 0 || (h->c_in % 32 != 0 && h->k > 512)) return NM_OK;
    h->wx_rows = (h->c_out + 31) / 32 * 32;
    const size_t bytes = static_cast<size_t>((h->k + 31) / 32) * h->wx_rows * 32 * sizeof(float);
    if (cudaMalloc(&h->wx, bytes) != cudaSuccess) {
        (void)cudaGetLastError();
        h->wx = nullptr;
        return fail(NM_ERR_ALLOC, "cannot allocate the expanded weights (%zu bytes)", bytes);
    }
    cudaError_t e = cudaMemsetAsync(h->wx, 0, bytes, st);
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "expanded layout memset: %s", cudaGetErrorString(e));
    const dim3 grid((h->kk + 127) / 128, h->c_out);
    k_expand<<<grid, 128, 0, st>>>(h->values, h->indices, h->wx_rows, h->kk, h->tile_t, h->wx);
    count_launch(1);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(NM_ERR_CUDA, "expanded layout kernel: %s", cudaGetErrorString(e));
    return NM_OK;
}

nm_status_t build_from_compressed(const float* values, const uint16_t* indices, nm_weights* h, cudaStream_t st)
{
    nm_status_t st_out = NM_OK;
    int bad = 0;
    const dim3 blk(128);
    const dim3 grid_idx((h->kk + 127) / 128, h->n_tiles);
    const dim3 grid_vals((h->kk_pad + 127) / 128, h->c_out);
    NM_CUDA_TRY(cudaMemcpyAsync(h->values, values, static_cast<size_t>(h->c_out) * h->kk * sizeof(float),
                                cudaMemcpyDeviceToDevice, st));
    NM_CUDA_TRY(cudaMemcpyAsync(h->indices, indices, static_cast<size_t>(h->n_tiles) * h->kk * sizeof(uint16_t),
                                cudaMemcpyDeviceToDevice, st));
    NM_CUDA_TRY(cudaMemsetAsync(h->taps, 0xFF, static_cast<size_t>(h->n_tiles) * h->kk_pad * sizeof(uint32_t), st));
    NM_CUDA_TRY(cudaMemsetAsync(h->status + 3, 0, sizeof(int), st));
    if (h->kk > 0) {
        k_check_indices<<<grid_idx, blk, 0, st>>>(h->indices, h->kk, h->k, h->n_keep, h->m_group, h->status + 3);
        k_taps_from_indices<<<grid_idx, blk, 0, st>>>(h->indices, h->kk, h->kk_pad, h->c_in, h->kw, h->taps);
        count_launch(2);
    }
    k_round_values<<<grid_vals, blk, 0, st>>>(h->values, h->kk, h->kk_pad, h->wt);
    count_launch(1);
    NM_CUDA_TRY(cudaGetLastError());
    NM_CUDA_TRY(cudaMemcpyAsync(&bad, h->status + 3, sizeof(int), cudaMemcpyDeviceToHost, st));
    NM_CUDA_TRY(cudaStreamSynchronize(st));
    if (bad) st_out = fail(NM_ERR_INVALID_ARG, "nm_weights_import: an index row is not strictly ascending below K, or does not hold N columns per group of M");
done:
    return st_out;
}

}  // namespace nmhost
