// nm_prune_noalloc: the pruning pass for callers that cannot allocate device memory.
//
// Some users of this library run inside a process whose device memory is already spoken for: an
// inference server that hands the whole of HBM to its own pool at start-up, so that a raw
// cudaMalloc from a plug-in either fails or eats into a budget somebody else accounts for; or a
// latency-bound loop in which cudaMalloc / cudaFree are unwelcome because they synchronise the
// device.  nm_prune needs two scratch arrays (the fp64 column scores and the keep flags) and
// gets them from cudaMalloc.  This variant keeps that scratch in a fixed array that is part of
// the library image instead, writes its results into buffers the caller supplies, and calls no
// allocator of any kind.
//
// The price: the array is sized at build time (NM_NOALLOC_MAX_CELLS (tile, column) cells,
// 9 bytes each, about 4.5 MiB) and is resident on every GPU that loads the library until the
// process exits; larger problems are refused.  All calls share the one array, so two calls whose
// kernels may overlap on the GPU (different streams, different host threads) race with each
// other; serialise them.  Every cell a call reads it has written first, so stale contents from an
// earlier call are harmless and nothing needs clearing.
//
// The array's name is only a host-side handle in host code; the device address is looked up once
// per device with cudaGetSymbolAddress while that device is current and cached.  That lookup
// happens on the first call for a device, which should therefore be made outside any stream
// capture.  With lazy module loading that first call is also the moment the CUDA runtime loads the
// module holding the array, i.e. when the 4.5 MiB are actually reserved on the device (and the
// load may synchronise): "allocates nothing" holds from the second call on, so make one warm-up
// call per device at start-up.  The cached address does not survive a cudaDeviceReset.
#include <mutex>

#include "nm_internal.h"

namespace {

constexpr size_t kBytesPerCell = sizeof(double) + 1;
static __device__ __align__(256) unsigned char g_prune_scratch[NM_NOALLOC_MAX_CELLS * kBytesPerCell];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device (looked up once per device).
nm_status_t scratch_for_current_device(unsigned char** out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return nmhost::fail(NM_ERR_CUDA, "nm_prune_noalloc: cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices)
        return nmhost::fail(NM_ERR_UNSUPPORTED, "nm_prune_noalloc: device ordinal %d not supported", dev);
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_prune_scratch);
        if (e != cudaSuccess || !p)
            return nmhost::fail(NM_ERR_CUDA, "nm_prune_noalloc: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        g_scratch_addr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_scratch_addr[dev];
    return NM_OK;
}

// The same three steps as the allocating pruner (Sec. 3.1), restated here so that this entry
// point shares no code path with it: L1 score per (tile, column) in fp64 over ascending rows (a NaN
// sum ranks as +infinity);
// keep a column iff fewer than N columns of its group beat it (greater score, or equal score and
// lower position); place each kept column at N * group + kept-before-it.
__global__ void k_static_score(const float* __restrict__ w, int c_out, int k, int tile_t, double* __restrict__ score)
{
    const int col = blockIdx.x * blockDim.x + threadIdx.x;
    const int r = blockIdx.y;
    if (col >= k) return;
    const int row0 = r * tile_t, row1 = min(row0 + tile_t, c_out);
    double s = 0.0;
    for (int o = row0; o < row1; ++o) s += fabs(static_cast<double>(w[static_cast<size_t>(o) * k + col]));
    score[static_cast<size_t>(r) * k + col] = (s == s) ? s : static_cast<double>(INFINITY);   // NaN ranks as +infinity
}

__global__ void k_static_select(const double* __restrict__ score, int k, int n_keep, int m_group,
                                unsigned char* __restrict__ keep)
{
    const int col = blockIdx.x * blockDim.x + threadIdx.x;
    const int r = blockIdx.y;
    if (col >= k) return;
    const double* s = score + static_cast<size_t>(r) * k;
    const int g0 = (col / m_group) * m_group, g1 = min(g0 + m_group, k);
    const double mine = s[col];
    int beaten_by = 0;
    for (int i = g0; i < g1; ++i) beaten_by += (s[i] > mine) || (s[i] == mine && i < col);
    keep[static_cast<size_t>(r) * k + col] = beaten_by < n_keep ? 1 : 0;
}

__global__ void k_static_place(const unsigned char* __restrict__ keep, int k, int kk, int n_keep, int m_group,
                               uint16_t* __restrict__ indices)
{
    const int col = blockIdx.x * blockDim.x + threadIdx.x;
    const int r = blockIdx.y;
    if (col >= k) return;
    const unsigned char* kp = keep + static_cast<size_t>(r) * k;
    if (!kp[col]) return;
    const int g = col / m_group;
    int pos = g * n_keep;
    for (int i = g * m_group; i < col; ++i) pos += kp[i];
    if (pos >= min(kk, (g + 1) * n_keep)) return;   // never outside the group's slots, whatever the input
    indices[static_cast<size_t>(r) * kk + pos] = static_cast<uint16_t>(col);
}

__global__ void k_static_values(const float* __restrict__ w, const uint16_t* __restrict__ indices, int k, int kk,
                                int tile_t, float* __restrict__ values)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int o = blockIdx.y;
    if (j >= kk) return;
    values[static_cast<size_t>(o) * kk + j] = w[static_cast<size_t>(o) * k + indices[static_cast<size_t>(o / tile_t) * kk + j]];
}

}  // namespace

extern "C" nm_status_t nm_prune_noalloc(const float* w_dense, int c_out, int kh, int kw, int c_in, int n_keep,
                                        int m_group, int tile_t, float* values, uint16_t* indices, void* cuda_stream)
{
    if (!w_dense || !values || !indices)
        return nmhost::fail(NM_ERR_INVALID_ARG, "nm_prune_noalloc: w_dense, values or indices is NULL");
    if (c_out < 1 || kh < 1 || kw < 1 || c_in < 1)
        return nmhost::fail(NM_ERR_INVALID_ARG, "nm_prune_noalloc: c_out, kh, kw, c_in must be >= 1");
    if (n_keep < 1 || m_group < 1 || n_keep > m_group)
        return nmhost::fail(NM_ERR_INVALID_ARG, "nm_prune_noalloc: need 1 <= n_keep <= m_group (got %d:%d)", n_keep, m_group);
    if (tile_t < 1) return nmhost::fail(NM_ERR_INVALID_ARG, "nm_prune_noalloc: tile_t must be >= 1");
    // the limits of nm_prune / nm_weights_import, so that whatever this call produces can be imported
    if (kh > 255 || kw > 255) return nmhost::fail(NM_ERR_UNSUPPORTED, "nm_prune_noalloc: kernel extent above 255");
    if (tile_t > 256) return nmhost::fail(NM_ERR_UNSUPPORTED, "nm_prune_noalloc: tile_t above 256");
    const long long k = static_cast<long long>(kh) * kw * c_in;
    if (k > 65535) return nmhost::fail(NM_ERR_UNSUPPORTED, "nm_prune_noalloc: K = %lld exceeds the uint16 index range", k);
    if (c_out > 65535) return nmhost::fail(NM_ERR_UNSUPPORTED, "nm_prune_noalloc: c_out above 65535");
    const long long n_tiles = (c_out + tile_t - 1) / tile_t;
    const long long cells = n_tiles * k;
    if (cells > static_cast<long long>(NM_NOALLOC_MAX_CELLS))
        return nmhost::fail(NM_ERR_UNSUPPORTED,
                            "nm_prune_noalloc: ceil(c_out / tile_t) * K = %lld cells exceeds the built-in scratch of %d "
                            "cells; use nm_prune, or a wider tile",
                            cells, NM_NOALLOC_MAX_CELLS);
    unsigned char* scratch = nullptr;
    nm_status_t s = scratch_for_current_device(&scratch);
    if (s != NM_OK) return s;
    double* score = reinterpret_cast<double*>(scratch);                       // [n_tiles][k], 256-byte aligned base
    unsigned char* keep = scratch + NM_NOALLOC_MAX_CELLS * sizeof(double);    // [n_tiles][k]

    const int ki = static_cast<int>(k);
    const int full = ki / m_group, tail = ki % m_group;
    const int kk = full * n_keep + (tail < n_keep ? tail : n_keep);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const dim3 blk(128);
    const dim3 grid_cols((ki + 127) / 128, static_cast<unsigned>(n_tiles));
    k_static_score<<<grid_cols, blk, 0, st>>>(w_dense, c_out, ki, tile_t, score);
    k_static_select<<<grid_cols, blk, 0, st>>>(score, ki, n_keep, m_group, keep);
    k_static_place<<<grid_cols, blk, 0, st>>>(keep, ki, kk, n_keep, m_group, indices);
    const dim3 grid_vals((kk + 127) / 128, c_out);
    k_static_values<<<grid_vals, blk, 0, st>>>(w_dense, indices, ki, kk, tile_t, values);
    nmhost::count_launch(4);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return nmhost::fail(NM_ERR_CUDA, "nm_prune_noalloc: launch failed: %s", cudaGetErrorString(e));
    return NM_OK;
}
