// Global rank selection across layers (Algorithm 1 of the paper, between the block scores and the
// pruning itself; Sec. III-C "Pruning Algorithm"):
//   K-R1  per layer: sort every row of the block-score grid increasingly and add the o-th smallest
//         score of every row tile into the rank-column sum c_o (128-bit: sums can pass 2^64);
//   K-R2  global order of all c_o of all layers by their real value c * 2^e (e = the layer's score
//         scale), ties to the lower layer, then the lower rank position; a rank position is pruned
//         while the weight of everything before it in that order is still below the target;
//   K-R3  kkeep = nblk - pruned rank positions, per layer.
// The order is not materialised: for every candidate one warp adds up the weight of the candidates that
// precede it (all pairs, tiled through shared memory).  The lists are small (one entry per rank position per
// layer: hundreds to a few thousand for the networks of Sec. IV), so the quadratic pass costs
// microseconds, is exact, and has no data-dependent control flow.
#include <climits>
#include <cmath>
#include <memory>
#include <new>

#include "crisp_internal.h"

namespace crisp {
namespace {

constexpr int kRankThreads = 256;
constexpr int kRankMaxBlocks = 4096;                 // k-blocks per row tile (one shared-memory row)

struct RankLayer {                                   // device copy of one crisp_rank_layer_t
    const unsigned long long *scores;
    const uint32_t *max_key;
    long long block_elems;
    int nrt, nblk, candidates, entry_off;
};

// One candidate rank position.  Its value c * 2^e is stored normalised, so that the global order is a
// plain lexicographic comparison: `top` = position of the leading bit of the real value (bit length of
// c plus e; INT_MIN for c = 0) and the 128-bit c shifted left until its leading bit is bit 127.  Two
// non-zero values with the same `top` compare like their left-aligned digits; nothing is rounded.
struct RankEntry {
    unsigned long long mhi, mlo;
    unsigned long long weight;                       // weights removed by pruning this rank position
    int top, layer, o, pad;
};

// Exponent of a positive finite float given by its bits (ilogb), denormals included; 0 for zero.
__device__ __forceinline__ int float_bits_exponent(uint32_t key) {
    if (!key) return 0;
    const int e = (int)(key >> 23);
    return e ? e - 127 : (31 - __clz(key)) - 149;
}

__device__ __forceinline__ RankEntry make_entry(unsigned long long lo, unsigned long long hi, int e, int layer, int o,
                                                unsigned long long weight) {
    RankEntry out;
    out.weight = weight; out.layer = layer; out.o = o; out.pad = 0;
    if ((lo | hi) == 0) { out.top = INT_MIN; out.mhi = out.mlo = 0; return out; }
    const int bits = hi ? 128 - __clzll(hi) : 64 - __clzll(lo);
    const int sh = 128 - bits;                       // 0..127
    if (sh >= 64) { out.mhi = lo << (sh - 64); out.mlo = 0; }
    else if (sh) { out.mhi = (hi << sh) | (lo >> (64 - sh)); out.mlo = lo << sh; }
    else { out.mhi = hi; out.mlo = lo; }
    out.top = bits + e;
    return out;
}

// a strictly before b in the global order: value, then layer, then rank position (branch-free, so that
// the loads of consecutive comparisons overlap)
__device__ __forceinline__ bool entry_before(const RankEntry &a, const RankEntry &b) {
    const bool by_pos = (a.layer < b.layer) | ((a.layer == b.layer) & (a.o < b.o));
    const bool by_lo = (a.mlo < b.mlo) | ((a.mlo == b.mlo) & by_pos);
    const bool by_hi = (a.mhi < b.mhi) | ((a.mhi == b.mhi) & by_lo);
    return (a.top < b.top) | ((a.top == b.top) & by_hi);
}

// Increasing bitonic sort of `padded` (a power of two) values in shared memory by `nthreads` threads that
// call it together; `sync` separates the exchange steps (the warp or the whole CTA).
template <typename Sync>
__device__ __forceinline__ void bitonic_sort(unsigned long long *v, int padded, int tid, int nthreads, Sync sync) {
    for (int k = 2; k <= padded; k <<= 1)
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = tid; i < padded; i += nthreads) {
                const int partner = i ^ j;
                if (partner > i) {
                    const unsigned long long a = v[i], b = v[partner];
                    if ((a > b) == ((i & k) == 0)) { v[i] = b; v[partner] = a; }
                }
            }
            sync();
        }
}

constexpr int kWarpRowMax = 512;                     // rows up to this (padded) length are sorted by one warp each

// K-R1.  One CTA per layer.  Rows of up to 512 blocks: each of the 8 warps sorts its own rows in its
// slice of shared memory and keeps its partial rank sums in registers (lane t owns positions t, t + 32,
// ...); the warps' sums are then added up in shared memory.  Longer rows: the whole CTA sorts one row
// at a time (thread t owns positions t, t + 256, ...).
__global__ void __launch_bounds__(kRankThreads)
rank_columns_kernel(const RankLayer *__restrict__ layers, RankEntry *__restrict__ entries) {
    __shared__ unsigned long long s_row[kRankMaxBlocks];
    __shared__ unsigned long long s_lo[kWarpRowMax], s_hi[kWarpRowMax];
    const RankLayer L = layers[blockIdx.x];
    int padded = 1;
    while (padded < L.nblk) padded <<= 1;
    const int e = float_bits_exponent(*L.max_key);
    const unsigned long long weight = (unsigned long long)L.nrt * (unsigned long long)L.block_elems;
    constexpr int kPerThread = kRankMaxBlocks / kRankThreads;        // = kWarpRowMax / 32
    unsigned long long lo[kPerThread], hi[kPerThread];
#pragma unroll
    for (int i = 0; i < kPerThread; ++i) lo[i] = hi[i] = 0;

    if (padded <= kWarpRowMax) {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        unsigned long long *mine = s_row + warp * kWarpRowMax;
        for (int rt = warp; rt < L.nrt; rt += kRankThreads / 32) {
            const unsigned long long *row = L.scores + (long long)rt * L.nblk;
            for (int i = lane; i < padded; i += 32) mine[i] = i < L.nblk ? row[i] : ~0ull;
            __syncwarp();
            bitonic_sort(mine, padded, lane, 32, [] { __syncwarp(); });
#pragma unroll
            for (int i = 0; i < kPerThread; ++i) {
                const int o = lane + i * 32;
                if (o < L.nblk) {
                    const unsigned long long v = mine[o];
                    lo[i] += v;
                    hi[i] += lo[i] < v;              // carry
                }
            }
            __syncwarp();
        }
        for (int i = threadIdx.x; i < kWarpRowMax; i += kRankThreads) s_lo[i] = s_hi[i] = 0;
        __syncthreads();
        for (int w = 0; w < kRankThreads / 32; ++w) {
            if (warp == w) {
#pragma unroll
                for (int i = 0; i < kPerThread; ++i) {
                    const int o = lane + i * 32;
                    if (o < L.nblk) {
                        const unsigned long long before = s_lo[o];
                        s_lo[o] = before + lo[i];
                        s_hi[o] += hi[i] + (s_lo[o] < before);
                    }
                }
            }
            __syncthreads();
        }
        for (int o = threadIdx.x; o < L.candidates; o += kRankThreads)
            entries[L.entry_off + o] = make_entry(s_lo[o], s_hi[o], e, blockIdx.x, o, weight);
        return;
    }

    for (int rt = 0; rt < L.nrt; ++rt) {
        const unsigned long long *row = L.scores + (long long)rt * L.nblk;
        for (int i = threadIdx.x; i < padded; i += kRankThreads) s_row[i] = i < L.nblk ? row[i] : ~0ull;
        __syncthreads();
        bitonic_sort(s_row, padded, threadIdx.x, kRankThreads, [] { __syncthreads(); });
#pragma unroll
        for (int i = 0; i < kPerThread; ++i) {
            const int o = threadIdx.x + i * kRankThreads;
            if (o < L.nblk) {
                const unsigned long long v = s_row[o];
                lo[i] += v;
                hi[i] += lo[i] < v;                  // carry
            }
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < kPerThread; ++i) {
        const int o = threadIdx.x + i * kRankThreads;
        if (o < L.candidates) entries[L.entry_off + o] = make_entry(lo[i], hi[i], e, blockIdx.x, o, weight);
    }
}

// K-R2.  One warp per candidate i: the lanes share out the other candidates (tiled through shared memory),
// each adds up the weight of those that precede i in the global order, and a shuffle reduction gives the
// weight pruned before i.
__global__ void __launch_bounds__(kRankThreads)
global_select_kernel(const RankEntry *__restrict__ entries, int n, unsigned long long target,
                     int32_t *__restrict__ pruned) {
    __shared__ RankEntry s_tile[kRankThreads];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x * (kRankThreads / 32) + warp;
    RankEntry mine;
    mine.top = 0; mine.mhi = mine.mlo = 0; mine.layer = mine.o = 0;
    if (i < n) mine = entries[i];
    unsigned long long before = 0;
    for (int base = 0; base < n; base += kRankThreads) {
        if (base + (int)threadIdx.x < n) s_tile[threadIdx.x] = entries[base + threadIdx.x];
        __syncthreads();
        const int cnt = min(kRankThreads, n - base);
#pragma unroll 4
        for (int j = lane; j < cnt; j += 32) {
            const RankEntry other = s_tile[j];
            before += entry_before(other, mine) ? other.weight : 0ull;
        }
        __syncthreads();
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) before += __shfl_xor_sync(0xFFFFFFFFu, before, d);
    if (i < n && lane == 0 && before < target) atomicAdd(&pruned[mine.layer], 1);
}

// K-R3.
__global__ void kept_count_kernel(const RankLayer *__restrict__ layers, const int32_t *__restrict__ pruned,
                                  int n_layers, int32_t *__restrict__ kkeep) {
    const int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l < n_layers) kkeep[l] = layers[l].nblk - pruned[l];
}

struct RankLayout {
    size_t table_off, pruned_off, entries_off, total;
    long long n_entries;
};

crisp_status_t rank_layout(int32_t n_layers, const crisp_rank_layer_t *layers, RankLayout *out) {
    if (n_layers <= 0 || !layers) return CRISP_INVALID_ARG;
    long long n = 0;
    for (int l = 0; l < n_layers; ++l) {
        const crisp_rank_layer_t &L = layers[l];
        if (L.nrt <= 0 || L.nblk <= 0 || L.block_elems <= 0) return CRISP_BAD_SHAPE;
        if (L.min_keep < 0 || L.min_keep > L.nblk) return CRISP_INVALID_ARG;
        if (L.nblk > kRankMaxBlocks) return CRISP_UNSUPPORTED;
        n += L.nblk - L.min_keep;
    }
    if (n > 0x7FFFFFFF) return CRISP_UNSUPPORTED;
    out->n_entries = n;
    out->table_off = 0;
    out->pruned_off = align_up((size_t)n_layers * sizeof(RankLayer));
    out->entries_off = out->pruned_off + align_up((size_t)n_layers * sizeof(int32_t));
    out->total = out->entries_off + align_up((size_t)(n > 0 ? n : 1) * sizeof(RankEntry));
    return CRISP_OK;
}

}  // namespace
}  // namespace crisp

using crisp::RankEntry;
using crisp::RankLayer;
using crisp::RankLayout;

extern "C" {

CRISP_API crisp_status_t crisp_global_rank_sizes(int32_t n_layers, const crisp_rank_layer_t *layers,
                                                 size_t *workspace_bytes) {
    if (!workspace_bytes) return CRISP_INVALID_ARG;
    RankLayout lay;
    crisp_status_t s = crisp::rank_layout(n_layers, layers, &lay);
    if (s != CRISP_OK) return s;
    *workspace_bytes = lay.total;
    return CRISP_OK;
}

CRISP_API crisp_status_t crisp_global_rank(int32_t n_layers, const crisp_rank_layer_t *layers, double prune_fraction,
                                           void *d_workspace, int32_t *d_kkeep, void *stream) {
    RankLayout lay;
    crisp_status_t s = crisp::rank_layout(n_layers, layers, &lay);
    if (s != CRISP_OK) return s;
    if (!d_workspace || !d_kkeep || reinterpret_cast<uintptr_t>(d_workspace) % crisp::kAlign) return CRISP_INVALID_ARG;
    if (!(prune_fraction >= 0.0 && prune_fraction <= 1.0)) return CRISP_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    // The layer table is staged from a temporary host array, so the call cannot be part of a stream capture
    // (the graph would keep a pointer to memory that is gone when it is replayed).
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) return CRISP_CUDA_ERROR;
    if (cap != cudaStreamCaptureStatusNone) return CRISP_UNSUPPORTED;
    std::unique_ptr<RankLayer[]> table(new (std::nothrow) RankLayer[(size_t)n_layers]);
    if (!table) return CRISP_CUDA_ERROR;
    double total = 0.0;
    int off = 0;
    for (int l = 0; l < n_layers; ++l) {
        const crisp_rank_layer_t &L = layers[l];
        if (!L.d_scores || !L.d_max_key) return CRISP_INVALID_ARG;
        table[l].scores = L.d_scores;
        table[l].max_key = L.d_max_key;
        table[l].block_elems = L.block_elems;
        table[l].nrt = L.nrt; table[l].nblk = L.nblk;
        table[l].candidates = L.nblk - L.min_keep;
        table[l].entry_off = off;
        off += table[l].candidates;
        total += (double)L.nrt * (double)L.nblk * (double)L.block_elems;
    }
    const unsigned long long target = (unsigned long long)floor(prune_fraction * total + 0.5);
    uint8_t *ws = reinterpret_cast<uint8_t *>(d_workspace);
    RankLayer *d_table = reinterpret_cast<RankLayer *>(ws + lay.table_off);
    int32_t *d_pruned = reinterpret_cast<int32_t *>(ws + lay.pruned_off);
    RankEntry *d_entries = reinterpret_cast<RankEntry *>(ws + lay.entries_off);
    // the table is read from pageable host memory: the call returns once it has been staged
    if (cudaMemcpyAsync(d_table, table.get(), (size_t)n_layers * sizeof(RankLayer), cudaMemcpyHostToDevice, st) != cudaSuccess)
        return CRISP_CUDA_ERROR;
    if (cudaMemsetAsync(d_pruned, 0, (size_t)n_layers * sizeof(int32_t), st) != cudaSuccess) return CRISP_CUDA_ERROR;
    crisp::rank_columns_kernel<<<n_layers, crisp::kRankThreads, 0, st>>>(d_table, d_entries);
    const int n = (int)lay.n_entries;
    if (n > 0)
        crisp::global_select_kernel<<<(n + crisp::kRankThreads / 32 - 1) / (crisp::kRankThreads / 32), crisp::kRankThreads, 0, st>>>(
            d_entries, n, target, d_pruned);
    crisp::kept_count_kernel<<<(n_layers + 255) / 256, 256, 0, st>>>(d_table, d_pruned, n_layers, d_kkeep);
    return cudaGetLastError() == cudaSuccess ? CRISP_OK : CRISP_CUDA_ERROR;
}

CRISP_API crisp_status_t crisp_mask_scores(const crisp_layer_desc_t *desc, const void *d_workspace,
                                           const unsigned long long **d_scores, const uint32_t **d_max_key) {
    if (!desc || !d_workspace || !d_scores || !d_max_key) return CRISP_INVALID_ARG;
    size_t mask_bytes = 0, ws_bytes = 0;
    crisp_status_t s = crisp_mask_sizes(desc, &mask_bytes, &ws_bytes);
    if (s != CRISP_OK) return s;
    const uint8_t *ws = reinterpret_cast<const uint8_t *>(d_workspace);
    *d_max_key = reinterpret_cast<const uint32_t *>(ws);
    *d_scores = reinterpret_cast<const unsigned long long *>(ws + crisp::kAlign);
    return CRISP_OK;
}

}  // extern "C"
