// Walk lists of the tensor-core SpMM, built from the kept-block list of the mask.
//   walk of a CTA tile = ascending union of the kept block columns of its r = 128 / bm row tiles.
// One CTA (256 threads) per 128-row CTA tile.  Kept columns are marked in a shared bitmap and compacted
// with a prefix over the bitmap words.  The body is a device function so that it can run either as a
// kernel of its own or as extra CTAs of the encode kernel (it needs only the mask's block list).
#pragma once

#include "crisp_internal.h"

namespace crisp {

struct WalkArgs {
    const int32_t *blk_col;       // [nrt, kkeep] kept block columns of the mask, ascending per row tile
    int r, nst, wcap;
    int nctas;                    // CTAs that build walk lists (0: none), one per CTA tile
    int32_t *walk_col, *walk_len;
    uint32_t *header = nullptr;   // 64 words that CTA 0 of the kernel clears (the handle's status block), or nullptr
};

// The status block at the head of the execution buffer, cleared by the kernel that fills the buffer: a memset of
// its own in front of the kernel costs the stream about 2 us.
__device__ __forceinline__ void clear_header(const WalkArgs &a) {
    if (blockIdx.x == 0 && a.header != nullptr && threadIdx.x < 64) a.header[threadIdx.x] = 0u;
}

constexpr int kWalkBitmapWords = 128;                  // nblk <= 4096

struct WalkShared {
    uint32_t bits[kWalkBitmapWords];
    int prefix[kWalkBitmapWords + 1];
};

__device__ __forceinline__ void build_walks_body(const Geometry &g, const WalkArgs &a, int st, WalkShared &sh) {
    const int words = (g.nblk + 31) / 32;
    for (int i = threadIdx.x; i < kWalkBitmapWords; i += blockDim.x) sh.bits[i] = 0u;
    __syncthreads();
    const int first_rt = st * a.r;
    const int n_rt = min(a.r, g.nrt - first_rt);
    for (int i = threadIdx.x; i < n_rt * g.kkeep; i += blockDim.x) {
        const int jb = a.blk_col[(int64_t)first_rt * g.kkeep + i];
        atomicOr(&sh.bits[jb >> 5], 1u << (jb & 31));
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int i = 0; i < words; ++i) {
            sh.prefix[i] = run;
            run += __popc(sh.bits[i]);
        }
        a.walk_len[st] = run;
    }
    __syncthreads();
    for (int jb = threadIdx.x; jb < g.nblk; jb += blockDim.x) {
        const int w = jb >> 5;
        const uint32_t b = sh.bits[w];
        if ((b >> (jb & 31)) & 1u)
            a.walk_col[(int64_t)st * a.wcap + sh.prefix[w] + __popc(b & ((1u << (jb & 31)) - 1u))] = jb;
    }
}

}  // namespace crisp
