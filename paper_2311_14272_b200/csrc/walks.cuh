// Walk lists of the tensor-core SpMM, built from the kept-block list of the mask.
//   walk of a CTA tile  = ascending union of the kept block columns of its r = 128 / bm row tiles;
//   walk of the pair    = ascending union of its two CTA tiles' walks, with each side's entry index
//                         (or -1) for the CTA-pair kernel.
// One CTA (256 threads) per pair of adjacent 128-row CTA tiles.  Kept columns are marked in shared bitmaps
// and compacted with a prefix over the bitmap words.  The body is a device function so that it can run
// either as a kernel of its own or as extra CTAs of the encode kernel (it needs only the mask's block list).
#pragma once

#include "crisp_internal.h"

namespace crisp {

struct WalkArgs {
    const int32_t *blk_col;       // [nrt, kkeep] kept block columns of the mask, ascending per row tile
    int r, nst, wcap, pwcap;
    int npairs;                   // CTAs that build walk lists (0: none)
    int32_t *walk_col, *walk_len, *pair_col, *pair_len, *pair_src;
};

constexpr int kWalkBitmapWords = 128;                  // nblk <= 4096

struct WalkShared {
    uint32_t bits[2][kWalkBitmapWords];
    int prefix[3][kWalkBitmapWords + 1];
};

__device__ __forceinline__ void build_walks_body(const Geometry &g, const WalkArgs &a, int p, WalkShared &sh) {
    const int words = (g.nblk + 31) / 32;
    for (int i = threadIdx.x; i < 2 * kWalkBitmapWords; i += blockDim.x) sh.bits[i >> 7][i & 127] = 0u;
    __syncthreads();
    for (int side = 0; side < 2; ++side) {
        const int st = 2 * p + side;
        if (st >= a.nst) continue;
        const int first_rt = st * a.r;
        const int n_rt = min(a.r, g.nrt - first_rt);
        for (int i = threadIdx.x; i < n_rt * g.kkeep; i += blockDim.x) {
            const int jb = a.blk_col[(int64_t)first_rt * g.kkeep + i];
            atomicOr(&sh.bits[side][jb >> 5], 1u << (jb & 31));
        }
    }
    __syncthreads();
    if (threadIdx.x < 3) {                           // prefix of side 0, side 1 and of their union
        const int which = threadIdx.x;
        int run = 0;
        for (int i = 0; i < words; ++i) {
            sh.prefix[which][i] = run;
            const uint32_t b = which == 2 ? (sh.bits[0][i] | sh.bits[1][i]) : sh.bits[which][i];
            run += __popc(b);
        }
        if (which == 2) a.pair_len[p] = run;
        else if (2 * p + which < a.nst) a.walk_len[2 * p + which] = run;
    }
    __syncthreads();
    for (int jb = threadIdx.x; jb < g.nblk; jb += blockDim.x) {
        const int w = jb >> 5;
        const uint32_t below = (1u << (jb & 31)) - 1u;
        int pos[2] = {-1, -1};
        for (int side = 0; side < 2; ++side) {
            const uint32_t b = sh.bits[side][w];
            if ((b >> (jb & 31)) & 1u) {
                pos[side] = sh.prefix[side][w] + __popc(b & below);
                a.walk_col[(int64_t)(2 * p + side) * a.wcap + pos[side]] = jb;
            }
        }
        if (pos[0] >= 0 || pos[1] >= 0) {
            const int o = sh.prefix[2][w] + __popc((sh.bits[0][w] | sh.bits[1][w]) & below);
            a.pair_col[(int64_t)p * a.pwcap + o] = jb;
            a.pair_src[((int64_t)p * a.pwcap + o) * 2 + 0] = pos[0];
            a.pair_src[((int64_t)p * a.pwcap + o) * 2 + 1] = pos[1];
        }
    }
}

}  // namespace crisp
