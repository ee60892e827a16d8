// CTA-pair variant of the tensor-core SpMM (sm_100a, tcgen05 cta_group::2).
//
// The single-CTA kernel is bound by the bytes each SM pulls from L2 into shared memory, and three
// quarters of those bytes are the activation tile X[kept rows, 256 columns].  Here two CTAs of a
// cluster take two adjacent 128-row tiles and the same 256 output columns.  They walk the UNION of the
// two tiles' kept-block lists; for every block of the union each CTA loads only its half of the X tile
// (128 columns) and its own weight tile, and one tcgen05.mma.cta_group::2 (M = 256, N = 256) issued by
// the leader CTA reads both halves.  A tile that does not keep a block of the union contributes a
// zero weight tile (a TMA load from an out-of-bounds coordinate: zero fill, no memory traffic).
// Steps 1-3 of Sec. III-E are unchanged; only the staging of step 1 is shared between two row tiles.
//
// Synchronisation (all waits bounded):
//   full[s]   leader's barrier; both CTAs' loads signal it (cta_group::2 loads), leader expects both
//   empty[s]  per CTA; released for both CTAs by one multicast tcgen05.commit
//   tfull     per CTA; multicast tcgen05.commit after the last block of a tile
//   tempty    leader's barrier; the 4 epilogue warps of both CTAs arrive on it (remote arrive)
#include "crisp_internal.h"
#include "tc_common.cuh"

namespace crisp {

using namespace tc;

namespace {

constexpr int kPairTileN = 256;            // output columns of a pair tile
constexpr int kPairBoxes = 2;              // 64-column boxes of X per CTA (its half of the tile)
constexpr int kPairMaxStages = 16;

struct PairParams {
    const int32_t *pair_col;    // [npairs, pwcap] union block columns
    const int32_t *pair_len;    // [npairs]
    const int32_t *pair_src;    // [npairs, pwcap, 2] entry index in each side's own walk list, or -1
    int32_t *status;
    void *y;
    int64_t ldy, ncols;
    int nst, npairs, wcap, pwcap, bk, rows, num_tiles;
    int image_rows;             // rows (of 256 bytes) of the image: a load from there is all zeros
    uint32_t a_bytes, entry_bytes, box_bytes, stage_bytes, num_stages;
};

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t out;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(addr), "r"(rank));
    return out;
}
__device__ __forceinline__ void remote_arrive(uint32_t cluster_bar) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap *map, int x, int y, int z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// Arrive on the barrier at this offset in both CTAs once all earlier MMAs of the pair have completed.
__device__ __forceinline__ void mma_commit_pair(uint32_t bar) {
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void mma_dense_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void mma_sparse_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                uint32_t acc, uint32_t meta_tmem) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.sp.cta_group::2.kind::f16 [%0], %1, %2, [%5], %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc), "r"(meta_tmem) : "memory");
}
__device__ __forceinline__ void tmem_copy_128x128b_pair(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::2.128x128b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
// bf16 x bf16 -> fp32, A K-major, B MN-major, M = 256 across the pair, N = 256.
__host__ __device__ constexpr uint32_t make_idesc_pair(bool sparse) {
    return (sparse ? (1u << 2) : 0u) | (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) |
           ((uint32_t)(kPairTileN >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

#include "spmm_tc_pair_kernel.inl"

}  // namespace

#include "spmm_tc_pair_host.inl"

}  // namespace crisp
