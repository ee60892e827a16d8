// Host side of the CTA-pair SpMM (included by spmm_tc_pair.cu inside namespace crisp).

// The pair kernel needs whole 64-column boxes (its X load is the 3-D view) and at least two CTA tiles.
bool tc_pair_supported(const Geometry &g, int64_t ncols) {
    return ncols % kBoxN == 0 && (g.nrt * g.bm + kTileM - 1) / kTileM >= 2 && tensor_maps_available();
}

template <bool kSparse, typename OutT>
static cudaError_t launch_pair_variant(const CUtensorMap &mx, const CUtensorMap &my, const CUtensorMap &ma,
                                       const PairParams &p, int grid, size_t smem, cudaStream_t st) {
    auto kern = spmm_tc_pair_kernel<kSparse, OutT>;
    static size_t configured = 0;
    if (smem > configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured = smem;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, mx, my, ma, p);
}

cudaError_t launch_spmm_tc_pair(const Geometry &g, bool sparse, const uint8_t *d_exec, int32_t *d_status,
                                const uint16_t *d_x, int64_t ldx, int64_t ncols, void *d_y, int64_t ldy,
                                int y_dtype, cudaStream_t st) {
    const TcImageLayout L = tc_image_layout(g, sparse);
    static int sm_count = 0;
    if (!sm_count) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
        if (sm_count <= 0) sm_count = 148;
    }
    PairParams p;
    p.pair_col = reinterpret_cast<const int32_t *>(d_exec + L.pair_col_off);
    p.pair_len = reinterpret_cast<const int32_t *>(d_exec + L.pair_len_off);
    p.pair_src = reinterpret_cast<const int32_t *>(d_exec + L.pair_src_off);
    p.status = d_status;
    p.y = d_y; p.ldy = ldy; p.ncols = ncols;
    p.nst = L.nst; p.npairs = L.npairs; p.wcap = L.wcap; p.pwcap = L.pwcap; p.bk = g.bk; p.rows = g.rows;
    const int64_t tiles = (int64_t)L.npairs * ((ncols + kPairTileN - 1) / kPairTileN);
    if (tiles > 0x7FFFFFFF) return cudaErrorInvalidValue;
    p.num_tiles = (int)tiles;
    const uint64_t image_bytes = (uint64_t)L.nst * L.wcap * L.entry_bytes;
    p.image_rows = (int)(image_bytes >> 8);
    p.a_bytes = L.a_bytes; p.entry_bytes = L.entry_bytes;
    p.box_bytes = (uint32_t)(kBoxN * g.bk * 2);
    p.stage_bytes = p.entry_bytes + kPairBoxes * p.box_bytes;
    const uint32_t fixed = kEpiWarps * 2 * kStageTileBytes + 512;
    uint32_t stages = (kSmemBudget - fixed) / p.stage_bytes;
    if (stages > (uint32_t)kPairMaxStages) stages = kPairMaxStages;
    if (stages < 2) return cudaErrorInvalidValue;
    p.num_stages = stages;
    const size_t smem = (size_t)stages * p.stage_bytes + fixed + 1024;

    CUtensorMap mx, my, ma;
    if (!make_map_x3d(&mx, d_x, (uint64_t)ncols, (uint64_t)g.k, (uint64_t)ldx, (uint32_t)g.bk, kPairBoxes))
        return cudaErrorInvalidValue;
    if (!make_map_image(&ma, d_exec + L.image_off, image_bytes, L.entry_bytes)) return cudaErrorInvalidValue;
    const bool f32 = y_dtype != 0;
    if (!make_map_2d(&my, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, f32 ? 4 : 2, d_y,
                     (uint64_t)ncols, (uint64_t)g.rows, (uint64_t)ldy, f32 ? 32 : 64, 32))
        return cudaErrorInvalidValue;
    const int pairs_resident = sm_count / 2;
    const int grid = 2 * (int)(tiles < pairs_resident ? tiles : pairs_resident);
    if (sparse)
        return f32 ? launch_pair_variant<true, float>(mx, my, ma, p, grid, smem, st)
                   : launch_pair_variant<true, uint16_t>(mx, my, ma, p, grid, smem, st);
    return f32 ? launch_pair_variant<false, float>(mx, my, ma, p, grid, smem, st)
               : launch_pair_variant<false, uint16_t>(mx, my, ma, p, grid, smem, st);
}
