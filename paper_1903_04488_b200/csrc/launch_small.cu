// launch_small.cu -- instantiations and launch of the one-kernel tail of small problems (Algorithm 3 lines 9-13:
// small_tail.cuh).  The kernel's CTAs wait for one another at grid barriers, so the grid must be co-resident:
// it is sized from the occupancy query (one CTA per SM, whole clusters only) and launched cooperatively, which
// makes the runtime refuse the launch rather than start a grid that does not fit.
#include "ctx.cuh"

namespace ssgd {

// Cluster size (1, 2, 4 or 8 CTAs) whose combined shared memory holds the r x c table, split by columns: every CTA
// holds `cols` = 2^shift consecutive columns of every row.  0 if even 8 CTAs do not hold it.
static int small_cluster_for_table(const ssgd_ctx* x, int* shift_out) {
    for (int cs = 1; cs <= 8; cs *= 2) {
        int64_t cols = 1;
        int shift = 0;
        while (cols * cs < x->c) { cols <<= 1; ++shift; }
        if ((size_t)x->r * (size_t)cols * 4 <= SMALL_TABLE_SMEM_MAX) { *shift_out = shift; return cs; }
    }
    return 0;
}

bool small_tail_applicable(const ssgd_ctx* x, int64_t ncand) {
    return x->d <= SMALL_MAX_D && ncand <= SMALL_MAX_NCAND;
}

template <int R, bool POW2>
static int launch_small_tail_t(ssgd_ctx* x, SmallArgs& A, cudaStream_t st) {
    auto kern = k_small_tail<R, POW2>;
    int shift = 0;
    const int cs_table = small_cluster_for_table(x, &shift);
    const int cs = cs_table ? cs_table : 1;
    A.use_smem = cs_table ? 1 : 0;
    A.col_shift = shift;
    const size_t slice = cs_table ? (size_t)x->r * ((size_t)1 << shift) * 4 : 0;
    const size_t lists = (size_t)A.ncand * 8;              // the last CTA's candidates and sums
    const size_t smem = slice > lists ? slice : lists;
    cudaLaunchConfig_t cfg{};
    cfg.blockDim = dim3(ST_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)cs; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeCooperative;
    at[1].val.cooperative = 1;
    cfg.attrs = at;
    if (x->small_grid == 0 || x->small_smem != smem || x->small_cs != cs) {
        CU(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem), "smem attribute");
        // co-resident clusters: the occupancy query wants a grid that is a multiple of the cluster size
        cfg.gridDim = dim3((unsigned)(x->sm_count / cs * cs));
        cfg.numAttrs = 1;
        int nclusters = 0;
        CU(cudaOccupancyMaxActiveClusters(&nclusters, kern, &cfg), "cluster occupancy query");
        int grid = nclusters * cs;
        if (grid > x->sm_count / cs * cs) grid = x->sm_count / cs * cs;      // one CTA per SM is all the kernel can use
        if (grid < cs) { x->last_error = "the small-problem kernel does not fit this device"; return SSGD_ECUDA; }
        x->small_grid = grid; x->small_smem = smem; x->small_cs = cs;
    }
    cfg.gridDim = dim3((unsigned)x->small_grid);
    cfg.numAttrs = 2;
    CU(cudaLaunchKernelEx(&cfg, kern, A), "launch k_small_tail");
    LAUNCHED("k_small_tail");
    return SSGD_OK;
}

int launch_small_tail(ssgd_ctx* x, SmallArgs& A, cudaStream_t st) {
    DISPATCH_R(launch_small_tail_t, x, A, st)
}

}  // namespace ssgd
