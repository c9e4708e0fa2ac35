// launch_small.cu -- instantiations and launch of the one-kernel tail of small problems (Algorithm 3 lines 9-13:
// small_tail.cuh).  The kernel's CTAs wait for one another at grid barriers, so the grid must be co-resident:
// one CTA per SM, checked against the occupancy query, and launched cooperatively, which makes the runtime refuse
// the launch rather than start a grid that does not fit.
#include "ctx.cuh"

namespace ssgd {

bool small_tail_applicable(const ssgd_ctx* x, int64_t ncand) {
    return x->d <= SMALL_MAX_D && ncand <= SMALL_MAX_NCAND;
}

template <int R, bool POW2>
static int launch_small_tail_t(ssgd_ctx* x, SmallArgs& A, cudaStream_t st) {
    auto kern = k_small_tail<R, POW2>;
    // As many rows of the table as fit go to every CTA's shared memory, if the copy pays: a CTA saves about 0.6
    // clocks per lookup (1 / 1.1 - 1 / 3.5) on d / ctas lookups per row and spends about c / 8 clocks copying a
    // row, so the copy is worth it from d = c * ctas / 4 coordinates on
    const int ctas = x->small_grid ? x->small_grid : x->sm_count;
    int rows = (int)(SMALL_TABLE_SMEM_MAX / ((size_t)x->c * 4));
    if (rows > x->r) rows = x->r;
    if (x->d < x->c * (int64_t)ctas / 4) rows = 0;
    A.rows_smem = rows;
    const size_t table_bytes = (size_t)rows * x->c * 4;
    const size_t lists = (size_t)A.ncand * 8;              // the last CTA's candidates and sums
    const size_t smem = table_bytes > lists ? table_bytes : lists;
    cudaLaunchConfig_t cfg{};
    cfg.blockDim = dim3(ST_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeCooperative;
    at[0].val.cooperative = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (x->small_grid == 0) {
        // the same limit from every context (the attribute belongs to the kernel, not to the context)
        constexpr size_t SMEM_LIMIT = SMALL_TABLE_SMEM_MAX > (size_t)SMALL_MAX_NCAND * 8 ? SMALL_TABLE_SMEM_MAX : (size_t)SMALL_MAX_NCAND * 8;
        CU(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_LIMIT), "smem attribute");
        int per_sm = 0;
        CU(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, ST_THREADS, SMEM_LIMIT), "occupancy query");
        if (per_sm < 1) { x->last_error = "the small-problem kernel does not fit this device"; return SSGD_ECUDA; }
        x->small_grid = x->sm_count;                       // one CTA per SM: co-resident by the query above
    }
    cfg.gridDim = dim3((unsigned)x->small_grid);
    const cudaError_t le = A.withhold < 0 ? cudaErrorCooperativeLaunchTooLarge : cudaLaunchKernelEx(&cfg, kern, A);
    if (le == cudaErrorCooperativeLaunchTooLarge || le == cudaErrorLaunchOutOfResources) {
        // the device cannot hold one block per SM at once right now (SMs taken by another context, or the test
        // hook): nothing was launched; the caller takes the chain of ordinary launches instead
        if (A.withhold >= 0) cudaGetLastError();
        return SMALL_TAIL_REFUSED;
    }
    if (le != cudaSuccess) return cuda_fail(x, le, "launch k_small_tail");
    LAUNCHED("k_small_tail");
    return SSGD_OK;
}

int launch_small_tail(ssgd_ctx* x, SmallArgs& A, cudaStream_t st) {
    DISPATCH_R(launch_small_tail_t, x, A, st)
}

}  // namespace ssgd
