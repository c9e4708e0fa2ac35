// launch_accum.cu -- instantiations and launches of the accumulate+insert kernels (Algorithm 3 lines 5-7).
#include "ctx.cuh"

namespace ssgd {

// ---- K1 dispatch over (R, POW2, MODE) ------------------------------------------------------------
template <int R, bool POW2, int MODE>
int launch_accum_t(ssgd_ctx* x, const AccumArgs& A, cudaStream_t st) {
    const int64_t groups = (A.d + 3) / 4;
    if (MODE == INS_MERGED_SMEM) {
        const size_t smem = (size_t)R * A.c * 4;
        CU(cudaFuncSetAttribute(k_accum_insert<R, POW2, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)smem), "smem attribute");
        const int grid = grid_for(groups, K1_THREADS, x->sm_count);
        k_accum_insert<R, POW2, MODE><<<grid, K1_THREADS, smem, st>>>(A);
    } else {
        const int grid = grid_for(groups, K1_THREADS, (int64_t)1 << 30);
        bool few = false;
        if constexpr (MODE == INS_MERGED_GLOBAL) {
            if (A.W <= K1_UNROLL_FEW) {
                few = true;
                CU(launch_pdl_w(st, L2Window{A.table, x->persist_bytes}, k_accum_insert<R, POW2, MODE, K1_UNROLL_FEW>, grid,
                                K1_THREADS, 0, A), "launch k_accum_insert");
            }
        }
        if (!few)
            CU(launch_pdl_w(st, L2Window{MODE == INS_MERGED_GLOBAL ? A.table : nullptr, x->persist_bytes},
                            k_accum_insert<R, POW2, MODE>, grid, K1_THREADS, 0, A), "launch k_accum_insert");
    }
    LAUNCHED("k_accum_insert");
    return SSGD_OK;
}

template <int R, bool POW2>
int launch_accum_m(ssgd_ctx* x, const AccumArgs& A, int mode, cudaStream_t st) {
    switch (mode) {
        case INS_MERGED_GLOBAL: return launch_accum_t<R, POW2, INS_MERGED_GLOBAL>(x, A, st);
        case INS_PER_WORKER: return launch_accum_t<R, POW2, INS_PER_WORKER>(x, A, st);
        default: return launch_accum_t<R, POW2, INS_MERGED_SMEM>(x, A, st);
    }
}

int launch_accum(ssgd_ctx* x, const AccumArgs& A, int mode, cudaStream_t st) {
    DISPATCH_R(launch_accum_m, x, A, mode, st)
}

template <int R, bool POW2>
int launch_accum_tma_t(ssgd_ctx* x, const AccumArgs& A, cudaStream_t st) {
    auto kern = k_accum_insert_tma<R, POW2>;
    const size_t smem = sizeof(KtShared);
    if (x->kt_blocks_per_sm == 0) {
        CU(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem), "smem attribute");
        int nb = 0;
        CU(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, kern, KT_THREADS, smem), "occupancy query");
        x->kt_blocks_per_sm = nb < 1 ? 1 : nb;
    }
    const int64_t ntiles = ((A.d & ~(int64_t)3) + KT_TC - 1) / KT_TC;
    const int grid = grid_for(ntiles, 1, (int64_t)x->sm_count * x->kt_blocks_per_sm);
    CU(launch_pdl_w(st, L2Window{A.table, x->persist_bytes}, kern, grid, KT_THREADS, smem, A,
                    reinterpret_cast<int32_t*>(x->ws + x->off_err)), "launch k_accum_insert_tma");
    LAUNCHED("k_accum_insert_tma");
    return SSGD_OK;
}

int launch_accum_tma(ssgd_ctx* x, const AccumArgs& A, cudaStream_t st) {
    DISPATCH_R(launch_accum_tma_t, x, A, st)
}

template <int R, bool POW2>
int launch_insert_rows_t(ssgd_ctx* x, const float* xsum, float* table, int lo, int hi, cudaStream_t st) {
    const int64_t groups = (x->d + 3) / 4;
    CU(launch_pdl(st, k_insert_rows<R, POW2>, grid_for(groups, 256, (int64_t)x->sm_count * 8), 256, 0, xsum, x->d, table, x->c,
                  x->hp, x->bk, lo, hi), "launch k_insert_rows");
    LAUNCHED("k_insert_rows");
    return SSGD_OK;
}

int launch_insert_rows(ssgd_ctx* x, const float* xsum, float* table, int lo, int hi, cudaStream_t st) {
    DISPATCH_R(launch_insert_rows_t, x, xsum, table, lo, hi, st)
}

}  // namespace ssgd
