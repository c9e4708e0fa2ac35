// launch_unsketch.cu -- instantiations and launches of the kernels that evaluate Algorithm 4's estimate for
// every coordinate (Algorithm 3 line 9; Algorithm 1 line 2).
#include "ctx.cuh"

namespace ssgd {

template <int R, bool POW2>
int launch_unsketch_t(ssgd_ctx* x, const UnsketchArgs& A, cudaStream_t st) {
    const int64_t groups = (A.d + K3_NC - 1) / K3_NC;
    // a few blocks per SM: each block pays one histogram flush
    const int grid = grid_for(groups, K3_THREADS, (int64_t)x->sm_count * K3_GRID);
    CU(launch_pdl(st, k_unsketch<R, POW2>, grid, K3_THREADS, 0, A), "launch k_unsketch");
    LAUNCHED("k_unsketch");
    return SSGD_OK;
}

int launch_unsketch(ssgd_ctx* x, const UnsketchArgs& A, cudaStream_t st) {
    DISPATCH_R(launch_unsketch_t, x, A, st)
}

// The first pass over all coordinates: the bit-per-bucket filter when the (folded) bitmap fits an SM's shared
// memory, else the early-exit kernel that reads the table.
bool use_filter(const ssgd_ctx* x) {
    return x->prune_mode != SSGD_PRUNE_EARLY_EXIT && (x->bm_fold >= 0 || x->rowbits) &&
           sizeof(SelShared) + FILTER_QUEUE_BYTES + (size_t)FILTER_MAX_WORDS * 4 <= (size_t)x->max_smem_optin;
}

template <int R, bool POW2>
int launch_sparse_t(ssgd_ctx* x, const SparseArgs& A, cudaStream_t st) {
    const int64_t groups = (A.d + 3) / 4;
    const int64_t windows = (groups + (1 << SPARSE_SAMPLE_SHIFT) - 1) >> SPARSE_SAMPLE_SHIFT;
    CU(launch_pdl(st, k_unsketch_sample<R, POW2>, grid_for(windows, SEL_THREADS, (int64_t)x->sm_count * 4), SEL_THREADS, 0, A),
       "launch k_unsketch_sample");
    LAUNCHED("k_unsketch_sample");
    const int pruned_grid = grid_for((A.d + PRUNED_NC - 1) / PRUNED_NC, SEL_THREADS, (int64_t)x->sm_count * PRUNED_GRID);
    if (use_filter(x)) {
        FilterArgs F;
        F.A = A;
        F.bm_full = reinterpret_cast<uint32_t*>(x->ws + x->off_bm_full);
        F.bm_fold = reinterpret_cast<uint32_t*>(x->ws + x->off_bm_fold);
        F.stride_full = x->bm_stride_full; F.stride_fold = x->bm_stride_fold; F.fold = x->bm_fold; F.r = x->r;
        F.decide_in_build = x->rowbits ? 1 : 0; F.max_pass = ROWBITS_MAX_PASS;
        const int64_t build_tasks = (int64_t)x->r * ((x->bm_stride_full + 31) / 32);
        CU(launch_pdl(st, k_bitmap_build, grid_for(build_tasks, SEL_WARPS, (int64_t)x->sm_count * 8), SEL_THREADS, 0, F),
           "launch k_bitmap_build");
        LAUNCHED("k_bitmap_build");
        if (x->rowbits) {
            // the bitmap row by row: r x (SMs / r) blocks each hold one row, then the r bits of every coordinate are counted
            RowBitsArgs B;
            B.F = F;
            B.rowbits = reinterpret_cast<uint32_t*>(x->ws + x->off_rowbits);
            B.words_per_row = (x->d + 31) / 32;
            B.slices = x->rb_slices; B.slice_words = x->rb_slice_words;
            // two blocks per SM when two rows fit its shared memory (32 registers per thread: 2048 threads are resident)
            const size_t row_bytes = B.slices > 1 ? (size_t)B.slice_words * 4 + 16 : (size_t)F.stride_full * 4;   // + the zero word
            const int per_sm = 2 * (row_bytes + 1024) <= (size_t)x->max_smem_optin ? 2 : 1;
            const int row_blocks = x->r * B.slices;
            B.ranges = x->sm_count * per_sm / row_blocks > 0 ? x->sm_count * per_sm / row_blocks : 1;
            auto kern = B.slices > 1 ? k_row_bits<POW2, true> : k_row_bits<POW2, false>;
            if (!x->rowbits_ready) {
                CU(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)((size_t)FILTER_MAX_WORDS * 4 + 16)),
                   "smem attribute");
                CU(cudaFuncSetAttribute(k_rowbits_combine<R, POW2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)RBC_SMEM),
                   "smem attribute");
                x->rowbits_ready = true;
            }
            CU(launch_pdl(st, kern, row_blocks * B.ranges, RB_MAX_THREADS, row_bytes, B), "launch k_row_bits");
            LAUNCHED("k_row_bits");
            CU(launch_pdl(st, k_rowbits_combine<R, POW2>, grid_for(B.words_per_row, SEL_THREADS, (int64_t)x->sm_count * 2),
                          SEL_THREADS, RBC_SMEM, B), "launch k_rowbits_combine");
            LAUNCHED("k_rowbits_combine");
            SparseArgs G = A;
            G.gated = 1;                                 // runs only if the bitmap turned out too dense (plain stream order)
            k_unsketch_pruned<R, POW2><<<pruned_grid, SEL_THREADS, 0, st>>>(G);
            LAUNCHED("k_unsketch_pruned");
        } else {
        if (F.fold) {
            CU(launch_pdl(st, k_bitmap_fold, grid_for((int64_t)x->r * F.stride_fold, SEL_THREADS, (int64_t)x->sm_count * 8),
                          SEL_THREADS, 0, F), "launch k_bitmap_fold");
            LAUNCHED("k_bitmap_fold");
        }
        auto kern = F.fold ? k_unsketch_filter<R, POW2, true> : k_unsketch_filter<R, POW2, false>;
        const size_t smem = (size_t)x->r * (F.fold ? F.stride_fold : F.stride_full) * 4 + FILTER_QUEUE_BYTES;
        if (!x->filter_ready) {
            CU(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)((size_t)FILTER_MAX_WORDS * 4 + FILTER_QUEUE_BYTES)), "smem attribute");
            x->filter_ready = true;
        }
        CU(launch_pdl(st, kern, grid_for(A.d, FILTER_THREADS, (int64_t)x->sm_count), FILTER_THREADS, smem, F),
           "launch k_unsketch_filter");
        LAUNCHED("k_unsketch_filter");
        if (F.fold) {                                    // runs only if the folded bitmap turned out too dense
            SparseArgs G = A;
            G.gated = 1;
            // plain stream order, no programmatic launch: measured on B200, blocks of this kernel that become
            // resident while the declining filter kernel drains cost 4 ms (d = 9e7)
            k_unsketch_pruned<R, POW2><<<pruned_grid, SEL_THREADS, 0, st>>>(G);
            LAUNCHED("k_unsketch_pruned");
        }
        }
    } else {
        CU(launch_pdl(st, k_unsketch_pruned<R, POW2>, pruned_grid, SEL_THREADS, 0, A), "launch k_unsketch_pruned");
        LAUNCHED("k_unsketch_pruned");
    }
    SparseArgs B = A;
    B.rerun = 1;                                         // returns at once unless the first pass kept too few
    CU(launch_pdl(st, k_unsketch_pruned<R, POW2>, pruned_grid, SEL_THREADS, 0, B), "launch k_unsketch_pruned (unpruned rerun)");
    LAUNCHED("k_unsketch_pruned");
    return SSGD_OK;
}

int launch_sparse(ssgd_ctx* x, const SparseArgs& A, cudaStream_t st) {
    DISPATCH_R(launch_sparse_t, x, A, st)
}

template <int R, bool POW2>
int launch_heavymix_keys_t(ssgd_ctx* x, const HeavymixArgs& A, cudaStream_t st) {
    const int64_t groups = (A.d + 3) / 4;
    k_heavymix_keys<R, POW2><<<grid_for(groups, SEL_THREADS, (int64_t)x->sm_count * 4), SEL_THREADS, 0, st>>>(A);
    LAUNCHED("k_heavymix_keys");
    return SSGD_OK;
}

int launch_heavymix_keys(ssgd_ctx* x, const HeavymixArgs& A, cudaStream_t st) {
    DISPATCH_R(launch_heavymix_keys_t, x, A, st)
}

}  // namespace ssgd
