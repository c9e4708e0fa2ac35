// ctx.cuh -- what the translation units of the library share on the host side: the context object, the error
// and launch helpers, and the launch functions that one unit defines and another calls.  The kernels that
// are instantiated per (rows, power-of-two columns) live in units of their own so that they compile in parallel:
//   launch_accum.cu     Algorithm 3 lines 5-7 (k_accum_insert, k_accum_insert_tma, k_insert_rows)
//   launch_unsketch.cu  Algorithm 3 line 9 (k_unsketch, k_unsketch_sample, k_unsketch_filter, k_unsketch_pruned)
//                       and Algorithm 1's key kernel
//   launch_small.cu     Algorithm 3 lines 9-13 in one cooperative kernel (k_small_tail)
//   ssgd.cu             the C ABI, workspace layout, the selections and everything else
#pragma once
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdlib>
#include <string>

#include "../../include/ssgd.h"
#include "hash.cuh"
#include "select.cuh"
#include "accum_tma.cuh"
#include "estimate.cuh"
#include "sparse_select.cuh"
#include "filter_unsketch.cuh"
#include "rowbits_unsketch.cuh"
#include "heavymix.cuh"
#include "step_kernels.cuh"
#include "small_tail.cuh"

struct ssgd_ctx {
    int64_t d, c, k;
    int32_t r, W;
    uint64_t seed;
    ssgd::HashParams hp;
    ssgd::Bucketizer bk;
    bool pow2;
    int32_t insert_mode;
    // binding
    float* u; float* v; int64_t ld;
    char* ws; size_t ws_bytes; int64_t ncand_max;
    // workspace layout (byte offsets)
    size_t off_table, off_hist_c, off_hist_f, off_state_c, off_state_f, off_err, zero_bytes;
    size_t off_h19_c, off_h19_f, off_small, zero_small_bytes;
    size_t off_sp_hist, off_sp_state, off_maps, off_map_chunks, off_list_idx, off_list_est;   // early-exit path
    size_t map_bytes;
    int64_t list_cap, nchunk_map;
    size_t off_bm_full, off_bm_fold;                       // bit-per-bucket filter (filter_unsketch.cuh)
    int32_t bm_stride_full, bm_stride_fold, bm_fold;       // bm_fold < 0: the bitmap cannot be folded into shared memory
    bool filter_ready;                                     // shared-memory attribute of the filter kernel set
    bool rowbits;                                          // the bitmap does not fit as a whole but row by row (rowbits_unsketch.cuh)
    int rb_slices, rb_slice_words;                         // pieces each of its rows is cut into for that, words per piece
    bool rowbits_ready;                                    // shared-memory attribute of k_row_bits set
    size_t off_rowbits;                                    // [r][ceil(d/32)] result words of k_row_bits (rowbits only)
    uint32_t sample_rank;   // 0: derive the sample rank from ncand; else use this one (tests)
    size_t off_pending;     // d-bit map of the deferred zero-out; survives from step to step
    int32_t zero_mode;      // SSGD_ZERO_DEFERRED / SSGD_ZERO_EAGER
    int32_t sched_mode;     // SSGD_SCHED_*: how ssgd_sketch_accumulate walks workers and coordinates
    bool pending_dirty;     // a deferred ssgd_step has run since the last flush: u, v may await their zero-out
    size_t off_hm;
    int32_t prune_mode;
    size_t persist_bytes;   // > 0: launches that touch the table carry an L2 access-policy window of this size
    size_t split_bytes;     // > 0: ssgd_step inserts at most this many bytes of table rows per kernel
    int stream_loads;       // SSGD_STREAM_*: cache operator of the plain-load kernel's reads of g, u, v
    size_t off_xsum;        // per-coordinate sums over the workers of the new v, written by ssgd_step's accumulate kernel
    size_t off_est, off_chunk_c, off_chunk_f, off_cand, off_xs, off_oidx, off_oval, total_bytes;
    int64_t nchunk_c, nchunk_f;
    // device facts
    int device; int sm_count; int max_smem_optin;
    int kt_blocks_per_sm;   // residency of the bulk-copy pipeline kernel (0 = not queried yet)
    int small_grid;         // CTAs of the one-kernel tail (0 = not queried yet)
    bool small_refused;     // a cooperative launch was refused: AUTO stays with the chain of ordinary launches
    uint64_t wait_ns;       // limit of every device-side wait (grid barriers, mbarriers)
    int32_t withhold;       // test hook: this CTA (1-based; 0 = none) never arrives, so the others' waits run out
    int64_t launches;
    // optional per-stage timing of ssgd_step (CUDA events on the caller's stream)
    bool timing;
    cudaEvent_t* ev;        // [TIMING_SLOTS][SSGD_NSTAGES + 1]
    int32_t ev_steps;       // steps recorded since the last collection
    std::string last_error;
};

namespace ssgd {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int cuda_fail(ssgd_ctx* x, cudaError_t e, const char* what) {
    x->last_error = std::string(what) + ": " + cudaGetErrorString(e);
    return SSGD_ECUDA;
}

#define CU(call, what)                                                   \
    do {                                                                 \
        cudaError_t e_ = (call);                                         \
        if (e_ != cudaSuccess) return cuda_fail(x, e_, what);            \
    } while (0)

#define LAUNCHED(what)                                                   \
    do {                                                                 \
        x->launches++;                                                   \
        cudaError_t e_ = cudaGetLastError();                             \
        if (e_ != cudaSuccess) return cuda_fail(x, e_, what);            \
    } while (0)

// Launch with programmatic stream serialization: the kernel may become resident while its predecessor
// drains; it orders itself with pdl_wait().

// An L2 access-policy window for one launch: accesses inside [base, base+bytes) are kept (persisting),
// everything else the kernel touches is treated as streaming.
struct L2Window { const void* base; size_t bytes; };

template <typename... P, typename... A>
cudaError_t launch_pdl_w(cudaStream_t st, L2Window win, void (*kern)(P...), int grid, int block, size_t smem, A... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    int n = 0;
    at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
    if (win.base && win.bytes) {
        at[n].id = cudaLaunchAttributeAccessPolicyWindow;
        at[n].val.accessPolicyWindow.base_ptr = const_cast<void*>(win.base);
        at[n].val.accessPolicyWindow.num_bytes = win.bytes;
        at[n].val.accessPolicyWindow.hitRatio = 1.0f;
        at[n].val.accessPolicyWindow.hitProp = cudaAccessPropertyPersisting;
        at[n].val.accessPolicyWindow.missProp = cudaAccessPropertyStreaming;
        ++n;
    }
    cfg.attrs = at;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kern, P(args)...);
}

template <typename... P, typename... A>
cudaError_t launch_pdl(cudaStream_t st, void (*kern)(P...), int grid, int block, size_t smem, A... args) {
    return launch_pdl_w(st, L2Window{nullptr, 0}, kern, grid, block, smem, args...);
}

inline int grid_for(int64_t items, int threads, int64_t cap) {
    int64_t b = (items + threads - 1) / threads;
    if (b < 1) b = 1;
    if (b > cap) b = cap;
    return (int)b;
}

// Instantiation switch over the row count (odd, 1..15) and "c is a power of two".
#define DISPATCH_R(fn, ...)                                                       \
    switch (x->r) {                                                               \
        case 1: return x->pow2 ? fn<1, true>(__VA_ARGS__) : fn<1, false>(__VA_ARGS__);    \
        case 3: return x->pow2 ? fn<3, true>(__VA_ARGS__) : fn<3, false>(__VA_ARGS__);    \
        case 5: return x->pow2 ? fn<5, true>(__VA_ARGS__) : fn<5, false>(__VA_ARGS__);    \
        case 7: return x->pow2 ? fn<7, true>(__VA_ARGS__) : fn<7, false>(__VA_ARGS__);    \
        case 9: return x->pow2 ? fn<9, true>(__VA_ARGS__) : fn<9, false>(__VA_ARGS__);    \
        case 11: return x->pow2 ? fn<11, true>(__VA_ARGS__) : fn<11, false>(__VA_ARGS__); \
        case 13: return x->pow2 ? fn<13, true>(__VA_ARGS__) : fn<13, false>(__VA_ARGS__); \
        case 15: return x->pow2 ? fn<15, true>(__VA_ARGS__) : fn<15, false>(__VA_ARGS__); \
        default: return SSGD_EINVAL;                                              \
    }

// defined in launch_accum.cu
int launch_accum(ssgd_ctx* x, const AccumArgs& A, int mode, cudaStream_t st);
int launch_accum_tma(ssgd_ctx* x, const AccumArgs& A, cudaStream_t st);
int launch_insert_rows(ssgd_ctx* x, const float* xsum, float* table, int lo, int hi, cudaStream_t st);
// defined in launch_unsketch.cu
int launch_unsketch(ssgd_ctx* x, const UnsketchArgs& A, cudaStream_t st);
bool use_filter(const ssgd_ctx* x);
int launch_sparse(ssgd_ctx* x, const SparseArgs& A, cudaStream_t st);
int launch_heavymix_keys(ssgd_ctx* x, const HeavymixArgs& A, cudaStream_t st);
// defined in launch_small.cu
constexpr int SMALL_TAIL_REFUSED = 1;    // launch_small_tail: the cooperative launch does not fit the device right now
bool small_tail_applicable(const ssgd_ctx* x, int64_t ncand);
int launch_small_tail(ssgd_ctx* x, SmallArgs& A, cudaStream_t st);

}  // namespace ssgd
