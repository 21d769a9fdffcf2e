// Shared declarations of the CUDA side: control block layout, launch bookkeeping, small
// device helpers.  Nothing here is seen by the CPU oracle.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "vocabtrim.h"

namespace vt {

// First VT_CTRL_BYTES of every workspace.  Cleared once by vt_workspace_init; every kernel
// leaves `ticket` words at zero when it finishes.
struct Ctrl {
    uint32_t flags;               // sticky VT_FLAG_* bits
    uint32_t head_ticket;         // "last CTA merges" ticket of the head kernels (wraps to 0)
    unsigned long long n_bad;     // ids skipped by the histogram
    unsigned long long wait_ns;   // bound of a device-side wait in nanoseconds (0 = the built-in default)
    uint32_t pad[58];
};
static_assert(sizeof(Ctrl) == VT_CTRL_BYTES, "control block size");

constexpr int kNumSMsFallback = 148;

int num_sms();                    // SM count of the current device (cached per device)
void count_launch(int n = 1);     // host-side launch counter behind vt_launch_count

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
#ifdef __CUDACC__
__device__ __forceinline__ size_t align_up_dev(size_t x, size_t a) { return (x + a - 1) / a * a; }
#endif

// ---- launchers implemented in the .cu files (host functions) --------------------------------
struct HistPlan {
    bool small;            // all bins fit in one CTA's shared memory
    size_t off_sample;     // uint32 [V]   sampled counts
    size_t off_packed;     // uint32 [V]   what the packed kernel counted (only when three bins per word fit)
    size_t off_gate;       // uint32 [4]   {recount, -, skipped ids (64 bits)} of the packed kernel
    size_t clear_bytes;    // the scratch prefix every call zeroes
    size_t off_table;      // uint2  [ceil(V/32)] hot-bin table {bitmap word, slot base}
    size_t bytes;          // scratch after the control block
};
HistPlan hist_plan(int32_t V);
bool hist_supported(int32_t V);   // V the counting kernels take (bins or lookup table fit shared memory)
cudaError_t launch_histogram(const int32_t* ids, int64_t n, int32_t V, uint32_t* counts,
                             int accumulate, Ctrl* ctrl, uint8_t* scratch, cudaStream_t s);

cudaError_t launch_hist_fold(const int32_t* ids, int64_t n, int32_t V, int32_t bins, uint32_t* counts, cudaStream_t s);

size_t select_scratch_bytes(int32_t V);
cudaError_t launch_select_topk(const uint32_t* counts, int32_t V, int32_t K, int32_t* map,
                               int32_t* inv_map, uint8_t* scratch, cudaStream_t s);

size_t select_cut_scratch_bytes(int32_t V);
cudaError_t launch_select_cut(const uint32_t* counts, int32_t V, int mode, double pfrac, uint32_t min_count,
                              int32_t* map, int32_t* inv_map, int32_t* k_out, uint8_t* scratch, cudaStream_t s);

cudaError_t launch_verify_greedy(const int32_t* token, const int32_t* parent, const int32_t* target, int32_t S,
                                 int32_t N, int32_t* n_accept, int32_t* path, int32_t* emitted,
                                 unsigned long long* tokens_total, cudaStream_t st);

// One depth of the draft-tree expansion (vt_tree_expand's arguments); pool_token == nullptr: none.
struct TreeArgs {
    const int32_t* frontier;      // [B] pool index of each hidden row's node, or nullptr (the prefix)
    int32_t* pool_token;
    int32_t* pool_parent;
    float* pool_score;
    int32_t pool_base, n_front;
    int32_t* next_frontier;       // [n_front]
};

int tree_max_nodes();
cudaError_t launch_tree_expand(const int32_t* cand_ids, const float* cand_lp, int32_t B, int32_t topk, int32_t ld,
                               int32_t col0, const TreeArgs& t, cudaStream_t st);
cudaError_t launch_tree_rerank(const int32_t* pool_token, const int32_t* pool_parent, const float* pool_score,
                               int32_t n, int32_t budget, int32_t* out_nodes, int32_t* out_token,
                               int32_t* out_parent, cudaStream_t st);

cudaError_t launch_gather_rows(const uint16_t* W_full, const int32_t* map, uint16_t* W_trim,
                               int32_t V, int32_t K, int32_t d, Ctrl* ctrl, cudaStream_t s);

struct HeadArgs {
    const uint16_t* h;
    const uint16_t* W;
    const int32_t* map;
    int32_t B, K, d;
    const float* temp;
    int32_t topk;
    const float* uniforms;
    int32_t* out_ids;
    float* out_logprobs;
    float* dbg_logits;
    float* dbg_lse;
    int32_t overlap;       // launch with programmatic stream serialization (weights may be fetched early)
    TreeArgs tree;         // expansion to run on the merged top-k (pool_token == nullptr: none)
};
bool head_skinny_supported(int32_t B, int32_t d);
size_t head_skinny_scratch_bytes(int32_t B, int32_t K, int32_t topk);
cudaError_t launch_head_skinny(const HeadArgs& a, Ctrl* ctrl, uint8_t* scratch, cudaStream_t s);
#ifdef VT_STAMPS
size_t head_skinny_stamps_offset(int32_t B, int32_t topk);   // offset of the phase stamps in the head scratch
size_t head_dense_stamps_offset(int32_t B, int32_t topk);    // the same for the batched head
#endif

bool head_dense_supported(int32_t B, int32_t K, int32_t d);
bool head_dense_topk_ok(int32_t topk);
size_t head_dense_scratch_bytes(int32_t B, int32_t K, int32_t topk);
cudaError_t launch_head_dense(const HeadArgs& a, Ctrl* ctrl, uint8_t* scratch, cudaStream_t s);

// ---- device helpers ----------------------------------------------------------------------------
#ifdef __CUDACC__
// Streaming 128-bit load: read-only path, do not keep the line in L1 (data is used once).
__device__ __forceinline__ uint4 ld_stream_u4(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::128B.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream_u4(void* p, uint4 v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y),
                 "r"(v.z), "r"(v.w)
                 : "memory");
}
// Load that bypasses L1 (partials written by other CTAs of the same grid).
__device__ __forceinline__ float ld_cg_f32(const float* p) {
    float v;
    asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ int ld_cg_s32(const int* p) {
    int v;
    asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ unsigned lanemask_lt() {
    unsigned m;
    asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
    return m;
}
#endif

}  // namespace vt
