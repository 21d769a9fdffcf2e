// Batched-serving head (17 <= B <= 256 hidden rows): the projection is a real dense contraction
// and runs on the 5th-generation tensor cores (Algorithm 2, lines 5-6, with many sequences and
// tree nodes drafted at once).
//
//   D[b, j] = sum_i h[b, i] * W_trim[j, i]      M = hidden rows (128 per MMA, two M tiles),
//                                               N = 128 vocabulary rows per tile, K-loop over d
//
// One persistent CTA per SM walks vocabulary tiles.  Warp 0 feeds a 4-stage shared-memory ring with
// TMA tensor copies (128-byte swizzle, no multicast): per 64-column step the two halves of h and one
// tile of W_trim.  One thread of warp 1 issues tcgen05.mma (bf16 x bf16 -> fp32) with the operands
// described in place by shared-memory descriptors and the accumulators in tensor memory: two
// accumulator stages of 2 x 128 columns, so the epilogue of tile t overlaps the MMAs of tile t+1.
// Eight epilogue warps read the accumulators back with tcgen05.ld -- TMEM lane = hidden row, so every
// thread owns one hidden row and walks its 128 logits of the tile, 16 at a time: running max / sum-exp of
// z = logit / T_b, Gumbel-max candidate from the caller's uniforms, and a sorted top-k list kept in
// registers.  Logits never go to HBM.  Per CTA and hidden row one record goes to scratch; a second
// small kernel (one warp per hidden row) merges the records, applies the index mapper and writes
// the outputs.  Every wait is bounded; on expiry the CTA raises VT_FLAG_TIMEOUT and leaves after
// releasing its tensor memory.
#include <cuda.h>

#include <mutex>

#include "vt_common.cuh"
#include "vt_head_common.cuh"

namespace vt {

namespace {

constexpr int kBM = 128;                  // hidden rows per MMA (TMEM lanes)
constexpr int kBN = 128;                  // vocabulary rows per tile (TMEM columns per accumulator)
constexpr int kBK = 64;                   // columns of d per ring stage: 128 bytes, one swizzle row
constexpr int kStages = 4;
constexpr int kTileBytes = kBM * kBK * 2; // 16 KB: one operand tile of a stage
constexpr int kStageBytes = 3 * kTileBytes;
constexpr int kEpiWarps = 8;
constexpr int kThreads = (2 + kEpiWarps) * 32;
constexpr int kCh = 16;                   // accumulator columns per epilogue step (keeps the row state in registers)
constexpr int kTmemCols = 512;            // 2 accumulator stages x 2 M tiles x 128 columns
constexpr int kMaxTopk = 16;              // top-k list lives in registers
constexpr unsigned long long kWaitLimitNs = 2000000000ull;
constexpr size_t kDynSmem = (size_t)kStages * kStageBytes + 1024;   // + slack to align to 1024 bytes

// ---- PTX wrappers ----------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* b, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* b, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try(b, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 128; ++i)
            if (mbar_try(b, parity)) return true;
        if (*abort_flag) return false;
        if (global_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
    }
}
// Same, called by all 32 lanes of a warp: the outcome is voted on so the lanes never part ways
// before a warp-collective instruction.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* b, uint32_t parity, volatile int* abort_flag) {
    return __all_sync(0xffffffffu, mbar_wait(b, parity, abort_flag));
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, 128 x N x 16, bf16 inputs, fp32 accumulation
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p; }"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
// 16 consecutive accumulator columns of this thread's TMEM lane
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory operand descriptor: K-major tile of 128-byte rows, 128-byte swizzle, 8-row groups
// 1024 bytes apart (the layout a TMA tensor copy with SWIZZLE_128B and a 64-column bf16 box writes).
// Fields: start address >> 4 [0,14); leading byte offset >> 4 [16,30) (unused for swizzled K-major: 1);
// stride byte offset >> 4 [32,46); descriptor version 1 at [46,48); layout type 2 = 128B swizzle at [61,64).
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr) {
    return (uint64_t)((smem_addr >> 4) & 0x3fffu) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Instruction descriptor of kind::f16: fp32 accumulator (1 at [4,6)), A and B bf16 (1 at [7,10) and
// [10,13)), both K-major (0 at bits 15 and 16), N >> 3 at [17,23), M >> 4 at [24,29).
__host__ __device__ constexpr uint32_t make_idesc(int M, int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

struct DenseGeo {
    int n_tiles;      // vocabulary tiles of kBN rows
    int n_kc;         // ring steps per tile: ceil(d / kBK)
    int n_mt;         // M tiles: 1 (B <= 128) or 2
};

// KT: capacity of the register top-k list (8 or kMaxTopk)
template <int KT>
__global__ void __launch_bounds__(kThreads, 1)
k_head_dense(const HeadArgs a, Ctrl* ctrl, float* __restrict__ recs, const DenseGeo geo,
             const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ CUtensorMap tm_w) {
    extern __shared__ uint8_t s_dyn[];
    __shared__ uint64_t s_full[kStages], s_empty[kStages], s_acc_full[2], s_acc_empty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(s_dyn) + 1023) & ~(uintptr_t)1023);
    const uint32_t ring_u32 = smem_u32(ring);
    const int B = a.B, K = a.K, topk = a.topk;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&s_full[s], 1); mbar_init(&s_empty[s], 1); }
        for (int p = 0; p < 2; ++p) { mbar_init(&s_acc_full[p], 1); mbar_init(&s_acc_empty[p], kEpiWarps); }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // tensor memory: the whole SM's 512 columns (one CTA per SM by shared-memory size)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&s_tmem_base)), "r"((uint32_t)kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    volatile int* abort_flag = &s_abort;

    if (warp == 0) {
        // ================= TMA producer ================================================================
        if (lane == 0) {
            int s = 0, issued = 0;
            uint32_t ph = 0;
            const uint32_t bytes = (uint32_t)(geo.n_mt + 1) * kTileBytes;
            bool alive = true;
            for (int tile = blockIdx.x; tile < geo.n_tiles && alive; tile += gridDim.x) {
                for (int kc = 0; kc < geo.n_kc; ++kc) {
                    if (issued >= kStages && !mbar_wait(&s_empty[s], ph ^ 1, abort_flag)) { alive = false; break; }
                    const uint32_t base = ring_u32 + (uint32_t)s * kStageBytes;
                    mbar_expect_tx(&s_full[s], bytes);
                    tma_load_2d(base, &tm_h, kc * kBK, 0, &s_full[s]);
                    if (geo.n_mt == 2) tma_load_2d(base + kTileBytes, &tm_h, kc * kBK, kBM, &s_full[s]);
                    tma_load_2d(base + 2 * kTileBytes, &tm_w, kc * kBK, tile * kBN, &s_full[s]);
                    ++issued;
                    if (++s == kStages) { s = 0; ph ^= 1; }
                }
            }
            if (!alive || *abort_flag) {
                // drain: every stage that was filled must have landed before the CTA may leave
                const int back = min(issued, kStages);
                for (int i = 1; i <= back; ++i) {
                    const int it = issued - i;
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try(&s_full[it % kStages], (uint32_t)((it / kStages) & 1)) &&
                           global_ns() - t0 < kWaitLimitNs) {}
                }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer ==================================================================
        if (lane == 0) {
            const uint32_t idesc = make_idesc(kBM, kBN);
            int s = 0, t_local = 0;
            uint32_t ph = 0;
            bool alive = true;
            for (int tile = blockIdx.x; tile < geo.n_tiles && alive; tile += gridDim.x, ++t_local) {
                const int as = t_local & 1;
                const uint32_t use = (uint32_t)(t_local >> 1);
                if (t_local >= 2 && !mbar_wait(&s_acc_empty[as], (use - 1) & 1, abort_flag)) break;
                tc_fence_after();
                for (int kc = 0; kc < geo.n_kc; ++kc) {
                    if (!mbar_wait(&s_full[s], ph, abort_flag)) { alive = false; break; }
                    tc_fence_after();
                    const uint32_t base = ring_u32 + (uint32_t)s * kStageBytes;
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt) {
                        if (mt < geo.n_mt) {
                            const uint32_t d_tmem = tmem_base + (uint32_t)(as * 2 * kBN + mt * kBN);
#pragma unroll
                            for (int k = 0; k < kBK / 16; ++k)
                                tc_mma(d_tmem, make_desc(base + mt * kTileBytes + k * 32),
                                       make_desc(base + 2 * kTileBytes + k * 32), idesc, (kc | k) != 0 ? 1u : 0u);
                        }
                    }
                    tc_commit(&s_empty[s]);                  // the stage is free once these MMAs have read it
                    if (++s == kStages) { s = 0; ph ^= 1; }
                }
                if (alive) tc_commit(&s_acc_full[as]);       // accumulators of this tile are complete
            }
        }
    } else {
        // ================= epilogue warps: one hidden row per thread ===================================
        const int ew = warp - 2;
        const int quad = warp & 3;                            // TMEM lanes this warp may read
        const int mt = ew >> 2;
        const int b = mt * kBM + quad * 32 + lane;
        const bool row_live = b < B && mt < geo.n_mt;
        float invT = 1.f;
        if (row_live) {
            const float T = a.temp[b];
            invT = (T > 0.f && T < CUDART_INF_F) ? 1.f / T : CUDART_NAN_F;
        }
        float st_m = -CUDART_INF_F, st_s = 0.f, gb_s = -CUDART_INF_F, gb_z = 0.f, thr = -CUDART_INF_F;
        int gb_j = -1;
        float tv[KT];
        int tj[KT];
#pragma unroll
        // the list sits at the END of the arrays (slots KT-topk .. KT-1, descending), behind +inf
        // sentinels: its last entry -- the insertion threshold -- is then always slot KT-1, a register
        for (int i = 0; i < KT; ++i) { tv[i] = (i < KT - topk) ? CUDART_INF_F : -CUDART_INF_F; tj[i] = -1; }
        const bool vec_u = a.uniforms && ((K & 3) == 0);
        const bool use_u = row_live && a.uniforms != nullptr;
        float u[kCh];
#pragma unroll
        for (int i = 0; i < kCh; ++i) u[i] = 0.5f;
        int t_local = 0;
        for (int tile = blockIdx.x; tile < geo.n_tiles; tile += gridDim.x, ++t_local) {
            const int as = t_local & 1;
            if (!mbar_wait_warp(&s_acc_full[as], (uint32_t)((t_local >> 1) & 1), abort_flag)) break;
            tc_fence_after();
            if (mt < geo.n_mt) {
#pragma unroll 1
                for (int ch = 0; ch < kBN / kCh; ++ch) {
                    const int j0 = tile * kBN + ch * kCh;
                    // this chunk's uniforms are requested first (they are needed last), and the next
                    // chunk's line is pulled into L2 meanwhile
                    if (use_u && j0 < K) {
                        const float* up = a.uniforms + (size_t)b * K + j0;
                        if (vec_u && j0 + kCh <= K) {
#pragma unroll
                            for (int i = 0; i < kCh / 4; ++i) {
                                const float4 q = __ldg(reinterpret_cast<const float4*>(up) + i);
                                u[4 * i] = q.x; u[4 * i + 1] = q.y; u[4 * i + 2] = q.z; u[4 * i + 3] = q.w;
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < kCh; ++i) u[i] = (j0 + i < K) ? __ldg(up + i) : 0.5f;
                        }
                    }
                    const int jn = (ch + 2 < kBN / kCh) ? j0 + 2 * kCh : (tile + (int)gridDim.x) * kBN;
                    if (use_u && jn < K && (ch & 1) == 0)
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(a.uniforms + (size_t)b * K + jn));
                    uint32_t r[kCh];
                    tc_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(as * 2 * kBN + mt * kBN + ch * kCh), r);
                    // Warp-uniform from here on (j0 and K are): rows that do not exist simply carry nv = 0,
                    // i.e. columns of -inf, so the warp votes below always see all 32 lanes.
                    if (j0 < K) {
                        const int nv = row_live ? min(kCh, K - j0) : 0;
                        float z[kCh];
                        float cmax = -CUDART_INF_F;
#pragma unroll
                        for (int i = 0; i < kCh; ++i) {
                            z[i] = (i < nv) ? __uint_as_float(r[i]) * invT : -CUDART_INF_F;
                            cmax = fmaxf(cmax, z[i]);
                        }
                        if (a.dbg_logits && row_live) {
#pragma unroll
                            for (int i = 0; i < kCh; ++i)
                                if (i < nv) a.dbg_logits[(size_t)b * K + j0 + i] = __uint_as_float(r[i]);
                        }
                        // running max / sum-exp: one rescale per chunk, independent exponentials
                        const float m_new = fmaxf(st_m, cmax);
                        const float m_ref = (m_new == -CUDART_INF_F) ? 0.f : m_new;
                        float acc = 0.f;
#pragma unroll
                        for (int i = 0; i < kCh; ++i) acc += __expf(z[i] - m_ref);
                        st_s = st_s * __expf(st_m - m_ref) + acc;
                        st_m = m_new;
                        if (a.uniforms) {
#pragma unroll
                            for (int i = 0; i < kCh; ++i) {
                                // g = -log(-log u): -log u from a short series in 1-u near 1 (where the fast
                                // logarithm's absolute error would dominate), fast logarithms elsewhere
                                const float uc = fminf(fmaxf(u[i], 0x1p-24f), 1.f - 0x1p-24f);
                                const float t = 1.f - uc;
                                const float lp = t * (1.f + t * (0.5f + t * (0.33333334f + t * (0.25f + t * 0.2f))));
                                const float L = uc > 0.95f ? lp : -__logf(uc);
                                const float sc = z[i] - __logf(L);
                                const bool win = sc > gb_s;               // invalid columns carry z = -inf
                                gb_s = win ? sc : gb_s;
                                gb_j = win ? j0 + i : gb_j;
                                gb_z = win ? z[i] : gb_z;
                            }
                        }
                        // top-k: pull the chunk's maxima out in descending order while they beat the list's
                        // last entry.  The loop is warp-uniform (it runs while any row of the warp still has
                        // a candidate) and everything inside is select-based: one row's insertions never
                        // make the other 31 rows branch.
                        float mx = z[0];
                        int mi = 0;
#pragma unroll
                        for (int i = 1; i < kCh; ++i) {
                            const bool gt = z[i] > mx;                    // strict: ties keep the lower column
                            mx = gt ? z[i] : mx;
                            mi = gt ? i : mi;
                        }
                        while (__any_sync(0xffffffffu, mx > thr)) {
                            const bool take = mx > thr;
                            float cv = take ? mx : -CUDART_INF_F;
                            int cj = j0 + mi;
#pragma unroll
                            for (int p = 0; p < KT; ++p) {                // the +inf sentinels in front never move
                                const bool sw = cv > tv[p];               // equal values keep the lower index first
                                const float ov = tv[p];
                                const int oj = tj[p];
                                tv[p] = sw ? cv : ov;
                                tj[p] = sw ? cj : oj;
                                cv = sw ? ov : cv;
                                cj = sw ? oj : cj;
                            }
                            thr = tj[KT - 1] >= 0 ? tv[KT - 1] : -CUDART_INF_F;   // a threshold only once the list is full
                            // drop the extracted element, find the next maximum
                            float nmx = -CUDART_INF_F;
                            int nmi = 0;
#pragma unroll
                            for (int i = 0; i < kCh; ++i) {
                                z[i] = (take && i == mi) ? -CUDART_INF_F : z[i];
                                const bool gt = z[i] > nmx;
                                nmx = gt ? z[i] : nmx;
                                nmi = gt ? i : nmi;
                            }
                            mx = nmx;
                            mi = nmi;
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_acc_empty[as]);
        }
        // ---- this CTA's record of hidden row b ---------------------------------------------------------
        if (row_live && !*abort_flag) {
            int* irecs = reinterpret_cast<int*>(recs);
            const int c = blockIdx.x;
            recs[rec_at(b, 0, topk) + c] = st_m;
            recs[rec_at(b, 1, topk) + c] = st_s;
            recs[rec_at(b, 2, topk) + c] = gb_s;
            irecs[rec_at(b, 3, topk) + c] = gb_j;
            recs[rec_at(b, 4, topk) + c] = gb_z;
#pragma unroll
            for (int p = 0; p < KT; ++p)
                if (p >= KT - topk) {
                    recs[rec_at(b, 5 + p - (KT - topk), topk) + c] = tv[p];
                    irecs[rec_at(b, 5 + topk + p - (KT - topk), topk) + c] = tj[p];
                }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
    }
    if (threadIdx.x == 0 && s_abort) atomicOr(&ctrl->flags, (uint32_t)VT_FLAG_TIMEOUT);
}

// One warp per hidden row: merge the CTA records, remap, write the outputs.
__global__ void __launch_bounds__(32)
k_head_merge(const HeadArgs a, Ctrl* ctrl, const float* __restrict__ recs, int G) {
    __shared__ float s_stage[kMergeStageWords];
    const int b = blockIdx.x;
    const float T = a.temp[b];
    const bool row_ok = (T > 0.f) && (T < CUDART_INF_F);
    merge_records(a.map, a.out_ids, a.out_logprobs, a.dbg_lse, a.topk, a.uniforms != nullptr, ctrl, recs, b, row_ok, G,
                  s_stage);
}

// ---- host side ----------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static std::mutex mu;
    static EncodeTiledFn fn = nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 matrix [rows, cols] row-major -> boxes of kBK columns x box_rows rows, 128-byte swizzle
bool encode_map(CUtensorMap* tm, const void* base, int rows, int cols, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t gstr[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstr, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool head_dense_supported(int32_t B, int32_t K, int32_t d) {
    return B >= 1 && B <= 2 * kBM && K >= 1 && d >= 8 && (d & 7) == 0;
}

bool head_dense_topk_ok(int32_t topk) { return topk >= 1 && topk <= kMaxTopk; }

size_t head_dense_scratch_bytes(int32_t B, int32_t K, int32_t topk) {
    (void)K;
    return align_up((size_t)kMaxGrid * B * rec_fields(topk) * 4, 256);
}

cudaError_t launch_head_dense(const HeadArgs& a, Ctrl* ctrl, uint8_t* scratch, cudaStream_t s) {
    if (!head_dense_supported(a.B, a.K, a.d) || !head_dense_topk_ok(a.topk)) return cudaErrorInvalidValue;
    CUtensorMap tm_h, tm_w;
    if (!encode_map(&tm_h, a.h, a.B, a.d, kBM) || !encode_map(&tm_w, a.W, a.K, a.d, kBN)) return cudaErrorInvalidValue;
    DenseGeo geo{};
    geo.n_tiles = (a.K + kBN - 1) / kBN;
    geo.n_kc = (a.d + kBK - 1) / kBK;
    geo.n_mt = a.B > kBM ? 2 : 1;
    int grid = num_sms();
    if (grid > kMaxGrid) grid = kMaxGrid;
    if (grid > geo.n_tiles) grid = geo.n_tiles;
    static int attr_done[64] = {0};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !attr_done[dev]) {
        cudaError_t e = cudaFuncSetAttribute(k_head_dense<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDynSmem);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(k_head_dense<kMaxTopk>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDynSmem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_done[dev] = 1;
    }
    float* recs = reinterpret_cast<float*>(scratch);
    if (a.topk <= 8) k_head_dense<8><<<grid, kThreads, kDynSmem, s>>>(a, ctrl, recs, geo, tm_h, tm_w);
    else k_head_dense<kMaxTopk><<<grid, kThreads, kDynSmem, s>>>(a, ctrl, recs, geo, tm_h, tm_w);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    k_head_merge<<<a.B, 32, 0, s>>>(a, ctrl, recs, grid);
    count_launch(2);
    return cudaGetLastError();
}

}  // namespace vt
