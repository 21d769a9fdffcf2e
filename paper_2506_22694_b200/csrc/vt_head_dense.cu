// Batched-serving head (17 <= B <= 256 hidden rows): the projection is a real dense contraction
// and runs on the 5th-generation tensor cores (Algorithm 2, the drafter-forward and index-mapping steps, with many sequences and
// tree nodes drafted at once).
//
//   D[b, j] = sum_i h[b, i] * W_trim[j, i]      M = hidden rows (the TMEM lanes), N = vocabulary rows
//                                               of a tile (TMEM columns), K-loop over d in 64-column steps
//
// B <= 128: one persistent CTA per SM walks vocabulary tiles (M = 128, tcgen05.mma.cta_group::1).
// B  > 128: the two CTAs of a cluster act as one MMA of M = 256 (cta_group::2).  Each CTA stages its
// own 128 hidden rows and HALF of the tile's vocabulary rows; the tensor cores of both SMs read the
// two halves of the B operand from both shared memories.  Per SM and flop this halves the operand
// bytes staged and read compared with two M tiles in one CTA, which is what bounded that form.
//
// Warp 0 feeds a shared-memory ring with TMA tensor copies (128-byte swizzle, every CTA fetches its own tiles); in a pair
// both CTAs' copies count their bytes on the leader's barrier.  A ring stage holds one or two 64-column steps of d
// (two where three such stages fit): the two threads that drive the ring wait and release once per stage, and their
// turn-around is on its critical path, so they also move their cursors by additions only.  One thread of warp 1 (of the leader)
// issues the MMAs (bf16 x bf16 -> fp32) with the operands described in place by shared-memory
// descriptors and the accumulators in tensor memory: two accumulator stages of up to 256 columns, so
// the epilogue of tile t overlaps the MMAs of tile t+1.  tcgen05.commit releases ring stages and
// publishes accumulators (to both CTAs of a pair).  Eight epilogue warps read the accumulators back
// with tcgen05.ld -- TMEM lane = hidden row; the two warps of a lane quadrant take one half of a tile's
// columns each -- 16 columns at a time: running max / sum-exp of z = logit / T_b, Gumbel-max candidate
// from the caller's uniforms, and a sorted top-k list kept in registers.  Logits never go to HBM.  The
// two column halves of a row are merged through shared memory; per CTA (pair) and hidden row one
// record goes to scratch; a second small kernel (one warp per hidden row) merges the records,
// applies the index mapper and writes the outputs.  Every wait is bounded; on expiry the CTA raises
// VT_FLAG_TIMEOUT and leaves after releasing its tensor memory.
#include <cuda.h>

#include <mutex>

#include "vt_common.cuh"
#include "vt_head_common.cuh"

namespace vt {

namespace {

constexpr int kBM = 128;                  // hidden rows per CTA (TMEM lanes)
constexpr int kMaxBN = 256;               // vocabulary rows per tile at most (TMEM columns per accumulator)
constexpr int kBK = 64;                   // columns of d per ring stage: 128 bytes, one swizzle row
constexpr int kMaxSub = 2;                // d-steps of kBK columns one ring stage holds at most
constexpr int kMaxStages = 8;
constexpr int kHTileBytes = kBM * kBK * 2; // 16 KB: the hidden-row operand of a stage
constexpr int kParts8 = 2, kParts16 = 2;  // epilogue warps per TMEM lane quadrant for lists of 8 / 16 (3 and 4 were no
                                          // faster: the epilogue is bound by the instructions it issues, not by latency)
constexpr int epi_threads(int parts) { return (2 + 4 * parts) * 32; }   // TMA producer, MMA issuer, epilogue warps
constexpr int kCh = 16;                   // accumulator columns per epilogue step (keeps the row state in registers)
constexpr int kTmemCols = 512;            // 2 accumulator stages x kMaxBN columns
constexpr int kMaxTopk = 16;              // top-k list lives in registers
constexpr unsigned long long kWaitLimitNs = 2000000000ull;
constexpr size_t kRingBudget = 225 * 1024;   // ring bytes at most (227 KB per CTA less alignment slack and statics)

// Phase stamps (-DVT_STAMPS builds only): one thread per role writes %globaltimer into a region behind the
// records; bench.py --case stamps reads them back.  Slots per CTA: 0 entry, 1 set up (barriers, tensor
// memory), 2 producer released by the launch dependency, 3 first stage landed (MMA issuer), 4 / 5 MMAs of the
// CTA's first / last tile issued, 6 / 7 accumulators of the first / last tile complete (epilogue warp 0),
// 8 / 9 first / last tile's epilogue done, 10 record written, 11 leaving; CTA 0 also carries the merge
// kernel's 12 start (records complete) and 13 end for hidden row 0.
#ifdef VT_STAMPS
#define VT_DSTAMP(slot) do { stamps[(size_t)blockIdx.x * kStampSlots + (slot)] = global_ns(); } while (0)
#else
#define VT_DSTAMP(slot) do {} while (0)
#endif

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
// Same, called by all 32 lanes of a warp that expects to wait long (a whole tile of MMAs): lane 0
// polls with pauses -- 256 spinning threads cost issue slots and power the tensor pipe wants -- then
// every lane observes the completed phase itself.  The outcome is voted on so the lanes never part
// ways before a warp-collective instruction.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* b, uint32_t parity, volatile int* abort_flag) {
    bool ok = true;
    if ((threadIdx.x & 31) == 0 && !mbar_try(b, parity)) {
        const unsigned long long t0 = global_ns();
        for (;;) {
            __nanosleep(128);
            if (mbar_try(b, parity)) break;
            if (*abort_flag) { ok = false; break; }
            if (global_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; ok = false; break; }
        }
    }
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (ok) ok = mbar_try(b, parity) || mbar_wait(b, parity, abort_flag);
    return __all_sync(0xffffffffu, ok);
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

// Programmatic dependent launch: let the next launch on the stream become resident / wait until the
// work this launch depends on has completed and its writes are visible (no-ops in a plain launch).
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---- CTA-pair forms (cta_group::2): two CTAs of a cluster act as one 256-row MMA ---------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same variable in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// tensor copy into THIS CTA's shared memory whose bytes are counted on a barrier of either CTA of the pair
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar_cluster), "r"(x), "r"(y) : "memory");
}
// arrives on the barrier at this shared-memory offset in both CTAs once the MMAs issued so far are done:
// one commit per CTA of the pair (the peer's barrier by its shared::cluster address)
__device__ __forceinline__ void tc_commit_pair(uint64_t* bar) {
    const uint32_t own = smem_u32(bar);
    const uint32_t peer = mapa_u32(own, 1);
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(own) : "memory");
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(peer) : "memory");
}
// D[tmem of both CTAs] (+)= A * B^T, 256 x N x 16: each CTA supplies 128 rows of A and N/2 rows of B
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    const uint32_t z = 0;
    asm volatile(
        "{ .reg .pred p; setp.ne.b32 p, %4, 0;"
        " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p; }"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc), "r"(z) : "memory");
}

struct DenseGeo {
    int n_tiles;      // vocabulary tiles of bn rows
    int n_kc;         // ring steps per tile: ceil(d / kBK)
    int bn;           // vocabulary rows per tile (per CTA pair when paired); a multiple of 32, <= kMaxBN
    int n_stages;     // ring depth
    int stage_bytes;  // bytes one CTA stages per step: hidden rows + its share of the vocabulary rows
    int n_groups;     // CTAs (or CTA pairs) walking the tiles round-robin
    int sub;          // d-steps per ring stage (1 or 2): one wait and one release per stage, so two steps per stage halve
                      // what the two single threads that drive the ring spend per MMA; taken when three such stages fit
};

// Per-thread state of one hidden row over the columns the thread has seen.
template <int KT>
struct RowState {
    float m, s;               // running max and sum of exp(z - m)
    float gb_s, gb_z;         // best Gumbel score and its z
    int gb_j;
    float tv[KT];             // top-k list at the END of the arrays (slots KT-topk .. KT-1, descending)
    int tj[KT];               // behind +inf sentinels: the insertion threshold is always slot KT-1
};

// Insert (cv, cj) into the sorted list with selects only; equal values keep the entry already there.
template <int KT>
__device__ __forceinline__ void list_insert(float (&tv)[KT], int (&tj)[KT], float cv, int cj) {
#pragma unroll
    for (int p = 0; p < KT; ++p) {
        const bool sw = cv > tv[p];
        const float ov = tv[p];
        const int oj = tj[p];
        tv[p] = sw ? cv : ov;
        tj[p] = sw ? cj : oj;
        cv = sw ? ov : cv;
        cj = sw ? oj : cj;
    }
}

// KT: capacity of the register top-k list (8 or kMaxTopk).  PAIR: two CTAs of a cluster form one MMA.
// PARTS: epilogue warps per TMEM lane quadrant; each takes a contiguous share of a tile's 16-column chunks.
// The epilogue is a long chain of dependent arithmetic per column: it runs at the rate the schedulers can
// interleave warps, so more warps per scheduler shorten it almost in proportion.
template <int KT, bool PAIR, int PARTS>
__global__ void __launch_bounds__(epi_threads(PARTS), 1)
k_head_dense(const HeadArgs a, Ctrl* ctrl, float* __restrict__ recs, const DenseGeo geo,
             const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ CUtensorMap tm_w) {
    extern __shared__ uint8_t s_dyn[];
    __shared__ uint64_t s_full[kMaxStages], s_empty[kMaxStages], s_acc_full[2], s_acc_empty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#ifdef VT_STAMPS
    unsigned long long* stamps = reinterpret_cast<unsigned long long*>(
        reinterpret_cast<uint8_t*>(recs) + align_up_dev((size_t)kMaxGrid * a.B * rec_fields(a.topk) * 4, 256));
    if (threadIdx.x == 0) VT_DSTAMP(0);
#endif
    // identical in both CTAs of a pair: the MMA addresses the peer's operands by the leader's offsets
    uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(s_dyn) + 1023) & ~(uintptr_t)1023);
    const uint32_t ring_u32 = smem_u32(ring);
    const int B = a.B, K = a.K, topk = a.topk;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;          // 0 = leader: issues the MMAs, owns the full barriers
    const int group = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int bn = geo.bn, n_stages = geo.n_stages;
    const int w_rows = PAIR ? bn / 2 : bn;                         // vocabulary rows this CTA stages per step

    if (threadIdx.x == 0) {
        // the two tensor maps are fetched now, not by the first copy that needs them
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_h)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_w)) : "memory");
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(&s_full[s], 1); mbar_init(&s_empty[s], 1); }
        for (int p = 0; p < 2; ++p) { mbar_init(&s_acc_full[p], 1); mbar_init(&s_acc_empty[p], (PAIR ? 2 : 1) * 4 * PARTS); }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // tensor memory: all 512 columns of the SM (one CTA per SM by shared-memory size)
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(&s_tmem_base)), "r"((uint32_t)kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(&s_tmem_base)), "r"((uint32_t)kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    if (PAIR) cluster_sync_all(); else __syncthreads();           // barriers initialised in both CTAs before any signal
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    volatile int* abort_flag = &s_abort;
    griddep_launch_dependents();                                  // the merge kernel may take its seats
#ifdef VT_STAMPS
    if (threadIdx.x == 0) VT_DSTAMP(1);
#endif

    if (warp == 0) {
        // ================= TMA producer (both CTAs of a pair) ==========================================
        if (lane == 0) {
            // fills are numbered g = 0 .. total-1 over (tile, step in d); fill g uses stage g % n_stages
            const int my_tiles = (geo.n_tiles - group + geo.n_groups - 1) / geo.n_groups;
            const int sub = geo.sub;
            const int n_ks = (geo.n_kc + sub - 1) / sub;               // ring stages per tile
            const int total = my_tiles * n_ks;
            const uint32_t sub_bytes = (uint32_t)geo.stage_bytes / (uint32_t)sub;
            const uint32_t full0 = PAIR ? mapa_u32(smem_u32(&s_full[0]), 0) : 0u;      // the leader's full barriers
            auto subs_of = [&](int g) { return min(sub, geo.n_kc - (g % n_ks) * sub); };
            auto load_w = [&](int g) {
                const int s = g % n_stages, tile = group + (g / n_ks) * geo.n_groups;
                for (int u = 0; u < subs_of(g); ++u) {
                    const int kc = (g % n_ks) * sub + u;
                    const uint32_t dst = ring_u32 + (uint32_t)s * (uint32_t)geo.stage_bytes + (uint32_t)u * sub_bytes + kHTileBytes;
                    if (PAIR) tma_load_2d_pair(dst, &tm_w, kc * kBK, tile * bn + (int)rank * w_rows, full0 + (uint32_t)(s * sizeof(uint64_t)));
                    else tma_load_2d(dst, &tm_w, kc * kBK, tile * bn, &s_full[s]);
                }
            };
            auto load_h = [&](int g) {
                const int s = g % n_stages;
                for (int u = 0; u < subs_of(g); ++u) {
                    const int kc = (g % n_ks) * sub + u;
                    const uint32_t dst = ring_u32 + (uint32_t)s * (uint32_t)geo.stage_bytes + (uint32_t)u * sub_bytes;
                    if (PAIR) tma_load_2d_pair(dst, &tm_h, kc * kBK, (int)rank * kBM, full0 + (uint32_t)(s * sizeof(uint64_t)));
                    else tma_load_2d(dst, &tm_h, kc * kBK, 0, &s_full[s]);
                }
            };
            auto bytes_of = [&](int g) { return (uint32_t)(PAIR ? 2 : 1) * sub_bytes * (uint32_t)subs_of(g); };
            // The weights are static: the first ring of them is requested before the work this launch
            // depends on has finished; everything that work may have produced is touched after the wait.
            const int pre = min(n_stages, total);
            for (int g = 0; g < pre; ++g) {
                if (rank == 0) mbar_expect_tx(&s_full[g], bytes_of(g));
                load_w(g);
            }
            griddep_wait();
            VT_DSTAMP(2);
            for (int g = 0; g < pre; ++g) load_h(g);
            int done = pre;
            {
                // steady state: the cursor over (stage, step in d, tile) moves by additions only -- this thread's
                // turn-around between "stage free" and "copies asked for" is on the ring's critical path
                int sc = pre % n_stages, ks = pre % n_ks, tl = pre / n_ks;
                uint32_t par = (uint32_t)((pre / n_stages) & 1) ^ 1u;
                const uint32_t pair_mul = PAIR ? 2u : 1u;
                for (int g = pre; g < total; ++g, ++done) {
                    if (!mbar_wait(&s_empty[sc], par, abort_flag)) break;
                    const int subs = min(sub, geo.n_kc - ks * sub);
                    if (rank == 0) mbar_expect_tx(&s_full[sc], pair_mul * sub_bytes * (uint32_t)subs);
                    const uint32_t dst0 = ring_u32 + (uint32_t)sc * (uint32_t)geo.stage_bytes;
                    const uint32_t bar = full0 + (uint32_t)(sc * sizeof(uint64_t));
                    const int row_w = (group + tl * geo.n_groups) * bn + (PAIR ? (int)rank * w_rows : 0);
#pragma unroll
                    for (int u = 0; u < kMaxSub; ++u) {
                        if (u < subs) {
                            const int x = (ks * sub + u) * kBK;
                            if (PAIR) {
                                tma_load_2d_pair(dst0 + (uint32_t)u * sub_bytes, &tm_h, x, (int)rank * kBM, bar);
                                tma_load_2d_pair(dst0 + (uint32_t)u * sub_bytes + kHTileBytes, &tm_w, x, row_w, bar);
                            } else {
                                tma_load_2d(dst0 + (uint32_t)u * sub_bytes, &tm_h, x, 0, &s_full[sc]);
                                tma_load_2d(dst0 + (uint32_t)u * sub_bytes + kHTileBytes, &tm_w, x, row_w, &s_full[sc]);
                            }
                        }
                    }
                    if (++sc == n_stages) { sc = 0; par ^= 1u; }
                    if (++ks == n_ks) { ks = 0; ++tl; }
                }
            }
            if (done == total && !*abort_flag) {
                // every fill consumed: all copies have landed and every commit aimed at this CTA's
                // barriers has arrived before the CTA may leave
                for (int g = max(0, total - n_stages); g < total; ++g)
                    if (!mbar_wait(&s_empty[g % n_stages], (uint32_t)((g / n_stages) & 1), abort_flag)) break;
            }
            if (*abort_flag) {
                // something timed out: give copies still in flight time to land before the memory goes away
                const unsigned long long t0 = global_ns();
                while (global_ns() - t0 < 200000ull) {}
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer (leader CTA only) ================================================
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = make_idesc(PAIR ? 2 * kBM : kBM, bn);
            const uint64_t desc_a0 = make_desc(ring_u32);                       // (the ring is 1024-byte aligned and under 256 KB:
            const uint64_t sub16 = (uint64_t)(((uint32_t)geo.stage_bytes / (uint32_t)geo.sub) >> 4);   //  adding byte offsets >> 4 stays inside the address field)
            int s = 0, t_local = 0;
            uint32_t ph = 0;
            bool alive = true;
            for (int tile = group; tile < geo.n_tiles && alive; tile += geo.n_groups, ++t_local) {
                const int as = t_local & 1;
                const uint32_t use = (uint32_t)(t_local >> 1);
                if (t_local >= 2 && !mbar_wait(&s_acc_empty[as], (use - 1) & 1, abort_flag)) { alive = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(as * kMaxBN);
                const int n_ks = (geo.n_kc + geo.sub - 1) / geo.sub;
                for (int ks = 0; ks < n_ks; ++ks) {
                    const int kc = ks * geo.sub;
                    if (!mbar_wait(&s_full[s], ph, abort_flag)) { alive = false; break; }
#ifdef VT_STAMPS
                    if (t_local == 0 && kc == 0) VT_DSTAMP(3);
#endif
                    tc_fence_after();
                    const int subs = min(geo.sub, geo.n_kc - kc);
                    const uint64_t da0 = desc_a0 + (uint64_t)(((uint32_t)s * (uint32_t)geo.stage_bytes) >> 4);
                    const uint64_t db0 = da0 + (uint64_t)(kHTileBytes >> 4);
#pragma unroll
                    for (int u = 0; u < kMaxSub; ++u) {
                        if (u < subs) {
#pragma unroll
                            for (int k = 0; k < kBK / 16; ++k) {
                                const uint64_t step = (uint64_t)u * sub16 + (uint64_t)(k * 2);
                                if (PAIR) tc_mma_pair(d_tmem, da0 + step, db0 + step, idesc, (kc | u | k) != 0 ? 1u : 0u);
                                else tc_mma(d_tmem, da0 + step, db0 + step, idesc, (kc | u | k) != 0 ? 1u : 0u);
                            }
                        }
                    }
                    // the stage is free (in both CTAs) once these MMAs have read it
                    if (PAIR) tc_commit_pair(&s_empty[s]); else tc_commit(&s_empty[s]);
                    if (++s == n_stages) { s = 0; ph ^= 1; }
                }
                if (alive) {                                      // accumulators of this tile are complete
                    if (PAIR) tc_commit_pair(&s_acc_full[as]); else tc_commit(&s_acc_full[as]);
#ifdef VT_STAMPS
                    if (t_local == 0) VT_DSTAMP(4);
                    VT_DSTAMP(5);
#endif
                }
            }
            // the last accumulators have been read (every arrival of the peer has landed) before leaving
            for (int t = max(0, t_local - 2); t < t_local && alive; ++t)
                if (!mbar_wait(&s_acc_empty[t & 1], (uint32_t)((t >> 1) & 1), abort_flag)) break;
        }
    } else {
        // ================= epilogue warps: one hidden row and one share of the tile's columns per thread =
        const int ew = warp - 2;
        const int quad = warp & 3;                            // TMEM lanes this warp may read
        const int part = ew >> 2;                             // which share of the tile's chunks
        const int n_ch_tile = bn / kCh;
        const int ch_lo = part * n_ch_tile / PARTS, ch_hi = (part + 1) * n_ch_tile / PARTS;
        const int b = (int)rank * kBM + quad * 32 + lane;
        const bool row_live = b < B;
        griddep_wait();                                       // temp, uniforms and the record scratch belong to earlier work until here
        float invT = 1.f;
        if (row_live) {
            const float T = a.temp[b];
            invT = (T > 0.f && T < CUDART_INF_F) ? 1.f / T : CUDART_NAN_F;
        }
        RowState<KT> st;
        st.m = -CUDART_INF_F; st.s = 0.f; st.gb_s = -CUDART_INF_F; st.gb_z = 0.f; st.gb_j = -1;
        float thr = -CUDART_INF_F;
#pragma unroll
        for (int i = 0; i < KT; ++i) { st.tv[i] = (i < KT - topk) ? CUDART_INF_F : -CUDART_INF_F; st.tj[i] = -1; }
        const bool vec_u = a.uniforms && ((K & 3) == 0) && ((reinterpret_cast<uintptr_t>(a.uniforms) & 15) == 0);
        const bool use_u = row_live && a.uniforms != nullptr;
        const uint32_t acc_empty_bar = PAIR ? mapa_u32(smem_u32(&s_acc_empty[0]), 0) : 0u;
        float u[kCh];
#pragma unroll
        for (int i = 0; i < kCh; ++i) u[i] = 0.5f;
        int t_local = 0;
        for (int tile = group; tile < geo.n_tiles; tile += geo.n_groups, ++t_local) {
            const int as = t_local & 1;
            if (!mbar_wait_warp(&s_acc_full[as], (uint32_t)((t_local >> 1) & 1), abort_flag)) break;
#ifdef VT_STAMPS
            if (warp == 2 && lane == 0) { if (t_local == 0) VT_DSTAMP(6); VT_DSTAMP(7); }
#endif
            tc_fence_after();
            const int jt = tile * bn;                         // first vocabulary row of the tile
#pragma unroll 1
            for (int ch = ch_lo; ch < ch_hi; ++ch) {
                const int j0 = jt + ch * kCh;
                // this chunk's uniforms are requested first (they are needed last), and a later
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
                const int jn = (ch + 2 < ch_hi) ? j0 + 2 * kCh : jt + geo.n_groups * bn + ch_lo * kCh;
                if (use_u && jn < K && (ch & 1) == 0)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(a.uniforms + (size_t)b * K + jn));
                uint32_t r[kCh];
                tc_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(as * kMaxBN + ch * kCh), r);
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
                    const float m_new = fmaxf(st.m, cmax);
                    const float m_ref = (m_new == -CUDART_INF_F) ? 0.f : m_new;
                    float acc = 0.f;
#pragma unroll
                    for (int i = 0; i < kCh; ++i) acc += __expf(z[i] - m_ref);
                    st.s = st.s * __expf(st.m - m_ref) + acc;
                    st.m = m_new;
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
                            const bool win = sc > st.gb_s;            // invalid columns carry z = -inf
                            st.gb_s = win ? sc : st.gb_s;
                            st.gb_j = win ? j0 + i : st.gb_j;
                            st.gb_z = win ? z[i] : st.gb_z;
                        }
                    }
                    // top-k: pull the chunk's maxima out in descending order while they beat the list's
                    // last entry.  The loop is warp-uniform (it runs while any row of the warp still has
                    // a candidate) and everything inside is select-based: one row's insertions never
                    // make the other 31 rows branch.
                    // a NaN logit poisons the row's lse (reported through VT_FLAG_NAN_ROW) but must not hide the
                    // chunk's other candidates: it competes as -inf
#pragma unroll
                    for (int i = 0; i < kCh; ++i) z[i] = (z[i] == z[i]) ? z[i] : -CUDART_INF_F;
                    // candidates: the columns that beat the list's last entry as it stands; they go in by
                    // ascending column (equal values keep the lower column ahead), one per trip of a warp-
                    // uniform loop that runs while any row still has one.  A candidate that has fallen under
                    // the entry that moved up meanwhile simply finds no slot.
                    uint32_t cand = 0;
#pragma unroll
                    for (int i = 0; i < kCh; ++i) cand |= (z[i] > thr) ? (1u << i) : 0u;
                    while (__any_sync(0xffffffffu, cand != 0)) {
                        const bool take = cand != 0;
                        const int i = take ? __ffs(cand) - 1 : 0;
                        float q8[8], q4[4], q2[2];
#pragma unroll
                        for (int k = 0; k < 8; ++k) q8[k] = (i & 1) ? z[2 * k + 1] : z[2 * k];
#pragma unroll
                        for (int k = 0; k < 4; ++k) q4[k] = (i & 2) ? q8[2 * k + 1] : q8[2 * k];
#pragma unroll
                        for (int k = 0; k < 2; ++k) q2[k] = (i & 4) ? q4[2 * k + 1] : q4[2 * k];
                        const float v = (i & 8) ? q2[1] : q2[0];
                        list_insert<KT>(st.tv, st.tj, take ? v : -CUDART_INF_F, j0 + i);
                        thr = st.tj[KT - 1] >= 0 ? st.tv[KT - 1] : -CUDART_INF_F;   // a threshold only once the list is full
                        cand &= cand - 1;
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (PAIR) mbar_arrive_cluster(acc_empty_bar + (uint32_t)(as * sizeof(uint64_t)));
                else mbar_arrive(&s_acc_empty[as]);
            }
#ifdef VT_STAMPS
            if (warp == 2 && lane == 0) { if (t_local == 0) VT_DSTAMP(8); VT_DSTAMP(9); }
#endif
        }
        // ---- the column shares of a row meet in shared memory (the ring is idle by now: the last
        // accumulators were complete, so every MMA has read its operands and every copy has landed) ----
        float* xch = reinterpret_cast<float*>(ring);
        constexpr int kXchFields = 5 + 2 * KT;
        const int slot = quad * 32 + lane;                    // row within the CTA
        const bool ok = !*abort_flag;
        if (part > 0 && ok) {
            float* x = xch + (size_t)(part - 1) * kXchFields * kBM + slot;     // field-major: conflict-free
            x[0 * kBM] = st.m; x[1 * kBM] = st.s; x[2 * kBM] = st.gb_s; x[3 * kBM] = __int_as_float(st.gb_j); x[4 * kBM] = st.gb_z;
#pragma unroll
            for (int p = 0; p < KT; ++p) { x[(5 + p) * kBM] = st.tv[p]; x[(5 + KT + p) * kBM] = __int_as_float(st.tj[p]); }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(4 * PARTS * 32) : "memory");
        if (part == 0 && ok && row_live) {
#pragma unroll 1
            for (int o = 0; o < PARTS - 1; ++o) {
                const float* x = xch + (size_t)o * kXchFields * kBM + slot;
                lse_merge(st.m, st.s, x[0 * kBM], x[1 * kBM]);
                const float os = x[2 * kBM];
                const int oj = __float_as_int(x[3 * kBM]);
                if (better(os, oj, st.gb_s, st.gb_j) && oj >= 0) { st.gb_s = os; st.gb_j = oj; st.gb_z = x[4 * kBM]; }
#pragma unroll
                for (int p = 0; p < KT; ++p) {
                    // entries of the other share: equal values must still order by index, so compare keys
                    float cv = x[(5 + p) * kBM];
                    int cj = __float_as_int(x[(5 + KT + p) * kBM]);
                    if (p < KT - topk) continue;              // its sentinels
#pragma unroll
                    for (int q = 0; q < KT; ++q) {
                        const bool sw = key64(cv, cj) > key64(st.tv[q], st.tj[q]) && q >= KT - topk;
                        const float ov = st.tv[q];
                        const int oj2 = st.tj[q];
                        st.tv[q] = sw ? cv : ov;
                        st.tj[q] = sw ? cj : oj2;
                        cv = sw ? ov : cv;
                        cj = sw ? oj2 : cj;
                    }
                }
            }
            // ---- this CTA's record of hidden row b ---------------------------------------------------------
            unsigned long long* kp = rec_keys(recs, b, topk);
            float* fp = rec_f32(recs, b, topk);
            const int c = group;
            fp[c] = st.m;
            fp[kMaxGrid + c] = st.s;
            fp[2 * kMaxGrid + c] = st.gb_z;
            kp[c] = st.gb_j >= 0 ? key64(st.gb_s, st.gb_j) : 0ull;
#pragma unroll
            for (int p = 0; p < KT; ++p)
                if (p >= KT - topk)
                    kp[(size_t)(1 + p - (KT - topk)) * kMaxGrid + c] = st.tj[p] >= 0 ? key64(st.tv[p], st.tj[p]) : 0ull;
        }
#ifdef VT_STAMPS
        if (warp == 2 && lane == 0) VT_DSTAMP(10);
#endif
    }
    tc_fence_before();
    __syncwarp();                                                 // lanes of the single-thread roles rejoin their warps
    if (PAIR) cluster_sync_all(); else __syncthreads();           // nobody leaves while its peer may still signal it
    if (warp == 1) {
        tc_fence_after();
        if (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
    }
    if (threadIdx.x == 0 && s_abort) atomicOr(&ctrl->flags, (uint32_t)VT_FLAG_TIMEOUT);
#ifdef VT_STAMPS
    if (threadIdx.x == 0) VT_DSTAMP(11);
#endif
}

// Two warps per hidden row (candidates / statistics): merge the CTA records, remap, write the outputs.
__global__ void __launch_bounds__(64)
k_head_merge(const HeadArgs a, Ctrl* ctrl, float* __restrict__ recs, int G) {
    __shared__ __align__(8) float s_stage[kMergeStageWords];
    __shared__ float s_xch;
    const int b = blockIdx.x;
    griddep_launch_dependents();                                  // the next step may start fetching its weights
    griddep_wait();                                               // the records are complete
#ifdef VT_STAMPS
    unsigned long long* stamps = reinterpret_cast<unsigned long long*>(
        reinterpret_cast<uint8_t*>(recs) + align_up_dev((size_t)kMaxGrid * a.B * rec_fields(a.topk) * 4, 256));
    if (b == 0 && threadIdx.x == 0) stamps[12] = global_ns();
#endif
    const float T = a.temp[b];
    const bool row_ok = (T > 0.f) && (T < CUDART_INF_F);
    const MergeOut mo{a.map, a.out_ids, a.out_logprobs, a.dbg_lse, a.topk, a.uniforms != nullptr};
    merge_records(mo, ctrl, recs, b, row_ok, G, s_stage, threadIdx.x < 32 ? kRoleCand : kRoleStats, &s_xch, 1);
#ifdef VT_STAMPS
    if (b == 0 && threadIdx.x == 0) stamps[13] = global_ns();
#endif
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

// Tile width: the vocabulary is dealt to `groups` CTAs (pairs) in tiles of bn rows; the slowest group
// works ceil(tiles / groups) * bn rows.  Smallest such makespan wins, the wider tile on equal terms
// (fewer re-reads of the hidden rows).
DenseGeo make_geo(int32_t K, int32_t d, bool pair, int max_groups) {
    DenseGeo g{};
    long best = -1;
    for (int bn = kMaxBN; bn >= 32; bn -= 32) {
        const long tiles = (K + bn - 1) / bn;
        const long span = ((tiles + max_groups - 1) / max_groups) * bn;
        if (best < 0 || span < best) { best = span; g.bn = bn; }
    }
    g.n_tiles = (K + g.bn - 1) / g.bn;
    g.n_kc = (d + kBK - 1) / kBK;
    g.n_groups = g.n_tiles < max_groups ? g.n_tiles : max_groups;
    const int step_bytes = kHTileBytes + (pair ? g.bn / 2 : g.bn) * kBK * 2;
    g.sub = (3 * kMaxSub * (size_t)step_bytes <= kRingBudget && g.n_kc >= kMaxSub) ? kMaxSub : 1;
    g.stage_bytes = step_bytes * g.sub;
    g.n_stages = (int)(kRingBudget / (size_t)g.stage_bytes);
    if (g.n_stages > kMaxStages) g.n_stages = kMaxStages;
    return g;
}

template <int KT, bool PAIR, int PARTS>
cudaError_t launch_variant(const HeadArgs& a, Ctrl* ctrl, float* recs, const DenseGeo& geo, const CUtensorMap& tm_h,
                           const CUtensorMap& tm_w, cudaStream_t s) {
    static int attr_done[64] = {0};
    const size_t smem = (size_t)geo.n_stages * geo.stage_bytes + 1024;   // + slack to align the ring to 1024 bytes
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !attr_done[dev]) {
        cudaError_t e = cudaFuncSetAttribute(k_head_dense<KT, PAIR, PARTS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)(kRingBudget + 1024));
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_done[dev] = 1;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(PAIR ? 2 * geo.n_groups : geo.n_groups));
    cfg.blockDim = dim3(epi_threads(PARTS));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = PAIR ? 2 : 1;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = a.overlap ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, k_head_dense<KT, PAIR, PARTS>, a, ctrl, recs, geo, tm_h, tm_w);
}

}  // namespace

bool head_dense_supported(int32_t B, int32_t K, int32_t d) {
    return B >= 1 && B <= 2 * kBM && K >= 1 && d >= 8 && (d & 7) == 0;
}

bool head_dense_topk_ok(int32_t topk) { return topk >= 1 && topk <= kMaxTopk; }

size_t head_dense_scratch_bytes(int32_t B, int32_t K, int32_t topk) {
    (void)K;
    return align_up((size_t)kMaxGrid * B * rec_fields(topk) * 4, 256) + kStampBytes;
}

#ifdef VT_STAMPS
size_t head_dense_stamps_offset(int32_t B, int32_t topk) {
    return align_up((size_t)kMaxGrid * B * rec_fields(topk) * 4, 256);
}
#endif

cudaError_t launch_head_dense(const HeadArgs& a, Ctrl* ctrl, uint8_t* scratch, cudaStream_t s) {
    if (!head_dense_supported(a.B, a.K, a.d) || !head_dense_topk_ok(a.topk)) return cudaErrorInvalidValue;
    const bool pair = a.B > kBM;                       // more than one MMA's worth of hidden rows: CTA pairs
    int max_groups = pair ? num_sms() / 2 : num_sms();
    if (max_groups > kMaxGrid) max_groups = kMaxGrid;
    if (max_groups < 1) return cudaErrorInvalidValue;
    const DenseGeo geo = make_geo(a.K, a.d, pair, max_groups);
    CUtensorMap tm_h, tm_w;
    if (!encode_map(&tm_h, a.h, a.B, a.d, kBM) || !encode_map(&tm_w, a.W, a.K, a.d, pair ? geo.bn / 2 : geo.bn))
        return cudaErrorInvalidValue;
    float* recs = reinterpret_cast<float*>(scratch);
    cudaError_t e;
    if (a.topk <= 8) e = pair ? launch_variant<8, true, kParts8>(a, ctrl, recs, geo, tm_h, tm_w, s)
                              : launch_variant<8, false, kParts8>(a, ctrl, recs, geo, tm_h, tm_w, s);
    else e = pair ? launch_variant<kMaxTopk, true, kParts16>(a, ctrl, recs, geo, tm_h, tm_w, s)
                  : launch_variant<kMaxTopk, false, kParts16>(a, ctrl, recs, geo, tm_h, tm_w, s);
    if (e != cudaSuccess) return e;
    // the merge always follows its own producer closely: it takes its seats early and waits on the device
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)a.B);
    cfg.blockDim = dim3(64);
    cfg.stream = s;
    cudaLaunchAttribute at{};
    at.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &at;
    cfg.numAttrs = 1;
    count_launch(2);
    e = cudaLaunchKernelEx(&cfg, k_head_merge, a, ctrl, recs, geo.n_groups);
    if (e != cudaSuccess || !a.tree.pool_token) return e;
    // tree drafting: the expansion needs every row's merge, i.e. the whole merge grid: one more launch
    return launch_tree_expand(a.out_ids, a.out_logprobs, a.B, a.topk, 1 + a.topk, 1, a.tree, s);
}

}  // namespace vt
