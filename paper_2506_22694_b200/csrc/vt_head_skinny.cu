// Trimmed LM head for a few hidden rows (B <= 16), fused with its sampling epilogue
// (Algorithm 2, lines 5-6: drafter head over the trimmed vocabulary, then the index mapper).
//
// HBM-bound: the only large operand is W_trim [K,d] bf16, read exactly once.  The vocabulary rows
// are split over one persistent CTA per SM (contiguous slabs of 8-row blocks); inside a CTA the 16
// warps split the hidden dimension, every lane keeping a ring of independent 128-bit streaming
// loads of W in flight (no shared-memory staging of W).  The inner product runs on the warp-level
// tensor instruction mma.m16n8k16 (bf16 in, fp32 accumulate) with the hidden rows as the 16-row
// operand and 8 vocabulary rows as the 8-column operand: a dot product does not care in which
// order k is visited, so the 16 contiguous bytes a lane loads from a W row serve directly as its
// fragment as long as the h fragment is taken from the same k positions.  This only off-loads the
// FMAs (at B = 10 the fp32 pipe could not keep up with HBM); the kernel remains a streaming read.
//
// Per 8-row block the 16 partial sums are reduced through shared memory and one warp per hidden
// row updates, on chip: running max / sum-exp of z = logit / T, the row's top-k list, and the
// Gumbel-max candidate from the caller's uniforms.  Logits never go to HBM.  Each CTA leaves one
// small record per hidden row; the last CTA to finish (atomic ticket, no spinning) merges the
// records in CTA order, remaps trimmed indices through `map` and writes the outputs.
#include <math_constants.h>

#include "vt_common.cuh"

namespace vt {

namespace {

constexpr int kNW = 16;                 // warps per CTA: split of the hidden dimension
constexpr int kThreads = kNW * 32;
constexpr int kPartStride = 136;        // floats per warp partial tile: 16 x 8 + pad (bank spread)
constexpr int kMaxB = 16;
constexpr int kMaxGrid = 160;           // merge: each lane owns at most kMaxOwn CTA records
constexpr int kMaxOwn = kMaxGrid / 32;
constexpr size_t kMaxDynSmem = 227 * 1024 - 1024;   // opt-in limit minus static shared memory
constexpr int kRecHdr = 8;              // record: m, s, gumbel score, gumbel j, gumbel z, pad[3]

__host__ __device__ inline int rec_words(int topk) { return kRecHdr + 2 * topk; }

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                         uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ bool better(float v, int j, float bv, int bj) {
    return v > bv || (v == bv && j < bj);
}

// (m, s) <- (m, s) (+) (m2, s2) for running max / sum of exponentials
__device__ __forceinline__ void lse_merge(float& m, float& s, float m2, float s2) {
    const float M = fmaxf(m, m2);
    if (M == -CUDART_INF_F) { m = M; s = 0.f; return; }
    s = s * __expf(m - M) + s2 * __expf(m2 - M);
    m = M;
}

struct Smem {
    float* part;       // [2][kNW][kPartStride]
    float* topv;       // [kMaxB][VT_MAX_TOPK]
    int* topj;         // [kMaxB][VT_MAX_TOPK]
    uint4* h;          // [KBpad][halves][32]
};

template <int U, int NBUF, bool TWO>
__global__ void __launch_bounds__(kThreads, 1)
k_head_skinny(const HeadArgs a, Ctrl* ctrl, float* __restrict__ recs, int RB, int KBW) {
    extern __shared__ __align__(16) uint8_t s_raw[];
    __shared__ int s_last;
    constexpr int HALVES = TWO ? 2 : 1;
    Smem sm;
    sm.part = reinterpret_cast<float*>(s_raw);
    sm.topv = sm.part + 2 * kNW * kPartStride;
    sm.topj = reinterpret_cast<int*>(sm.topv + kMaxB * VT_MAX_TOPK);
    sm.h = reinterpret_cast<uint4*>(sm.topj + kMaxB * VT_MAX_TOPK);

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int B = a.B, K = a.K, d = a.d, topk = a.topk;
    const int NG = KBW / U;                              // groups of U k-blocks per warp and row block
    const int KBpad = KBW * kNW;
    const int rb0 = (int)((long long)RB * blockIdx.x / gridDim.x);
    const int rb1 = (int)((long long)RB * (blockIdx.x + 1) / gridDim.x);
    const int n_items = (rb1 - rb0) * NG;

    // ---- ring of W loads: start streaming before anything else --------------------------------
    uint4 buf[NBUF][U];
    int ld_rb = rb0, ld_grp = 0, ld_item = 0;
    auto load_item = [&](uint4 (&bf)[U]) {
        if (ld_item < n_items) {
            const int row = min(ld_rb * 8 + g, K - 1);
            const uint16_t* base = a.W + (size_t)row * d + 8 * t;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int kb = warp + kNW * (ld_grp * U + u);
                bf[u] = (kb * 32 + 8 * t < d) ? ld_stream_u4(base + kb * 32) : make_uint4(0, 0, 0, 0);
            }
            ++ld_item;
            if (++ld_grp == NG) { ld_grp = 0; ++ld_rb; }
        }
    };
#pragma unroll
    for (int s = 0; s < NBUF; ++s) load_item(buf[s]);

    // ---- stage h as ready-made fragments, init the per-row state ---------------------------------
    for (int i = threadIdx.x; i < KBpad * HALVES * 32; i += kThreads) {
        const int ln = i & 31, half = (i >> 5) % HALVES, kb = (i >> 5) / HALVES;
        const int brow = half * 8 + (ln >> 2), k0 = kb * 32 + 8 * (ln & 3);
        uint4 v = make_uint4(0, 0, 0, 0);
        if (brow < B && k0 < d) v = *reinterpret_cast<const uint4*>(a.h + (size_t)brow * d + k0);
        sm.h[i] = v;
    }
    for (int i = threadIdx.x; i < kMaxB * VT_MAX_TOPK; i += kThreads) {
        sm.topv[i] = -CUDART_INF_F;
        sm.topj[i] = -1;
    }
    // per-row state lives in the registers of warp b (identical in its four 8-lane groups)
    const int b = warp;
    float invT = 1.f;
    bool row_ok = true;
    if (b < B) {
        const float T = a.temp[b];
        row_ok = (T > 0.f) && (T < CUDART_INF_F);
        invT = row_ok ? 1.f / T : CUDART_NAN_F;
    }
    float st_m = -CUDART_INF_F, st_s = 0.f;                 // running max / sum exp (per lane)
    float gb_s = -CUDART_INF_F, gb_z = 0.f;                 // Gumbel best (per lane)
    int gb_j = -1;
    float thr = -CUDART_INF_F;                              // k-th best so far (warp uniform)
    int tk_cnt = 0;
    const int v8 = lane & 7, q = lane >> 3;
    float u_next = 0.5f;
    if (a.uniforms && b < B && rb0 < rb1) {
        const int j = rb0 * 8 + v8;
        if (j < K) u_next = __ldg(a.uniforms + (size_t)b * K + j);
    }
    __syncthreads();

    // ---- end of a row block: reduce the 16 partial tiles, update the row's running state ---------
    auto finish_row_block = [&](int rb, float (&acc0)[4], float (&acc1)[4]) {
        const int pb = (rb - rb0) & 1;
        float* mine = sm.part + (pb * kNW + warp) * kPartStride;
        *reinterpret_cast<float2*>(mine + g * 8 + 2 * t) = make_float2(acc0[0] + acc1[0], acc0[1] + acc1[1]);
        if (TWO)
            *reinterpret_cast<float2*>(mine + 64 + g * 8 + 2 * t) =
                make_float2(acc0[2] + acc1[2], acc0[3] + acc1[3]);
        __syncthreads();
        if (b >= B) return;
        const float* src = sm.part + pb * kNW * kPartStride + b * 8 + v8;
        float x = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) x += src[(q + 4 * i) * kPartStride];
        x += __shfl_xor_sync(0xffffffffu, x, 8);
        x += __shfl_xor_sync(0xffffffffu, x, 16);
        const int j = rb * 8 + v8;
        const bool valid = j < K;
        if (a.dbg_logits && valid && q == 0) a.dbg_logits[(size_t)b * K + j] = x;
        const float z = x * invT;
        if (valid) {
            if (z > st_m) { st_s = st_s * __expf(st_m - z) + 1.f; st_m = z; }
            else st_s += __expf(z - st_m);
        }
        if (a.uniforms) {
            const float uc = fminf(fmaxf(u_next, 0x1p-24f), 1.f - 0x1p-24f);
            const float sc = z - logf(-logf(uc));
            if (valid && sc > gb_s) { gb_s = sc; gb_j = j; gb_z = z; }
            const int jn = (rb + 1) * 8 + v8;
            if (rb + 1 < rb1 && jn < K) u_next = __ldg(a.uniforms + (size_t)b * K + jn);
        }
        unsigned cand = __ballot_sync(0xffffffffu, valid && q == 0 && z > thr);
        while (cand) {
            const int l = __ffs(cand) - 1;
            cand &= cand - 1;
            const float cz = __shfl_sync(0xffffffffu, z, l);
            if (!(cz > thr)) continue;                       // thr may have risen meanwhile
            const int cj = rb * 8 + l;
            float* tv = sm.topv + b * VT_MAX_TOPK;
            int* tj = sm.topj + b * VT_MAX_TOPK;
            const int p0 = lane, p1 = lane + 32;
            const float v0 = p0 < tk_cnt ? tv[p0] : -CUDART_INF_F;
            const float v1 = p1 < tk_cnt ? tv[p1] : -CUDART_INF_F;
            const int j0 = p0 < tk_cnt ? tj[p0] : -1, j1 = p1 < tk_cnt ? tj[p1] : -1;
            const int pos = __popc(__ballot_sync(0xffffffffu, p0 < tk_cnt && v0 >= cz)) +
                            __popc(__ballot_sync(0xffffffffu, p1 < tk_cnt && v1 >= cz));
            const int ncnt = min(tk_cnt + 1, topk);
            __syncwarp();
            if (p0 >= pos && p0 < tk_cnt && p0 + 1 < ncnt) { tv[p0 + 1] = v0; tj[p0 + 1] = j0; }
            if (p1 >= pos && p1 < tk_cnt && p1 + 1 < ncnt) { tv[p1 + 1] = v1; tj[p1 + 1] = j1; }
            if (lane == 0) { tv[pos] = cz; tj[pos] = cj; }
            __syncwarp();
            tk_cnt = ncnt;
            thr = (tk_cnt == topk) ? tv[topk - 1] : -CUDART_INF_F;
        }
    };

    // ---- main loop ---------------------------------------------------------------------------------
    float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
    int c_rb = rb0, c_grp = 0;
#pragma unroll 1
    for (int it = 0; it < n_items; it += NBUF) {
#pragma unroll
        for (int s = 0; s < NBUF; ++s) {
            if (it + s < n_items) {
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int kb = warp + kNW * (c_grp * U + u);
                    const uint4 w = buf[s][u];
                    const uint4 hlo = sm.h[(kb * HALVES) * 32 + lane];
                    uint4 hhi = make_uint4(0, 0, 0, 0);
                    if (TWO) hhi = sm.h[(kb * HALVES + 1) * 32 + lane];
                    mma_bf16(acc0, hlo.x, hhi.x, hlo.y, hhi.y, w.x, w.y);
                    mma_bf16(acc1, hlo.z, hhi.z, hlo.w, hhi.w, w.z, w.w);
                }
                load_item(buf[s]);
                if (++c_grp == NG) {
                    c_grp = 0;
                    finish_row_block(c_rb, acc0, acc1);
                    ++c_rb;
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc0[i] = acc1[i] = 0.f;
                }
            }
        }
    }

    // ---- this CTA's record per hidden row ----------------------------------------------------------
    const int RW = rec_words(topk);
    if (b < B) {
#pragma unroll
        for (int o = 1; o < 8; o <<= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, st_m, o);
            const float s2 = __shfl_xor_sync(0xffffffffu, st_s, o);
            lse_merge(st_m, st_s, m2, s2);
            const float gs2 = __shfl_xor_sync(0xffffffffu, gb_s, o);
            const float gz2 = __shfl_xor_sync(0xffffffffu, gb_z, o);
            const int gj2 = __shfl_xor_sync(0xffffffffu, gb_j, o);
            if (gj2 >= 0 && (gb_j < 0 || better(gs2, gj2, gb_s, gb_j))) { gb_s = gs2; gb_j = gj2; gb_z = gz2; }
        }
        float* rec = recs + ((size_t)blockIdx.x * B + b) * RW;
        if (lane == 0) {
            rec[0] = st_m; rec[1] = st_s; rec[2] = gb_s;
            reinterpret_cast<int*>(rec)[3] = gb_j;
            rec[4] = gb_z;
            reinterpret_cast<int*>(rec)[5] = row_ok ? 1 : 0;
        }
        for (int r = lane; r < topk; r += 32) {
            rec[kRecHdr + r] = sm.topv[b * VT_MAX_TOPK + r];
            reinterpret_cast<int*>(rec)[kRecHdr + topk + r] = sm.topj[b * VT_MAX_TOPK + r];
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0)
        s_last = (atomicInc(&ctrl->head_ticket, gridDim.x - 1) == gridDim.x - 1);
    __syncthreads();
    if (!s_last || b >= B) return;
    __threadfence();

    // ---- last CTA: merge all records of row b in CTA order ------------------------------------------
    const int G = gridDim.x;
    float M = -CUDART_INF_F, S = 0.f, GS = -CUDART_INF_F, GZ = 0.f;
    int GJ = -1;
    for (int c = lane; c < G; c += 32) {
        const float* rec = recs + ((size_t)c * B + b) * RW;
        lse_merge(M, S, ld_cg_f32(rec + 0), ld_cg_f32(rec + 1));
        const float gs2 = ld_cg_f32(rec + 2), gz2 = ld_cg_f32(rec + 4);
        const int gj2 = ld_cg_s32(reinterpret_cast<const int*>(rec) + 3);
        if (gj2 >= 0 && (GJ < 0 || better(gs2, gj2, GS, GJ))) { GS = gs2; GJ = gj2; GZ = gz2; }
    }
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, M, o), s2 = __shfl_xor_sync(0xffffffffu, S, o);
        lse_merge(M, S, m2, s2);
        const float gs2 = __shfl_xor_sync(0xffffffffu, GS, o), gz2 = __shfl_xor_sync(0xffffffffu, GZ, o);
        const int gj2 = __shfl_xor_sync(0xffffffffu, GJ, o);
        if (gj2 >= 0 && (GJ < 0 || better(gs2, gj2, GS, GJ))) { GS = gs2; GJ = gj2; GZ = gz2; }
    }
    const float lse = M + logf(S);
    // stage the first `depth` entries of every CTA's list in shared memory (h is no longer needed)
    const int cap = (KBpad * HALVES * 32 * 16) / (B * 8);     // (value, index) pairs per row
    const int depth = min(topk, cap / G);
    float* stv = reinterpret_cast<float*>(sm.h) + (size_t)b * cap * 2;
    int* stj = reinterpret_cast<int*>(stv) + cap;
    for (int e = lane; e < G * depth; e += 32) {
        const int c = e / depth, r = e - c * depth;
        const float* rec = recs + ((size_t)c * B + b) * RW;
        stv[e] = ld_cg_f32(rec + kRecHdr + r);
        stj[e] = ld_cg_s32(reinterpret_cast<const int*>(rec) + kRecHdr + topk + r);
    }
    __syncwarp();
    int head[kMaxOwn];
#pragma unroll
    for (int o = 0; o < kMaxOwn; ++o) head[o] = 0;
    const int row_w = 1 + topk;
    int* oid = a.out_ids + (size_t)b * row_w;
    float* olp = a.out_logprobs + (size_t)b * row_w;
    int first_id = -1;
    float first_lp = CUDART_NAN_F;
    bool any_missing = false;
    for (int r = 0; r < topk; ++r) {
        float lv = -CUDART_INF_F;
        int lj = -1, lo = -1;
#pragma unroll
        for (int o = 0; o < kMaxOwn; ++o) {
            const int c = lane + 32 * o;
            if (c < G && head[o] < topk) {
                float v;
                int j;
                if (head[o] < depth) { v = stv[c * depth + head[o]]; j = stj[c * depth + head[o]]; }
                else {
                    const float* rec = recs + ((size_t)c * B + b) * RW;
                    v = ld_cg_f32(rec + kRecHdr + head[o]);
                    j = ld_cg_s32(reinterpret_cast<const int*>(rec) + kRecHdr + topk + head[o]);
                }
                if (j >= 0 && (lj < 0 || better(v, j, lv, lj))) { lv = v; lj = j; lo = o; }
            }
        }
        float wv = lv;
        int wj = lj;
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            const float v2 = __shfl_xor_sync(0xffffffffu, wv, o);
            const int j2 = __shfl_xor_sync(0xffffffffu, wj, o);
            if (j2 >= 0 && (wj < 0 || better(v2, j2, wv, wj))) { wv = v2; wj = j2; }
        }
#pragma unroll
        for (int o = 0; o < kMaxOwn; ++o)
            if (o == lo && lj == wj && wj >= 0) ++head[o];
        const bool ok = row_ok && wj >= 0;
        const int id = ok ? (a.map ? __ldg(a.map + wj) : wj) : -1;
        const float lp = ok ? wv - lse : CUDART_NAN_F;
        if (r == 0) { first_id = id; first_lp = lp; }
        if (!ok) any_missing = true;
        if (lane == 0) { oid[1 + r] = id; olp[1 + r] = lp; }
    }
    if (lane == 0) {
        if (a.uniforms) {
            const bool ok = row_ok && GJ >= 0;
            oid[0] = ok ? (a.map ? __ldg(a.map + GJ) : GJ) : -1;
            olp[0] = ok ? GZ - lse : CUDART_NAN_F;
            if (!ok) any_missing = true;
        } else {
            oid[0] = first_id;
            olp[0] = first_lp;
        }
        if (a.dbg_lse) a.dbg_lse[b] = lse;
        if (!row_ok) atomicOr(&ctrl->flags, (uint32_t)VT_FLAG_BAD_TEMP);
        else if (any_missing) atomicOr(&ctrl->flags, (uint32_t)VT_FLAG_NAN_ROW);
    }
}

size_t skinny_smem_bytes(int KBW, bool two) {
    return (size_t)2 * kNW * kPartStride * 4 + (size_t)kMaxB * VT_MAX_TOPK * 8 +
           (size_t)KBW * kNW * (two ? 2 : 1) * 512;
}

int skinny_kbw(int d) { return ((d + 31) / 32 + kNW - 1) / kNW; }

template <int U, int NBUF, bool TWO>
cudaError_t launch_variant(const HeadArgs& a, Ctrl* ctrl, float* recs, int grid, int RB, int KBW,
                           size_t smem, cudaStream_t s) {
    static int attr_done[64] = {0};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !attr_done[dev]) {
        cudaError_t e = cudaFuncSetAttribute(k_head_skinny<U, NBUF, TWO>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxDynSmem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_done[dev] = 1;
    }
    k_head_skinny<U, NBUF, TWO><<<grid, kThreads, smem, s>>>(a, ctrl, recs, RB, KBW);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

bool head_skinny_supported(int32_t B, int32_t d) {
    if (B < 1 || B > kMaxB || d < 8 || (d & 7)) return false;
    return skinny_smem_bytes(skinny_kbw(d), B > 8) <= kMaxDynSmem;
}

size_t head_skinny_scratch_bytes(int32_t B, int32_t K, int32_t topk) {
    (void)K;
    return align_up((size_t)kMaxGrid * B * rec_words(topk) * 4, 256);
}

cudaError_t launch_head_skinny(const HeadArgs& a, Ctrl* ctrl, uint8_t* scratch, cudaStream_t s) {
    const int RB = (a.K + 7) / 8;
    int grid = num_sms();
    if (grid > kMaxGrid) grid = kMaxGrid;
    if (grid > RB) grid = RB;
    const int KBW = skinny_kbw(a.d);
    const bool two = a.B > 8;
    const size_t smem = skinny_smem_bytes(KBW, two);
    float* recs = reinterpret_cast<float*>(scratch);
#define VT_LAUNCH(U, NBUF)                                                                       \
    (two ? launch_variant<U, NBUF, true>(a, ctrl, recs, grid, RB, KBW, smem, s)                  \
         : launch_variant<U, NBUF, false>(a, ctrl, recs, grid, RB, KBW, smem, s))
    if (KBW % 4 == 0) return VT_LAUNCH(4, 3);
    if (KBW % 3 == 0) return VT_LAUNCH(3, 4);
    if (KBW % 2 == 0) return VT_LAUNCH(2, 6);
    return VT_LAUNCH(1, 8);
#undef VT_LAUNCH
}

}  // namespace vt
