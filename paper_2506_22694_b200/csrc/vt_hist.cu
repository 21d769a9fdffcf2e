// Token-frequency histogram (Algorithm 1: c[t_i] += 1 over the calibration stream).
//
// The stream is read once from HBM (4 bytes per token); everything else is arranged so that the
// per-token work stays in shared memory:
//   * V * 4 bytes fit in one CTA's shared memory  -> every CTA keeps a private copy of all bins
//     (k_hist_small) and flushes the non-zero ones at the end.
//   * ceil(V / 3) * 4 bytes fit (Llama-3: 128256 bins = 171 KB)  -> every CTA still keeps all bins,
//     three 10-bit fields to a word (k_hist_packed): one shared-memory add per token and nothing else.
//     A field hands 512 counts on to global memory whenever it gets there; the add that would wrap a
//     field notices, and the stream is then counted again by the kernels of the next case.
//   * otherwise a short pre-pass samples the stream, picks the hottest bins that fit (about 49.8 K of
//     them for 128256 bins), and the main pass keeps those in shared memory; the rare cold tokens go
//     to L2 with one red.global each.  The hot set only steers traffic: counts are exact whichever
//     bins were picked.
//       hot lookup: entry[id >> 4] = {16 membership bits, 16-bit slot of the group's first member};
//       slot = base + popc(bits & below(id)), one 4-byte shared load per token.
#include "vt_common.cuh"

namespace vt {

namespace {

constexpr int kThreads = 1024;
constexpr size_t kDynSmem = 224 * 1024;        // dynamic shared memory of the counting kernels
constexpr size_t kMaxTableBytes = 160 * 1024;  // lookup table (8 bytes per 32 ids) at most: leaves 64 KB of hot bins;
                                               // the one limit behind hist_supported and both kernels' launches
constexpr int kMaxDevices = 64;
constexpr int kSampleSlots = 4096;             // aggregating cache of the sampling pre-pass
constexpr int kSamplePerCta = 16384;           // ids sampled per CTA
constexpr int kPickBins = 1024;                // sampled counts are clipped to kPickBins-1
static_assert(kPickBins == kThreads, "one pick bin per thread");
constexpr int kPickLoads = 16;                 // loads each thread of the one-CTA pick keeps in flight

// ---- streaming loop shared by the counting kernels ---------------------------------------------
// The CTA's share of the 16-byte-aligned body is read with four independent 128-bit loads per
// thread per trip; the unaligned head/tail (at most 3 + 3 ids) is handled by CTA 0.
template <class F>
__device__ __forceinline__ void stream_ids(const int32_t* __restrict__ ids, int64_t n, F&& tally) {
    const uintptr_t addr = reinterpret_cast<uintptr_t>(ids);
    int64_t head = ((16 - (addr & 15)) & 15) >> 2;
    if (head > n) head = n;
    const int64_t nvec = (n - head) >> 2;
    const int64_t tail0 = head + nvec * 4;
    if (blockIdx.x == 0) {
        if ((int64_t)threadIdx.x < head) tally((uint32_t)ids[threadIdx.x]);
        const int64_t t = tail0 + threadIdx.x;
        if (t < n) tally((uint32_t)ids[t]);
    }
    const uint4* vec = reinterpret_cast<const uint4*>(ids + head);
    const int64_t v0 = nvec * blockIdx.x / gridDim.x;
    const int64_t v1 = nvec * (blockIdx.x + 1) / gridDim.x;
    for (int64_t v = v0 + threadIdx.x; v < v1; v += 4 * kThreads) {
        uint4 a = ld_stream_u4(vec + v), b, c, d;
        const bool pb = v + kThreads < v1, pc = v + 2 * kThreads < v1, pd = v + 3 * kThreads < v1;
        if (pb) b = ld_stream_u4(vec + v + kThreads);
        if (pc) c = ld_stream_u4(vec + v + 2 * kThreads);
        if (pd) d = ld_stream_u4(vec + v + 3 * kThreads);
        tally(a.x); tally(a.y); tally(a.z); tally(a.w);
        if (pb) { tally(b.x); tally(b.y); tally(b.z); tally(b.w); }
        if (pc) { tally(c.x); tally(c.y); tally(c.z); tally(c.w); }
        if (pd) { tally(d.x); tally(d.y); tally(d.z); tally(d.w); }
    }
}

// Same walk, handing whole 128-bit loads (4 ids) to `tally4` and the ragged ends to `tally1`.
template <class F4, class F1>
__device__ __forceinline__ void stream_ids4(const int32_t* __restrict__ ids, int64_t n, F4&& tally4, F1&& tally1) {
    const uintptr_t addr = reinterpret_cast<uintptr_t>(ids);
    int64_t head = ((16 - (addr & 15)) & 15) >> 2;
    if (head > n) head = n;
    const int64_t nvec = (n - head) >> 2;
    const int64_t tail0 = head + nvec * 4;
    if (blockIdx.x == 0) {
        if ((int64_t)threadIdx.x < head) tally1((uint32_t)ids[threadIdx.x]);
        const int64_t t = tail0 + threadIdx.x;
        if (t < n) tally1((uint32_t)ids[t]);
    }
    const uint4* vec = reinterpret_cast<const uint4*>(ids + head);
    const int64_t v0 = nvec * blockIdx.x / gridDim.x;
    const int64_t v1 = nvec * (blockIdx.x + 1) / gridDim.x;
    for (int64_t v = v0 + threadIdx.x; v < v1; v += 4 * kThreads) {
        uint4 a = ld_stream_u4(vec + v), b, c, d;
        const bool pb = v + kThreads < v1, pc = v + 2 * kThreads < v1, pd = v + 3 * kThreads < v1;
        if (pb) b = ld_stream_u4(vec + v + kThreads);
        if (pc) c = ld_stream_u4(vec + v + 2 * kThreads);
        if (pd) d = ld_stream_u4(vec + v + 3 * kThreads);
        tally4(a.x, a.y, a.z, a.w);
        if (pb) tally4(b.x, b.y, b.z, b.w);
        if (pc) tally4(c.x, c.y, c.z, c.w);
        if (pd) tally4(d.x, d.y, d.z, d.w);
    }
}

__device__ __forceinline__ void report_bad(unsigned long long bad, Ctrl* ctrl) {
    for (int o = 16; o; o >>= 1) bad += __shfl_xor_sync(0xffffffffu, bad, o);
    if ((threadIdx.x & 31) == 0 && bad) {
        atomicAdd(&ctrl->n_bad, bad);
        atomicOr(&ctrl->flags, (uint32_t)VT_FLAG_BAD_ID);
    }
}

// ---- all bins private to each CTA ----------------------------------------------------------------
// Same walk as the packed kernel below: whole trips of kRows 128-bit loads per thread without a bounds test,
// one range test per load, then the guarded rest; CTA 0 takes the ragged ends.
constexpr int kRows = 6;                       // 128-bit loads a thread has in flight per trip (96 KB per CTA): four
                                               // leave HBM waiting, seven leave no registers for the tally
__global__ void __launch_bounds__(kThreads, 1)
k_hist_small(const int32_t* __restrict__ ids, int64_t n, int32_t V, uint32_t* __restrict__ counts,
             Ctrl* ctrl) {
    extern __shared__ __align__(16) uint32_t s_bins[];
    for (int i = threadIdx.x; i < V; i += kThreads) s_bins[i] = 0;
    __syncthreads();
    unsigned long long bad = 0;
    auto tally1 = [&](uint32_t id) {
        if (id < (uint32_t)V) atomicAdd(&s_bins[id], 1u);
        else ++bad;
    };
    auto tally4 = [&](uint4 x) {
        if (max(max(x.x, x.y), max(x.z, x.w)) < (uint32_t)V) {
            atomicAdd(&s_bins[x.x], 1u); atomicAdd(&s_bins[x.y], 1u); atomicAdd(&s_bins[x.z], 1u); atomicAdd(&s_bins[x.w], 1u);
        } else {
            tally1(x.x); tally1(x.y); tally1(x.z); tally1(x.w);
        }
    };
    const uintptr_t addr = reinterpret_cast<uintptr_t>(ids);
    int64_t head = ((16 - (addr & 15)) & 15) >> 2;
    if (head > n) head = n;
    const int64_t nvec = (n - head) >> 2;
    const int64_t tail0 = head + nvec * 4;
    if (blockIdx.x == 0) {
        if ((int64_t)threadIdx.x < head) tally1((uint32_t)ids[threadIdx.x]);
        const int64_t t = tail0 + threadIdx.x;
        if (t < n) tally1((uint32_t)ids[t]);
    }
    const uint4* vec = reinterpret_cast<const uint4*>(ids + head);
    const int64_t v0 = nvec * blockIdx.x / gridDim.x;
    const int64_t v1 = nvec * (blockIdx.x + 1) / gridDim.x;
    const int64_t trips = (v1 - v0) / (kRows * kThreads);
    const uint4* p = vec + v0 + threadIdx.x;
    for (int64_t t = 0; t < trips; ++t, p += kRows * kThreads) {
        uint4 x[kRows];
#pragma unroll
        for (int r = 0; r < kRows; ++r) x[r] = ld_stream_u4(p + r * kThreads);
#pragma unroll
        for (int r = 0; r < kRows; ++r) tally4(x[r]);
    }
    for (int64_t v = v0 + trips * (kRows * kThreads) + threadIdx.x; v < v1; v += kThreads) tally4(ld_stream_u4(vec + v));
    __syncthreads();
    for (int i = threadIdx.x; i < V; i += kThreads) {
        const int v = (i + blockIdx.x * (V / (int)gridDim.x)) % V;   // the CTAs' flushes spread over the whole array
        const uint32_t c = s_bins[v];
        if (c) atomicAdd(&counts[v], c);
    }
    report_bad(bad, ctrl);
}

// ---- pre-pass 1: sample the stream into sample[V] through a per-CTA aggregating cache -----------
__device__ __forceinline__ void sample_stream(const int32_t* __restrict__ ids, int64_t n, int32_t V,
                                              uint32_t* __restrict__ sample, int* s_tag, uint32_t* s_cnt) {
    for (int i = threadIdx.x; i < kSampleSlots; i += kThreads) { s_tag[i] = -1; s_cnt[i] = 0; }
    __syncthreads();
    const int64_t lo = n * blockIdx.x / gridDim.x;
    const int64_t hi = n * (blockIdx.x + 1) / gridDim.x;
    const int64_t end = (hi - lo > kSamplePerCta) ? lo + kSamplePerCta : hi;
    for (int64_t i = lo + threadIdx.x; i < end; i += kThreads) {
        const uint32_t id = (uint32_t)ids[i];
        if (id >= (uint32_t)V) continue;
        const uint32_t slot = (id * 2654435761u) >> 20;            // 12 bits -> kSampleSlots
        const int old = atomicCAS(&s_tag[slot], -1, (int)id);
        if (old == -1 || old == (int)id) atomicAdd(&s_cnt[slot], 1u);
        else atomicAdd(&sample[id], 1u);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kSampleSlots; i += kThreads)
        if (s_tag[i] >= 0) atomicAdd(&sample[s_tag[i]], s_cnt[i]);
}

__global__ void __launch_bounds__(kThreads, 1)
k_hist_sample(const int32_t* __restrict__ ids, int64_t n, int32_t V, uint32_t* __restrict__ sample) {
    __shared__ int s_tag[kSampleSlots];
    __shared__ uint32_t s_cnt[kSampleSlots];
    sample_stream(ids, n, V, sample, s_tag, s_cnt);
}

// Exclusive scan over one value per thread (kThreads threads); returns the prefix, *total the sum.
__device__ uint32_t block_excl_scan(uint32_t x, uint32_t* s_warp /*[33]*/, uint32_t* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t incl = x;
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    __syncthreads();                                   // s_warp may still be read from a previous scan
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = s_warp[lane], wi = w;
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += y;
        }
        s_warp[lane] = wi - w;
        if (lane == 31) s_warp[32] = wi;
    }
    __syncthreads();
    *total = s_warp[32];
    return s_warp[warp] + incl - x;
}

// ---- pre-pass 2: choose at most H hot bins from the sampled counts, build the lookup table ------
// hot = sampled count >= tau, plus (in id order) as many bins with count == tau-1 as still fit.
__global__ void __launch_bounds__(kThreads, 1)
k_hist_pick(const uint32_t* __restrict__ sample, int32_t V, int32_t H, uint2* __restrict__ table,
            const uint32_t* __restrict__ gate) {
    extern __shared__ __align__(16) uint8_t s_dyn[];
    if (gate && *gate == 0) return;                        // the packed count stood: nothing to recount
    __shared__ uint32_t s_hist[kPickBins];
    __shared__ uint32_t s_warp[33];
    __shared__ uint32_t s_definite;
    const int T32 = (V + 31) >> 5;
    uint2* s_tbl = reinterpret_cast<uint2*>(s_dyn);         // [T32] {definite, tie}, then {bits, slot base}
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    s_hist[threadIdx.x] = 0;
    __syncthreads();
    {   // most bins were sampled a handful of times: count those in registers, one atomic per warp
        uint32_t small[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        // sixteen loads in flight per thread: one CTA walking 128K counts one load at a time is all latency
        for (int v0 = threadIdx.x; v0 < V; v0 += kThreads * kPickLoads) {
            uint32_t cs[kPickLoads];
#pragma unroll
            for (int q = 0; q < kPickLoads; ++q) {
                const int v = v0 + q * kThreads;
                cs[q] = v < V ? __ldg(sample + v) : 0xffffffffu;
            }
#pragma unroll
            for (int q = 0; q < kPickLoads; ++q) {
                if (cs[q] == 0xffffffffu) continue;                     // past the end (a count never gets there)
                const uint32_t c = min(cs[q], (uint32_t)(kPickBins - 1));
                if (c < 8) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) small[k] += (c == (uint32_t)k);
                } else {
                    atomicAdd(&s_hist[c], 1u);
                }
            }
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            uint32_t x = small[k];
            for (int o = 16; o; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
            if (lane == 0 && x) atomicAdd(&s_hist[k], x);
        }
    }
    __syncthreads();
    // P[t] = #{bins with clipped count >= kPickBins-1-t}; tau = kPickBins - #{t : P[t] <= H}
    uint32_t tot;
    const uint32_t mine = s_hist[kPickBins - 1 - threadIdx.x];
    const uint32_t P = block_excl_scan(mine, s_warp, &tot) + mine;
    const int n_ok = __syncthreads_count(P <= (uint32_t)H);
    const uint32_t tau = kPickBins - n_ok;
    if (n_ok == 0 && threadIdx.x == 0) s_definite = 0;
    if (n_ok > 0 && (int)threadIdx.x == n_ok - 1) s_definite = P;
    __syncthreads();
    const uint32_t quota = (uint32_t)H - s_definite;
    // pass A: one coalesced load per 32 ids, the membership words come out of warp ballots
    for (int w0 = warp; w0 < T32; w0 += (kThreads / 32) * kPickLoads) {          // again sixteen loads in flight
        uint32_t cs[kPickLoads];
#pragma unroll
        for (int q = 0; q < kPickLoads; ++q) {
            const int v = (w0 + q * (kThreads / 32)) * 32 + lane;
            cs[q] = v < V ? min(__ldg(sample + v), (uint32_t)(kPickBins - 1)) : 0xffffffffu;
        }
#pragma unroll
        for (int q = 0; q < kPickLoads; ++q) {
            const int w = w0 + q * (kThreads / 32);
            if (w >= T32) break;                                        // warp-uniform
            const bool in = cs[q] != 0xffffffffu;
            const uint32_t def = __ballot_sync(0xffffffffu, in && cs[q] >= tau);
            const uint32_t tie = __ballot_sync(0xffffffffu, in && cs[q] + 1 == tau);
            if (lane == 0) s_tbl[w] = make_uint2(def, tie);
        }
    }
    __syncthreads();
    // pass B: admit ties in id order while the quota lasts; every thread owns wpt consecutive words
    const int wpt = (T32 + kThreads - 1) / kThreads;
    const int w_lo = min(T32, (int)threadIdx.x * wpt), w_hi = min(T32, w_lo + wpt);
    uint32_t tsum = 0;
    for (int w = w_lo; w < w_hi; ++w) tsum += __popc(s_tbl[w].y);
    uint32_t tbase = block_excl_scan(tsum, s_warp, &tot);
    uint32_t hsum = 0;
    for (int w = w_lo; w < w_hi; ++w) {
        const uint2 e = s_tbl[w];
        uint32_t tie = e.y, keep = 0;
        const uint32_t room = tbase < quota ? quota - tbase : 0u;
        const int admit = (int)min(room, (uint32_t)__popc(tie));
        tbase += __popc(tie);
        for (int a = 0; a < admit; ++a) {
            const uint32_t low = tie & (0u - tie);
            keep |= low;
            tie ^= low;
        }
        const uint32_t bits = e.x | keep;
        s_tbl[w].x = bits;
        hsum += __popc(bits);
    }
    uint32_t hbase = block_excl_scan(hsum, s_warp, &tot);
    for (int w = w_lo; w < w_hi; ++w) {
        s_tbl[w].y = hbase;
        hbase += __popc(s_tbl[w].x);
    }
    __syncthreads();
    for (int w = threadIdx.x; w < T32; w += kThreads) table[w] = s_tbl[w];
}

// ---- main pass: hot bins in shared memory, cold bins through L2 ----------------------------------
__global__ void __launch_bounds__(kThreads, 1)
k_hist_hot(const int32_t* __restrict__ ids, int64_t n, int32_t V, uint32_t* __restrict__ counts,
           const uint2* __restrict__ table, int32_t H, Ctrl* ctrl, const uint32_t* __restrict__ gate) {
    extern __shared__ __align__(16) uint8_t s_raw[];
    if (gate && *gate == 0) return;
    const int T32 = (V + 31) >> 5;
    // The lookup is repacked for the main pass: one 4-byte word per 16 ids = {16 membership bits,
    // 16-bit slot of the first member} -- a 4-byte gather costs half the shared-memory wavefronts of
    // an 8-byte one, and the lookup is one of the two shared-memory operations every token pays.
    uint32_t* s_t16 = reinterpret_cast<uint32_t*>(s_raw);                       // [2 * T32]
    uint32_t* s_cnt = reinterpret_cast<uint32_t*>(s_raw + (size_t)T32 * 8);
    for (int i = threadIdx.x; i < T32; i += kThreads) {
        const uint2 e = table[i];
        s_t16[2 * i] = (e.x & 0xffffu) | (e.y << 16);
        s_t16[2 * i + 1] = (e.x >> 16) | ((e.y + __popc(e.x & 0xffffu)) << 16);
    }
    for (int i = threadIdx.x; i < H; i += kThreads) s_cnt[i] = 0;
    __syncthreads();
    unsigned long long bad = 0;
    const uint32_t tbl_addr = (uint32_t)__cvta_generic_to_shared(s_t16);
    const uint32_t cnt_addr = (uint32_t)__cvta_generic_to_shared(s_cnt);
    // One token, id < V known: a handful of integer instructions, one shared-memory load and one
    // reduction -- into the token's shared-memory counter when its id is hot, into global memory
    // when it is not -- chosen by a predicate: no branch, the warp never splits.
    auto tally_in_range = [&](uint32_t id) {
        asm volatile(
            "{\n\t"
            ".reg .pred ph;\n\t"
            ".reg .b32 w, e, sh, bit, m, r, sl;\n\t"
            ".reg .b64 ga;\n\t"
            "shr.u32 w, %0, 4;\n\t"
            "mad.lo.u32 w, w, 4, %1;\n\t"
            "ld.shared.u32 e, [w];\n\t"
            "and.b32 sh, %0, 15;\n\t"
            "shl.b32 bit, 1, sh;\n\t"
            "and.b32 r, e, bit;\n\t"
            "setp.ne.u32 ph, r, 0;\n\t"
            "add.u32 m, bit, -1;\n\t"
            "and.b32 r, e, m;\n\t"
            "popc.b32 r, r;\n\t"
            "shr.u32 sl, e, 16;\n\t"
            "add.u32 sl, sl, r;\n\t"
            "mad.lo.u32 sl, sl, 4, %2;\n\t"
            "@ph red.shared.add.u32 [sl], 1;\n\t"
            "mad.wide.u32 ga, %0, 4, %3;\n\t"
            "@!ph red.global.add.u32 [ga], 1;\n\t"
            "}" ::"r"(id), "r"(tbl_addr), "r"(cnt_addr), "l"(counts) : "memory");
    };
    // Four tokens at once, all in range: the four lookups are requested back to back before anything waits
    // for one of them, so a warp has four shared-memory loads in flight instead of one.
    auto tally4_in_range = [&](uint32_t i0, uint32_t i1, uint32_t i2, uint32_t i3) {
        asm volatile(
            "{\n\t"
            ".reg .pred p0, p1, p2, p3;\n\t"
            ".reg .b32 w0, w1, w2, w3, e0, e1, e2, e3, b0, b1, b2, b3, r0, r1, r2, r3, s0, s1, s2, s3;\n\t"
            ".reg .b64 g0, g1, g2, g3;\n\t"
            "shr.u32 w0, %0, 4;\n\t shr.u32 w1, %1, 4;\n\t shr.u32 w2, %2, 4;\n\t shr.u32 w3, %3, 4;\n\t"
            "mad.lo.u32 w0, w0, 4, %4;\n\t mad.lo.u32 w1, w1, 4, %4;\n\t mad.lo.u32 w2, w2, 4, %4;\n\t mad.lo.u32 w3, w3, 4, %4;\n\t"
            "ld.shared.u32 e0, [w0];\n\t ld.shared.u32 e1, [w1];\n\t ld.shared.u32 e2, [w2];\n\t ld.shared.u32 e3, [w3];\n\t"
            "and.b32 b0, %0, 15;\n\t and.b32 b1, %1, 15;\n\t and.b32 b2, %2, 15;\n\t and.b32 b3, %3, 15;\n\t"
            "shl.b32 b0, 1, b0;\n\t shl.b32 b1, 1, b1;\n\t shl.b32 b2, 1, b2;\n\t shl.b32 b3, 1, b3;\n\t"
            "mad.wide.u32 g0, %0, 4, %6;\n\t mad.wide.u32 g1, %1, 4, %6;\n\t mad.wide.u32 g2, %2, 4, %6;\n\t mad.wide.u32 g3, %3, 4, %6;\n\t"
            "and.b32 r0, e0, b0;\n\t and.b32 r1, e1, b1;\n\t and.b32 r2, e2, b2;\n\t and.b32 r3, e3, b3;\n\t"
            "setp.ne.u32 p0, r0, 0;\n\t setp.ne.u32 p1, r1, 0;\n\t setp.ne.u32 p2, r2, 0;\n\t setp.ne.u32 p3, r3, 0;\n\t"
            "add.u32 b0, b0, -1;\n\t add.u32 b1, b1, -1;\n\t add.u32 b2, b2, -1;\n\t add.u32 b3, b3, -1;\n\t"
            "and.b32 r0, e0, b0;\n\t and.b32 r1, e1, b1;\n\t and.b32 r2, e2, b2;\n\t and.b32 r3, e3, b3;\n\t"
            "popc.b32 r0, r0;\n\t popc.b32 r1, r1;\n\t popc.b32 r2, r2;\n\t popc.b32 r3, r3;\n\t"
            "shr.u32 s0, e0, 16;\n\t shr.u32 s1, e1, 16;\n\t shr.u32 s2, e2, 16;\n\t shr.u32 s3, e3, 16;\n\t"
            "add.u32 s0, s0, r0;\n\t add.u32 s1, s1, r1;\n\t add.u32 s2, s2, r2;\n\t add.u32 s3, s3, r3;\n\t"
            "mad.lo.u32 s0, s0, 4, %5;\n\t mad.lo.u32 s1, s1, 4, %5;\n\t mad.lo.u32 s2, s2, 4, %5;\n\t mad.lo.u32 s3, s3, 4, %5;\n\t"
            "@p0 red.shared.add.u32 [s0], 1;\n\t @p1 red.shared.add.u32 [s1], 1;\n\t"
            "@p2 red.shared.add.u32 [s2], 1;\n\t @p3 red.shared.add.u32 [s3], 1;\n\t"
            "@!p0 red.global.add.u32 [g0], 1;\n\t @!p1 red.global.add.u32 [g1], 1;\n\t"
            "@!p2 red.global.add.u32 [g2], 1;\n\t @!p3 red.global.add.u32 [g3], 1;\n\t"
            "}" ::"r"(i0), "r"(i1), "r"(i2), "r"(i3), "r"(tbl_addr), "r"(cnt_addr), "l"(counts) : "memory");
    };
    stream_ids4(ids, n, [&](uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
        // one range test per 128-bit load; ids outside [0, V) are rare and take the careful path
        if (max(max(a, b), max(c, d)) < (uint32_t)V) {
            tally4_in_range(a, b, c, d);
        } else {
            if (a < (uint32_t)V) tally_in_range(a); else ++bad;
            if (b < (uint32_t)V) tally_in_range(b); else ++bad;
            if (c < (uint32_t)V) tally_in_range(c); else ++bad;
            if (d < (uint32_t)V) tally_in_range(d); else ++bad;
        }
    }, [&](uint32_t id) {
        if (id < (uint32_t)V) tally_in_range(id); else ++bad;
    });
    __syncthreads();
    for (int i = threadIdx.x; i < 2 * T32; i += kThreads) {
        const int g = (i + blockIdx.x * 53) % (2 * T32);   // de-phase the CTAs' flushes
        const uint32_t e = s_t16[g];
        uint32_t bits = e & 0xffffu, slot = e >> 16;
        while (bits) {
            const int b = __ffs(bits) - 1;
            bits &= bits - 1;
            const uint32_t c = s_cnt[slot++];
            if (c) atomicAdd(&counts[g * 16 + b], c);
        }
    }
    report_bad(bad, ctrl);
}

// ---- every bin in shared memory, three 10-bit fields to a word -----------------------------------------
// Word w holds the counters of ids w, W + w and 2W + w (W >= ceil(V / 3)).  Each token is one returning
// shared-memory add of 1 << (10 * field).  The add that takes a field from kSpill-1 to kSpill subtracts
// kSpill again and credits them to out[id] in global memory, so a field holds fewer than kSpill counts plus
// whatever other threads add between those two operations.  With four adds in flight per thread that keeps
// a field from wrapping as long as no token makes up an eighth of the stream, so the most frequent token is
// taken out of the fields: the first id of a CTA that hands counts on becomes its hot id (the most frequent
// token gets to kSpill first), and from then on a lane that meets it adds 1 to a 32-bit word of its own
// instead (one per lane, so those adds never collide).  Until the hot id is known (kCarefulTrips trips)
// every add is tested before the thread's next one is issued.  An add that finds kFieldMax in its field has
// carried into the neighbour: it raises the gate, and the launcher's next kernels throw this count away
// and count the stream again with the hot / cold kernels.
constexpr uint32_t kFieldBits = 10, kFieldMax = (1u << kFieldBits) - 1, kSpill = 512;
constexpr uint32_t kNoId = 0xffffffffu;        // no token id: ids are tallied only when < V <= 2^31
constexpr int kCarefulTrips = 2;               // trips a CTA counts one add at a time, until its hot id is known
constexpr int kGateWords = 4;                  // {recount, unused, skipped ids (64 bits)}

// Words per CTA for V bins, 0 when they do not fit: the smallest W >= ceil(V / 3) for which
// field = (id * M) >> 32 with M = 2^32 / W + 1 is exact for every id < 3W (the quotient steps at W and 2W:
// it is monotone, so the four ids around the steps decide).
static uint32_t packed_words(int32_t V, uint32_t* magic) {
    for (uint64_t W = ((uint64_t)V + 2) / 3; W >= 2 && W * 4 <= kDynSmem; ++W) {
        const uint64_t M = (1ull << 32) / W + 1;
        if (M >> 32) continue;
        if ((((W - 1) * M) >> 32) == 0 && ((W * M) >> 32) == 1 && (((2 * W - 1) * M) >> 32) == 1 &&
            (((2 * W) * M) >> 32) == 2 && (((3 * W - 1) * M) >> 32) == 2) {
            if (magic) *magic = (uint32_t)M;
            return (uint32_t)W;
        }
    }
    return 0;
}

__global__ void __launch_bounds__(kThreads, 1)
k_hist_packed(const int32_t* __restrict__ ids, int64_t n, int32_t V, uint32_t W, uint32_t M,
              uint32_t* __restrict__ out, uint32_t* __restrict__ gate) {
    extern __shared__ __align__(16) uint32_t s_fields[];
    __shared__ uint32_t s_hot;
    __shared__ uint32_t s_own[32];                           // the hot id's counts, one word per lane
    for (uint32_t i = threadIdx.x; i < W; i += kThreads) s_fields[i] = 0;
    if (threadIdx.x == 0) s_hot = kNoId;
    if (threadIdx.x < 32) s_own[threadIdx.x] = 0;
    __syncthreads();
    unsigned long long bad = 0;
    uint32_t wrapped = 0, hot = kNoId;
    const uint32_t base = (uint32_t)__cvta_generic_to_shared(s_fields);
    const uint32_t own = (uint32_t)__cvta_generic_to_shared(&s_own[threadIdx.x & 31]);
    const uint32_t neg_w = 0u - W;
    // One token with id < V: the add, and what its test needs.  `low` is the field's low nine bits in place;
    // for the hot id it is bit 31 of the lane's own word, which is never set, so the test never fires there.
    auto add_one = [&](uint32_t id, uint32_t& low) -> uint32_t {
        uint32_t old;
        asm volatile("{\n\t"
            ".reg .pred ph;\n\t"
            ".reg .b32 f, w, sh, a, inc;\n\t"
            "mul.hi.u32 f, %2, %3;\n\t"
            "mad.lo.u32 w, f, %4, %2;\n\t"
            "mul.lo.u32 sh, f, 10;\n\t"
            "shl.b32 inc, 1, sh;\n\t"
            "shl.b32 %1, 511, sh;\n\t"
            "mad.lo.u32 a, w, 4, %5;\n\t"
            "setp.eq.u32 ph, %2, %6;\n\t"
            "selp.u32 a, %7, a, ph;\n\t"
            "selp.u32 inc, 1, inc, ph;\n\t"
            "selp.u32 %1, 0x80000000, %1, ph;\n\t"
            "atom.shared.add.u32 %0, [a], inc;\n\t"
            "}" : "=&r"(old), "=&r"(low)
                : "r"(id), "r"(M), "r"(neg_w), "r"(base), "r"(hot), "r"(own) : "memory");
        return old;
    };
    static_assert(kFieldBits == 10 && kSpill == 512, "written into the instructions above");
    // The add found the low nine bits of its field set: kSpill-1 (hand kSpill counts on) or kFieldMax (wrapped).
    auto settle_field = [&](uint32_t id, uint32_t old) {
        const uint32_t f = __umulhi(id, M), inc = 1u << (f * kFieldBits);
        if ((old & (inc * kFieldMax)) == inc * kFieldMax) {
            wrapped = 1;
        } else {
            atomicSub(&s_fields[id - f * W], inc * kSpill);
            atomicAdd(&out[id], kSpill);
            if (*reinterpret_cast<volatile uint32_t*>(&s_hot) == kNoId) atomicCAS(&s_hot, kNoId, id);
        }
    };
    auto tally_in_range = [&](uint32_t id) {
        uint32_t low;
        const uint32_t old = add_one(id, low);
        if ((~old & low) == 0) settle_field(id, old);
    };
    auto tally1 = [&](uint32_t id) {
        if (id < (uint32_t)V) tally_in_range(id); else ++bad;
    };
    // Four tokens of one 128-bit load: four adds in flight, their tests folded into one branch (taken once
    // in about kSpill / 4 loads).
    auto tally4 = [&](uint4 x) {
        if (max(max(x.x, x.y), max(x.z, x.w)) < (uint32_t)V) {       // one range test per 128-bit load
            uint32_t la, lb, lc, ld;
            const uint32_t oa = add_one(x.x, la);
            const uint32_t ob = add_one(x.y, lb);
            const uint32_t oc = add_one(x.z, lc);
            const uint32_t od = add_one(x.w, ld);
            const uint32_t za = ~oa & la, zb = ~ob & lb, zc = ~oc & lc, zd = ~od & ld;
            if (min(min(za, zb), min(zc, zd)) == 0) {
                if (za == 0) settle_field(x.x, oa);
                if (zb == 0) settle_field(x.y, ob);
                if (zc == 0) settle_field(x.z, oc);
                if (zd == 0) settle_field(x.w, od);
            }
        } else {
            tally1(x.x); tally1(x.y); tally1(x.z); tally1(x.w);
        }
    };
    // the same, each add tested before the next is issued (one add in flight per thread)
    auto tally4_in_turn = [&](uint4 x) { tally1(x.x); tally1(x.y); tally1(x.z); tally1(x.w); };
    // The walk over the CTA's share of the 16-byte-aligned body: whole trips of kRows rows (kThreads 128-bit
    // loads each) without a bounds test, then guarded rows; CTA 0 takes the ragged ends.
    const uintptr_t addr = reinterpret_cast<uintptr_t>(ids);
    int64_t head = ((16 - (addr & 15)) & 15) >> 2;
    if (head > n) head = n;
    const int64_t nvec = (n - head) >> 2;
    const int64_t tail0 = head + nvec * 4;
    if (blockIdx.x == 0) {
        if ((int64_t)threadIdx.x < head) tally1((uint32_t)ids[threadIdx.x]);
        const int64_t t = tail0 + threadIdx.x;
        if (t < n) tally1((uint32_t)ids[t]);
    }
    const uint4* vec = reinterpret_cast<const uint4*>(ids + head);
    const int64_t v0 = nvec * blockIdx.x / gridDim.x;
    const int64_t v1 = nvec * (blockIdx.x + 1) / gridDim.x;
    const int64_t trips = (v1 - v0) / (kRows * kThreads);
    const uint4* p = vec + v0 + threadIdx.x;
    for (int64_t t = 0; t < trips; ++t, p += kRows * kThreads) {
        uint4 x[kRows];
#pragma unroll
        for (int r = 0; r < kRows; ++r) x[r] = ld_stream_u4(p + r * kThreads);
        if (hot == kNoId) hot = *reinterpret_cast<volatile uint32_t*>(&s_hot);   // once set it stays
        if (t < kCarefulTrips) {
#pragma unroll
            for (int r = 0; r < kRows; ++r) tally4_in_turn(x[r]);
        } else {
#pragma unroll
            for (int r = 0; r < kRows; ++r) tally4(x[r]);
        }
    }
    for (int64_t v = v0 + trips * (kRows * kThreads) + threadIdx.x; v < v1; v += kThreads) tally4_in_turn(ld_stream_u4(vec + v));
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < W; i += kThreads) {
        const uint32_t w = (i + blockIdx.x * (W / gridDim.x)) % W;   // the CTAs' flushes spread over the whole array
        const uint32_t x = s_fields[w];
#pragma unroll
        for (uint32_t f = 0; f < 3; ++f) {
            const uint32_t c = (x >> (f * kFieldBits)) & kFieldMax, id = f * W + w;
            if (c && id < (uint32_t)V) atomicAdd(&out[id], c);
        }
    }
    if (threadIdx.x < 32) {                                  // (only lanes that had read s_hot added to s_own)
        uint32_t c = s_own[threadIdx.x];
        for (int o = 16; o; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
        if (threadIdx.x == 0 && c) atomicAdd(&out[s_hot], c);
    }
    if (wrapped) atomicOr(&gate[0], 1u);
    for (int o = 16; o; o >>= 1) bad += __shfl_xor_sync(0xffffffffu, bad, o);
    if ((threadIdx.x & 31) == 0 && bad) atomicAdd(reinterpret_cast<unsigned long long*>(gate + 2), bad);
}

// After the packed count: if it stood, counts (+)= packed and the skipped ids are reported; if a field
// wrapped, counts is left as the recount needs it (zero unless accumulating) and the recount's sampling
// pre-pass runs here.
__global__ void __launch_bounds__(kThreads, 1)
k_hist_settle(const int32_t* __restrict__ ids, int64_t n, int32_t V, const uint32_t* __restrict__ packed,
              uint32_t* __restrict__ counts, int accumulate, uint32_t* __restrict__ sample,
              const uint32_t* __restrict__ gate, Ctrl* ctrl) {
    __shared__ int s_tag[kSampleSlots];
    __shared__ uint32_t s_cnt[kSampleSlots];
    const bool recount = gate[0] != 0;
    for (int v = blockIdx.x * kThreads + threadIdx.x; v < V; v += gridDim.x * kThreads) {
        const uint32_t c = recount ? 0u : packed[v];
        counts[v] = accumulate ? counts[v] + c : c;
    }
    if (!recount) {
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            const unsigned long long bad = *reinterpret_cast<const unsigned long long*>(gate + 2);
            if (bad) {
                atomicAdd(&ctrl->n_bad, bad);
                atomicOr(&ctrl->flags, (uint32_t)VT_FLAG_BAD_ID);
            }
        }
        return;
    }
    sample_stream(ids, n, V, sample, s_tag, s_cnt);
}

// ---- measurement aid: directly indexed 32-bit bins, one shared-memory reduction per token, nothing else ----
// counts[id mod bins] over the ids inside [0, V): a plain second kernel over the same stream, timed beside
// the histogram by the benchmark.
__global__ void __launch_bounds__(kThreads, 1)
k_hist_fold(const int32_t* __restrict__ ids, int64_t n, int32_t V, int32_t bins, uint32_t* __restrict__ counts) {
    extern __shared__ __align__(16) uint32_t s_bins[];
    for (int i = threadIdx.x; i < bins; i += kThreads) s_bins[i] = 0;
    __syncthreads();
    const uint32_t nb = (uint32_t)bins;
    const bool two_steps = (uint32_t)V <= 3u * nb;           // id mod bins by at most two subtractions
    stream_ids(ids, n, [&](uint32_t id) {
        if (id < (uint32_t)V) {
            uint32_t b = id;
            if (two_steps) { b = b >= nb ? b - nb : b; b = b >= nb ? b - nb : b; }
            else b = b % nb;
            atomicAdd(&s_bins[b], 1u);
        }
    });
    __syncthreads();
    for (int i = threadIdx.x; i < bins; i += kThreads) {
        const int v = (i + blockIdx.x * 61) % bins;
        const uint32_t c = s_bins[v];
        if (c) atomicAdd(&counts[v], c);
    }
}

}  // namespace

// opt-in shared-memory sizes are per device: remember which devices have been set up
static cudaError_t set_smem_once(const void* fn, size_t bytes, int (&done)[kMaxDevices]) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < kMaxDevices && done[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess && dev >= 0 && dev < kMaxDevices) done[dev] = 1;
    return e;
}

cudaError_t launch_hist_fold(const int32_t* ids, int64_t n, int32_t V, int32_t bins, uint32_t* counts, cudaStream_t s) {
    if (bins < 1 || (size_t)bins * 4 > kDynSmem) return cudaErrorInvalidValue;
    cudaError_t e = cudaMemsetAsync(counts, 0, (size_t)bins * 4, s);
    if (e != cudaSuccess || n == 0) return e;
    static int done_fold[kMaxDevices] = {0};
    e = set_smem_once(reinterpret_cast<const void*>(k_hist_fold), kDynSmem, done_fold);
    if (e != cudaSuccess) return e;
    int grid = (int)((n + 4095) / 4096);
    if (grid > num_sms()) grid = num_sms();
    k_hist_fold<<<grid, kThreads, (size_t)bins * 4, s>>>(ids, n, V, bins, counts);
    count_launch();
    return cudaGetLastError();
}

bool hist_supported(int32_t V) {
    if (V < 1) return false;
    if ((size_t)V * 4 <= kDynSmem) return true;
    return ((size_t)V + 31) / 32 * 8 <= kMaxTableBytes;
}

static bool packed_fits(int32_t V) { return packed_words(V, nullptr) != 0; }

HistPlan hist_plan(int32_t V) {
    HistPlan p{};
    p.small = (size_t)V * 4 <= kDynSmem;
    if (p.small) { p.off_sample = p.off_packed = p.off_gate = p.off_table = 0; p.bytes = 0; return p; }
    const size_t T32 = ((size_t)V + 31) / 32;
    // sample, packed counts and gate lie together: one memset clears all three
    p.off_sample = 0;
    p.off_packed = (size_t)V * 4;
    p.off_gate = packed_fits(V) ? 2 * (size_t)V * 4 : p.off_packed;
    p.clear_bytes = packed_fits(V) ? p.off_gate + kGateWords * 4 : (size_t)V * 4;
    p.off_table = align_up(p.clear_bytes, 256);
    p.bytes = p.off_table + align_up(T32 * 8, 256);
    return p;
}

cudaError_t launch_histogram(const int32_t* ids, int64_t n, int32_t V, uint32_t* counts,
                             int accumulate, Ctrl* ctrl, uint8_t* scratch, cudaStream_t s) {
    cudaError_t e;
    const HistPlan p = hist_plan(V);
    const bool packed_path = !p.small && packed_fits(V) && n != 0;
    if (!accumulate && !packed_path) {                     // (the packed path's second kernel writes every count)
        e = cudaMemsetAsync(counts, 0, (size_t)V * 4, s);
        if (e != cudaSuccess) return e;
    }
    if (n == 0) return cudaSuccess;
    const int sms = num_sms();
    // enough CTAs to fill the chip, never more than one per 4096 ids
    int grid = (int)((n + 4095) / 4096);
    if (grid > sms) grid = sms;
    if (grid < 1) grid = 1;
    if (p.small) {
        static int done_small[kMaxDevices] = {0};
        e = set_smem_once(reinterpret_cast<const void*>(k_hist_small), kDynSmem, done_small);
        if (e != cudaSuccess) return e;
        k_hist_small<<<grid, kThreads, (size_t)V * 4, s>>>(ids, n, V, counts, ctrl);
        count_launch();
        return cudaGetLastError();
    }
    const size_t T32 = ((size_t)V + 31) / 32;
    if (T32 * 8 > kMaxTableBytes) return cudaErrorInvalidValue;   // rejected earlier by the API
    int32_t H = (int32_t)((kDynSmem - T32 * 8) / 4);
    if (H > 65535) H = 65535;                          // slots are 16-bit in the main pass's lookup
    uint32_t* sample = reinterpret_cast<uint32_t*>(scratch + p.off_sample);
    uint2* table = reinterpret_cast<uint2*>(scratch + p.off_table);
    e = cudaMemsetAsync(scratch, 0, p.clear_bytes, s);
    if (e != cudaSuccess) return e;
    static int done_pick[kMaxDevices] = {0}, done_hot[kMaxDevices] = {0}, done_packed[kMaxDevices] = {0};
    e = set_smem_once(reinterpret_cast<const void*>(k_hist_pick), kMaxTableBytes, done_pick);
    if (e != cudaSuccess) return e;
    e = set_smem_once(reinterpret_cast<const void*>(k_hist_hot), kDynSmem, done_hot);
    if (e != cudaSuccess) return e;
    // a refused launch must stop the chain: the main pass would count through an unwritten table
    const uint32_t* gate = nullptr;
    if (packed_path) {
        // all bins in shared memory, packed; the three kernels after it return at once unless a field wrapped
        e = set_smem_once(reinterpret_cast<const void*>(k_hist_packed), kDynSmem, done_packed);
        if (e != cudaSuccess) return e;
        uint32_t M = 0;
        const uint32_t W = packed_words(V, &M);
        uint32_t* packed = reinterpret_cast<uint32_t*>(scratch + p.off_packed);
        uint32_t* g = reinterpret_cast<uint32_t*>(scratch + p.off_gate);
        k_hist_packed<<<grid, kThreads, (size_t)W * 4, s>>>(ids, n, V, W, M, packed, g);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        k_hist_settle<<<grid, kThreads, 0, s>>>(ids, n, V, packed, counts, accumulate, sample, g, ctrl);
        gate = g;
    } else {
        k_hist_sample<<<grid, kThreads, 0, s>>>(ids, n, V, sample);
    }
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    k_hist_pick<<<1, kThreads, T32 * 8, s>>>(sample, V, H, table, gate);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    k_hist_hot<<<grid, kThreads, kDynSmem, s>>>(ids, n, V, counts, table, H, ctrl, gate);
    count_launch();
    return cudaGetLastError();
}

}  // namespace vt
