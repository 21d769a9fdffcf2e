// Head reconstruction (Eq. 1, second line: W_trim = W[Top-K(c,k), :]): a gather of K bf16 rows.
// Pure HBM traffic, 2 * K * d * 2 bytes.  One warp copies one row at a time with 128-bit
// streaming loads/stores, several in flight per lane; rows are dealt round-robin over a grid
// that fills the chip.
#include "vt_common.cuh"

namespace vt {

namespace {

constexpr int kThreads = 256;
constexpr int kCtasPerSm = 8;

__global__ void __launch_bounds__(kThreads)
k_gather_rows(const uint16_t* __restrict__ W_full, const int32_t* __restrict__ map,
              uint16_t* __restrict__ W_trim, int32_t V, int32_t K, int32_t d, Ctrl* ctrl) {
    const int lane = threadIdx.x & 31;
    const int warps_total = gridDim.x * (kThreads / 32);
    const int gw = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    const int nvec = d >> 3;                                     // 16-byte vectors per row
    for (int j = gw; j < K; j += warps_total) {
        const int32_t src = map[j];
        uint4* dst = reinterpret_cast<uint4*>(W_trim + (size_t)j * d);
        if ((uint32_t)src >= (uint32_t)V) {                      // bad entry: flag, zero the row
            if (lane == 0 && ctrl) atomicOr(&ctrl->flags, (uint32_t)VT_FLAG_BAD_MAP);
            for (int i = lane; i < nvec; i += 32) dst[i] = make_uint4(0, 0, 0, 0);
            continue;
        }
        const uint4* from = reinterpret_cast<const uint4*>(W_full + (size_t)src * d);
        int i = lane;
        for (; i + 224 < nvec; i += 256) {                       // 8 loads in flight per lane
            uint4 r[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) r[u] = ld_stream_u4(from + i + 32 * u);
#pragma unroll
            for (int u = 0; u < 8; ++u) st_stream_u4(dst + i + 32 * u, r[u]);
        }
        for (; i < nvec; i += 32) st_stream_u4(dst + i, ld_stream_u4(from + i));
    }
}

}  // namespace

cudaError_t launch_gather_rows(const uint16_t* W_full, const int32_t* map, uint16_t* W_trim,
                               int32_t V, int32_t K, int32_t d, Ctrl* ctrl, cudaStream_t s) {
    const int warps_per_cta = kThreads / 32;
    int grid = (K + warps_per_cta - 1) / warps_per_cta;
    const int cap = num_sms() * kCtasPerSm;
    if (grid > cap) grid = cap;
    k_gather_rows<<<grid, kThreads, 0, s>>>(W_full, map, W_trim, V, K, d, ctrl);
    count_launch();
    return cudaGetLastError();
}

}  // namespace vt
