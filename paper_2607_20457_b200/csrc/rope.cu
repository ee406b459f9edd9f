// Position ids of the assembled Phase-1 inputs and the rotary embedding they feed (Appendix E).
//
//   assemble_positions_kernel  one CTA column per assembled input: the prefix entries keep their
//                              global positions (sparse) or everything is renumbered (contiguous)
//   rope_kernel                a CTA takes eight rows at a time: each row's d/2 (cos, sin) pairs are
//                              formed once in shared memory -- angle in float64, reduced to [-pi, pi],
//                              then sincosf -- and applied to every head with 16-byte loads and
//                              stores.  A pure stream over the rows: HBM-bound.
#include <cmath>

#include "common.cuh"

namespace pulsar {
namespace {

constexpr int kMaxHalf = 128;                       // d <= 256
struct RopeFreq {
    double inv_freq[kMaxHalf];                      // theta^(-2j/d), from the host's libm
};

__global__ void __launch_bounds__(256)
assemble_positions_kernel(const int32_t* __restrict__ prefix_idx, const int32_t* __restrict__ prefix_len,
                          int prefix_total, int n_blocks, int block_size, int mode, int32_t* __restrict__ pos_out,
                          int64_t capacity, int32_t* status) {
    const int i = blockIdx.y;
    __shared__ int64_t s_base;
    __shared__ int s_len;
    if (threadIdx.x == 0) {
        int64_t base = 0;
        bool bad = false;
        for (int b = 0; b <= i; ++b) {
            int pl = prefix_len[b];
            if (pl < 0 || pl > prefix_total) { bad = true; pl = max(0, min(pl, prefix_total)); }
            if (b < i) base += pl + block_size;
            else s_len = pl;
        }
        if (bad && blockIdx.x == 0) report(status, PULSAR_DEV_BAD_LENGTH);
        s_base = base;
    }
    __syncthreads();
    const int P = s_len, n = P + block_size;
    for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < n; j += gridDim.x * blockDim.x) {
        const int64_t at = s_base + j;
        if (at >= capacity) break;
        int v;
        if (mode == PULSAR_POS_CONTIGUOUS) v = j;
        else v = j < P ? prefix_idx[j] : i * block_size + (j - P);
        pos_out[at] = v;
    }
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Measured on B200 (80,320 rows of 32 + 8 heads, d = 128, two launches): 8 rows, 2 loads in flight,
// 4 CTAs per SM 5.25 TB/s; 16 rows 5.09; 4 loads in flight (spills at 64 registers) 4.88; 6 CTAs per SM
// 4.77.  The 32-head pass alone streams at 6.4 TB/s; the 8-head pass is bound by the sines and cosines
// (same work per row, a quarter of the bytes), which is why Q and K can share one launch.
constexpr int kRopeRows = 8;                        // rows a CTA takes at a time
constexpr int kRopeUnroll = 2;                      // tasks (2 x 16-byte loads each) in flight per thread
constexpr int kRopeCtasPerSm = 4;

// X2/Y2/H2 describe an optional second tensor with the same rows and head size (K beside Q): it
// shares the rows' cosines and sines; H2 = 0 when there is none.
__global__ void __launch_bounds__(256, kRopeCtasPerSm)
rope_kernel(const uint4* __restrict__ X1, uint4* __restrict__ Y1, int H1, const uint4* __restrict__ X2,
            uint4* __restrict__ Y2, int H2, int64_t rows, int d, const int32_t* __restrict__ positions,
            const __grid_constant__ RopeFreq f, int32_t* status) {
    __shared__ float s_cos[kRopeRows][kMaxHalf], s_sin[kRopeRows][kMaxHalf];
    const int half = d >> 1;
    const int vec_half = half >> 3;                 // 16-byte vectors per half row of a head
    const int head_vecs = d >> 3;
    const int tasks1 = H1 * vec_half;               // per row: one task = vector v of both halves of head h
    const int tasks = tasks1 + H2 * vec_half;
    const int64_t n_groups = (rows + kRopeRows - 1) / kRopeRows;
    for (int64_t grp = blockIdx.x; grp < n_groups; grp += gridDim.x) {
        const int64_t row0 = grp * kRopeRows;
        const int nr = static_cast<int>(min(static_cast<int64_t>(kRopeRows), rows - row0));
        for (int e = threadIdx.x; e < nr * half; e += blockDim.x) {
            const int r = e / half, j = e - r * half;
            int p = positions[row0 + r];
            if (p < 0) {
                report(status, PULSAR_DEV_BAD_POSITION);
                p = 0;
            }
            // angle / 2pi in float64, reduced to [-1/2, 1/2] turns, then float32 sincos of at most pi
            const double turns = static_cast<double>(p) * f.inv_freq[j] * 0.15915494309189535;
            const double frac = turns - rint(turns);
            float sn, cs;
            sincosf(static_cast<float>(frac * 6.283185307179586), &sn, &cs);
            s_cos[r][j] = cs;
            s_sin[r][j] = sn;
        }
        __syncthreads();
        const int total = nr * tasks;
        for (int t0 = threadIdx.x; t0 < total; t0 += blockDim.x * kRopeUnroll) {
            uint4 a[kRopeUnroll], b[kRopeUnroll];
            int rr[kRopeUnroll], vv[kRopeUnroll];
            uint4* dst[kRopeUnroll];
#pragma unroll
            for (int u = 0; u < kRopeUnroll; ++u) {
                const int t = t0 + u * blockDim.x;
                if (t < total) {
                    const int r = t / tasks;
                    int rem = t - r * tasks;
                    const bool second = rem >= tasks1;
                    if (second) rem -= tasks1;
                    const int h = rem / vec_half, v = rem - h * vec_half;
                    const int64_t lo = (row0 + r) * (static_cast<int64_t>(second ? H2 : H1) * head_vecs) + h * head_vecs + v;
                    const uint4* src = (second ? X2 : X1) + lo;
                    rr[u] = r;
                    vv[u] = v;
                    dst[u] = (second ? Y2 : Y1) + lo;
                    a[u] = src[0];
                    b[u] = src[vec_half];
                }
            }
#pragma unroll
            for (int u = 0; u < kRopeUnroll; ++u) {
                const int t = t0 + u * blockDim.x;
                if (t < total) {
                    const uint32_t aw[4] = {a[u].x, a[u].y, a[u].z, a[u].w}, bw[4] = {b[u].x, b[u].y, b[u].z, b[u].w};
                    uint32_t ya[4], yb[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int j = vv[u] * 8 + 2 * k;
                        const float c0 = s_cos[rr[u]][j], s0 = s_sin[rr[u]][j];
                        const float c1 = s_cos[rr[u]][j + 1], s1 = s_sin[rr[u]][j + 1];
                        const float a0 = bf16_lo(aw[k]), a1 = bf16_hi(aw[k]), b0 = bf16_lo(bw[k]), b1 = bf16_hi(bw[k]);
                        ya[k] = pack_bf16x2(a0 * c0 - b0 * s0, a1 * c1 - b1 * s1);
                        yb[k] = pack_bf16x2(b0 * c0 + a0 * s0, b1 * c1 + a1 * s1);
                    }
                    dst[u][0] = make_uint4(ya[0], ya[1], ya[2], ya[3]);
                    dst[u][vec_half] = make_uint4(yb[0], yb[1], yb[2], yb[3]);
                }
            }
        }
        __syncthreads();
    }
}

int32_t launch_rope(const uint16_t* X1, uint16_t* Y1, int32_t H1, const uint16_t* X2, uint16_t* Y2, int32_t H2,
                    int64_t rows, int32_t d, const int32_t* positions, double theta, int32_t* device_status,
                    void* stream) {
    if (rows < 0 || H1 <= 0 || H2 < 0 || d <= 0 || !(theta > 0.0)) return PULSAR_ERR_INVALID_ARG;
    if (d % 16 != 0 || d > 2 * kMaxHalf || H1 > 65535 || H2 > 65535) return PULSAR_ERR_SHAPE;
    if (rows == 0) return PULSAR_OK;
    if (!X1 || !Y1 || !positions || (H2 > 0 && (!X2 || !Y2))) return PULSAR_ERR_INVALID_ARG;
    if (!aligned(X1, 16) || !aligned(Y1, 16) || !aligned(X2, 16) || !aligned(Y2, 16) || !aligned(positions, 4))
        return PULSAR_ERR_ALIGNMENT;
    int32_t rc = check_device();
    if (rc != PULSAR_OK) return rc;
    RopeFreq f;
    for (int j = 0; j < d / 2; ++j) f.inv_freq[j] = std::pow(theta, -2.0 * static_cast<double>(j) / static_cast<double>(d));
    const int64_t ctas = std::min<int64_t>((rows + kRopeRows - 1) / kRopeRows, static_cast<int64_t>(sm_count()) * kRopeCtasPerSm);
    rope_kernel<<<static_cast<unsigned>(ctas), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<const uint4*>(X1), reinterpret_cast<uint4*>(Y1), H1, reinterpret_cast<const uint4*>(X2),
        reinterpret_cast<uint4*>(Y2), H2, rows, d, positions, f, device_status);
    PULSAR_CUDA_OK(cudaGetLastError());
    count_launch();
    return PULSAR_OK;
}

}  // namespace
}  // namespace pulsar

using namespace pulsar;

extern "C" int32_t pulsar_assemble_positions(const int32_t* prefix_idx, const int32_t* prefix_len,
                                             int32_t prefix_total, int32_t n_blocks, int32_t block_size,
                                             int32_t mode, int32_t* pos_out, int64_t pos_capacity,
                                             int32_t* device_status, void* stream) {
    if (n_blocks <= 0 || block_size <= 0 || prefix_total < 0 || pos_capacity < 0) return PULSAR_ERR_INVALID_ARG;
    if (mode != PULSAR_POS_SPARSE && mode != PULSAR_POS_CONTIGUOUS) return PULSAR_ERR_INVALID_ARG;
    if (n_blocks > 65535) return PULSAR_ERR_SHAPE;
    if (!prefix_len || !pos_out || (prefix_total > 0 && !prefix_idx)) return PULSAR_ERR_INVALID_ARG;
    if (!aligned(prefix_len, 4) || !aligned(pos_out, 4) || !aligned(prefix_idx, 4)) return PULSAR_ERR_ALIGNMENT;
    int32_t rc = check_device();
    if (rc != PULSAR_OK) return rc;
    const int64_t longest = static_cast<int64_t>(prefix_total) + block_size;
    const unsigned gx = static_cast<unsigned>(std::min<int64_t>((longest + 255) / 256, 64));
    assemble_positions_kernel<<<dim3(gx, n_blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        prefix_idx, prefix_len, prefix_total, n_blocks, block_size, mode, pos_out, pos_capacity, device_status);
    PULSAR_CUDA_OK(cudaGetLastError());
    count_launch();
    return PULSAR_OK;
}

extern "C" int32_t pulsar_rope_apply(const uint16_t* X, uint16_t* Y, int64_t rows, int32_t H, int32_t d,
                                     const int32_t* positions, double theta, int32_t* device_status,
                                     void* stream) {
    return launch_rope(X, Y, H, nullptr, nullptr, 0, rows, d, positions, theta, device_status, stream);
}

extern "C" int32_t pulsar_rope_apply_qk(const uint16_t* Q, uint16_t* Q_out, int32_t Hq, const uint16_t* K,
                                        uint16_t* K_out, int32_t Hkv, int64_t rows, int32_t d,
                                        const int32_t* positions, double theta, int32_t* device_status,
                                        void* stream) {
    if (Hkv <= 0) return PULSAR_ERR_INVALID_ARG;
    return launch_rope(Q, Q_out, Hq, K, K_out, Hkv, rows, d, positions, theta, device_status, stream);
}
