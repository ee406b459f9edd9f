// Online-softmax merge of attention partials (Appendix H, Eq. 12-13) in closed form:
//   l = m + ln sum_j exp(l_j - m),  O = sum_j exp(l_j - l) A_j,  m = max_j l_j.
// One thread per four consecutive output elements: 128-bit loads of the fp32 partials, one
// 64-bit store of bf16.  The kernel is a pure stream over J*rows*(d+1) floats.
#include "common.cuh"

namespace pulsar {

// stride_O / stride_L: floats between consecutive parts of part_O / part_LSE.  kF32: the merged
// output stays float32 (a partial for a later merge) instead of being rounded to bf16.
template <bool kF32>
__global__ void __launch_bounds__(256)
lse_merge_kernel(const float* __restrict__ part_O, const float* __restrict__ part_LSE, int n_parts,
                 int64_t stride_O, int64_t stride_L, int64_t rows, int d, void* __restrict__ O_,
                 float* __restrict__ LSE) {
    grid_dependency_wait();        // launched beside the attention kernel that writes the partials: wait for it
    const int vec_per_row = d >> 2;
    const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= rows * vec_per_row) return;
    const int64_t row = idx / vec_per_row;
    const int v = static_cast<int>(idx - row * vec_per_row);

    // The loads of a group of parts are independent: issue them together (a decode-shaped merge is
    // a few CTAs whose run time is a chain of load latencies).
    float m = -INFINITY;
#pragma unroll 8
    for (int j = 0; j < n_parts; ++j) m = fmaxf(m, part_LSE[static_cast<size_t>(j) * stride_L + row]);

    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float denom = 0.f;
    if (m > -INFINITY) {
#pragma unroll 8
        for (int j = 0; j < n_parts; ++j) {
            const float w = __expf(part_LSE[static_cast<size_t>(j) * stride_L + row] - m);
            const float4 o = *reinterpret_cast<const float4*>(part_O + static_cast<size_t>(j) * stride_O + row * d + v * 4);
            denom += w;
            acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
        }
        const float inv = 1.f / denom;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    }
    if (kF32) {
        *reinterpret_cast<float4*>(static_cast<float*>(O_) + row * d + v * 4) = acc;
    } else {
        uint2 packed;
        packed.x = pack_bf16x2(acc.x, acc.y);
        packed.y = pack_bf16x2(acc.z, acc.w);
        *reinterpret_cast<uint2*>(static_cast<uint16_t*>(O_) + row * d + v * 4) = packed;
    }
    if (LSE != nullptr && v == 0) LSE[row] = (m > -INFINITY) ? m + logf(denom) : -INFINITY;
}

// The same merge for few output rows and many parts (decode shapes), where one thread per output
// vector would run a long chain of load latencies on a handful of CTAs: kLanes consecutive lanes
// share an output vector, lane i takes parts i, i + kLanes, ...; the maximum and the sums are
// combined by butterfly shuffles (a fixed order, so the result is reproducible).  A lane issues
// the loads of all its parts -- the l_j and the output vectors, which do not depend on them --
// before it uses any (up to kMaxInFlight parts at a time), so the kernel lasts about one memory
// round trip however many parts there are.
constexpr int kMergeLanes = 8;          // moderate part counts
constexpr int kMergeLanesWide = 32;     // decode shapes: 4 partials per KV part, dozens of parts
// Outputs (rows x d/4) up to which the lane form is used.  Measured: 72 parts into 32 or 256 rows 3.5 us
// faster than one thread per output; 16 parts into 2048 rows 2.6 us and 64 parts into 1024 rows 6 us slower.
constexpr int64_t kMergeLanesMaxThreads = 8192;
// ... and up to which a whole warp shares an output vector.  Measured at 72 parts: 32 rows (1024 outputs)
// 3 us faster than with 8 lanes, 256 rows (8192 outputs) no faster.
constexpr int64_t kMergeWideMaxThreads = 1024;

template <bool kF32, int kLanes>
__global__ void __launch_bounds__(256)
lse_merge_lanes_kernel(const float* __restrict__ part_O, const float* __restrict__ part_LSE, int n_parts,
                       int64_t stride_O, int64_t stride_L, int64_t rows, int d, void* __restrict__ O_,
                       float* __restrict__ LSE) {
    grid_dependency_wait();        // launched beside the attention kernel that writes the partials: wait for it
    constexpr int kMaxInFlight = 4;
    const int vec_per_row = d >> 2;
    const int64_t tid = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const int sub = static_cast<int>(tid % kLanes);
    const int64_t idx = tid / kLanes;
    const bool valid = idx < rows * vec_per_row;
    const int64_t row = valid ? idx / vec_per_row : 0;
    const int v = valid ? static_cast<int>(idx - row * vec_per_row) : 0;

    // running maximum, weight sum and weighted sum over this lane's parts (ascending part order)
    float m = -INFINITY, denom = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (valid) {
        for (int j0 = sub; j0 < n_parts; j0 += kLanes * kMaxInFlight) {
            float l[kMaxInFlight];
            float4 o[kMaxInFlight];
#pragma unroll
            for (int b = 0; b < kMaxInFlight; ++b) {
                const int j = j0 + b * kLanes;
                const int jc = j < n_parts ? j : j0;                 // a slot past the end repeats a load and weighs nothing
                l[b] = part_LSE[static_cast<size_t>(jc) * stride_L + row];
                o[b] = *reinterpret_cast<const float4*>(part_O + static_cast<size_t>(jc) * stride_O + row * d + v * 4);
                if (j >= n_parts) l[b] = -INFINITY;
            }
            float m_new = m;
#pragma unroll
            for (int b = 0; b < kMaxInFlight; ++b) m_new = fmaxf(m_new, l[b]);
            if (m_new > -INFINITY) {
                const float keep = (m == -INFINITY) ? 0.f : __expf(m - m_new);
                denom *= keep;
                acc.x *= keep; acc.y *= keep; acc.z *= keep; acc.w *= keep;
#pragma unroll
                for (int b = 0; b < kMaxInFlight; ++b) {
                    const float w = (l[b] == -INFINITY) ? 0.f : __expf(l[b] - m_new);
                    denom += w;
                    acc.x += w * o[b].x; acc.y += w * o[b].y; acc.z += w * o[b].z; acc.w += w * o[b].w;
                }
                m = m_new;
            }
        }
    }
    // bring the lanes to the common maximum, then add them up
    float m_all = m;
#pragma unroll
    for (int o = 1; o < kLanes; o <<= 1) m_all = fmaxf(m_all, __shfl_xor_sync(0xffffffffu, m_all, o));
    const float mine = (m == -INFINITY) ? 0.f : __expf(m - m_all);
    denom *= mine;
    acc.x *= mine; acc.y *= mine; acc.z *= mine; acc.w *= mine;
#pragma unroll
    for (int o = 1; o < kLanes; o <<= 1) {
        denom += __shfl_xor_sync(0xffffffffu, denom, o);
        acc.x += __shfl_xor_sync(0xffffffffu, acc.x, o);
        acc.y += __shfl_xor_sync(0xffffffffu, acc.y, o);
        acc.z += __shfl_xor_sync(0xffffffffu, acc.z, o);
        acc.w += __shfl_xor_sync(0xffffffffu, acc.w, o);
    }
    if (!valid || sub != 0) return;
    if (m_all > -INFINITY) {
        const float inv = 1.f / denom;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    }
    if (kF32) {
        *reinterpret_cast<float4*>(static_cast<float*>(O_) + row * d + v * 4) = acc;
    } else {
        uint2 packed;
        packed.x = pack_bf16x2(acc.x, acc.y);
        packed.y = pack_bf16x2(acc.z, acc.w);
        *reinterpret_cast<uint2*>(static_cast<uint16_t*>(O_) + row * d + v * 4) = packed;
    }
    if (LSE != nullptr && v == 0) LSE[row] = (m_all > -INFINITY) ? m_all + logf(denom) : -INFINITY;
}

// The merge with every part at its own address: part j is the buffer parts[j], laid out
// [rows_total * d outputs | rows_total LSE] like the Phase-2 exchange buffer of a GPU, and only rows
// [row0, row0 + rows) are merged.  The addresses may be peer-mapped memory of other GPUs: the kernel
// then pulls its slice of every GPU's partial over NVLink with plain loads while it merges (no copy
// engine, no TMA) -- the all-gather and the merge in one pass, each GPU reducing 1/H of
// the rows.
constexpr int kMaxMergePeers = 64;
struct PartTable {
    const float* base[kMaxMergePeers];
};

template <bool kF32>
__global__ void __launch_bounds__(256)
lse_merge_table_kernel(const __grid_constant__ PartTable parts, int n_parts, int64_t rows_total, int64_t row0,
                       int64_t rows, int d, void* __restrict__ O_, float* __restrict__ LSE) {
    const int vec_per_row = d >> 2;
    const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= rows * vec_per_row) return;
    const int64_t r = idx / vec_per_row;
    const int v = static_cast<int>(idx - r * vec_per_row);
    const int64_t row = row0 + r;
    const int64_t lse_at = rows_total * d + row;

    float m = -INFINITY;
#pragma unroll 8
    for (int j = 0; j < n_parts; ++j) m = fmaxf(m, parts.base[j][lse_at]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float denom = 0.f;
    if (m > -INFINITY) {
#pragma unroll 8
        for (int j = 0; j < n_parts; ++j) {
            const float w = __expf(parts.base[j][lse_at] - m);
            const float4 o = *reinterpret_cast<const float4*>(parts.base[j] + row * d + v * 4);
            denom += w;
            acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
        }
        const float inv = 1.f / denom;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    }
    if (kF32) {
        *reinterpret_cast<float4*>(static_cast<float*>(O_) + r * d + v * 4) = acc;
    } else {
        uint2 packed;
        packed.x = pack_bf16x2(acc.x, acc.y);
        packed.y = pack_bf16x2(acc.z, acc.w);
        *reinterpret_cast<uint2*>(static_cast<uint16_t*>(O_) + r * d + v * 4) = packed;
    }
    if (LSE != nullptr && v == 0) LSE[r] = (m > -INFINITY) ? m + logf(denom) : -INFINITY;
}

namespace {
// Launch with or without programmatic stream serialization (see launch_lse_merge).
template <typename Kernel, typename... Args>
cudaError_t launch_maybe_dependent(Kernel kernel, unsigned blocks, cudaStream_t stream, bool dependent, Args... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(blocks);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

int32_t launch_merge(const float* part_O, const float* part_LSE, int32_t n_parts, int64_t stride_O, int64_t stride_L,
                     int64_t rows, int32_t d, void* O, bool f32, float* LSE, cudaStream_t stream,
                     bool dependent = false) {
    if (rows == 0) return PULSAR_OK;
    const int64_t threads = rows * (d >> 2);
    if (n_parts >= 2 * kMergeLanes && threads <= kMergeLanesMaxThreads) {
        // few outputs, many parts: spread the parts of an output over lanes
        const bool wide = n_parts >= 2 * kMergeLanesWide && threads <= kMergeWideMaxThreads;
        const int lanes = wide ? kMergeLanesWide : kMergeLanes;
        const unsigned blocks = static_cast<unsigned>((threads * lanes + 255) / 256);
        auto kernel = wide ? (f32 ? lse_merge_lanes_kernel<true, kMergeLanesWide> : lse_merge_lanes_kernel<false, kMergeLanesWide>)
                           : (f32 ? lse_merge_lanes_kernel<true, kMergeLanes> : lse_merge_lanes_kernel<false, kMergeLanes>);
        PULSAR_CUDA_OK(launch_maybe_dependent(kernel, blocks, stream, dependent, part_O, part_LSE, static_cast<int>(n_parts),
                                              stride_O, stride_L, rows, static_cast<int>(d), O, LSE));
        PULSAR_CUDA_OK(cudaGetLastError());
        count_launch();
        return PULSAR_OK;
    }
    const int64_t blocks = (threads + 255) / 256;
    if (blocks > 0x7fffffffll) return PULSAR_ERR_SHAPE;
    auto kernel = f32 ? lse_merge_kernel<true> : lse_merge_kernel<false>;
    PULSAR_CUDA_OK(launch_maybe_dependent(kernel, static_cast<unsigned>(blocks), stream, dependent, part_O, part_LSE,
                                          static_cast<int>(n_parts), stride_O, stride_L, rows, static_cast<int>(d), O, LSE));
    PULSAR_CUDA_OK(cudaGetLastError());
    count_launch();
    return PULSAR_OK;
}
}  // namespace

// after_attention: launched right behind the attention kernel that writes the partials, with
// programmatic stream serialization: its CTAs are placed as that kernel's CTAs leave and wait
// (grid_dependency_wait) until it has finished, so no launch gap separates the two.
int32_t launch_lse_merge(const float* part_O, const float* part_LSE, int32_t n_parts, int64_t rows, int32_t d,
                         uint16_t* O, float* LSE, cudaStream_t stream, bool after_attention) {
    return launch_merge(part_O, part_LSE, n_parts, rows * d, rows, rows, d, O, false, LSE, stream, after_attention);
}

}  // namespace pulsar

using namespace pulsar;

extern "C" int32_t pulsar_lse_merge(const float* part_O, const float* part_LSE, int32_t n_parts, int64_t rows,
                                    int32_t d, uint16_t* O, float* LSE, void* stream) {
    if (n_parts < 1 || rows < 0 || d <= 0) return PULSAR_ERR_INVALID_ARG;
    if (d % 4 != 0 || d > 1024) return PULSAR_ERR_SHAPE;
    if (rows > 0 && (!part_O || !part_LSE || !O)) return PULSAR_ERR_INVALID_ARG;
    if (!aligned(part_O, 16) || !aligned(part_LSE, 4) || !aligned(O, 8)) return PULSAR_ERR_ALIGNMENT;
    int32_t rc = check_device();
    if (rc != PULSAR_OK) return rc;
    return launch_lse_merge(part_O, part_LSE, n_parts, rows, d, O, LSE, static_cast<cudaStream_t>(stream), false);
}

extern "C" int32_t pulsar_lse_merge_strided(const float* part_O, const float* part_LSE, int32_t n_parts,
                                            int64_t part_stride_O, int64_t part_stride_LSE, int64_t rows, int32_t d,
                                            void* O, int32_t out_is_f32, float* LSE, void* stream) {
    if (n_parts < 1 || rows < 0 || d <= 0) return PULSAR_ERR_INVALID_ARG;
    if (d % 4 != 0 || d > 1024) return PULSAR_ERR_SHAPE;
    if (part_stride_O < rows * d || part_stride_LSE < rows || part_stride_O % 4 != 0) return PULSAR_ERR_SHAPE;
    if (rows > 0 && (!part_O || !part_LSE || !O)) return PULSAR_ERR_INVALID_ARG;
    if (!aligned(part_O, 16) || !aligned(part_LSE, 4) || !aligned(O, out_is_f32 ? 16 : 8)) return PULSAR_ERR_ALIGNMENT;
    int32_t rc = check_device();
    if (rc != PULSAR_OK) return rc;
    return launch_merge(part_O, part_LSE, n_parts, part_stride_O, part_stride_LSE, rows, d, O, out_is_f32 != 0, LSE,
                        static_cast<cudaStream_t>(stream));
}

extern "C" int32_t pulsar_lse_merge_peers(const float* const* part_bases_host, int32_t n_parts, int64_t rows_total,
                                          int64_t row_begin, int64_t rows, int32_t d, void* O, int32_t out_is_f32,
                                          float* LSE, void* stream) {
    if (n_parts < 1 || n_parts > kMaxMergePeers || rows_total < 0 || row_begin < 0 || rows < 0 || d <= 0 ||
        !part_bases_host)
        return PULSAR_ERR_INVALID_ARG;
    if (d % 4 != 0 || d > 1024 || row_begin + rows > rows_total) return PULSAR_ERR_SHAPE;
    if (rows == 0) return PULSAR_OK;
    if (!O) return PULSAR_ERR_INVALID_ARG;
    PartTable t{};
    for (int j = 0; j < n_parts; ++j) {
        if (!part_bases_host[j]) return PULSAR_ERR_INVALID_ARG;
        if (!aligned(part_bases_host[j], 16)) return PULSAR_ERR_ALIGNMENT;
        t.base[j] = part_bases_host[j];
    }
    if (!aligned(O, out_is_f32 ? 16 : 8) || !aligned(LSE, 4)) return PULSAR_ERR_ALIGNMENT;
    int32_t rc = check_device();
    if (rc != PULSAR_OK) return rc;
    const int64_t blocks = (rows * (d >> 2) + 255) / 256;
    if (blocks > 0x7fffffffll) return PULSAR_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (out_is_f32)
        lse_merge_table_kernel<true><<<static_cast<unsigned>(blocks), 256, 0, st>>>(t, n_parts, rows_total, row_begin, rows,
                                                                                   d, O, LSE);
    else
        lse_merge_table_kernel<false><<<static_cast<unsigned>(blocks), 256, 0, st>>>(t, n_parts, rows_total, row_begin,
                                                                                    rows, d, O, LSE);
    PULSAR_CUDA_OK(cudaGetLastError());
    count_launch();
    return PULSAR_OK;
}
