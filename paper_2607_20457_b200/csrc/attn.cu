// Phase-1 prefix-block attention and Phase-2 split-KV attention (Eq. 1 over Eq. 4; Section 3.2).
//
// One FlashAttention-form kernel serves both phases.  A CTA owns a tile of 128 query rows and
// walks a list of 128-key tiles: S = Q K^T and O += P V run on the tensor cores (tcgen05.mma,
// accumulators in TMEM), operands are staged by TMA into 128-byte-swizzled shared memory, the
// softmax runs one thread per query row straight out of TMEM, and the probabilities go back to
// TMEM as the bf16 A operand of the PV product.
//
//   Phase 1: rows = 128 consecutive tokens of one block and one query head.  Key tiles: first
//            the gathered prefix rows [0, P_i) (fully visible, last tile possibly partial), then
//            the block's own rows up to the diagonal tile (causal mask on that tile only).
//   Phase 2: rows = (128/g tokens) x (the g query heads of one KV head); key tiles = one
//            contiguous part of the retained KV, no mask; output is the fp32 partial (A_j, l_j)
//            or, with a single part, the final bf16 result.
#include <cuda.h>

#include "common.cuh"

namespace pulsar {

int32_t launch_lse_merge(const float* part_O, const float* part_LSE, int32_t n_parts, int64_t rows, int32_t d,
                         uint16_t* O, float* LSE, cudaStream_t stream);

namespace {

constexpr int kTileM = 128;   // query rows per CTA
constexpr int kTileN = 128;   // keys per tile
constexpr int kPanelBytes = kTileN * 128;   // one 64-column panel of a 128-row bf16 tile (128-byte lines)

enum : int { kModePhase1 = 0, kModePhase2 = 1 };

struct AttnArgs {
    int mode;
    int n_tokens;          // L (phase 1) or nq (phase 2): tokens that exist, for the store guard
    int Hq, g, pack;       // query heads, heads per KV head, rows per token in a tile (1 or g)
    int block_size;        // phase 1: tokens per block
    int tiles_per_block;   // phase 1: ceil(block_size / 128)
    int prefix_total;      // phase 1: rows in the gathered prefix buffers
    const int32_t* prefix_len;
    int split_len;         // phase 2: keys per KV part
    float scale_log2;      // softmax scale * log2(e)
    uint16_t* O;           // bf16 [tokens, Hq, d]   (final output mode)
    float* LSE;            // f32  [tokens, Hq] or null
    float* part_O;         // f32  [parts, tokens, Hq, d] (partial output mode) or null
    float* part_LSE;       // f32  [parts, tokens, Hq]
    int32_t* status;
};

// ---------------------------------------------------------------------------------------------
// Gather of the prefix rows: Kp[j] = K[prefix_idx[j]], Vp[j] = V[prefix_idx[j]] for j < total.
// One CTA per prefix row; also checks that the row lies before the first block that uses it.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
gather_prefix_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V, const int32_t* __restrict__ prefix_idx,
                     const int32_t* __restrict__ prefix_len, int n_blocks, int block_size, int64_t L,
                     int row_vecs, uint4* __restrict__ Kp, uint4* __restrict__ Vp, int32_t* status) {
    const int j = blockIdx.x;
    __shared__ int s_src;
    if (threadIdx.x == 0) {
        int64_t limit = L;
        for (int i = 0; i < n_blocks; ++i)
            if (prefix_len[i] > j) { limit = static_cast<int64_t>(i) * block_size; break; }
        int src = prefix_idx[j];
        if (src < 0 || src >= limit) {
            report(status, PULSAR_DEV_BAD_PREFIX);
            src = 0;
        }
        s_src = src;
    }
    __syncthreads();
    const size_t src = static_cast<size_t>(s_src) * row_vecs, dst = static_cast<size_t>(j) * row_vecs;
    for (int v = threadIdx.x; v < row_vecs; v += blockDim.x) {
        Kp[dst + v] = K[src + v];
        Vp[dst + v] = V[src + v];
    }
}

// ---------------------------------------------------------------------------------------------
// Attention kernel
// ---------------------------------------------------------------------------------------------
template <int D>
struct SmemLayout {
    static constexpr int kPanels = D / 64;
    static constexpr int kTileBytes = kPanels * kPanelBytes;
    static constexpr int kQ = 0;
    static constexpr int kK = kTileBytes;
    static constexpr int kV = 2 * kTileBytes;
    static constexpr int kBars = 3 * kTileBytes;      // 4 mbarriers
    static constexpr int kTmemPtr = kBars + 4 * 8;
    static constexpr int kAbort = kTmemPtr + 4;
    static constexpr int kTotal = kAbort + 4;
    static constexpr int kDynBytes = kTotal + 1024;   // room to align the base to 1024 bytes
};

struct KvTile {
    int from_prefix;   // 1: gathered prefix buffer, 0: K/V themselves
    int row0;          // first key row of the tile in that tensor
    int valid;         // keys of the tile that exist for this work item (<= 128)
    int causal_base;   // >= 0: key c is visible to row r iff causal_base + c <= r_in_block; < 0: no causal mask
};

template <int D>
__global__ void __launch_bounds__(128)
attn_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
            const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmKp,
            const __grid_constant__ CUtensorMap tmVp, const AttnArgs a) {
    using SL = SmemLayout<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem + SL::kQ;
    uint8_t* sK = smem + SL::kK;
    uint8_t* sV = smem + SL::kV;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SL::kBars);
    uint64_t* bar_q = bars + 0;
    uint64_t* bar_kv = bars + 1;
    uint64_t* bar_s = bars + 2;
    uint64_t* bar_o = bars + 3;
    uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(smem + SL::kTmemPtr);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + SL::kAbort);

    const int tid = threadIdx.x, warp = tid >> 5;

    // ---- work item ---------------------------------------------------------------------
    int token0, head0, kvh, part = 0;
    int n_pref_tiles = 0, pref_len = 0, n_main_tiles, main_row0, main_len, row0_in_block = 0;
    if (a.mode == kModePhase1) {
        const int blk = blockIdx.x / a.tiles_per_block, qt = blockIdx.x - blk * a.tiles_per_block;
        row0_in_block = qt * kTileM;
        token0 = blk * a.block_size + row0_in_block;
        head0 = blockIdx.y;
        kvh = head0 / a.g;
        pref_len = a.prefix_len[blk];
        if (pref_len < 0 || pref_len > a.prefix_total) {
            if (tid == 0) report(a.status, PULSAR_DEV_BAD_LENGTH);
            pref_len = max(0, min(pref_len, a.prefix_total));
        }
        n_pref_tiles = (pref_len + kTileN - 1) / kTileN;
        n_main_tiles = qt + 1;
        main_row0 = blk * a.block_size;
        main_len = a.block_size;
    } else {
        token0 = blockIdx.x * (kTileM / a.pack);
        kvh = blockIdx.y;
        head0 = kvh * a.g;
        part = blockIdx.z;
        main_row0 = part * a.split_len;
        main_len = a.split_len;
        n_main_tiles = (a.split_len + kTileN - 1) / kTileN;
    }
    const int n_tiles = n_pref_tiles + n_main_tiles;

    // ---- set-up --------------------------------------------------------------------------
    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar_q, 1);
        mbar_init(bar_kv, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_o, 1);
        mbar_fence_init();
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
    }
    if (warp == 0) {
        tmem_alloc(tmem_ptr, 256);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr;
    const uint32_t tS = tmem_base;              // S: columns [0,128); P (bf16 pairs) reuses [0,64)
    const uint32_t tO = tmem_base + 128;        // O: columns [128, 128+D)
    const uint32_t lane_sel = static_cast<uint32_t>(warp * 32) << 16;

    constexpr uint32_t kIdescQK = umma_idesc_bf16(kTileM, kTileN, false, false);
    constexpr uint32_t kIdescPV = umma_idesc_bf16(kTileM, D, false, true);

    if (tid == 0) {
        mbar_expect_tx(bar_q, SL::kTileBytes);
        for (int p = 0; p < SL::kPanels; ++p)
            tma_load_3d(sQ + p * kPanelBytes, &tmQ, bar_q, p * 64, head0, token0);
    }

    float m_run = -INFINITY, l_run = 0.f;
    const int my_row_in_block = row0_in_block + tid;    // phase 1 only
    bool ok = true;

    for (int t = 0; t < n_tiles; ++t) {
        // ---- which keys ----------------------------------------------------------------
        KvTile kt;
        if (t < n_pref_tiles) {
            kt.from_prefix = 1;
            kt.row0 = t * kTileN;
            kt.valid = min(kTileN, pref_len - kt.row0);
            kt.causal_base = -1;
        } else {
            const int j = t - n_pref_tiles;
            kt.from_prefix = 0;
            kt.row0 = main_row0 + j * kTileN;
            kt.valid = min(kTileN, main_len - j * kTileN);
            kt.causal_base = (a.mode == kModePhase1 && j == n_main_tiles - 1) ? j * kTileN : -1;
        }

        // ---- load K and V tiles ----------------------------------------------------------
        if (tid == 0 && ok) {
            mbar_expect_tx(bar_kv, 2 * SL::kTileBytes);
            const CUtensorMap* mk = kt.from_prefix ? &tmKp : &tmK;
            const CUtensorMap* mv = kt.from_prefix ? &tmVp : &tmV;
            for (int p = 0; p < SL::kPanels; ++p) {
                tma_load_2d(sK + p * kPanelBytes, mk, bar_kv, kvh * D + p * 64, kt.row0);
                tma_load_2d(sV + p * kPanelBytes, mv, bar_kv, kvh * D + p * 64, kt.row0);
            }
        }
        if (t == 0) ok = ok && mbar_wait(bar_q, 0, abort_flag, a.status);
        ok = ok && mbar_wait(bar_kv, t & 1, abort_flag, a.status);

        // ---- S = Q K^T --------------------------------------------------------------------
        if (tid == 0 && ok) {
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t off = (kk >> 2) * kPanelBytes + (kk & 3) * 32;
                const uint64_t da = umma_smem_desc_sw128(smem_u32(sQ) + off, 16, 1024);
                const uint64_t db = umma_smem_desc_sw128(smem_u32(sK) + off, 16, 1024);
                umma_ss(tS, da, db, kIdescQK, kk > 0 ? 1u : 0u);
            }
            umma_commit(bar_s);
        }
        ok = ok && mbar_wait(bar_s, t & 1, abort_flag, a.status);
        tc_fence_after();

        // ---- softmax on this thread's row -------------------------------------------------
        // visible key columns of the tile for this row: [0, n_vis)
        int n_vis = kt.valid;
        if (kt.causal_base >= 0) n_vis = min(n_vis, my_row_in_block - kt.causal_base + 1);

        float m_tile = -INFINITY;
#pragma unroll
        for (int c0 = 0; c0 < kTileN; c0 += 32) {
            uint32_t r[32];
            tmem_ld32(tS + lane_sel + c0, r);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < 32; ++c)
                if (c0 + c < n_vis) m_tile = fmaxf(m_tile, __uint_as_float(r[c]));
        }
        const float m_new = fmaxf(m_run, m_tile * a.scale_log2);
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
        const float alpha = ex2(m_run - m_use);          // 0 on the first tile (m_run = -inf)
        float l_tile = 0.f;
#pragma unroll
        for (int c0 = 0; c0 < kTileN; c0 += 32) {
            uint32_t r[32];
            tmem_ld32(tS + lane_sel + c0, r);
            tmem_wait_ld();
            uint32_t pk[16];
#pragma unroll
            for (int c = 0; c < 32; c += 2) {
                float p0 = (c0 + c < n_vis) ? ex2(fmaf(__uint_as_float(r[c]), a.scale_log2, -m_use)) : 0.f;
                float p1 = (c0 + c + 1 < n_vis) ? ex2(fmaf(__uint_as_float(r[c + 1]), a.scale_log2, -m_use)) : 0.f;
                l_tile += p0 + p1;
                pk[c >> 1] = pack_bf16x2(p0, p1);
            }
            tmem_st16(tS + lane_sel + (c0 >> 1), pk);     // P column c/2 holds keys c, c+1
        }
        l_run = l_run * alpha + l_tile;
        m_run = m_new;

        // ---- rescale the running output ------------------------------------------------------
        if (t > 0) {
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tO + lane_sel + c0, r);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 32; ++c) r[c] = __float_as_uint(__uint_as_float(r[c]) * alpha);
                tmem_st32(tO + lane_sel + c0, r);
            }
        }
        tmem_wait_st();
        tc_fence_before();
        __syncthreads();
        ok = ok && (*abort_flag == 0);

        // ---- O += P V -----------------------------------------------------------------------
        if (tid == 0 && ok) {
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < kTileN / 16; ++kk) {
                const uint64_t db = umma_smem_desc_sw128(smem_u32(sV) + kk * 2048, kPanelBytes, 1024);
                umma_ts(tO, tS + kk * 8, db, kIdescPV, (t > 0 || kk > 0) ? 1u : 0u);
            }
            umma_commit(bar_o);
        }
        ok = ok && mbar_wait(bar_o, t & 1, abort_flag, a.status);
        tc_fence_after();
        // After a failed wait the loop keeps its shape (barriers and warp-collective TMEM
        // accesses stay convergent) but issues no further copies or MMAs and stores nothing.
    }

    // ---- epilogue: normalise and store this thread's row ---------------------------------------
    {
        const int token = token0 + tid / a.pack;
        const int head = head0 + tid % a.pack;
        bool store = ok && token < a.n_tokens;
        if (a.mode == kModePhase1) store = store && my_row_in_block < a.block_size;
        const float inv_l = l_run > 0.f ? 1.f / l_run : 0.f;
        const float lse = (l_run > 0.f) ? (m_run + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
        const size_t row = static_cast<size_t>(token) * a.Hq + head;
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += 32) {
            uint32_t r[32];
            tmem_ld32(tO + lane_sel + c0, r);      // every thread of the warp takes part in the load
            tmem_wait_ld();
            if (!store) continue;
            if (a.part_O != nullptr) {
                float4* dst = reinterpret_cast<float4*>(
                    a.part_O + (static_cast<size_t>(part) * a.n_tokens * a.Hq + row) * D + c0);
#pragma unroll
                for (int c = 0; c < 32; c += 4)
                    dst[c >> 2] = make_float4(__uint_as_float(r[c]) * inv_l, __uint_as_float(r[c + 1]) * inv_l,
                                              __uint_as_float(r[c + 2]) * inv_l, __uint_as_float(r[c + 3]) * inv_l);
            } else {
                uint4* dst = reinterpret_cast<uint4*>(a.O + row * D + c0);
#pragma unroll
                for (int c = 0; c < 32; c += 8) {
                    uint4 v;
                    v.x = pack_bf16x2(__uint_as_float(r[c]) * inv_l, __uint_as_float(r[c + 1]) * inv_l);
                    v.y = pack_bf16x2(__uint_as_float(r[c + 2]) * inv_l, __uint_as_float(r[c + 3]) * inv_l);
                    v.z = pack_bf16x2(__uint_as_float(r[c + 4]) * inv_l, __uint_as_float(r[c + 5]) * inv_l);
                    v.w = pack_bf16x2(__uint_as_float(r[c + 6]) * inv_l, __uint_as_float(r[c + 7]) * inv_l);
                    dst[c >> 3] = v;
                }
            }
        }
        if (store) {
            if (a.part_O != nullptr) a.part_LSE[static_cast<size_t>(part) * a.n_tokens * a.Hq + row] = lse;
            else if (a.LSE != nullptr) a.LSE[row] = lse;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, 256);
}

// ---------------------------------------------------------------------------------------------
// Host side: tensor maps, planning, launches
// ---------------------------------------------------------------------------------------------
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// [rows, heads, d] bf16 viewed as (d, heads, rows); box = (64, box_heads, box_rows), 128-byte swizzle.
bool make_map_3d(CUtensorMap* m, const void* base, int64_t rows, int heads, int d, int box_heads, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(heads), static_cast<cuuint64_t>(rows)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(d) * 2, static_cast<cuuint64_t>(heads) * d * 2};
    cuuint32_t box[3] = {64, static_cast<cuuint32_t>(box_heads), static_cast<cuuint32_t>(box_rows)};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// [rows, width] bf16; box = (64, 128), 128-byte swizzle.
bool make_map_2d(CUtensorMap* m, const void* base, int64_t rows, int64_t width) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {static_cast<cuuint64_t>(width), static_cast<cuuint64_t>(rows)};
    cuuint64_t strides[1] = {static_cast<cuuint64_t>(width) * 2};
    cuuint32_t box[2] = {64, kTileN};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D>
int32_t launch_attn(const CUtensorMap& q, const CUtensorMap& k, const CUtensorMap& v, const CUtensorMap& kp,
                    const CUtensorMap& vp, const AttnArgs& a, dim3 grid, cudaStream_t stream) {
    constexpr int smem = SmemLayout<D>::kDynBytes;
    static bool configured = false;
    if (!configured) {
        PULSAR_CUDA_OK(cudaFuncSetAttribute(attn_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        configured = true;
    }
    attn_kernel<D><<<grid, 128, smem, stream>>>(q, k, v, kp, vp, a);
    PULSAR_CUDA_OK(cudaGetLastError());
    count_launch();
    return PULSAR_OK;
}

struct Phase1Plan {
    int n_blocks, tiles_per_block;
    size_t pref_rows, pref_bytes, total;
};

int32_t plan_phase1(int64_t L, int32_t Hq, int32_t Hkv, int32_t d, int32_t block_size, int32_t prefix_total,
                    Phase1Plan& p) {
    if (L <= 0 || Hq <= 0 || Hkv <= 0 || block_size <= 0 || prefix_total < 0) return PULSAR_ERR_INVALID_ARG;
    if ((d != 64 && d != 128) || Hq % Hkv != 0 || L % block_size != 0 || L >= (1ll << 31)) return PULSAR_ERR_SHAPE;
    if (L / block_size > 65535 || Hq > 65535) return PULSAR_ERR_SHAPE;
    p.n_blocks = static_cast<int>(L / block_size);
    p.tiles_per_block = (block_size + kTileM - 1) / kTileM;
    p.pref_rows = static_cast<size_t>(prefix_total > 0 ? prefix_total : 1);
    p.pref_bytes = round_up(p.pref_rows * Hkv * d * 2, 256);
    p.total = 2 * p.pref_bytes;
    return PULSAR_OK;
}

int32_t choose_splits(int32_t nq, int64_t L, int32_t Hq, int32_t Hkv) {
    const int g = Hq / Hkv;
    const int64_t row_tiles = (static_cast<int64_t>(nq) * g + kTileM - 1) / kTileM;
    const int64_t items = row_tiles * Hkv;
    const int64_t want = 2ll * sm_count();
    if (L % kTileN != 0) return 1;
    const int64_t kv_tiles = L / kTileN;
    int64_t best = 1;
    for (int64_t j = 1; j <= kv_tiles && j <= 1024; ++j) {
        if (kv_tiles % j != 0) continue;
        best = j;
        if (items * j >= want) break;
    }
    return static_cast<int32_t>(best);
}

}  // namespace
}  // namespace pulsar

using namespace pulsar;

// =============================================================================================
// Phase 1
// =============================================================================================
extern "C" size_t pulsar_phase1_workspace_bytes(int64_t L, int32_t Hq, int32_t Hkv, int32_t d, int32_t block_size,
                                                int32_t prefix_total) {
    Phase1Plan p;
    if (plan_phase1(L, Hq, Hkv, d, block_size, prefix_total, p) != PULSAR_OK) return 0;
    return p.total;
}

extern "C" int32_t pulsar_phase1_attn(const uint16_t* Q, const uint16_t* K, const uint16_t* V, int64_t L, int32_t Hq,
                                      int32_t Hkv, int32_t d, int32_t block_size, const int32_t* prefix_idx,
                                      const int32_t* prefix_len, int32_t prefix_total, float softmax_scale,
                                      uint16_t* O, float* LSE, uint16_t* K_ret, uint16_t* V_ret, void* workspace,
                                      size_t workspace_bytes, int32_t* device_status, void* stream_) {
    Phase1Plan p;
    int32_t rc = plan_phase1(L, Hq, Hkv, d, block_size, prefix_total, p);
    if (rc != PULSAR_OK) return rc;
    if (!Q || !K || !V || !O || !prefix_len || !workspace || (prefix_total > 0 && !prefix_idx))
        return PULSAR_ERR_INVALID_ARG;
    if ((K_ret == nullptr) != (V_ret == nullptr)) return PULSAR_ERR_INVALID_ARG;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) || !aligned(prefix_len, 4) ||
        !aligned(prefix_idx, 4) || (LSE && !aligned(LSE, 4)) || (K_ret && !aligned(K_ret, 16)) ||
        (V_ret && !aligned(V_ret, 16)) || !aligned(workspace, 256))
        return PULSAR_ERR_ALIGNMENT;
    if (workspace_bytes < p.total) return PULSAR_ERR_WORKSPACE;
    rc = check_device();
    if (rc != PULSAR_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    uint16_t* Kp = static_cast<uint16_t*>(workspace);
    uint16_t* Vp = reinterpret_cast<uint16_t*>(static_cast<char*>(workspace) + p.pref_bytes);

    CUtensorMap tmQ, tmK, tmV, tmKp, tmVp;
    if (!make_map_3d(&tmQ, Q, L, Hq, d, 1, kTileM) || !make_map_2d(&tmK, K, L, static_cast<int64_t>(Hkv) * d) ||
        !make_map_2d(&tmV, V, L, static_cast<int64_t>(Hkv) * d) ||
        !make_map_2d(&tmKp, Kp, static_cast<int64_t>(p.pref_rows), static_cast<int64_t>(Hkv) * d) ||
        !make_map_2d(&tmVp, Vp, static_cast<int64_t>(p.pref_rows), static_cast<int64_t>(Hkv) * d))
        return PULSAR_ERR_CUDA;

    if (prefix_total > 0) {
        gather_prefix_kernel<<<prefix_total, 128, 0, stream>>>(
            reinterpret_cast<const uint4*>(K), reinterpret_cast<const uint4*>(V), prefix_idx, prefix_len, p.n_blocks,
            block_size, L, Hkv * d * 2 / 16, reinterpret_cast<uint4*>(Kp), reinterpret_cast<uint4*>(Vp),
            device_status);
        PULSAR_CUDA_OK(cudaGetLastError());
        count_launch();
    }

    AttnArgs a{};
    a.mode = kModePhase1;
    a.n_tokens = static_cast<int>(L);
    a.Hq = Hq;
    a.g = Hq / Hkv;
    a.pack = 1;
    a.block_size = block_size;
    a.tiles_per_block = p.tiles_per_block;
    a.prefix_total = prefix_total;
    a.prefix_len = prefix_len;
    a.scale_log2 = (softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf(static_cast<float>(d))) * 1.4426950408889634f;
    a.O = O;
    a.LSE = LSE;
    a.status = device_status;
    dim3 grid(static_cast<unsigned>(p.tiles_per_block) * p.n_blocks, Hq, 1);
    rc = d == 128 ? launch_attn<128>(tmQ, tmK, tmV, tmKp, tmVp, a, grid, stream)
                  : launch_attn<64>(tmQ, tmK, tmV, tmKp, tmVp, a, grid, stream);
    if (rc != PULSAR_OK) return rc;

    if (K_ret) {
        const size_t bytes = static_cast<size_t>(L) * Hkv * d * 2;
        PULSAR_CUDA_OK(cudaMemcpyAsync(K_ret, K, bytes, cudaMemcpyDeviceToDevice, stream));
        PULSAR_CUDA_OK(cudaMemcpyAsync(V_ret, V, bytes, cudaMemcpyDeviceToDevice, stream));
    }
    return PULSAR_OK;
}

// =============================================================================================
// Phase 2
// =============================================================================================
namespace {
int32_t plan_phase2(int32_t nq, int32_t B, int32_t block_size, int32_t Hq, int32_t Hkv, int32_t d, int32_t& n_splits,
                    size_t& part_o_bytes, size_t& part_l_bytes) {
    if (nq <= 0 || B <= 0 || block_size <= 0 || Hq <= 0 || Hkv <= 0 || n_splits < 0) return PULSAR_ERR_INVALID_ARG;
    if ((d != 64 && d != 128) || Hq % Hkv != 0) return PULSAR_ERR_SHAPE;
    const int g = Hq / Hkv;
    if (g != 1 && g != 2 && g != 4 && g != 8 && g != 16) return PULSAR_ERR_SHAPE;
    const int64_t L = static_cast<int64_t>(B) * block_size;
    if (L >= (1ll << 31) || Hkv > 65535) return PULSAR_ERR_SHAPE;
    if (n_splits == 0) n_splits = choose_splits(nq, L, Hq, Hkv);
    if (L % n_splits != 0 || n_splits > 65535) return PULSAR_ERR_SHAPE;
    part_o_bytes = round_up(static_cast<size_t>(n_splits) * nq * Hq * d * 4, 256);
    part_l_bytes = round_up(static_cast<size_t>(n_splits) * nq * Hq * 4, 256);
    return PULSAR_OK;
}
}  // namespace

extern "C" int32_t pulsar_phase2_choose_splits(int32_t nq, int32_t B, int32_t block_size, int32_t Hq, int32_t Hkv,
                                               int32_t d) {
    int32_t n = 0;
    size_t a, b;
    if (plan_phase2(nq, B, block_size, Hq, Hkv, d, n, a, b) != PULSAR_OK) return 0;
    return n;
}

extern "C" size_t pulsar_phase2_workspace_bytes(int32_t nq, int32_t B, int32_t block_size, int32_t Hq, int32_t Hkv,
                                                int32_t d, int32_t n_splits) {
    size_t a, b;
    if (plan_phase2(nq, B, block_size, Hq, Hkv, d, n_splits, a, b) != PULSAR_OK) return 0;
    return n_splits == 1 ? 256 : a + b;
}

extern "C" int32_t pulsar_phase2_attn(const uint16_t* Qq, int32_t nq, const uint16_t* Kb, const uint16_t* Vb,
                                      int32_t B, int32_t block_size, int32_t Hq, int32_t Hkv, int32_t d,
                                      float softmax_scale, int32_t n_splits, uint16_t* O, float* LSE, float* part_O,
                                      float* part_LSE, void* workspace, size_t workspace_bytes,
                                      int32_t* device_status, void* stream_) {
    size_t po_bytes, pl_bytes;
    const bool user_parts = part_O != nullptr;
    if ((part_O == nullptr) != (part_LSE == nullptr)) return PULSAR_ERR_INVALID_ARG;
    if (user_parts && n_splits <= 0) return PULSAR_ERR_INVALID_ARG;
    int32_t rc = plan_phase2(nq, B, block_size, Hq, Hkv, d, n_splits, po_bytes, pl_bytes);
    if (rc != PULSAR_OK) return rc;
    if (!Qq || !Kb || !Vb || !O) return PULSAR_ERR_INVALID_ARG;
    if (!aligned(Qq, 16) || !aligned(Kb, 16) || !aligned(Vb, 16) || !aligned(O, 16) || (LSE && !aligned(LSE, 4)) ||
        (part_O && !aligned(part_O, 16)) || (part_LSE && !aligned(part_LSE, 4)) ||
        (workspace && !aligned(workspace, 256)))
        return PULSAR_ERR_ALIGNMENT;
    const bool need_ws = n_splits > 1 && !user_parts;
    if (need_ws && (!workspace || workspace_bytes < po_bytes + pl_bytes)) return PULSAR_ERR_WORKSPACE;
    rc = check_device();
    if (rc != PULSAR_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    const int64_t L = static_cast<int64_t>(B) * block_size;
    const int g = Hq / Hkv;
    CUtensorMap tmQ, tmK, tmV;
    if (!make_map_3d(&tmQ, Qq, nq, Hq, d, g, kTileM / g) || !make_map_2d(&tmK, Kb, L, static_cast<int64_t>(Hkv) * d) ||
        !make_map_2d(&tmV, Vb, L, static_cast<int64_t>(Hkv) * d))
        return PULSAR_ERR_CUDA;

    const bool partial_out = n_splits > 1 || user_parts;
    float* pO = user_parts ? part_O : (need_ws ? static_cast<float*>(workspace) : nullptr);
    float* pL = user_parts ? part_LSE
                           : (need_ws ? reinterpret_cast<float*>(static_cast<char*>(workspace) + po_bytes) : nullptr);

    AttnArgs a{};
    a.mode = kModePhase2;
    a.n_tokens = nq;
    a.Hq = Hq;
    a.g = g;
    a.pack = g;
    a.split_len = static_cast<int>(L / n_splits);
    a.scale_log2 = (softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf(static_cast<float>(d))) * 1.4426950408889634f;
    a.O = O;
    a.LSE = LSE;
    a.part_O = partial_out ? pO : nullptr;
    a.part_LSE = partial_out ? pL : nullptr;
    a.status = device_status;
    const int tokens_per_tile = kTileM / g;
    dim3 grid((nq + tokens_per_tile - 1) / tokens_per_tile, Hkv, n_splits);
    rc = d == 128 ? launch_attn<128>(tmQ, tmK, tmV, tmK, tmV, a, grid, stream)
                  : launch_attn<64>(tmQ, tmK, tmV, tmK, tmV, a, grid, stream);
    if (rc != PULSAR_OK) return rc;
    if (partial_out)
        return launch_lse_merge(pO, pL, n_splits, static_cast<int64_t>(nq) * Hq, d, O, LSE, stream);
    return PULSAR_OK;
}
