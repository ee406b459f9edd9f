// Max-IDF summary selection (Section 3.1, Eq. 2-4; Algorithm 1 lines 3 and 6).
//
// Four launches on one stream, no host synchronisation:
//   presence_kernel   one CTA per block: a V-bit presence set of the block's token ids, built
//                     with shared-memory atomicOr and written to the workspace
//   df_idf_kernel     one thread per vocabulary entry: df(t) = number of blocks whose set holds
//                     t, IDF(t) = ln(B / max(df, 1))   (Eq. 3)
//   chunk_level_kernel one warp per chunk: the minimum df of its tokens (the chunk with the largest
//                     IDF is the one with the smallest df, Eq. 2)
//   topk_kernel       one CTA per block: a counting select of the k best chunks with ties to the
//                     lower index, then the block's part of the prefix list (Eq. 4)
// Ranking uses the integer df only, so the selection is exact.
//
// pulsar_chunk_select runs the same first two launches, then chunk_score_kernel (a float64 score
// per chunk under TF-IDF, BM25, the type-token ratio or Max-IDF, Appendix C Eq. 6-9) and
// topk_score_kernel (rank by score, ties to the lower index).
#include <cmath>
#include <mutex>

#include <math_constants.h>

#include "common.cuh"

namespace pulsar {
namespace {

constexpr int kPresenceThreads = 1024;
constexpr int kTopkThreads = 256;
constexpr size_t kMaxDynSmem = 227 * 1024;

__global__ void __launch_bounds__(kPresenceThreads)
presence_kernel(const uint32_t* __restrict__ ids, int64_t L, int block_size, int vocab_size, int words,
                uint32_t* __restrict__ bitmaps, int32_t* status) {
    extern __shared__ uint32_t bits[];
    grid_launch_dependents();          // the next launch of the chain may be placed; it waits for this grid itself
    const int b = blockIdx.x;
    for (int w = threadIdx.x; w < words; w += blockDim.x) bits[w] = 0u;
    __syncthreads();
    const uint32_t* blk = ids + static_cast<size_t>(b) * block_size;
    const int len = static_cast<int>(min(static_cast<int64_t>(block_size), L - static_cast<int64_t>(b) * block_size));
    for (int i = threadIdx.x; i < len; i += blockDim.x) {
        const uint32_t t = blk[i];
        if (t < static_cast<uint32_t>(vocab_size)) atomicOr(&bits[t >> 5], 1u << (t & 31));
        else report(status, PULSAR_DEV_BAD_TOKEN);
    }
    __syncthreads();
    uint32_t* out = bitmaps + static_cast<size_t>(b) * words;
    for (int w = threadIdx.x; w < words; w += blockDim.x) out[w] = bits[w];
}

__global__ void df_idf_kernel(const uint32_t* __restrict__ bitmaps, int n_blocks, int words, int vocab_size,
                              uint16_t* __restrict__ df_table, uint32_t* __restrict__ df_out,
                              float* __restrict__ idf_out) {
    grid_launch_dependents();
    grid_dependency_wait();            // the presence sets are complete
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= vocab_size) return;
    const int w = t >> 5, bit = t & 31;
    uint32_t df = 0;
    for (int b = 0; b < n_blocks; ++b) df += (bitmaps[static_cast<size_t>(b) * words + w] >> bit) & 1u;
    df_table[t] = static_cast<uint16_t>(df);
    if (df_out) df_out[t] = df;
    if (idf_out) idf_out[t] = logf(static_cast<float>(n_blocks) / static_cast<float>(df > 0 ? df : 1));
}

// Exclusive block-wide prefix sum of one int per thread; returns the thread's offset and the
// block total through `total`.  warp_sums: kTopkThreads/32 ints of shared scratch.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    int base = 0;
    total = 0;
    for (int i = 0; i < kTopkThreads / 32; ++i) {
        int s = warp_sums[i];
        if (i < warp) base += s;
        total += s;
    }
    __syncthreads();
    return base + incl - v;
}

// level[b*C + c] = min over the chunk's tokens of df.  Slot c of block b covers the tokens
// [b*block_size + c*chunk, +chunk) that lie inside the block and the sequence: the last chunk of
// a block may be shorter, and a slot past the end of a short last block holds no chunk at all.
// Ranks: a chunk whose ids all lie outside the vocabulary gets `worst` (after every real df), a
// slot without a chunk worst + 1 (never selected).
__global__ void __launch_bounds__(256)
chunk_level_kernel(const uint32_t* __restrict__ ids, const uint16_t* __restrict__ df_table, int64_t L,
                   int block_size, int chunks_per_block, int n_slots_total, int chunk, int vocab_size, int worst,
                   uint16_t* __restrict__ level) {
    grid_launch_dependents();
    grid_dependency_wait();            // the df table is complete
    const int lane = threadIdx.x & 31;
    const int slot = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (slot >= n_slots_total) return;
    const int b = slot / chunks_per_block, c = slot - b * chunks_per_block;
    const int64_t lo = static_cast<int64_t>(b) * block_size;
    const int64_t block_end = min(lo + block_size, L);
    const int64_t start = lo + static_cast<int64_t>(c) * chunk;
    const int len = static_cast<int>(max(static_cast<int64_t>(0), min(static_cast<int64_t>(chunk), block_end - start)));
    int mn = len > 0 ? worst : worst + 1;
    for (int p = lane; p < len; p += 32) {
        const uint32_t t = ids[start + p];
        if (t < static_cast<uint32_t>(vocab_size)) mn = min(mn, static_cast<int>(df_table[t]));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mn = min(mn, __shfl_xor_sync(0xffffffffu, mn, o));
    if (lane == 0) level[slot] = static_cast<uint16_t>(mn);
}

// Where a block's part of the prefix list goes and how long it is when lengths do not divide.
struct PrefixGeometry {
    int k_b;          // chunks this block contributes: min(k, chunks it has)
    int sink_eff;     // min(sink, tokens of block 0)
    int tail;         // tokens of the last chunk slot of a full block (= chunk when chunk divides block_size)
    int cap;          // entries of prefix_idx: sink + (n_blocks - 1) * k * chunk
};

__device__ __forceinline__ PrefixGeometry prefix_geometry(int b, int n_blocks, int64_t L, int block_size, int chunk,
                                                          int k, int sink) {
    PrefixGeometry g;
    const int64_t lo = static_cast<int64_t>(b) * block_size;
    const int len_b = static_cast<int>(min(static_cast<int64_t>(block_size), L - lo));
    const int chunks_b = (len_b + chunk - 1) / chunk;
    g.k_b = min(k, chunks_b);
    g.sink_eff = static_cast<int>(min(static_cast<int64_t>(sink), min(static_cast<int64_t>(block_size), L)));
    const int C = (block_size + chunk - 1) / chunk;
    g.tail = block_size - (C - 1) * chunk;
    g.cap = sink + (n_blocks - 1) * k * chunk;
    return g;
}

// Block b's part of the prefix list (Eq. 4): its chosen chunks (ascending, in shared memory) as
// global token positions starting at entry `offset`, the sink entries (written by block 0), the
// unused entries at the end (-1, written by the last block) and prefix_len[b] = offset (0 for
// block 0).  Only the last chosen chunk can be a short one (the last slot of the block), so the
// block's entries are the leading ones of k_b * chunk: those whose position lies inside the block.
__device__ __forceinline__ void write_block_prefix(int b, int n_blocks, int block_size, int chunk, int k,
                                                   const PrefixGeometry& g, int offset, const int* chosen,
                                                   int32_t* __restrict__ sel_chunks, int32_t* __restrict__ prefix_idx,
                                                   int32_t* __restrict__ prefix_len) {
    for (int j = g.k_b + threadIdx.x; j < k; j += blockDim.x) sel_chunks[static_cast<size_t>(b) * k + j] = -1;
    if (b < n_blocks - 1) {
        int32_t* dst = prefix_idx + offset;
        const int n = g.k_b * chunk;
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            const int j = i / chunk, p = i - j * chunk;
            const int pos = chosen[j] * chunk + p;
            if (pos < block_size) dst[i] = b * block_size + pos;
        }
    } else {
        for (int i = offset + threadIdx.x; i < g.cap; i += blockDim.x) prefix_idx[i] = -1;
    }
    if (b == 0)
        for (int i = threadIdx.x; i < g.sink_eff; i += blockDim.x) prefix_idx[i] = i;
    if (threadIdx.x == 0) prefix_len[b] = b == 0 ? 0 : offset;
}

// Entry of prefix_idx at which block b's summary starts: the sink plus the tokens of the
// summaries of blocks 0..b-1.  Those blocks are full ones; each contributes k chunks of `chunk`
// tokens, except that a block which selected its last chunk slot contributes only that slot's
// `tail` tokens for it.  The last slot (index C-1) is selected iff fewer than k of the other slots
// rank at or before it, i.e. have a level <= its own (they all have a lower index).  Only needed
// when chunk does not divide block_size; one warp per earlier block.
__device__ __forceinline__ int prefix_offset(int b, const uint16_t* __restrict__ level_all, int C, int chunk, int k,
                                             const PrefixGeometry& g, int* s_short) {
    if (g.tail == chunk || k == 0 || b == 0) return g.sink_eff + b * k * chunk;
    if (threadIdx.x == 0) *s_short = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    for (int j = warp; j < b; j += n_warps) {
        const uint16_t* lv = level_all + static_cast<size_t>(j) * C;
        const int last = lv[C - 1];
        int before = 0;
        for (int c = lane; c < C - 1; c += 32) before += (lv[c] <= last) ? 1 : 0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
        if (lane == 0 && before < k) atomicAdd(s_short, 1);
    }
    __syncthreads();
    return g.sink_eff + b * k * chunk - *s_short * (chunk - g.tail);
}

__global__ void __launch_bounds__(kTopkThreads)
topk_kernel(const uint16_t* __restrict__ level_all, int n_blocks, int64_t L, int block_size, int chunk, int k_all,
            int sink, int32_t* __restrict__ sel_chunks, int32_t* __restrict__ prefix_idx,
            int32_t* __restrict__ prefix_len) {
    extern __shared__ int smem[];
    const int C = (block_size + chunk - 1) / chunk;
    int* level = smem;                       // [C]   min df of the chunk
    int* hist = level + C;                   // [n_blocks + 3]
    int* chosen = hist + n_blocks + 3;       // [k]   selected chunk ids, ascending
    __shared__ int warp_sums[kTopkThreads / 32];
    __shared__ int s_threshold, s_need, s_short;

    const int b = blockIdx.x;
    const PrefixGeometry geo = prefix_geometry(b, n_blocks, L, block_size, chunk, k_all, sink);
    const int k = geo.k_b;                   // a short last block may have fewer than k_all chunks

    for (int i = threadIdx.x; i < n_blocks + 3; i += blockDim.x) hist[i] = 0;
    grid_dependency_wait();                  // the chunk levels are complete
    __syncthreads();
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        const int lv = level_all[static_cast<size_t>(b) * C + c];
        level[c] = lv;
        atomicAdd(&hist[lv], 1);
    }
    __syncthreads();

    // threshold level T: all chunks below T are taken, `need` more at T (lowest indices first)
    if (threadIdx.x == 0) {
        int cum = 0, T = 0;
        for (; T <= n_blocks + 1; ++T) {
            if (cum + hist[T] >= k) break;
            cum += hist[T];
        }
        s_threshold = T;
        s_need = k - cum;
    }
    __syncthreads();
    const int T = s_threshold, need = s_need;

    // ordered compaction over the chunks, a tile of blockDim chunks at a time
    int at_T_before = 0, taken_before = 0;
    for (int c0 = 0; c0 < C; c0 += kTopkThreads) {
        const int c = c0 + threadIdx.x;
        const int lv = c < C ? level[c] : n_blocks + 3;
        const int is_T = (lv == T) ? 1 : 0;
        int tot_T;
        const int rank_T = at_T_before + block_exclusive_scan(is_T, warp_sums, tot_T);
        const int take = (lv < T || (is_T && rank_T < need)) ? 1 : 0;
        int tot_take;
        const int pos = taken_before + block_exclusive_scan(take, warp_sums, tot_take);
        if (take && pos < k) {
            chosen[pos] = c;
            sel_chunks[static_cast<size_t>(b) * k_all + pos] = c;
        }
        at_T_before += tot_T;
        taken_before += tot_take;
    }
    __syncthreads();

    const int offset = prefix_offset(b, level_all, C, chunk, k_all, geo, &s_short);
    write_block_prefix(b, n_blocks, block_size, chunk, k_all, geo, offset, chosen, sel_chunks, prefix_idx, prefix_len);
}

// ---------------------------------------------------------------------------------------------
// Selection under the other chunk scores of Appendix C (Eq. 6-8) and Max-IDF as a score (Eq. 9).
// Scores are float64 and every operation is an explicitly rounded add, multiply or divide in
// the order the equations are written (positions left to right, types by first occurrence), so
// two chunks tie exactly when their scores are the same double.  The logarithms are a table over
// df = 0..B that the host fills (B + 1 values) and passes as a kernel parameter.  |C| is the number
// of tokens the chunk has (the last chunk of a block may be short), the mean chunk length of the
// BM25 normaliser is L over the number of chunks of the sequence.
// ---------------------------------------------------------------------------------------------
constexpr int kMaxScoreBlocks = 1024;
constexpr int kMaxScoreChunk = 1024;
constexpr int kMaxScoreChunksPerBlock = 4096;
struct ScoreTable {
    double by_df[kMaxScoreBlocks + 1];   // Eq. 5 (TF-IDF, Max-IDF) or the BM25 IDF of Eq. 7, per df
    double k1_plus_1, k1, b, one_minus_b, mean_len;   // BM25: D(C) = (1 - b) + b * (|C| / mean chunk length)
};

// One thread per chunk slot.  Slot c of block b covers the tokens [b*block_size + c*chunk, +chunk)
// that lie inside the block and the sequence (|C| = len); a slot without a chunk scores -inf.
__global__ void __launch_bounds__(128)
chunk_score_kernel(const uint32_t* __restrict__ ids, const uint16_t* __restrict__ df_table, int64_t L,
                   int block_size, int chunks_per_block, int n_slots_total, int chunk, int vocab_size, int mode,
                   const __grid_constant__ ScoreTable tab, double* __restrict__ score) {
    const int slot = blockIdx.x * blockDim.x + threadIdx.x;
    if (slot >= n_slots_total) return;
    const int b = slot / chunks_per_block, c = slot - b * chunks_per_block;
    const int64_t lo = static_cast<int64_t>(b) * block_size;
    const int64_t start = lo + static_cast<int64_t>(c) * chunk;
    const int len = static_cast<int>(max(static_cast<int64_t>(0),
                                         min(static_cast<int64_t>(chunk), min(lo + block_size, L) - start)));
    const uint32_t* tok = ids + start;
    const uint32_t V = static_cast<uint32_t>(vocab_size);
    double s = 0.0;
    if (len == 0) {
        s = -CUDART_INF;
    } else if (mode == PULSAR_SCORE_MAX_IDF) {
        s = -CUDART_INF;
        for (int p = 0; p < len; ++p) {
            const uint32_t t = tok[p];
            if (t < V) s = fmax(s, tab.by_df[df_table[t]]);
        }
    } else if (mode == PULSAR_SCORE_TF_IDF) {
        for (int p = 0; p < len; ++p) {
            const uint32_t t = tok[p];
            if (t < V) s = __dadd_rn(s, tab.by_df[df_table[t]]);
        }
        s = __ddiv_rn(s, static_cast<double>(len));
    } else {
        // D(C) = (1 - b) + b * (|C| / mean chunk length), then k1 * D(C): one rounding per operation
        const double k1_times_D =
            __dmul_rn(tab.k1, __dadd_rn(tab.one_minus_b, __dmul_rn(tab.b, __ddiv_rn(static_cast<double>(len), tab.mean_len))));
        int distinct = 0;
        for (int p = 0; p < len; ++p) {
            const uint32_t t = tok[p];
            bool first = true;
            for (int q = 0; q < p; ++q) first = first && (tok[q] != t);
            if (!first) continue;
            ++distinct;
            if (mode == PULSAR_SCORE_BM25 && t < V) {
                int tf = 0;
                for (int q = p; q < len; ++q) tf += (tok[q] == t) ? 1 : 0;
                const double tfd = static_cast<double>(tf);
                const double num = __dmul_rn(tab.by_df[df_table[t]], __dmul_rn(tfd, tab.k1_plus_1));
                s = __dadd_rn(s, __ddiv_rn(num, __dadd_rn(tfd, k1_times_D)));
            }
        }
        if (mode == PULSAR_SCORE_TYPE_TOKEN) s = __ddiv_rn(static_cast<double>(distinct), static_cast<double>(len));
    }
    score[slot] = s;
}

// One CTA per block: chunk c is taken when fewer than k chunks beat it (a larger score, or the
// same score at a lower index); the taken chunks are compacted in index order.
__global__ void __launch_bounds__(kTopkThreads)
topk_score_kernel(const double* __restrict__ score_all, int n_blocks, int64_t L, int block_size, int chunk, int k_all,
                  int sink, int32_t* __restrict__ sel_chunks, int32_t* __restrict__ prefix_idx,
                  int32_t* __restrict__ prefix_len) {
    extern __shared__ double smem_d[];
    const int C = (block_size + chunk - 1) / chunk;
    double* sc = smem_d;                                   // [C]
    int* chosen = reinterpret_cast<int*>(sc + C);          // [k]
    __shared__ int warp_sums[kTopkThreads / 32];
    __shared__ int s_short;
    const int b = blockIdx.x;
    const PrefixGeometry geo = prefix_geometry(b, n_blocks, L, block_size, chunk, k_all, sink);
    const int k = geo.k_b;                                 // a short last block may have fewer than k_all chunks
    const int64_t lo = static_cast<int64_t>(b) * block_size;
    const int Cb = static_cast<int>((min(static_cast<int64_t>(block_size), L - lo) + chunk - 1) / chunk);
    for (int c = threadIdx.x; c < C; c += blockDim.x) sc[c] = score_all[static_cast<size_t>(b) * C + c];
    __syncthreads();
    int taken_before = 0;
    for (int c0 = 0; c0 < C; c0 += kTopkThreads) {
        const int c = c0 + threadIdx.x;
        int take = 0;
        if (c < Cb) {
            const double mine = sc[c];
            int better = 0;
            for (int o = 0; o < Cb; ++o) {
                const double v = sc[o];
                better += (v > mine || (v == mine && o < c)) ? 1 : 0;
            }
            take = better < k ? 1 : 0;
        }
        int tot;
        const int pos = taken_before + block_exclusive_scan(take, warp_sums, tot);
        if (take && pos < k) {
            chosen[pos] = c;
            sel_chunks[static_cast<size_t>(b) * k_all + pos] = c;
        }
        taken_before += tot;
    }
    __syncthreads();
    // Entry of prefix_idx at which this block's summary starts: as in prefix_offset, with the scores
    // deciding whether an earlier (full) block selected its short last chunk -- it did iff fewer
    // than k of its other chunks, which all have a lower index, score at least as much.
    int offset = geo.sink_eff + b * k_all * chunk;
    if (geo.tail != chunk && k_all > 0 && b > 0) {
        if (threadIdx.x == 0) s_short = 0;
        __syncthreads();
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
        for (int j = warp; j < b; j += n_warps) {
            const double* sj = score_all + static_cast<size_t>(j) * C;
            const double last = sj[C - 1];
            int before = 0;
            for (int c = lane; c < C - 1; c += 32) before += (sj[c] >= last) ? 1 : 0;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
            if (lane == 0 && before < k_all) atomicAdd(&s_short, 1);
        }
        __syncthreads();
        offset -= s_short * (chunk - geo.tail);
    }
    write_block_prefix(b, n_blocks, block_size, chunk, k_all, geo, offset, chosen, sel_chunks, prefix_idx, prefix_len);
}

struct SelectPlan {
    int n_blocks, words, C;
    size_t bitmap_bytes, df_bytes, level_bytes, total;
    size_t presence_smem, topk_smem;
};

int32_t plan_select(int64_t L, int32_t vocab_size, int32_t block_size, int32_t chunk, int32_t k, int32_t sink,
                    SelectPlan& p) {
    if (L <= 0 || vocab_size <= 0 || block_size <= 0 || chunk <= 0 || k < 0 || sink < 0) return PULSAR_ERR_INVALID_ARG;
    if (L >= (1ll << 31)) return PULSAR_ERR_SHAPE;
    const int64_t B = (L + block_size - 1) / block_size;
    p.C = (block_size + chunk - 1) / chunk;
    // chunk levels are 16-bit: the real df values 0..B and the two ranks after them, B + 1 and B + 2
    if (B > 65533 || k > p.C || sink > block_size || p.C > 32768) return PULSAR_ERR_SHAPE;
    if (sink + (B - 1) * static_cast<int64_t>(k) * chunk >= (1ll << 31)) return PULSAR_ERR_SHAPE;
    p.n_blocks = static_cast<int>(B);
    p.words = (vocab_size + 31) / 32;
    p.presence_smem = static_cast<size_t>(p.words) * 4;
    p.topk_smem = (static_cast<size_t>(p.C) + p.n_blocks + 3 + k) * 4;
    if (p.presence_smem > kMaxDynSmem || p.topk_smem > kMaxDynSmem) return PULSAR_ERR_SHAPE;
    p.bitmap_bytes = round_up(static_cast<size_t>(p.n_blocks) * p.words * 4, 256);
    p.df_bytes = round_up(static_cast<size_t>(vocab_size) * 2, 256);
    p.level_bytes = round_up(static_cast<size_t>(p.n_blocks) * p.C * 2, 256);
    p.total = p.bitmap_bytes + p.df_bytes + p.level_bytes;
    return PULSAR_OK;
}

}  // namespace
}  // namespace pulsar

using namespace pulsar;

extern "C" size_t pulsar_maxidf_select_workspace_bytes(int64_t L, int32_t vocab_size, int32_t block_size,
                                                       int32_t chunk, int32_t k, int32_t sink) {
    SelectPlan p;
    if (plan_select(L, vocab_size, block_size, chunk, k, sink, p) != PULSAR_OK) return 0;
    return p.total;
}

extern "C" int32_t pulsar_maxidf_select(const uint32_t* token_ids, int64_t L, int32_t vocab_size,
                                        int32_t block_size, int32_t chunk, int32_t k, int32_t sink,
                                        int32_t* sel_chunks, int32_t* prefix_idx, int32_t* prefix_len,
                                        uint32_t* df_out, float* idf_out, void* workspace,
                                        size_t workspace_bytes, int32_t* device_status, void* stream_) {
    SelectPlan p;
    int32_t rc = plan_select(L, vocab_size, block_size, chunk, k, sink, p);
    if (rc != PULSAR_OK) return rc;
    if (!token_ids || !sel_chunks || !prefix_idx || !prefix_len || !workspace) return PULSAR_ERR_INVALID_ARG;
    if (!aligned(token_ids, 16) || !aligned(sel_chunks, 16) || !aligned(prefix_idx, 16) || !aligned(prefix_len, 16) ||
        (df_out && !aligned(df_out, 16)) || (idf_out && !aligned(idf_out, 16)) || !aligned(workspace, 256))
        return PULSAR_ERR_ALIGNMENT;
    if (workspace_bytes < p.total) return PULSAR_ERR_WORKSPACE;
    rc = check_device();
    if (rc != PULSAR_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    uint32_t* bitmaps = static_cast<uint32_t*>(workspace);
    uint16_t* df_table = reinterpret_cast<uint16_t*>(static_cast<char*>(workspace) + p.bitmap_bytes);
    uint16_t* level = reinterpret_cast<uint16_t*>(static_cast<char*>(workspace) + p.bitmap_bytes + p.df_bytes);

    if (p.presence_smem > 48 * 1024)
        PULSAR_CUDA_OK(cudaFuncSetAttribute(presence_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            static_cast<int>(p.presence_smem)));
    if (p.topk_smem > 48 * 1024)
        PULSAR_CUDA_OK(cudaFuncSetAttribute(topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            static_cast<int>(p.topk_smem)));

    presence_kernel<<<p.n_blocks, kPresenceThreads, p.presence_smem, stream>>>(
        token_ids, L, block_size, vocab_size, p.words, bitmaps, device_status);
    PULSAR_CUDA_OK(cudaGetLastError());
    count_launch();
    // The three launches that follow are programmatic dependents of the one before them: they are placed
    // while it runs and wait for it on the device, which takes the launch gaps out of the chain.
    PULSAR_CUDA_OK(launch_kernel(df_idf_kernel, dim3((vocab_size + 255) / 256), dim3(256), 0, stream, true, bitmaps,
                                 p.n_blocks, p.words, vocab_size, df_table, df_out, idf_out));
    count_launch();
    const int n_chunks_total = p.n_blocks * p.C;
    PULSAR_CUDA_OK(launch_kernel(chunk_level_kernel, dim3((n_chunks_total + 7) / 8), dim3(256), 0, stream, true, token_ids,
                                 df_table, L, block_size, p.C, n_chunks_total, chunk, vocab_size, p.n_blocks + 1, level));
    count_launch();
    PULSAR_CUDA_OK(launch_kernel(topk_kernel, dim3(p.n_blocks), dim3(kTopkThreads), p.topk_smem, stream, true, level,
                                 p.n_blocks, L, block_size, chunk, k, sink, sel_chunks, prefix_idx, prefix_len));
    count_launch();
    return PULSAR_OK;
}

// =============================================================================================
// Selection under a chosen chunk score
// =============================================================================================
namespace {
struct ScorePlan {
    SelectPlan base;
    size_t score_bytes, total, topk_smem;
};
int32_t plan_score(int64_t L, int32_t vocab_size, int32_t block_size, int32_t chunk, int32_t k, int32_t sink,
                   int32_t mode, ScorePlan& p) {
    if (mode < PULSAR_SCORE_MAX_IDF || mode > PULSAR_SCORE_TYPE_TOKEN) return PULSAR_ERR_INVALID_ARG;
    int32_t rc = plan_select(L, vocab_size, block_size, chunk, k, sink, p.base);
    if (rc != PULSAR_OK) return rc;
    if (p.base.n_blocks > kMaxScoreBlocks || chunk > kMaxScoreChunk || p.base.C > kMaxScoreChunksPerBlock)
        return PULSAR_ERR_SHAPE;
    p.score_bytes = round_up(static_cast<size_t>(p.base.n_blocks) * p.base.C * 8, 256);
    p.total = p.base.bitmap_bytes + p.base.df_bytes + p.score_bytes;
    p.topk_smem = static_cast<size_t>(p.base.C) * 8 + static_cast<size_t>(k) * 4;
    return PULSAR_OK;
}
}  // namespace

extern "C" size_t pulsar_chunk_select_workspace_bytes(int64_t L, int32_t vocab_size, int32_t block_size,
                                                      int32_t chunk, int32_t k, int32_t sink, int32_t score_mode) {
    ScorePlan p;
    if (plan_score(L, vocab_size, block_size, chunk, k, sink, score_mode, p) != PULSAR_OK) return 0;
    return p.total;
}

extern "C" int32_t pulsar_chunk_select(const uint32_t* token_ids, int64_t L, int32_t vocab_size, int32_t block_size,
                                       int32_t chunk, int32_t k, int32_t sink, int32_t score_mode,
                                       int32_t* sel_chunks, int32_t* prefix_idx, int32_t* prefix_len,
                                       double* score_out, void* workspace, size_t workspace_bytes,
                                       int32_t* device_status, void* stream_) {
    ScorePlan p;
    int32_t rc = plan_score(L, vocab_size, block_size, chunk, k, sink, score_mode, p);
    if (rc != PULSAR_OK) return rc;
    if (!token_ids || !sel_chunks || !prefix_idx || !prefix_len || !workspace) return PULSAR_ERR_INVALID_ARG;
    if (!aligned(token_ids, 16) || !aligned(sel_chunks, 16) || !aligned(prefix_idx, 16) || !aligned(prefix_len, 16) ||
        (score_out && !aligned(score_out, 16)) || !aligned(workspace, 256))
        return PULSAR_ERR_ALIGNMENT;
    if (workspace_bytes < p.total) return PULSAR_ERR_WORKSPACE;
    rc = check_device();
    if (rc != PULSAR_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const SelectPlan& b = p.base;

    uint32_t* bitmaps = static_cast<uint32_t*>(workspace);
    uint16_t* df_table = reinterpret_cast<uint16_t*>(static_cast<char*>(workspace) + b.bitmap_bytes);
    double* score = score_out ? score_out
                              : reinterpret_cast<double*>(static_cast<char*>(workspace) + b.bitmap_bytes + b.df_bytes);

    // The logarithms of Eq. 5 / Eq. 7 for every possible df, in float64 from the host's libm.
    ScoreTable tab;
    const double N = static_cast<double>(b.n_blocks);
    for (int f = 0; f <= b.n_blocks; ++f) {
        const double fd = static_cast<double>(f);
        tab.by_df[f] = score_mode == PULSAR_SCORE_BM25 ? std::log((N - fd + 0.5) / (fd + 0.5) + 1.0)
                                                       : std::log(N / static_cast<double>(f > 1 ? f : 1));
    }
    const double k1 = 1.2, bb = 0.75;
    // mean chunk length over the sequence: full blocks have C chunks, a short last block what it needs
    const int64_t last_len = L - static_cast<int64_t>(b.n_blocks - 1) * block_size;
    const int64_t n_chunks = static_cast<int64_t>(b.n_blocks - 1) * b.C + (last_len + chunk - 1) / chunk;
    tab.k1_plus_1 = k1 + 1.0;
    tab.k1 = k1;
    tab.b = bb;
    tab.one_minus_b = 1.0 - bb;
    tab.mean_len = static_cast<double>(L) / static_cast<double>(n_chunks);

    if (b.presence_smem > 48 * 1024)
        PULSAR_CUDA_OK(cudaFuncSetAttribute(presence_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            static_cast<int>(b.presence_smem)));
    presence_kernel<<<b.n_blocks, kPresenceThreads, b.presence_smem, stream>>>(token_ids, L, block_size, vocab_size,
                                                                               b.words, bitmaps, device_status);
    PULSAR_CUDA_OK(cudaGetLastError());
    count_launch();
    df_idf_kernel<<<(vocab_size + 255) / 256, 256, 0, stream>>>(bitmaps, b.n_blocks, b.words, vocab_size, df_table,
                                                                nullptr, nullptr);
    PULSAR_CUDA_OK(cudaGetLastError());
    count_launch();
    const int n_chunks_total = b.n_blocks * b.C;
    chunk_score_kernel<<<(n_chunks_total + 127) / 128, 128, 0, stream>>>(token_ids, df_table, L, block_size, b.C,
                                                                         n_chunks_total, chunk, vocab_size, score_mode,
                                                                         tab, score);
    PULSAR_CUDA_OK(cudaGetLastError());
    count_launch();
    topk_score_kernel<<<b.n_blocks, kTopkThreads, p.topk_smem, stream>>>(score, b.n_blocks, L, block_size, chunk, k,
                                                                         sink, sel_chunks, prefix_idx, prefix_len);
    PULSAR_CUDA_OK(cudaGetLastError());
    count_launch();
    return PULSAR_OK;
}

// =============================================================================================
// Selection without a caller workspace
// =============================================================================================
namespace {

// Scratch shared by every pulsar_maxidf_select_noalloc call on a device.  It is part of the
// library image: each GPU that loads the library holds these bytes until the process exits.
constexpr size_t kStaticScratchBytes = 4u << 20;
static __device__ __align__(256) unsigned char g_select_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of g_select_scratch on the current device.  In host code the symbol's name is
// only a stand-in; the address a kernel can use comes from cudaGetSymbolAddress, looked up once
// per device with that device current and remembered for the life of the process.  (A device
// reset, or a primary context torn down and created again, would leave the remembered address
// stale: the header tells callers not to use this entry point across one.)
int32_t static_scratch(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return PULSAR_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (g_scratch_ptr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_select_scratch) != cudaSuccess || p == nullptr) {
            (void)cudaGetLastError();
            return PULSAR_ERR_CUDA;
        }
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return PULSAR_OK;
}

}  // namespace

extern "C" size_t pulsar_maxidf_select_noalloc_max_scratch(void) { return kStaticScratchBytes; }

extern "C" int32_t pulsar_maxidf_select_noalloc(const uint32_t* token_ids, int64_t L, int32_t vocab_size,
                                                int32_t block_size, int32_t chunk, int32_t k, int32_t sink,
                                                int32_t* sel_chunks, int32_t* prefix_idx, int32_t* prefix_len,
                                                uint32_t* df_out, float* idf_out, int32_t* device_status,
                                                void* stream) {
    SelectPlan p;
    int32_t rc = plan_select(L, vocab_size, block_size, chunk, k, sink, p);
    if (rc != PULSAR_OK) return rc;
    if (p.total > kStaticScratchBytes) return PULSAR_ERR_WORKSPACE;      // problem too large for the built-in scratch
    rc = check_device();
    if (rc != PULSAR_OK) return rc;
    void* scratch = nullptr;
    rc = static_scratch(&scratch);
    if (rc != PULSAR_OK) return rc;
    // Same kernels, same order as pulsar_maxidf_select; every scratch region is fully written
    // before it is read, so nothing needs clearing between calls.
    return pulsar_maxidf_select(token_ids, L, vocab_size, block_size, chunk, k, sink, sel_chunks, prefix_idx,
                                prefix_len, df_out, idf_out, scratch, kStaticScratchBytes, device_status, stream);
}
