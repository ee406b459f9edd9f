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
//            or, with a single part, the final bf16 result.  With at most 32 such rows (decode)
//            the rows are replicated into the four lane quarters of the tile and each softmax
//            warp takes a quarter of the keys; the generation shard of Algorithm 1 l.11-16 is
//            one more part, causal by token.
//   Assembled inputs (Algorithm 1 l.8 as the paper runs it): sequences of any lengths packed back
//            to back, every token a query, plain causal attention inside each.
#include <cuda.h>

#include "common.cuh"

namespace pulsar {

// after_attention: the merge follows the attention launch that wrote the partials and may be
// scheduled while that launch drains (it waits for it before it reads).
int32_t launch_lse_merge(const float* part_O, const float* part_LSE, int32_t n_parts, int64_t rows, int32_t d,
                         uint16_t* O, float* LSE, cudaStream_t stream, bool after_attention = false);

namespace {

constexpr int kTileM = 128;   // query rows per CTA
constexpr int kTileN = 128;   // keys per tile
constexpr int kPanelBytes = kTileN * 128;   // one 64-column panel of a 128-row bf16 tile (128-byte lines)

enum : int { kModePhase1 = 0, kModePhase2 = 1, kModeVarlen = 2 };

// Sequence table of the variable-length causal mode (passed by value with the launch).
constexpr int kMaxVarlenSeqs = 64;
struct VarlenTable {
    int start[kMaxVarlenSeqs + 1];      // first row of sequence j; start[n] = total rows
    int pair_cum[kMaxVarlenSeqs + 1];   // tile pairs of the sequences n-1, n-2, ... j summed (scheduling order)
    int n_seq;
};

struct AttnArgs {
    int mode;
    int n_tokens;          // L (phase 1) or nq (phase 2): tokens that exist, for the store guard
    int Hq, g, pack;       // query heads, heads per KV head, rows per token in a tile (1 or g)
    int block_size;        // phase 1: tokens per block
    int tiles_per_block;   // phase 1: ceil(block_size / 128)
    int prefix_total;      // phase 1: rows in the gathered prefix buffers
    const int32_t* prefix_len;
    int split_len;         // phase 2: keys per KV part (the last part may be shorter)
    int kv_len;            // phase 2: context keys in total
    int n_ctx_parts;       // phase 2: parts of the context KV; part n_ctx_parts (if any) is the generation shard
    int gen_len;           // phase 2: rows of the generation shard that precede the new tokens
    int gen_total;         // phase 2: gen_len + new tokens (0 = no generation shard)
    int loader_waits;      // the launch before this one wrote rows the loader reads (the appended shard rows) and this
                           // launch was allowed to start beside it: the loader waits for it first
    int quad;              // phase 2, at most 32 query rows per KV head: the rows are replicated into the four
                           // lane quarters of the tile and each softmax warp takes one quarter of the keys
    int single;            // phase 2, one query tile per KV head (at most 128 rows): the tile's logits alternate
                           // between the two S buffers so that S of the next key tile is formed during the softmax
                           // of this one (set with quad as well)
    int Hkv;
    int pairs;             // phase 1: query-tile pairs per full block; phase 2: query-tile pairs per KV head
    int last_len;          // phase 1: tokens of the last block (block_size unless the sequence ends inside it)
    int pairs_last;        // phase 1: query-tile pairs of the last block
    int n_items;           // work items in total
    int n_blocks;          // phase 1
    int32_t* counter;      // work counter (zeroed before the launch): items are drawn in index order as CTAs
                           // become free; null = fixed round order
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
        int64_t limit = -1;                 // stays -1 when no block uses entry j (the list may be shorter than its buffer)
        for (int i = 0; i < n_blocks; ++i)
            if (prefix_len[i] > j) { limit = static_cast<int64_t>(i) * block_size; break; }
        int src = -1;
        if (limit >= 0) {
            src = prefix_idx[j];
            if (src < 0 || src >= limit) {
                report(status, PULSAR_DEV_BAD_PREFIX);
                src = 0;
            }
        }
        s_src = src;
    }
    __syncthreads();
    const size_t dst = static_cast<size_t>(j) * row_vecs;
    if (s_src < 0) {
        // An entry no block uses still shares a key tile with used ones: the attention kernel masks
        // its logits, but the PV product multiplies whatever the row holds by zero, and 0 * NaN
        // is NaN.  The workspace is the caller's and may hold anything, so the row is cleared.
        for (int v = threadIdx.x; v < row_vecs; v += blockDim.x) {
            Kp[dst + v] = make_uint4(0u, 0u, 0u, 0u);
            Vp[dst + v] = make_uint4(0u, 0u, 0u, 0u);
        }
        return;
    }
    const size_t src = static_cast<size_t>(s_src) * row_vecs;
    for (int v = threadIdx.x; v < row_vecs; v += blockDim.x) {
        Kp[dst + v] = K[src + v];
        Vp[dst + v] = V[src + v];
    }
}

// KV(q) of the new tokens appended to the generation shard: one launch for both tensors.  The
// attention launch that follows may start beside it; its loader waits for this grid before it
// reads the shard.
__global__ void __launch_bounds__(256)
append_kv_kernel(const uint4* __restrict__ Knew, const uint4* __restrict__ Vnew, uint4* __restrict__ Kdst,
                 uint4* __restrict__ Vdst, int vecs) {
    grid_launch_dependents();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < vecs) {
        Kdst[i] = Knew[i];
        Vdst[i] = Vnew[i];
    }
}

// KV discard (Section 3.1, Appendix F): of every assembled input only the last block_size rows -- the
// block's own keys and values -- are kept.  first[j] = first kept row of input j.
struct RetainTable {
    int first[kMaxVarlenSeqs];
};
__global__ void __launch_bounds__(128)
retain_block_kv_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V, const __grid_constant__ RetainTable tab,
                       int block_size, int row_vecs, uint4* __restrict__ Kret, uint4* __restrict__ Vret) {
    const int row = blockIdx.x;                              // retained row: input row / block_size, offset row % block_size
    const int j = row / block_size;
    const size_t src = static_cast<size_t>(tab.first[j] + (row - j * block_size)) * row_vecs;
    const size_t dst = static_cast<size_t>(row) * row_vecs;
    for (int v = threadIdx.x; v < row_vecs; v += blockDim.x) {
        Kret[dst + v] = K[src + v];
        Vret[dst + v] = V[src + v];
    }
}

// Row gather without the prefix check: Kout[j] = K[idx[j]], Vout[j] = V[idx[j]].  An index outside
// [0, rows_in) is reported and row 0 used.
__global__ void __launch_bounds__(128)
gather_rows_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V, const int32_t* __restrict__ idx,
                   int64_t rows_in, int row_vecs, uint4* __restrict__ Kout, uint4* __restrict__ Vout,
                   int32_t* status) {
    const int j = blockIdx.x;
    int src_row = idx[j];
    if (src_row < 0 || src_row >= rows_in) {
        if (threadIdx.x == 0) report(status, PULSAR_DEV_BAD_PREFIX);
        src_row = 0;
    }
    const size_t src = static_cast<size_t>(src_row) * row_vecs, dst = static_cast<size_t>(j) * row_vecs;
    for (int v = threadIdx.x; v < row_vecs; v += blockDim.x) {
        Kout[dst + v] = K[src + v];
        Vout[dst + v] = V[src + v];
    }
}

// What one GPU contributes to the prefix exchange: row j < sink is row j of its first local block
// (meaningful only on the GPU that holds logical block 0); row sink + (s*k + c)*chunk + p is token
// p of the c-th selected chunk of local block s (logical block block_ids[s]).
__global__ void __launch_bounds__(128)
pack_summary_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V, const int32_t* __restrict__ sel_chunks,
                    const int32_t* __restrict__ block_ids, int n_local, int n_blocks, int block_size, int chunk,
                    int k, int sink, int row_vecs, uint4* __restrict__ Kout, uint4* __restrict__ Vout,
                    int32_t* status) {
    const int j = blockIdx.x;
    int src_row;
    if (j < sink) {
        src_row = j;
    } else {
        const int t = j - sink, sigma = k * chunk;
        const int s = t / sigma, r = t - s * sigma;
        const int c = r / chunk, p = r - c * chunk;
        const int blk = block_ids[s];
        int ch = 0;
        if (blk < 0 || blk >= n_blocks) {
            if (threadIdx.x == 0) report(status, PULSAR_DEV_BAD_PREFIX);
        } else {
            ch = sel_chunks[static_cast<size_t>(blk) * k + c];
            if (ch < 0 || (ch + 1) * chunk > block_size) {
                if (threadIdx.x == 0) report(status, PULSAR_DEV_BAD_PREFIX);
                ch = 0;
            }
        }
        src_row = s * block_size + ch * chunk + p;
    }
    const size_t src = static_cast<size_t>(src_row) * row_vecs, dst = static_cast<size_t>(j) * row_vecs;
    for (int v = threadIdx.x; v < row_vecs; v += blockDim.x) {
        Kout[dst + v] = K[src + v];
        Vout[dst + v] = V[src + v];
    }
}

// ---------------------------------------------------------------------------------------------
// Attention kernel: persistent, warp-specialised.
//
//   warps 0-3   softmax of query tile 0 (one thread per query row, TMEM lane = row)
//   warps 4-7   softmax of query tile 1
//   warp  8     MMA issuer (one elected lane): S_s = Q_s K^T, O_s += P_s V
//   warp  9     TMA loader (one elected lane): Q tiles and the K/V ring
//
// A work item is two 128-row query tiles sharing one list of 128-key tiles.  The two tiles
// ping-pong on the tensor pipe: while the softmax warpgroup of one tile works on S, the pipe
// runs the other tile's PV and next S.  TMEM: S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512);
// P_s (bf16 pairs) overwrites the first 64 columns of S_s.  The running maximum is only moved
// when it grows by more than 2^8 (the stale maximum is used consistently for P, O and the row
// sum, so the result is unchanged); the rare rescale of O is done by the softmax warpgroup.
// P goes to the issuer in two halves of 64 keys (two barriers), so the first half of PV runs while
// the second half of the row is exponentiated.  The loader publishes the CTA's work items through
// a small shared-memory queue; all device waits are bounded (see mbar_wait).
// ---------------------------------------------------------------------------------------------
// Stages of the key/value ring (one K or V tile each).  For the decode-shaped launches, which stream K and V
// from HBM, 4 and 5 stages measure the same (93 / 99 us for 1 / 8 query tokens at the 128K key/value set), 3
// stages 120 / 126 us, and a sixth stage in the unused second query tile's memory 95 / 101 us: more loads in
// flight than the latency needs only add contention in the memory system.
constexpr int kStages = 5;
constexpr int kItemQueue = 4;     // work items the loader may publish ahead of the slowest consumer
constexpr int kAttnThreads = 384;             // warps 10 and 11 only take part in the register hand-back
constexpr int kMmaWarp = 8;
constexpr int kLoadWarp = 9;
constexpr float kRescaleThreshold = 8.0f;      // in log2 units
// Tuning knobs (overridable at build time with -D).  Measured on a 1000 W B200 running the 128K
// step back to back (power-capped, SM clock ~1.56 GHz): without the polynomial exponential 1060 TFLOP/s,
// with one pair in four 1032 -- under the power cap the variant that executes the fewest instructions
// wins, although the option shortens the per-tile latency in short runs.  (Forming the first half of P
// with the maximum in use while the tile maximum is computed alongside was a second such option: 1048,
// and 1020 with both; taken out of the source.)
#ifndef PULSAR_POLY_PAIRS
#define PULSAR_POLY_PAIRS 0
#endif
#ifndef PULSAR_EARLY_RELEASE
#define PULSAR_EARLY_RELEASE 1
#endif
// Hand a query tile's shared memory back to the loader when its last S product has been issued (the PV
// products that follow do not read Q), and the O accumulator back to the issuer as soon as the epilogue has
// read it into registers (before the rows are scaled and stored): both shorten the gap between work items.
constexpr bool kEarlyRelease = PULSAR_EARLY_RELEASE;
// Two more variants were built, measured at the 128K step and taken out again: the two softmax warps of a
// scheduler taking turns at a key tile's exponentials instead of interleaving them on the MUFU pipe (Phase 1
// 17.09 ms against 15.75 ms: one warp alone does not fill the pipe, two interleaved warps hide each other's
// latencies), and reading S from TMEM in two halves with the first half's maximum formed while the second
// arrives (0.6-1 % slower at the power limit).
constexpr int kPolyPairs128 = PULSAR_POLY_PAIRS;  // of every four column pairs, how many use the polynomial exp2 (d = 128)
// Head dimension 64 halves the tensor work per exponential, the GPU stays below its power limit there,
// and one polynomial pair in four is 3.6 % faster (32K shape with d = 64: 1.228 against 1.272 ms; two pairs
// in four: 1.309 ms).
#ifndef PULSAR_POLY_PAIRS_D64
#define PULSAR_POLY_PAIRS_D64 1
#endif
template <int D> constexpr int kPolyPairsFor = D == 64 ? PULSAR_POLY_PAIRS_D64 : kPolyPairs128;
// Registers per thread: the kernel is compiled for 168 (twelve warps).  setmaxnreg moves
// registers inside the CTA's own pool of 12 * 168 per lane slot and acts on whole warpgroups:
// warpgroup 2 (MMA issuer, TMA loader and two spare warps) hands back all but kRegsIssuer,
// the eight softmax warps grow to kRegsSoftmax:  4 * 88 + 8 * 208 = 2016 = 12 * 168.
constexpr int kRegsIssuer = 88;
constexpr int kRegsSoftmax = 208;

template <int D>
struct SmemLayout {
    static constexpr int kPanels = D / 64;
    static constexpr int kTileBytes = kPanels * kPanelBytes;
    static constexpr int kQ = 0;                                   // 2 query tiles
    static constexpr int kKV = 2 * kTileBytes;                     // kStages key/value tiles
    static constexpr int kBars = kKV + kStages * kTileBytes;
    // barrier indices
    static constexpr int bQFull = 0, bQEmpty = 2, bSFull = 4, bPFull = 6, bOFull = 8, bOEmpty = 10, bPFull2 = 12;
    static constexpr int bKvFull = 14, bKvEmpty = 14 + kStages;
    static constexpr int bItemFull = 14 + 2 * kStages, bItemEmpty = bItemFull + kItemQueue;
    static constexpr int kNumBars = bItemEmpty + kItemQueue;
    static constexpr int kTmemPtr = kBars + kNumBars * 8;
    static constexpr int kAbort = kTmemPtr + 4;
    static constexpr int kItemQ = kAbort + 4;                      // int [kItemQueue]: published work items
    static constexpr int kTotal = kItemQ + 4 * kItemQueue;
    static constexpr int kDynBytes = kTotal + 1024;                // room to align the base to 1024 bytes
};

// What one work item covers; every role decodes it the same way.
struct Item {
    int token0_a, token0_b;      // first token of each query tile
    int head0, kvh, part;
    int has1;                    // second query tile exists
    int n_tiles_a, n_tiles_b;    // key tiles each query tile walks
    int n_load;                  // key tiles to stage = max of the two
    int n_pref_tiles, pref_len;
    int main_row0, main_len;
    int row0_a, row0_b;          // first row of each query tile within its block (phase 1)
    int bad_length;              // phase 1: prefix_len of the block was outside [0, prefix_total] (clamped)
    int gen_base;                // >= 0: generation shard, token u sees its rows [0, gen_base + u]; -1 otherwise
};

// Work item of this CTA in a given round.  Items are sorted costliest first; rounds alternate
// direction (boustrophedon) so that no CTA always draws the costlier end of a round.  -1: none.
__device__ __forceinline__ int item_of_round(int round, int n_items) {
    const int G = static_cast<int>(gridDim.x), c = static_cast<int>(blockIdx.x);
    const int idx = round * G + ((round & 1) ? G - 1 - c : c);
    return idx < n_items ? idx : -1;
}

__device__ __forceinline__ void decode_item(const AttnArgs& a, const VarlenTable& vt, int idx, Item& it) {
    if (a.mode == kModeVarlen) {
        // Independent sequences of different lengths, plain causal attention inside each.
        // Items run from the last sequence down and, inside a sequence, from its last tile
        // pair down (for assembled Pulsar inputs the later blocks are the longer ones).
        const int rank = idx / a.Hq;
        it.head0 = idx - rank * a.Hq;
        it.kvh = it.head0 / a.g;
        it.part = 0;
        int k = 0;                                             // k-th sequence from the end
        while (k + 1 < vt.n_seq && vt.pair_cum[k + 1] <= rank) ++k;
        const int seq = vt.n_seq - 1 - k;
        const int start = vt.start[seq], len = vt.start[seq + 1] - start;
        const int tiles = (len + kTileM - 1) / kTileM, pairs = (tiles + 1) / 2;
        const int pair = pairs - 1 - (rank - vt.pair_cum[k]);
        const int qt0 = 2 * pair;
        it.has1 = (qt0 + 1 < tiles) ? 1 : 0;
        it.row0_a = qt0 * kTileM;
        it.row0_b = (qt0 + 1) * kTileM;
        it.token0_a = start + it.row0_a;
        it.token0_b = start + it.row0_b;
        it.bad_length = 0;
        it.pref_len = 0;
        it.n_pref_tiles = 0;
        it.main_row0 = start;
        it.main_len = len;
        it.gen_base = -1;
        it.n_tiles_a = qt0 + 1;
        it.n_tiles_b = it.has1 ? qt0 + 2 : 0;
    } else if (a.mode == kModePhase1) {
        // Items run block-major from the last block (longest prefix) down and, within a block,
        // from the last tile pair (most causal tiles) down; the heads of one (block, pair) are
        // adjacent.  CTAs that run at the same time therefore read the same K/V rows (L2 hits),
        // and the costliest items are handed out first.
        // The last block may be shorter than the others: it then has fewer tile pairs.
        const int rank = idx / a.Hq;
        it.head0 = idx - rank * a.Hq;
        it.kvh = it.head0 / a.g;
        it.part = 0;
        int blk, pair, len;
        if (rank < a.pairs_last) {
            blk = a.n_blocks - 1;
            pair = a.pairs_last - 1 - rank;
            len = a.last_len;
        } else {
            const int r2 = rank - a.pairs_last;
            blk = a.n_blocks - 2 - r2 / a.pairs;
            pair = a.pairs - 1 - r2 % a.pairs;
            len = a.block_size;
        }
        const int qt0 = 2 * pair;
        it.has1 = (qt0 + 1 < (len + kTileM - 1) / kTileM) ? 1 : 0;
        it.row0_a = qt0 * kTileM;
        it.row0_b = (qt0 + 1) * kTileM;
        it.token0_a = blk * a.block_size + it.row0_a;
        it.token0_b = blk * a.block_size + it.row0_b;
        int pl = a.prefix_len[blk];
        it.bad_length = (pl < 0 || pl > a.prefix_total) ? 1 : 0;
        pl = max(0, min(pl, a.prefix_total));
        it.pref_len = pl;
        it.n_pref_tiles = (pl + kTileN - 1) / kTileN;
        it.main_row0 = blk * a.block_size;
        it.main_len = len;
        it.gen_base = -1;
        it.n_tiles_a = it.n_pref_tiles + qt0 + 1;
        it.n_tiles_b = it.has1 ? it.n_pref_tiles + qt0 + 2 : 0;
    } else {
        const int rp = idx % a.pairs;
        const int rest = idx / a.pairs;
        it.kvh = rest % a.Hkv;
        it.part = rest / a.Hkv;
        it.head0 = it.kvh * a.g;
        const int tokens_per_tile = kTileM / a.pack;
        it.token0_a = (2 * rp) * tokens_per_tile;
        it.token0_b = (2 * rp + 1) * tokens_per_tile;
        it.has1 = (it.token0_b < a.n_tokens) ? 1 : 0;
        it.row0_a = it.row0_b = 0;
        it.bad_length = 0;
        int n;
        if (a.gen_total > 0 && it.part == a.n_ctx_parts) {
            // the generation shard: read through the second pair of tensor maps, causal by token
            it.pref_len = a.gen_total;
            it.n_pref_tiles = (a.gen_total + kTileN - 1) / kTileN;
            it.main_row0 = 0;
            it.main_len = 0;
            it.gen_base = a.gen_len;
            n = it.n_pref_tiles;
        } else {
            it.pref_len = 0;
            it.n_pref_tiles = 0;
            it.main_row0 = it.part * a.split_len;
            it.main_len = min(a.split_len, a.kv_len - it.main_row0);
            it.gen_base = -1;
            n = (it.main_len + kTileN - 1) / kTileN;
        }
        it.n_tiles_a = n;
        it.n_tiles_b = it.has1 ? n : 0;
    }
    it.n_load = max(it.n_tiles_a, it.n_tiles_b);
}

// Row maximum of 128 raw logits (3-input max, four independent chains).
__device__ __forceinline__ float row_max128(const uint32_t (&r)[kTileN]) {
    float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
    for (int c = 0; c < kTileN; c += 8) {
        m0 = max3(m0, __uint_as_float(r[c]), __uint_as_float(r[c + 1]));
        m1 = max3(m1, __uint_as_float(r[c + 2]), __uint_as_float(r[c + 3]));
        m2 = max3(m2, __uint_as_float(r[c + 4]), __uint_as_float(r[c + 5]));
        m3 = max3(m3, __uint_as_float(r[c + 6]), __uint_as_float(r[c + 7]));
    }
    return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
}

// p_c = 2^(s_c * scale + neg_m) for logits [kBegin, kEnd) of a row, rounded to bf16 pairs and written
// to TMEM as the A operand of the PV product; returns the fp32 row sum.  kPoly of every four
// column pairs take the polynomial exp2 (FMA pipe) instead of MUFU.  kPoly must be 0 when
// logits may be -inf (masked tiles).
template <int kPoly, int kBegin = 0, int kEnd = kTileN>
__device__ __forceinline__ float exp_row128(const uint32_t (&r)[kTileN], float scale, float neg_m, uint32_t tP) {
    float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
    const float2 sc = make_float2(scale, scale), nm = make_float2(neg_m, neg_m);
#pragma unroll
    for (int c0 = kBegin; c0 < kEnd; c0 += 32) {
        uint32_t pk[16];
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
            const float2 x =
                __ffma2_rn(make_float2(__uint_as_float(r[c0 + c]), __uint_as_float(r[c0 + c + 1])), sc, nm);
            float2 pv;
            if (((c >> 1) & 3) >= 4 - kPoly) {
                pv = ex2_poly2(x);
            } else {
                pv.x = ex2(x.x);
                pv.y = ex2(x.y);
            }
            if ((c >> 1) & 1) acc1 = __fadd2_rn(acc1, pv);
            else acc0 = __fadd2_rn(acc0, pv);
            pk[c >> 1] = pack_bf16x2(pv.x, pv.y);
        }
        tmem_st16(tP + (c0 >> 1), pk);                           // P column c/2 holds keys c, c+1
    }
    return (acc0.x + acc0.y) + (acc1.x + acc1.y);
}

// kQuad: the decode-shaped instance (AttnArgs::quad); a separate instantiation keeps its code out
// of the Phase-1 kernel's register allocation.
// kSingle: every work item of the launch has one query tile (AttnArgs::single).  With a second tile the
// tensor pipe forms one tile's products while the other tile is in its softmax; with one tile it would
// idle during the softmax and the softmax during the products (S_t -> softmax_t -> PV_t -> S_t+1 in a
// chain).  Here the logits of successive key tiles alternate between the S buffers of the two tiles
// (buffer = key-tile count of the CTA, parity), the issuer forms S_t+1 before it waits for P_t, and
// softmax warpgroup 0 walks all key tiles with both sets of barriers.  A rescale of O at key tile t
// needs PV_t-1 complete, which the completion of S_t no longer implies (it implies PV_t-2): the issuer
// commits every PV to the O barrier of the absent second tile, and a softmax warp that has to rescale
// waits for it first.  Measured against the 128K key/value set (131,072 keys, 18 parts, L2 flushed clean
// before each call): 9 to 32 query tokens of 4 heads per KV head 120-124 us -> 99-103 us (0.69 -> 0.83 of
// the HBM bandwidth), the 8-token decode shape 101.3 -> 99.4 us.
template <int D, bool kQuad, bool kSingle>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
            const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmKp,
            const __grid_constant__ CUtensorMap tmVp, const AttnArgs a,
            const __grid_constant__ VarlenTable vt) {
    using SL = SmemLayout<D>;
    static_assert(kSingle || !kQuad, "the decode-shaped instance has one query tile per item");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem + SL::kQ;
    uint8_t* sKV = smem + SL::kKV;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SL::kBars);
    uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(smem + SL::kTmemPtr);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + SL::kAbort);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // The launch that follows (the merge of this launch's partials, if any) may be scheduled as
    // SMs become free; it waits for this grid to finish before it reads anything.
    grid_launch_dependents();

    if (tid == 0) {
        *abort_flag = 0;
        for (int s = 0; s < 2; ++s) {
            mbar_init(bars + SL::bQFull + s, 1);
            mbar_init(bars + SL::bQEmpty + s, 1);
            mbar_init(bars + SL::bSFull + s, 1);
            mbar_init(bars + SL::bPFull + s, 4);        // first half of P: one arrival per softmax warp
            mbar_init(bars + SL::bPFull2 + s, 4);       // second half of P
            mbar_init(bars + SL::bOFull + s, 1);
            mbar_init(bars + SL::bOEmpty + s, 4);
        }
        for (int i = 0; i < kItemQueue; ++i) {
            mbar_init(bars + SL::bItemFull + i, 1);
            mbar_init(bars + SL::bItemEmpty + i, 9);        // MMA issuer + one lane of each softmax warp
        }
        for (int i = 0; i < kStages; ++i) {
            mbar_init(bars + SL::bKvFull + i, 1);
            mbar_init(bars + SL::bKvEmpty + i, 1);
        }
        mbar_fence_init();
    }
    if (warp == kLoadWarp && lane == 0) {
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
        tma_prefetch_desc(&tmKp);
        tma_prefetch_desc(&tmVp);
    }
    if (warp == kMmaWarp) {
        tmem_alloc(tmem_ptr, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr;

    if (warp >= 8) reg_dealloc<kRegsIssuer>();
    // Ring bookkeeping shared by the two issuer roles: `stage` walks 0..kStages-1, `phase`
    // flips at every wrap.  Barrier i lives at bar0 + 8 * i.
    const uint32_t bar0 = smem_u32(bars);
#define PULSAR_RING_NEXT(stage, phase) \
    do { if (++(stage) == kStages) { (stage) = 0; (phase) ^= 1u; } } while (0)

    if (warp == kLoadWarp) {
        // =============================== TMA loader ===============================
        // The whole warp walks the loops so that addresses, coordinates and barrier numbers stay
        // warp-uniform (the copy and barrier instructions take uniform operands); one elected
        // lane issues.
        {
            const bool leader = elect_one();
            const uint32_t q_smem = smem_u32(sQ), kv_smem = smem_u32(sKV);
            uint32_t stage = 0, phase = 0;           // next ring slot to fill
            uint32_t q_use0 = 0, q_use1 = 0;
            bool ok = true;
            volatile int* item_q = reinterpret_cast<volatile int*>(smem + SL::kItemQ);
            if (a.loader_waits) grid_dependency_wait();
            for (uint32_t seq = 0; ok; ++seq) {
                // Reconverge once per iteration: every barrier is waited on at most once per
                // iteration, so a lane that is still polling can never be more than one phase behind
                // the lanes that went ahead (two phases behind, its parity test would read "not yet"
                // again and it would stall until the bound expires).
                __syncwarp();
                // Next work item: drawn from the global counter (items differ in cost or outnumber the
                // CTAs, so they are handed out as CTAs become free) or the fixed round order.
                // It is published through a small queue for the MMA issuer and the softmax warps.
                const uint32_t slot = seq % kItemQueue;
                ok = mbar_wait_a(bar0 + 8 * (SL::bItemEmpty + slot), ((seq / kItemQueue) & 1) ^ 1, abort_flag, a.status);
                if (!ok) break;
                int idx;
                if (a.counter != nullptr) {
                    int v = 0;
                    if (lane == 0) v = atomicAdd(a.counter, 1);
                    idx = __shfl_sync(0xffffffffu, v, 0);
                    if (idx >= a.n_items) idx = -1;
                } else {
                    idx = static_cast<int>(seq) * static_cast<int>(gridDim.x) < a.n_items
                              ? item_of_round(static_cast<int>(seq), a.n_items) : -1;
                }
                if (lane == 0) {
                    item_q[slot] = idx;
                    mbar_arrive(bars + SL::bItemFull + slot);
                }
                if (idx < 0) break;
                Item it;
                decode_item(a, vt, idx, it);
                if (it.bad_length && lane == 0) report(a.status, PULSAR_DEV_BAD_LENGTH);
                const int x = it.kvh * D;
                // query tile 0
                ok = mbar_wait_a(bar0 + 8 * (SL::bQEmpty + 0), (q_use0 & 1) ^ 1, abort_flag, a.status);
                ++q_use0;
                if (!ok) break;
                if (leader) mbar_expect_tx_a(bar0 + 8 * (SL::bQFull + 0), SL::kTileBytes);
                if (kQuad) {
                    // the same 32 rows four times, at rows 0, 32, 64, 96 of the tile (the box of the
                    // tensor map is 32 rows here; 32 rows of a panel are 4096 bytes)
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int p = 0; p < SL::kPanels; ++p)
                            if (leader) tma_load_3d_a(q_smem + p * kPanelBytes + c * 4096, &tmQ, bar0 + 8 * (SL::bQFull + 0),
                                          p * 64, it.head0, it.token0_a);
                } else {
#pragma unroll
                    for (int p = 0; p < SL::kPanels; ++p)
                        if (leader) tma_load_3d_a(q_smem + p * kPanelBytes, &tmQ, bar0 + 8 * (SL::bQFull + 0), p * 64, it.head0,
                                      it.token0_a);
                }
                for (int t = 0; t < it.n_load && ok; ++t) {
                    __syncwarp();
                    const bool pref = t < it.n_pref_tiles;
                    const int row = pref ? t * kTileN : it.main_row0 + (t - it.n_pref_tiles) * kTileN;
                    // K_t
                    ok = mbar_wait_a(bar0 + 8 * (SL::bKvEmpty + stage), phase ^ 1, abort_flag, a.status);
                    if (!ok) break;
                    {
                        const uint32_t full = bar0 + 8 * (SL::bKvFull + stage), dst = kv_smem + stage * SL::kTileBytes;
                        if (leader) mbar_expect_tx_a(full, SL::kTileBytes);
#pragma unroll
                        for (int p = 0; p < SL::kPanels; ++p)
                            if (leader) tma_load_2d_a(dst + p * kPanelBytes, pref ? &tmKp : &tmK, full, x + p * 64, row);
                    }
                    PULSAR_RING_NEXT(stage, phase);
                    if (t == 0 && it.has1) {
                        ok = mbar_wait_a(bar0 + 8 * (SL::bQEmpty + 1), (q_use1 & 1) ^ 1, abort_flag, a.status);
                        ++q_use1;
                        if (!ok) break;
                        if (leader) mbar_expect_tx_a(bar0 + 8 * (SL::bQFull + 1), SL::kTileBytes);
#pragma unroll
                        for (int p = 0; p < SL::kPanels; ++p)
                            if (leader) tma_load_3d_a(q_smem + SL::kTileBytes + p * kPanelBytes, &tmQ, bar0 + 8 * (SL::bQFull + 1),
                                          p * 64, it.head0, it.token0_b);
                    }
                    // V_t
                    ok = mbar_wait_a(bar0 + 8 * (SL::bKvEmpty + stage), phase ^ 1, abort_flag, a.status);
                    if (!ok) break;
                    {
                        const uint32_t full = bar0 + 8 * (SL::bKvFull + stage), dst = kv_smem + stage * SL::kTileBytes;
                        if (leader) mbar_expect_tx_a(full, SL::kTileBytes);
#pragma unroll
                        for (int p = 0; p < SL::kPanels; ++p)
                            if (leader) tma_load_2d_a(dst + p * kPanelBytes, pref ? &tmVp : &tmV, full, x + p * 64, row);
                    }
                    PULSAR_RING_NEXT(stage, phase);
                }
            }
        }
        __syncwarp();
    } else if (warp == kMmaWarp) {
        // =============================== MMA issuer ===============================
        // Per key tile t the issue order is PV_0(t), S_0(t+1), PV_1(t), S_1(t+1): tile 0 gets its
        // next S about one PV + S ahead of tile 1, which keeps the two softmax warpgroups half a
        // period apart (one exponentiates while the tensor pipe works for the other).
        // Warp-uniform control flow, one elected lane issues: descriptors, TMEM addresses and
        // barrier numbers then live in uniform registers, which the MMA instructions read.
        {
            const bool leader = elect_one();
            constexpr uint32_t kIdescQK = umma_idesc_bf16(kTileM, kTileN, false, false);
            constexpr uint32_t kIdescPV = umma_idesc_bf16(kTileM, D, false, true);
            constexpr uint32_t kStageStep = SL::kTileBytes >> 4;         // descriptor address units (16 bytes)
            // Descriptors of stage 0 / query tile 0; other tiles add a multiple of kStageStep to the
            // address field (shared memory is below 256 KB, so the 14-bit field never carries).
            const uint64_t descQ0 = umma_smem_desc_sw128(smem_u32(sQ), 16, 1024);
            const uint64_t descQ1 = descQ0 + kStageStep;
            const uint64_t descK = umma_smem_desc_sw128(smem_u32(sKV), 16, 1024);
            const uint64_t descV = umma_smem_desc_sw128(smem_u32(sKV), kPanelBytes, 1024);
            const uint32_t tS0 = tmem_base, tS1 = tmem_base + 128, tO0 = tmem_base + 256, tO1 = tmem_base + 384;
            uint32_t stage = 0, phase = 0;           // next ring slot to consume
            uint32_t q_use0 = 0, q_use1 = 0, p_cnt0 = 0, p_cnt1 = 0, o_use0 = 0, o_use1 = 0;
            uint32_t g_tile = 0;                     // kSingle: key tiles this CTA has walked
            bool ok = true;

#define PULSAR_ISSUE_S(tS, dq, dk, s_)                                                                    \
    do {                                                                                                  \
        _Pragma("unroll") for (int kk = 0; kk < D / 16; ++kk) {                                           \
            const uint64_t off = static_cast<uint64_t>(((kk >> 2) * kPanelBytes + (kk & 3) * 32) >> 4);    \
            if (leader) umma_ss(tS, (dq) + off, (dk) + off, kIdescQK, kk > 0 ? 1u : 0u);                  \
        }                                                                                                 \
        if (leader) umma_commit_a(bar0 + 8 * (SL::bSFull + (s_)));                                        \
    } while (0)
// P arrives in two halves of 64 keys, each with its own barrier.
#define PULSAR_ISSUE_PV(tO, tP, dv, acc, s_, par)                                                         \
    do {                                                                                                  \
        _Pragma("unroll") for (int half = 0; half < 2; ++half) {                                          \
            ok = ok && mbar_wait_a(bar0 + 8 * ((half ? SL::bPFull2 : SL::bPFull) + (s_)), par, abort_flag, \
                                   a.status);                                                             \
            tc_fence_after();                                                                             \
            _Pragma("unroll") for (int kk = half * 4; kk < half * 4 + 4; ++kk)                            \
                if (leader && ok)                                                                         \
                    umma_ts(tO, (tP) + kk * 8, (dv) + static_cast<uint64_t>(kk * 128), kIdescPV,          \
                            ((acc) || kk > 0) ? 1u : 0u);                                                 \
        }                                                                                                 \
    } while (0)

            volatile int* item_q = reinterpret_cast<volatile int*>(smem + SL::kItemQ);
            for (uint32_t seq = 0; ok; ++seq) {
                __syncwarp();              // see the loader: lanes stay within one barrier phase of each other
                const uint32_t slot = seq % kItemQueue;
                ok = mbar_wait_a(bar0 + 8 * (SL::bItemFull + slot), (seq / kItemQueue) & 1, abort_flag, a.status);
                if (!ok) break;
                const int idx = item_q[slot];
                if (leader) mbar_arrive(bars + SL::bItemEmpty + slot);
                if (idx < 0) break;
                Item it;
                decode_item(a, vt, idx, it);
                const int n0 = it.n_tiles_a, n1 = it.n_tiles_b;
                if (kSingle) {
                    // Ring slots: K_t at position 2t of the item, V_t at 2t + 1 (the loader's order); the
                    // issuer consumes K_t+1 before V_t.
                    uint32_t kst = stage, kph = phase, vst = stage, vph = phase;
                    PULSAR_RING_NEXT(vst, vph);
                    ok = mbar_wait_a(bar0 + 8 * (SL::bQFull + 0), q_use0 & 1, abort_flag, a.status) &&
                         mbar_wait_a(bar0 + 8 * (SL::bKvFull + kst), kph, abort_flag, a.status);
                    ++q_use0;
                    if (!ok) break;
                    tc_fence_after();
                    {
                        const uint32_t b = g_tile & 1u;
                        PULSAR_ISSUE_S(tS0 + b * 128, descQ0, descK + static_cast<uint64_t>(kst * kStageStep), b);
                    }
                    if (leader) umma_commit_a(bar0 + 8 * (SL::bKvEmpty + kst));
                    if (n0 == 1 && leader) umma_commit_a(bar0 + 8 * (SL::bQEmpty + 0));
                    PULSAR_RING_NEXT(kst, kph);
                    PULSAR_RING_NEXT(kst, kph);
                    for (int t = 0; t < n0; ++t) {
                        __syncwarp();
                        const uint32_t b = g_tile & 1u, par = (g_tile >> 1) & 1u;
                        if (t + 1 < n0) {                                  // S_t+1 into the other buffer
                            ok = mbar_wait_a(bar0 + 8 * (SL::bKvFull + kst), kph, abort_flag, a.status);
                            if (!ok) break;
                            tc_fence_after();
                            PULSAR_ISSUE_S(tS0 + (b ^ 1u) * 128, descQ0, descK + static_cast<uint64_t>(kst * kStageStep), b ^ 1u);
                            if (leader) umma_commit_a(bar0 + 8 * (SL::bKvEmpty + kst));
                            if (t + 2 == n0 && leader) umma_commit_a(bar0 + 8 * (SL::bQEmpty + 0));
                            PULSAR_RING_NEXT(kst, kph);
                            PULSAR_RING_NEXT(kst, kph);
                        }
                        ok = mbar_wait_a(bar0 + 8 * (SL::bKvFull + vst), vph, abort_flag, a.status);
                        if (!ok) break;
                        if (t == 0) {
                            ok = mbar_wait_a(bar0 + 8 * (SL::bOEmpty + 0), (o_use0 & 1) ^ 1, abort_flag, a.status);
                            ++o_use0;
                        }
                        const uint64_t dv = descV + static_cast<uint64_t>(vst * kStageStep);
                        PULSAR_ISSUE_PV(tO0, tS0 + b * 128, dv, t > 0, b, par);
                        if (!ok) break;
                        if (leader) {
                            umma_commit_a(bar0 + 8 * (SL::bKvEmpty + vst));
                            umma_commit_a(bar0 + 8 * (SL::bOFull + 1));            // PV_t complete
                            if (t == n0 - 1) umma_commit_a(bar0 + 8 * (SL::bOFull + 0));
                        }
                        PULSAR_RING_NEXT(vst, vph);
                        PULSAR_RING_NEXT(vst, vph);
                        ++g_tile;
                    }
                    stage = kst;
                    phase = kph;
                    continue;
                }
                // K_0
                uint32_t ks = stage, kp = phase;
                PULSAR_RING_NEXT(stage, phase);
                ok = mbar_wait_a(bar0 + 8 * (SL::bQFull + 0), q_use0 & 1, abort_flag, a.status) &&
                     mbar_wait_a(bar0 + 8 * (SL::bKvFull + ks), kp, abort_flag, a.status);
                ++q_use0;
                if (!ok) break;
                tc_fence_after();
                PULSAR_ISSUE_S(tS0, descQ0, descK + static_cast<uint64_t>(ks * kStageStep), 0);
                if (kEarlyRelease && n0 == 1 && leader) umma_commit_a(bar0 + 8 * (SL::bQEmpty + 0));
                if (it.has1) {
                    ok = mbar_wait_a(bar0 + 8 * (SL::bQFull + 1), q_use1 & 1, abort_flag, a.status);
                    ++q_use1;
                    if (!ok) break;
                    tc_fence_after();
                    PULSAR_ISSUE_S(tS1, descQ1, descK + static_cast<uint64_t>(ks * kStageStep), 1);
                    if (kEarlyRelease && n1 == 1 && leader) umma_commit_a(bar0 + 8 * (SL::bQEmpty + 1));
                }
                if (leader) umma_commit_a(bar0 + 8 * (SL::bKvEmpty + ks));
                for (int t = 0; t < it.n_load; ++t) {
                    __syncwarp();
                    const uint32_t vs = stage, vp = phase;                 // V_t
                    PULSAR_RING_NEXT(stage, phase);
                    const bool more = t + 1 < it.n_load;
                    if (more) {                                            // K_{t+1}
                        ks = stage;
                        kp = phase;
                        PULSAR_RING_NEXT(stage, phase);
                    }
                    const uint64_t dv = descV + static_cast<uint64_t>(vs * kStageStep);
                    const uint64_t dk = descK + static_cast<uint64_t>(ks * kStageStep);
                    ok = mbar_wait_a(bar0 + 8 * (SL::bKvFull + vs), vp, abort_flag, a.status);
                    if (!ok) break;
                    if (t < n0) {
                        if (t == 0) {
                            ok = mbar_wait_a(bar0 + 8 * (SL::bOEmpty + 0), (o_use0 & 1) ^ 1, abort_flag, a.status);
                            ++o_use0;
                        }
                        PULSAR_ISSUE_PV(tO0, tS0, dv, t > 0, 0, p_cnt0 & 1);
                        ++p_cnt0;
                        if (!ok) break;
                        if (t == n0 - 1) {
                            if (leader) umma_commit_a(bar0 + 8 * (SL::bOFull + 0));
                            if (!kEarlyRelease && leader) umma_commit_a(bar0 + 8 * (SL::bQEmpty + 0));
                        }
                    }
                    if (more) {
                        ok = mbar_wait_a(bar0 + 8 * (SL::bKvFull + ks), kp, abort_flag, a.status);
                        if (!ok) break;
                        tc_fence_after();
                        if (t + 1 < n0) {
                            PULSAR_ISSUE_S(tS0, descQ0, dk, 0);
                            // the tile's last S: nothing reads its Q any more
                            if (kEarlyRelease && t + 2 == n0 && leader) umma_commit_a(bar0 + 8 * (SL::bQEmpty + 0));
                        }
                    }
                    if (t < n1) {
                        if (t == 0) {
                            ok = mbar_wait_a(bar0 + 8 * (SL::bOEmpty + 1), (o_use1 & 1) ^ 1, abort_flag, a.status);
                            ++o_use1;
                        }
                        PULSAR_ISSUE_PV(tO1, tS1, dv, t > 0, 1, p_cnt1 & 1);
                        ++p_cnt1;
                        if (!ok) break;
                        if (t == n1 - 1) {
                            if (leader) umma_commit_a(bar0 + 8 * (SL::bOFull + 1));
                            if (!kEarlyRelease && leader) umma_commit_a(bar0 + 8 * (SL::bQEmpty + 1));
                        }
                    }
                    if (leader) umma_commit_a(bar0 + 8 * (SL::bKvEmpty + vs));
                    if (more) {
                        if (t + 1 < n1) {
                            PULSAR_ISSUE_S(tS1, descQ1, dk, 1);
                            if (kEarlyRelease && t + 2 == n1 && leader) umma_commit_a(bar0 + 8 * (SL::bQEmpty + 1));
                        }
                        if (leader) umma_commit_a(bar0 + 8 * (SL::bKvEmpty + ks));
                    }
                }
            }
#undef PULSAR_ISSUE_S
#undef PULSAR_ISSUE_PV
        }
        __syncwarp();
    } else if (warp < 8) {
        // =============================== softmax warpgroups ===============================
        reg_alloc<kRegsSoftmax>();
        const int s = warp >> 2;                               // query tile of this warpgroup
        const int row = (warp & 3) * 32 + lane;                // row of the tile = TMEM lane
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS_own = tmem_base + s * 128 + lane_sel;
        const uint32_t tO = tmem_base + 256 + s * 128 + lane_sel;
        uint64_t* bar_of = bars + SL::bOFull + s;
        uint64_t* bar_pv = bars + SL::bOFull + 1;              // kSingle: one completion per PV product
        uint32_t g_tile = 0;                                   // kSingle: key tiles this CTA has walked
        uint64_t* bar_oe = bars + SL::bOEmpty + s;
        uint32_t s_cnt = 0, o_cnt = 0;
        bool ok = true;

        volatile int* item_q = reinterpret_cast<volatile int*>(smem + SL::kItemQ);
        for (uint32_t seq = 0; ok; ++seq) {
            const uint32_t slot = seq % kItemQueue;
            ok = __all_sync(0xffffffffu, mbar_wait(bars + SL::bItemFull + slot, (seq / kItemQueue) & 1, abort_flag, a.status));
            if (!ok) break;
            const int idx = item_q[slot];
            __syncwarp();
            if (lane == 0) mbar_arrive(bars + SL::bItemEmpty + slot);
            if (idx < 0) break;
            Item it;
            decode_item(a, vt, idx, it);
            const int n = s ? it.n_tiles_b : it.n_tiles_a;
            if (n == 0) continue;
            float m_used = -INFINITY, l_run = 0.f;
            const int my_row_in_block = (s ? it.row0_b : it.row0_a) + row;
            const int row_t = kQuad ? lane : row;             // row as far as token and head are concerned

            for (int t = 0; t < n; ++t) {
                // visible key columns of this tile for this row: [0, n_vis)
                int n_vis = kTileN;
                bool masked = false;
                if (t < it.n_pref_tiles) {
                    const int valid = it.pref_len - t * kTileN;
                    if (valid < kTileN) { n_vis = valid; masked = true; }
                    if (it.gen_base >= 0) {                   // generation shard: causal by token
                        const int token = (s ? it.token0_b : it.token0_a) + row_t / a.pack;
                        n_vis = min(n_vis, it.gen_base + token + 1 - t * kTileN);
                        masked = true;
                    }
                } else {
                    const int j = t - it.n_pref_tiles;
                    const int valid = it.main_len - j * kTileN;
                    if (valid < kTileN) { n_vis = valid; masked = true; }
                    if (a.mode != kModePhase2 && t == n - 1) {
                        n_vis = min(n_vis, my_row_in_block - j * kTileN + 1);
                        masked = true;
                    }
                }

                // kSingle: buffer and barriers alternate with the CTA's key-tile count
                const uint32_t gb = kSingle ? (g_tile & 1u) : 0u;
                const uint32_t tS = tS_own + gb * 128;
                uint64_t* bar_s = bars + SL::bSFull + s + gb;
                uint64_t* bar_p = bars + SL::bPFull + s + gb;
                uint64_t* bar_p2 = bars + SL::bPFull2 + s + gb;
                ok = __all_sync(0xffffffffu,
                                ok && mbar_wait(bar_s, kSingle ? ((g_tile >> 1) & 1u) : (s_cnt & 1u), abort_flag, a.status));
                ++s_cnt;
                ++g_tile;
                if (!ok) break;
                tc_fence_after();

                if (kQuad) {
                    // Few query rows (decode): this warp's lane quarter holds a copy of the rows and
                    // the warp takes keys [32q, 32q+32) of the tile only; the other keys get P = 0 in
                    // its copy.  Each copy ends as a partial of its own, merged with the KV parts.
                    const int q4 = warp & 3;
                    uint32_t rq[32];
                    tmem_ld32(tS + 32 * q4, rq);
                    tmem_wait_ld();
                    if (masked) {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (32 * q4 + c >= n_vis) rq[c] = 0xff800000u;          // -inf
                    }
                    float mq = -INFINITY;
#pragma unroll
                    for (int c = 0; c < 32; c += 2) mq = max3(mq, __uint_as_float(rq[c]), __uint_as_float(rq[c + 1]));
                    const float m_tile = mq * a.scale_log2;
                    const bool need = m_tile > m_used + kRescaleThreshold;
                    if (__any_sync(0xffffffffu, need)) {
                        if (kSingle && t > 0) {
                            // O may be rescaled once the PV product of the previous key tile is complete.
                            // This is key tile g_tile - 1 of the CTA; completions 0 .. g_tile - 3 are certain
                            // (this tile's S was issued after them), so the barrier is in phase g_tile - 2
                            // or g_tile - 1 and the parity of g_tile - 2 tells the two apart.
                            ok = __all_sync(0xffffffffu, mbar_wait(bar_pv, g_tile & 1u, abort_flag, a.status));
                            if (!ok) break;
                            tc_fence_after();
                        }
                        const float m_new = need ? m_tile : m_used;
                        const float alpha = (m_new == -INFINITY) ? 1.f : ex2(m_used - m_new);
                        l_run *= alpha;
                        m_used = m_new;
                        if (t > 0) {
#pragma unroll
                            for (int c0 = 0; c0 < D; c0 += 32) {
                                uint32_t o[32];
                                tmem_ld32(tO + c0, o);
                                tmem_wait_ld();
#pragma unroll
                                for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
                                tmem_st32(tO + c0, o);
                            }
                        }
                    }
                    const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
                    uint32_t pk[16];
                    float2 acc = make_float2(0.f, 0.f);
                    const float2 sc = make_float2(a.scale_log2, a.scale_log2), nm = make_float2(neg_m, neg_m);
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        const float2 x = __ffma2_rn(make_float2(__uint_as_float(rq[c]), __uint_as_float(rq[c + 1])), sc, nm);
                        float2 pv;
                        pv.x = ex2(x.x);
                        pv.y = ex2(x.y);
                        acc = __fadd2_rn(acc, pv);
                        pk[c >> 1] = pack_bf16x2(pv.x, pv.y);
                    }
                    l_run += acc.x + acc.y;
                    uint32_t zero[16];
#pragma unroll
                    for (int c = 0; c < 16; ++c) zero[c] = 0u;
#pragma unroll
                    for (int qq = 0; qq < 4; ++qq) {
                        if (qq == q4) tmem_st16(tS + 16 * qq, pk);          // P column c/2 holds keys c, c+1
                        else tmem_st16(tS + 16 * qq, zero);
                    }
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(bar_p);
                        mbar_arrive(bar_p2);
                    }
                    continue;
                }

                uint32_t r[kTileN];
                PULSAR_TMEM_LD32_AT(tS + 0, r, 0);
                PULSAR_TMEM_LD32_AT(tS + 32, r, 32);
                PULSAR_TMEM_LD32_AT(tS + 64, r, 64);
                PULSAR_TMEM_LD32_AT(tS + 96, r, 96);
                tmem_wait_ld();

                if (masked) {
#pragma unroll
                    for (int c = 0; c < kTileN; ++c)
                        if (c >= n_vis) r[c] = 0xff800000u;          // -inf
                }
                const float m_tile = row_max128(r) * a.scale_log2;
                const bool need = m_tile > m_used + kRescaleThreshold;   // always true on the first tile
                if (__any_sync(0xffffffffu, need)) {
                    if (kSingle && t > 0) {
                        // O may be rescaled once the PV product of the previous key tile is complete.
                        // This is key tile g_tile - 1 of the CTA; completions 0 .. g_tile - 3 are certain
                        // (this tile's S was issued after them), so the barrier is in phase g_tile - 2
                        // or g_tile - 1 and the parity of g_tile - 2 tells the two apart.
                        ok = __all_sync(0xffffffffu, mbar_wait(bar_pv, g_tile & 1u, abort_flag, a.status));
                        if (!ok) break;
                        tc_fence_after();
                    }
                    const float m_new = need ? m_tile : m_used;
                    const float alpha = (m_new == -INFINITY) ? 1.f : ex2(m_used - m_new);
                    l_run *= alpha;
                    m_used = m_new;
                    if (t > 0) {
#pragma unroll
                        for (int c0 = 0; c0 < D; c0 += 32) {
                            uint32_t o[32];
                            tmem_ld32(tO + c0, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
                            tmem_st32(tO + c0, o);
                        }
                    }
                }
                const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
                // P goes to the MMA issuer in two halves of 64 keys, so that the first half
                // of the PV product runs while the second half of the row is exponentiated.
                // (The rescale above has stored its O columns before the first hand-over.)
                if (masked) l_run += exp_row128<0, 0, 64>(r, a.scale_log2, neg_m, tS);
                else l_run += exp_row128<kPolyPairsFor<D>, 0, 64>(r, a.scale_log2, neg_m, tS);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_p);
                if (masked) l_run += exp_row128<0, 64, 128>(r, a.scale_log2, neg_m, tS);
                else l_run += exp_row128<kPolyPairsFor<D>, 64, 128>(r, a.scale_log2, neg_m, tS);

                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_p2);
            }
            if (!ok) break;

            // ---- epilogue: normalise and store this thread's row ----
            ok = __all_sync(0xffffffffu, ok && mbar_wait(bar_of, o_cnt & 1, abort_flag, a.status));
            ++o_cnt;
            if (!ok) break;
            tc_fence_after();
            {
                const int token = (s ? it.token0_b : it.token0_a) + row_t / a.pack;
                const int head = it.head0 + row_t % a.pack;
                const int part = kQuad ? it.part * 4 + (warp & 3) : it.part;
                bool store = token < a.n_tokens;
                if (a.mode != kModePhase2) store = store && my_row_in_block < it.main_len;
                const float inv_l = l_run > 0.f ? 1.f / l_run : 0.f;
                const float lse = (l_run > 0.f) ? (m_used + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
                const size_t orow = static_cast<size_t>(token) * a.Hq + head;
                // The whole accumulator row goes to registers first (the logits' registers are free by
                // now), so that the accumulator can be handed back before the row is scaled and stored.
                uint32_t o[D];
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += 32) PULSAR_TMEM_LD32_AT(tO + c0, o, c0);
                tmem_wait_ld();
                if (kEarlyRelease) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_oe);
                }
                if (store) {
                    if (a.part_O != nullptr) {
                        float4* dst = reinterpret_cast<float4*>(
                            a.part_O + (static_cast<size_t>(part) * a.n_tokens * a.Hq + orow) * D);
#pragma unroll
                        for (int c = 0; c < D; c += 4)
                            dst[c >> 2] = make_float4(__uint_as_float(o[c]) * inv_l, __uint_as_float(o[c + 1]) * inv_l,
                                                      __uint_as_float(o[c + 2]) * inv_l, __uint_as_float(o[c + 3]) * inv_l);
                        a.part_LSE[static_cast<size_t>(part) * a.n_tokens * a.Hq + orow] = lse;
                    } else {
                        uint4* dst = reinterpret_cast<uint4*>(a.O + orow * D);
#pragma unroll
                        for (int c = 0; c < D; c += 8) {
                            uint4 v;
                            v.x = pack_bf16x2(__uint_as_float(o[c]) * inv_l, __uint_as_float(o[c + 1]) * inv_l);
                            v.y = pack_bf16x2(__uint_as_float(o[c + 2]) * inv_l, __uint_as_float(o[c + 3]) * inv_l);
                            v.z = pack_bf16x2(__uint_as_float(o[c + 4]) * inv_l, __uint_as_float(o[c + 5]) * inv_l);
                            v.w = pack_bf16x2(__uint_as_float(o[c + 6]) * inv_l, __uint_as_float(o[c + 7]) * inv_l);
                            dst[c >> 3] = v;
                        }
                        if (a.LSE != nullptr) a.LSE[orow] = lse;
                    }
                }
            }
            if (!kEarlyRelease) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_oe);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tmem_base, 512);
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

// overlap_prior: launch with programmatic stream serialization, i.e. the kernel may start while the
// launch before it on the stream is still running (that launch must be this library's append
// kernel, which releases its dependent at once); the loader then waits for it before its first
// load (AttnArgs::loader_waits).
template <int D>
int32_t launch_attn(const CUtensorMap& q, const CUtensorMap& k, const CUtensorMap& v, const CUtensorMap& kp,
                    const CUtensorMap& vp, const AttnArgs& a, cudaStream_t stream,
                    const VarlenTable* table = nullptr, bool overlap_prior = false) {
    constexpr int smem = SmemLayout<D>::kDynBytes;
    // The opt-in to more than 48 KB of dynamic shared memory is a per-device function attribute;
    // setting it on every launch keeps multi-device processes correct and costs well under a microsecond.
    auto kernel = a.quad ? attn_kernel<D, true, true>
                         : (a.single ? attn_kernel<D, false, true> : attn_kernel<D, false, false>);
    PULSAR_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    const int grid = a.n_items < sm_count() ? a.n_items : sm_count();     // one persistent CTA per SM
    if (grid <= 0) return PULSAR_OK;
    static const VarlenTable kNoTable{};
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(kAttnThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_prior ? 1 : 0;
    PULSAR_CUDA_OK(cudaLaunchKernelEx(&cfg, kernel, q, k, v, kp, vp, a, table ? *table : kNoTable));
    PULSAR_CUDA_OK(cudaGetLastError());
    count_launch();
    return PULSAR_OK;
}

struct Phase1Plan {
    int n_blocks, tiles_per_block, pairs_per_block;
    int last_len, pairs_last;                 // the last block: its tokens and its tile pairs
    int n_items;
    size_t pref_rows, pref_bytes, total;
};

// whole_only: the entry point takes only sequences made of whole blocks.
int32_t plan_phase1(int64_t L, int32_t Hq, int32_t Hkv, int32_t d, int32_t block_size, int32_t prefix_total,
                    Phase1Plan& p, bool whole_only = false) {
    if (L <= 0 || Hq <= 0 || Hkv <= 0 || block_size <= 0 || prefix_total < 0) return PULSAR_ERR_INVALID_ARG;
    if ((d != 64 && d != 128) || Hq % Hkv != 0 || L >= (1ll << 31)) return PULSAR_ERR_SHAPE;
    if (whole_only && L % block_size != 0) return PULSAR_ERR_SHAPE;
    const int64_t B = (L + block_size - 1) / block_size;       // the last block holds the tokens that remain
    if (B > 65535 || Hq > 65535) return PULSAR_ERR_SHAPE;
    if (prefix_total > (1 << 30)) return PULSAR_ERR_SHAPE;
    p.n_blocks = static_cast<int>(B);
    p.tiles_per_block = (block_size + kTileM - 1) / kTileM;
    p.pref_rows = static_cast<size_t>(prefix_total > 0 ? prefix_total : 1);
    p.pairs_per_block = (p.tiles_per_block + 1) / 2;
    p.last_len = static_cast<int>(L - (B - 1) * block_size);
    p.pairs_last = ((p.last_len + kTileM - 1) / kTileM + 1) / 2;
    p.pref_bytes = round_up(p.pref_rows * Hkv * d * 2, 256);
    p.total = 2 * p.pref_bytes + 256;                        // gathered prefix K, V and the work counter
    const int64_t items = ((B - 1) * p.pairs_per_block + p.pairs_last) * Hq;
    if (items >= (1ll << 31)) return PULSAR_ERR_SHAPE;
    p.n_items = static_cast<int>(items);
    return PULSAR_OK;
}

// Number of KV parts for Phase 2 when the caller leaves the choice to the library: the J that
// minimises a simple time model --
//   rounds(J) * (tiles per part * t_tile + t_item)  +  partial traffic(J) / HBM bandwidth,
// rounds = ceil(items / CTAs).  More parts fill the last round better and shorten it, but every
// part writes and re-reads fp32 partials.  Constants are measured on B200 (one pair of query
// tiles against one 128-key tile: about 2 us; per-item prologue and epilogue: about 6 us).
int32_t choose_splits(int32_t nq, int64_t L, int32_t Hq, int32_t Hkv, int32_t d) {
    const int g = Hq / Hkv;
    const int64_t row_tiles = (static_cast<int64_t>(nq) * g + kTileM - 1) / kTileM;
    const int64_t items = (row_tiles + 1) / 2 * Hkv;               // a work item is a pair of row tiles
    const int64_t kv_tiles = (L + kTileN - 1) / kTileN;
    const double ctas = sm_count(), t_tile_us = 2.0, t_item_us = 6.0, hbm_bytes_per_us = 6.0e6;
    double best_t = 0;
    int64_t best = 1;
    for (int64_t j = 1; j <= kv_tiles && j <= 1024; ++j) {
        const int64_t tiles_per_part = (kv_tiles + j - 1) / j;
        if ((kv_tiles + tiles_per_part - 1) / tiles_per_part != j) continue;      // some part would be empty
        const double rounds = static_cast<double>((items * j + static_cast<int64_t>(ctas) - 1) / static_cast<int64_t>(ctas));
        const double partial = j > 1 ? 2.0 * j * nq * Hq * (d + 1) * 4.0 / hbm_bytes_per_us : 0.0;
        const double t = rounds * (static_cast<double>(tiles_per_part) * t_tile_us + t_item_us) + partial;
        if (best_t == 0 || t < best_t) { best_t = t; best = j; }
    }
    return static_cast<int32_t>(best);
}

// Decode shapes: all query rows of a KV head (tokens x heads per KV head) fit one quarter of a
// tile, so the kernel works on four copies of them, one key quarter each; every copy is a partial
// of its own (four times the partials, merged with the KV parts).
inline bool phase2_quad(int32_t nq, int32_t g) { return nq * g <= 32; }

// Keys per KV part: L / n_splits when that divides; otherwise the parts are whole 128-key tiles,
// ceil(tiles / n_splits) each, the last one shorter.  0 if some part would be empty.
int64_t phase2_split_len(int64_t L, int32_t n_splits) {
    if (n_splits <= 0) return 0;
    if (L % n_splits == 0) return L / n_splits;
    const int64_t kv_tiles = (L + kTileN - 1) / kTileN;
    const int64_t tiles_per_part = (kv_tiles + n_splits - 1) / n_splits;
    if ((kv_tiles + tiles_per_part - 1) / tiles_per_part != n_splits) return 0;
    return tiles_per_part * kTileN;
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
    int32_t* counter = reinterpret_cast<int32_t*>(static_cast<char*>(workspace) + 2 * p.pref_bytes);

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

    PULSAR_CUDA_OK(cudaMemsetAsync(counter, 0, sizeof(int32_t), stream));

    AttnArgs a{};
    a.mode = kModePhase1;
    a.Hkv = Hkv;
    a.pairs = p.pairs_per_block;
    a.last_len = p.last_len;
    a.pairs_last = p.pairs_last;
    a.n_items = p.n_items;
    a.n_blocks = p.n_blocks;
    a.counter = counter;
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
    rc = d == 128 ? launch_attn<128>(tmQ, tmK, tmV, tmKp, tmVp, a, stream)
                  : launch_attn<64>(tmQ, tmK, tmV, tmKp, tmVp, a, stream);
    if (rc != PULSAR_OK) return rc;

    if (K_ret) {
        const size_t bytes = static_cast<size_t>(L) * Hkv * d * 2;
        PULSAR_CUDA_OK(cudaMemcpyAsync(K_ret, K, bytes, cudaMemcpyDeviceToDevice, stream));
        PULSAR_CUDA_OK(cudaMemcpyAsync(V_ret, V, bytes, cudaMemcpyDeviceToDevice, stream));
    }
    return PULSAR_OK;
}

// =============================================================================================
// Phase 1 with the logical blocks spread over several GPUs (block-to-host mapping, Section 3 and
// Appendix J): what one GPU runs before and after the exchange of summary K/V rows.
// =============================================================================================
extern "C" int32_t pulsar_pack_summary_kv(const uint16_t* K, const uint16_t* V, int32_t n_local, int32_t block_size,
                                          int32_t Hkv, int32_t d, const int32_t* sel_chunks,
                                          const int32_t* block_ids, int32_t n_blocks, int32_t chunk, int32_t k,
                                          int32_t sink, uint16_t* K_send, uint16_t* V_send, int32_t* device_status,
                                          void* stream) {
    if (n_local <= 0 || block_size <= 0 || Hkv <= 0 || d <= 0 || n_blocks <= 0 || chunk <= 0 || k < 0 || sink < 0)
        return PULSAR_ERR_INVALID_ARG;
    if ((static_cast<int64_t>(Hkv) * d * 2) % 16 != 0 || block_size % chunk != 0 || k > block_size / chunk ||
        sink > block_size || n_local > n_blocks || static_cast<int64_t>(n_local) * block_size >= (1ll << 31))
        return PULSAR_ERR_SHAPE;
    if (!K || !V || !sel_chunks || !block_ids || !K_send || !V_send) return PULSAR_ERR_INVALID_ARG;
    if (!aligned(K, 16) || !aligned(V, 16) || !aligned(K_send, 16) || !aligned(V_send, 16) ||
        !aligned(sel_chunks, 4) || !aligned(block_ids, 4))
        return PULSAR_ERR_ALIGNMENT;
    int32_t rc = check_device();
    if (rc != PULSAR_OK) return rc;
    const int64_t rows = sink + static_cast<int64_t>(n_local) * k * chunk;
    if (rows == 0) return PULSAR_OK;
    if (rows > 0x7fffffffll) return PULSAR_ERR_SHAPE;
    pack_summary_kernel<<<static_cast<unsigned>(rows), 128, 0, static_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<const uint4*>(K), reinterpret_cast<const uint4*>(V), sel_chunks, block_ids, n_local, n_blocks,
        block_size, chunk, k, sink, Hkv * d * 2 / 16, reinterpret_cast<uint4*>(K_send),
        reinterpret_cast<uint4*>(V_send), device_status);
    PULSAR_CUDA_OK(cudaGetLastError());
    count_launch();
    return PULSAR_OK;
}

extern "C" int32_t pulsar_gather_kv_rows(const uint16_t* K, const uint16_t* V, int64_t rows_in, int32_t Hkv, int32_t d,
                                         const int32_t* idx, int32_t n_idx, uint16_t* K_out, uint16_t* V_out,
                                         int32_t* device_status, void* stream) {
    if (rows_in <= 0 || Hkv <= 0 || d <= 0 || n_idx < 0) return PULSAR_ERR_INVALID_ARG;
    if ((static_cast<int64_t>(Hkv) * d * 2) % 16 != 0 || rows_in >= (1ll << 31)) return PULSAR_ERR_SHAPE;
    if (n_idx == 0) return PULSAR_OK;
    if (!K || !V || !idx || !K_out || !V_out) return PULSAR_ERR_INVALID_ARG;
    if (!aligned(K, 16) || !aligned(V, 16) || !aligned(K_out, 16) || !aligned(V_out, 16) || !aligned(idx, 4))
        return PULSAR_ERR_ALIGNMENT;
    int32_t rc = check_device();
    if (rc != PULSAR_OK) return rc;
    gather_rows_kernel<<<n_idx, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<const uint4*>(K), reinterpret_cast<const uint4*>(V), idx, rows_in, Hkv * d * 2 / 16,
        reinterpret_cast<uint4*>(K_out), reinterpret_cast<uint4*>(V_out), device_status);
    PULSAR_CUDA_OK(cudaGetLastError());
    count_launch();
    return PULSAR_OK;
}

extern "C" int32_t pulsar_phase1_attn_sharded(const uint16_t* Q, const uint16_t* K, const uint16_t* V, int64_t L_local,
                                              int32_t Hq, int32_t Hkv, int32_t d, int32_t block_size,
                                              const uint16_t* K_prefix, const uint16_t* V_prefix,
                                              int32_t prefix_total, const int32_t* prefix_len_local,
                                              float softmax_scale, uint16_t* O, float* LSE, void* workspace,
                                              size_t workspace_bytes, int32_t* device_status, void* stream_) {
    Phase1Plan p;
    int32_t rc = plan_phase1(L_local, Hq, Hkv, d, block_size, prefix_total, p, /*whole_only=*/true);
    if (rc != PULSAR_OK) return rc;
    if (!Q || !K || !V || !O || !prefix_len_local || !workspace || (prefix_total > 0 && (!K_prefix || !V_prefix)))
        return PULSAR_ERR_INVALID_ARG;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) || !aligned(prefix_len_local, 4) ||
        !aligned(K_prefix, 16) || !aligned(V_prefix, 16) || (LSE && !aligned(LSE, 4)) || !aligned(workspace, 256))
        return PULSAR_ERR_ALIGNMENT;
    if (workspace_bytes < 256) return PULSAR_ERR_WORKSPACE;
    rc = check_device();
    if (rc != PULSAR_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int32_t* counter = static_cast<int32_t*>(workspace);

    // With no prefix at all the two prefix maps still have to describe valid memory: use K, V.
    const uint16_t* Kp = prefix_total > 0 ? K_prefix : K;
    const uint16_t* Vp = prefix_total > 0 ? V_prefix : V;
    CUtensorMap tmQ, tmK, tmV, tmKp, tmVp;
    if (!make_map_3d(&tmQ, Q, L_local, Hq, d, 1, kTileM) ||
        !make_map_2d(&tmK, K, L_local, static_cast<int64_t>(Hkv) * d) ||
        !make_map_2d(&tmV, V, L_local, static_cast<int64_t>(Hkv) * d) ||
        !make_map_2d(&tmKp, Kp, static_cast<int64_t>(p.pref_rows), static_cast<int64_t>(Hkv) * d) ||
        !make_map_2d(&tmVp, Vp, static_cast<int64_t>(p.pref_rows), static_cast<int64_t>(Hkv) * d))
        return PULSAR_ERR_CUDA;

    PULSAR_CUDA_OK(cudaMemsetAsync(counter, 0, sizeof(int32_t), stream));

    AttnArgs a{};
    a.mode = kModePhase1;
    a.Hkv = Hkv;
    a.pairs = p.pairs_per_block;
    a.last_len = p.last_len;
    a.pairs_last = p.pairs_last;
    a.n_items = p.n_items;
    a.n_blocks = p.n_blocks;
    a.counter = counter;
    a.n_tokens = static_cast<int>(L_local);
    a.Hq = Hq;
    a.g = Hq / Hkv;
    a.pack = 1;
    a.block_size = block_size;
    a.tiles_per_block = p.tiles_per_block;
    a.prefix_total = prefix_total;
    a.prefix_len = prefix_len_local;
    a.scale_log2 = (softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf(static_cast<float>(d))) * 1.4426950408889634f;
    a.O = O;
    a.LSE = LSE;
    a.status = device_status;
    return d == 128 ? launch_attn<128>(tmQ, tmK, tmV, tmKp, tmVp, a, stream)
                    : launch_attn<64>(tmQ, tmK, tmV, tmKp, tmVp, a, stream);
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
    if (n_splits == 0) n_splits = choose_splits(nq, L, Hq, Hkv, d);
    if (n_splits > 65535 || phase2_split_len(L, n_splits) == 0) return PULSAR_ERR_SHAPE;
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
    if (phase2_quad(nq, Hq / Hkv)) return 4 * (a + b);
    return n_splits == 1 ? 256 : a + b + 256;              // partials and the work counter
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
    const bool quad = !user_parts && phase2_quad(nq, Hq / Hkv);
    const int copies = quad ? 4 : 1;
    po_bytes *= copies;                                        // both stay multiples of 256
    pl_bytes *= copies;
    const bool need_ws = (n_splits > 1 || quad) && !user_parts;
    if (need_ws && (!workspace || workspace_bytes < po_bytes + pl_bytes + (quad ? 0 : 256))) return PULSAR_ERR_WORKSPACE;
    rc = check_device();
    if (rc != PULSAR_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    const int64_t L = static_cast<int64_t>(B) * block_size;
    const int g = Hq / Hkv;
    CUtensorMap tmQ, tmK, tmV;
    if (!make_map_3d(&tmQ, Qq, nq, Hq, d, g, (quad ? 32 : kTileM) / g) ||
        !make_map_2d(&tmK, Kb, L, static_cast<int64_t>(Hkv) * d) ||
        !make_map_2d(&tmV, Vb, L, static_cast<int64_t>(Hkv) * d))
        return PULSAR_ERR_CUDA;

    const bool partial_out = n_splits > 1 || user_parts || quad;
    float* pO = user_parts ? part_O : (need_ws ? static_cast<float*>(workspace) : nullptr);
    float* pL = user_parts ? part_LSE
                           : (need_ws ? reinterpret_cast<float*>(static_cast<char*>(workspace) + po_bytes) : nullptr);

    AttnArgs a{};
    a.mode = kModePhase2;
    a.n_tokens = nq;
    a.Hq = Hq;
    a.g = g;
    a.pack = g;
    a.split_len = static_cast<int>(phase2_split_len(L, n_splits));
    a.kv_len = static_cast<int>(L);
    a.n_ctx_parts = n_splits;
    a.quad = quad ? 1 : 0;
    a.scale_log2 = (softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf(static_cast<float>(d))) * 1.4426950408889634f;
    a.O = O;
    a.LSE = LSE;
    a.part_O = partial_out ? pO : nullptr;
    a.part_LSE = partial_out ? pL : nullptr;
    a.status = device_status;
    const int tokens_per_tile = kTileM / g;
    const int row_tiles = (nq + tokens_per_tile - 1) / tokens_per_tile;
    a.Hkv = Hkv;
    a.single = row_tiles == 1 ? 1 : 0;               // includes every decode shape (quad)
    a.pairs = (row_tiles + 1) / 2;
    a.n_items = a.pairs * Hkv * n_splits;
    if (a.n_items > sm_count() && need_ws && !quad && workspace_bytes >= po_bytes + pl_bytes + 256) {
        // More items than CTAs: hand them out as CTAs become free (the last part is shorter, and the
        // last round would otherwise leave CTAs idle behind the slowest one).  The result of an
        // item does not depend on which CTA computes it.
        a.counter = reinterpret_cast<int32_t*>(static_cast<char*>(workspace) + po_bytes + pl_bytes);
        PULSAR_CUDA_OK(cudaMemsetAsync(a.counter, 0, sizeof(int32_t), stream));
    }
    rc = d == 128 ? launch_attn<128>(tmQ, tmK, tmV, tmK, tmV, a, stream)
                  : launch_attn<64>(tmQ, tmK, tmV, tmK, tmV, a, stream);
    if (rc != PULSAR_OK) return rc;
    if (partial_out)
        return launch_lse_merge(pO, pL, n_splits * copies, static_cast<int64_t>(nq) * Hq, d, O, LSE, stream, true);
    return PULSAR_OK;
}

// =============================================================================================
// Phase 2, generation step (Algorithm 1 lines 11-16): context parts + the generation shard
// =============================================================================================
extern "C" size_t pulsar_phase2_generate_workspace_bytes(int32_t n_new, int32_t B, int32_t block_size, int32_t Hq,
                                                         int32_t Hkv, int32_t d, int32_t n_splits) {
    size_t a, b;
    if (plan_phase2(n_new, B, block_size, Hq, Hkv, d, n_splits, a, b) != PULSAR_OK) return 0;
    // one more part than the context has: the generation shard; four partials per part for decode shapes
    const size_t parts = static_cast<size_t>(n_splits + 1) * (phase2_quad(n_new, Hq / Hkv) ? 4 : 1);
    return round_up(parts * n_new * Hq * d * 4, 256) + round_up(parts * n_new * Hq * 4, 256);
}

extern "C" int32_t pulsar_phase2_generate_step(const uint16_t* Qnew, const uint16_t* Knew, const uint16_t* Vnew,
                                               int32_t n_new, const uint16_t* Kb, const uint16_t* Vb, int32_t B,
                                               int32_t block_size, uint16_t* Kgen, uint16_t* Vgen, int32_t gen_len,
                                               int32_t gen_capacity, int32_t Hq, int32_t Hkv, int32_t d,
                                               float softmax_scale, int32_t n_splits, uint16_t* O, float* LSE,
                                               void* workspace, size_t workspace_bytes, int32_t* device_status,
                                               void* stream_) {
    size_t unused_a, unused_b;
    if (gen_len < 0 || gen_capacity <= 0) return PULSAR_ERR_INVALID_ARG;
    int32_t rc = plan_phase2(n_new, B, block_size, Hq, Hkv, d, n_splits, unused_a, unused_b);
    if (rc != PULSAR_OK) return rc;
    if (static_cast<int64_t>(gen_len) + n_new > gen_capacity) return PULSAR_ERR_SHAPE;
    if (!Qnew || !Knew || !Vnew || !Kb || !Vb || !Kgen || !Vgen || !O || !workspace) return PULSAR_ERR_INVALID_ARG;
    if (!aligned(Qnew, 16) || !aligned(Knew, 16) || !aligned(Vnew, 16) || !aligned(Kb, 16) || !aligned(Vb, 16) ||
        !aligned(Kgen, 16) || !aligned(Vgen, 16) || !aligned(O, 16) || (LSE && !aligned(LSE, 4)) ||
        !aligned(workspace, 256))
        return PULSAR_ERR_ALIGNMENT;
    const int n_parts = n_splits + 1;
    const bool quad = phase2_quad(n_new, Hq / Hkv);
    const int copies = quad ? 4 : 1;
    const size_t po_bytes = round_up(static_cast<size_t>(n_parts) * copies * n_new * Hq * d * 4, 256);
    const size_t pl_bytes = round_up(static_cast<size_t>(n_parts) * copies * n_new * Hq * 4, 256);
    if (workspace_bytes < po_bytes + pl_bytes) return PULSAR_ERR_WORKSPACE;
    rc = check_device();
    if (rc != PULSAR_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    const int64_t L = static_cast<int64_t>(B) * block_size;
    const int g = Hq / Hkv;
    const size_t row_bytes = static_cast<size_t>(Hkv) * d * 2;
    CUtensorMap tmQ, tmK, tmV, tmKg, tmVg;
    if (!make_map_3d(&tmQ, Qnew, n_new, Hq, d, g, (quad ? 32 : kTileM) / g) ||
        !make_map_2d(&tmK, Kb, L, static_cast<int64_t>(Hkv) * d) ||
        !make_map_2d(&tmV, Vb, L, static_cast<int64_t>(Hkv) * d) ||
        // The shard's maps end at its live rows: TMA zero-fills the rest of the last key tile, so
        // whatever the unwritten rows [gen_len + n_new, gen_capacity) hold (NaN patterns of an
        // uninitialised cache included) never reaches the PV product as 0 * NaN.
        !make_map_2d(&tmKg, Kgen, static_cast<int64_t>(gen_len) + n_new, static_cast<int64_t>(Hkv) * d) ||
        !make_map_2d(&tmVg, Vgen, static_cast<int64_t>(gen_len) + n_new, static_cast<int64_t>(Hkv) * d))
        return PULSAR_ERR_CUDA;

    // append KV(q) to the generation shard (Algorithm 1 line 15), then attend
    {
        const int vecs = static_cast<int>(n_new * row_bytes / 16);
        append_kv_kernel<<<(vecs + 255) / 256, 256, 0, stream>>>(
            reinterpret_cast<const uint4*>(Knew), reinterpret_cast<const uint4*>(Vnew),
            reinterpret_cast<uint4*>(reinterpret_cast<char*>(Kgen) + gen_len * row_bytes),
            reinterpret_cast<uint4*>(reinterpret_cast<char*>(Vgen) + gen_len * row_bytes), vecs);
        PULSAR_CUDA_OK(cudaGetLastError());
        count_launch();
    }

    float* pO = static_cast<float*>(workspace);
    float* pL = reinterpret_cast<float*>(static_cast<char*>(workspace) + po_bytes);
    AttnArgs a{};
    a.mode = kModePhase2;
    a.n_tokens = n_new;
    a.Hq = Hq;
    a.g = g;
    a.pack = g;
    a.split_len = static_cast<int>(phase2_split_len(L, n_splits));
    a.kv_len = static_cast<int>(L);
    a.n_ctx_parts = n_splits;
    a.gen_len = gen_len;
    a.gen_total = gen_len + n_new;
    a.quad = quad ? 1 : 0;
    a.scale_log2 = (softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf(static_cast<float>(d))) * 1.4426950408889634f;
    a.O = O;
    a.LSE = LSE;
    a.part_O = pO;
    a.part_LSE = pL;
    a.status = device_status;
    const int tokens_per_tile = kTileM / g;
    const int row_tiles = (n_new + tokens_per_tile - 1) / tokens_per_tile;
    a.Hkv = Hkv;
    a.single = row_tiles == 1 ? 1 : 0;               // includes every decode shape (quad)
    a.pairs = (row_tiles + 1) / 2;
    a.n_items = a.pairs * Hkv * n_parts;
    a.loader_waits = 1;                                // the shard rows are written by the append launch
    rc = d == 128 ? launch_attn<128>(tmQ, tmK, tmV, tmKg, tmVg, a, stream, nullptr, true)
                  : launch_attn<64>(tmQ, tmK, tmV, tmKg, tmVg, a, stream, nullptr, true);
    if (rc != PULSAR_OK) return rc;
    return launch_lse_merge(pO, pL, n_parts * copies, static_cast<int64_t>(n_new) * Hq, d, O, LSE, stream, true);
}

// =============================================================================================
// Causal attention over assembled inputs of different lengths (Algorithm 1 line 8 as the paper
// runs it: every token of Input_i is a query, the keys and values are those of Input_i itself)
// =============================================================================================
extern "C" int32_t pulsar_causal_varlen_attn(const uint16_t* Q, const uint16_t* K, const uint16_t* V,
                                             int64_t total_rows, const int32_t* cu_seqlens_host, int32_t n_seq,
                                             int32_t Hq, int32_t Hkv, int32_t d, float softmax_scale, uint16_t* O,
                                             float* LSE, void* workspace, size_t workspace_bytes,
                                             int32_t* device_status, void* stream_) {
    if (total_rows <= 0 || n_seq <= 0 || Hq <= 0 || Hkv <= 0 || !cu_seqlens_host) return PULSAR_ERR_INVALID_ARG;
    if ((d != 64 && d != 128) || Hq % Hkv != 0 || total_rows >= (1ll << 31) || n_seq > kMaxVarlenSeqs || Hq > 65535)
        return PULSAR_ERR_SHAPE;
    if (cu_seqlens_host[0] != 0 || cu_seqlens_host[n_seq] != total_rows) return PULSAR_ERR_SHAPE;
    for (int j = 0; j < n_seq; ++j)
        if (cu_seqlens_host[j + 1] <= cu_seqlens_host[j]) return PULSAR_ERR_SHAPE;       // empty or descending
    if (!Q || !K || !V || !O || !workspace) return PULSAR_ERR_INVALID_ARG;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) || (LSE && !aligned(LSE, 4)) ||
        !aligned(workspace, 256))
        return PULSAR_ERR_ALIGNMENT;
    if (workspace_bytes < 256) return PULSAR_ERR_WORKSPACE;
    int32_t rc = check_device();
    if (rc != PULSAR_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    VarlenTable vt{};
    vt.n_seq = n_seq;
    for (int j = 0; j <= n_seq; ++j) vt.start[j] = cu_seqlens_host[j];
    int64_t pairs_total = 0;
    for (int k = 0; k < n_seq; ++k) {
        vt.pair_cum[k] = static_cast<int>(pairs_total);
        const int len = vt.start[n_seq - k] - vt.start[n_seq - 1 - k];
        pairs_total += ((len + kTileM - 1) / kTileM + 1) / 2;
    }
    vt.pair_cum[n_seq] = static_cast<int>(pairs_total);
    if (pairs_total * Hq >= (1ll << 31)) return PULSAR_ERR_SHAPE;

    CUtensorMap tmQ, tmK, tmV;
    if (!make_map_3d(&tmQ, Q, total_rows, Hq, d, 1, kTileM) ||
        !make_map_2d(&tmK, K, total_rows, static_cast<int64_t>(Hkv) * d) ||
        !make_map_2d(&tmV, V, total_rows, static_cast<int64_t>(Hkv) * d))
        return PULSAR_ERR_CUDA;

    int32_t* counter = static_cast<int32_t*>(workspace);
    PULSAR_CUDA_OK(cudaMemsetAsync(counter, 0, sizeof(int32_t), stream));

    AttnArgs a{};
    a.mode = kModeVarlen;
    a.n_tokens = static_cast<int>(total_rows);
    a.Hq = Hq;
    a.g = Hq / Hkv;
    a.pack = 1;
    a.Hkv = Hkv;
    a.n_items = static_cast<int>(pairs_total) * Hq;
    a.counter = counter;
    a.scale_log2 = (softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf(static_cast<float>(d))) * 1.4426950408889634f;
    a.O = O;
    a.LSE = LSE;
    a.status = device_status;
    return d == 128 ? launch_attn<128>(tmQ, tmK, tmV, tmK, tmV, a, stream, &vt)
                    : launch_attn<64>(tmQ, tmK, tmV, tmK, tmV, a, stream, &vt);
}

extern "C" int32_t pulsar_retain_block_kv(const uint16_t* K, const uint16_t* V, int64_t total_rows,
                                          const int32_t* cu_seqlens_host, int32_t n_seq, int32_t block_size,
                                          int32_t Hkv, int32_t d, uint16_t* K_ret, uint16_t* V_ret, void* stream) {
    if (total_rows <= 0 || n_seq <= 0 || block_size <= 0 || Hkv <= 0 || d <= 0 || !cu_seqlens_host)
        return PULSAR_ERR_INVALID_ARG;
    if (n_seq > kMaxVarlenSeqs || total_rows >= (1ll << 31) || (static_cast<int64_t>(Hkv) * d * 2) % 16 != 0 ||
        static_cast<int64_t>(n_seq) * block_size >= (1ll << 31))
        return PULSAR_ERR_SHAPE;
    if (cu_seqlens_host[0] != 0 || cu_seqlens_host[n_seq] != total_rows) return PULSAR_ERR_SHAPE;
    RetainTable tab{};
    for (int j = 0; j < n_seq; ++j) {
        if (cu_seqlens_host[j + 1] - cu_seqlens_host[j] < block_size) return PULSAR_ERR_SHAPE;   // shorter than a block
        tab.first[j] = cu_seqlens_host[j + 1] - block_size;
    }
    if (!K || !V || !K_ret || !V_ret) return PULSAR_ERR_INVALID_ARG;
    if (!aligned(K, 16) || !aligned(V, 16) || !aligned(K_ret, 16) || !aligned(V_ret, 16)) return PULSAR_ERR_ALIGNMENT;
    int32_t rc = check_device();
    if (rc != PULSAR_OK) return rc;
    retain_block_kv_kernel<<<n_seq * block_size, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<const uint4*>(K), reinterpret_cast<const uint4*>(V), tab, block_size, Hkv * d * 2 / 16,
        reinterpret_cast<uint4*>(K_ret), reinterpret_cast<uint4*>(V_ret));
    PULSAR_CUDA_OK(cudaGetLastError());
    count_launch();
    return PULSAR_OK;
}
