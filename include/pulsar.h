/*
 * pulsar.h -- C ABI of the B200 (sm_100a) Pulsar Attention context-encoding library.
 *
 * Three operations of the method, one call each, plus the merge on its own:
 *
 *   pulsar_maxidf_select   Max-IDF summary selection      (Section 3.1, Eq. 2-4; Alg. 1 l.3, l.6)
 *   pulsar_phase1_attn     Phase-1 prefix-block attention (Eq. 1 over Input_i of Eq. 4; Alg. 1 l.7-8)
 *   pulsar_phase2_attn     Phase-2 query attention + merge (Section 3.2; Alg. 1 l.12-13; App. H)
 *   pulsar_lse_merge       online-softmax merge alone      (Appendix H, Eq. 12-13)
 *   pulsar_causal_varlen_attn    causal attention over assembled inputs of any lengths (Alg. 1 l.8)
 *   pulsar_phase2_generate_step  one generation step: append KV(q), attend, merge (Alg. 1 l.11-16)
 *
 * Conventions that hold for every call
 * ------------------------------------
 *  - All data pointers are DEVICE pointers unless the comment says "host".  Tensors are
 *    contiguous in the stated layout, 16-byte aligned.  "bf16" is the raw 16-bit bfloat16
 *    pattern (uint16_t here).
 *  - The caller owns all memory.  The library allocates and frees no device memory and keeps
 *    no pointer after the work enqueued on `stream` has finished.  Scratch comes from the
 *    `workspace` argument, whose minimum size the matching *_workspace_bytes function returns
 *    (256-byte aligned base required).  The workspace may be reused by the next call on the
 *    same stream.  The one exception is pulsar_maxidf_select_noalloc, whose scratch is a fixed
 *    array inside the library image (see there).
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls
 *    only enqueue work and never synchronise the host; inputs and outputs must stay alive
 *    until the stream reaches the end of the call.
 *  - The return value is a pulsar_status_t.  Arguments are validated on the host before
 *    anything is launched: a call that returns non-zero has launched nothing.
 *  - Errors that depend on device data (a token id >= vocab_size, a prefix index that is not
 *    before its block, a device-side wait that ran out) are OR-ed into `*device_status`
 *    (device int32, may be NULL; the caller zeroes it and reads it after synchronising).
 *    The kernels never trap: offending elements are skipped or clamped, every wait is bounded.
 *  - Only compute capability 10.0 devices are accepted (PULSAR_ERR_UNSUPPORTED_DEVICE otherwise).
 *    There is no CPU path.
 */
#ifndef PULSAR_H_
#define PULSAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum pulsar_status {
    PULSAR_OK = 0,
    PULSAR_ERR_INVALID_ARG = 1,        /* NULL where data is required, negative size          */
    PULSAR_ERR_SHAPE = 2,              /* shape outside what the kernels cover                */
    PULSAR_ERR_ALIGNMENT = 3,          /* pointer not 16-byte (workspace: 256-byte) aligned   */
    PULSAR_ERR_WORKSPACE = 4,          /* workspace_bytes below the *_workspace_bytes value   */
    PULSAR_ERR_UNSUPPORTED_DEVICE = 5, /* current device is not sm_100                        */
    PULSAR_ERR_CUDA = 6,               /* a CUDA runtime/driver call failed (launch, tensor map) */
    PULSAR_ERR_TIMEOUT = 7,            /* device_status bit: a bounded device wait gave up    */
    PULSAR_ERR_DEVICE_CHECK = 8        /* device_status bit: data-dependent check failed      */
} pulsar_status_t;

/* Bits OR-ed into *device_status by the kernels. */
#define PULSAR_DEV_BAD_TOKEN   0x1 /* token id >= vocab_size (token ignored)                 */
#define PULSAR_DEV_BAD_PREFIX  0x2 /* prefix index outside [0, first row of its block) (row 0 used) */
#define PULSAR_DEV_TIMEOUT     0x4 /* an mbarrier wait exceeded its bound (results invalid)   */
#define PULSAR_DEV_BAD_LENGTH  0x8 /* prefix_len[i] outside [0, prefix_total] (clamped)       */
#define PULSAR_DEV_BAD_POSITION 0x10 /* negative position id (0 used)                          */

/* Static, human-readable name of a status code (host pointer, never NULL). */
const char *pulsar_status_string(int32_t status);

/* Version of this ABI (bumped on any signature change). */
int32_t pulsar_abi_version(void);

/* Number of kernels this library has launched in this process so far (all entry points, all
 * threads).  Bookkeeping for benchmarks; the paper has no counterpart. */
uint64_t pulsar_launch_count(void);

/* Self-test of the bounded device wait that every kernel of the library uses (the paper has no
 * counterpart).  Launches one small kernel that waits on a barrier nothing arrives on; after
 * limit_ns (1 .. 1e9 ns) the wait gives up, ORs PULSAR_DEV_TIMEOUT into *device_status and the
 * kernel ends normally, leaving the context usable.  *device_result (device int32, may be
 * NULL) receives 2 when the wait gave up as designed, 1 if it claimed success. */
int32_t pulsar_wait_selftest(int32_t *device_status, uint64_t limit_ns, int32_t *device_result,
                             void *stream);

/* ------------------------------------------------------------------------------------------
 * Max-IDF summary selection (Section 3.1; Algorithm 1 lines 3 and 6; Appendix C.1, C.5).
 *
 * The L context tokens form B = ceil(L / block_size) logical blocks.  df(t) = number of blocks
 * in which token t occurs; IDF(t) = ln(B / max(df(t),1)) (Eq. 3); each block is cut into
 * C = ceil(block_size / chunk) chunks scored by the largest IDF among their tokens (Eq. 2); the
 * k best chunks of a block, equal scores going to the lower chunk index, listed in positional
 * order, are its summary Sigma_b.  The prefix list is [0..sink-1 | Sigma_0 | ... | Sigma_{B-2}]
 * as global token positions; block i attends to its first prefix_len[i] entries, with
 * prefix_len[0] = 0 and prefix_len[i] = sink + i*k*chunk (Eq. 4, Eq. 14).  Ranking is done on
 * the integer df (IDF is strictly decreasing in df), so the result is exact.
 *
 * Lengths that do not divide (the paper cuts the context "into blocks" and the blocks into
 * chunks of `chunk` tokens and is silent on remainders; this is the reading taken): the last
 * block holds the L - (B-1)*block_size tokens that remain; the last chunk of a block holds the
 * tokens that remain and is scored on those; a block with fewer than k chunks contributes all
 * of them; the sink is the first min(sink, L) tokens.  A summary that includes a short chunk
 * has fewer than k*chunk tokens, so in general prefix_len[i] = sink + the tokens of
 * Sigma_0 .. Sigma_{i-1}; that is Eq. 14's sink + i*k*chunk whenever chunk divides block_size.
 *
 *   token_ids   in  [L] uint32, each < vocab_size
 *   sel_chunks  out [B*k] int32: a block's chunk indices, ascending, then -1 up to k entries
 *   prefix_idx  out [sink + (B-1)*k*chunk] int32; entries past prefix_len[B-1] (and past the
 *               sink when B = 1) are -1
 *   prefix_len  out [B] int32
 *   df_out      out [vocab_size] uint32, or NULL
 *   idf_out     out [vocab_size] float32 (natural log), or NULL
 *
 * Requirements (else PULSAR_ERR_SHAPE): 0 <= k <= C, 0 <= sink <= block_size, B <= 65533,
 * L < 2^31, vocab_size <= 1,800,000 (one block's presence bitmap must fit in shared memory),
 * C <= 32768, and C + B + k + 3 <= 58,112 (the top-k kernel's per-block tables, 4 bytes each,
 * must fit in 227 KB of shared memory).
 * ------------------------------------------------------------------------------------------ */
size_t pulsar_maxidf_select_workspace_bytes(int64_t L, int32_t vocab_size, int32_t block_size,
                                            int32_t chunk, int32_t k, int32_t sink);

int32_t pulsar_maxidf_select(const uint32_t *token_ids, int64_t L, int32_t vocab_size,
                             int32_t block_size, int32_t chunk, int32_t k, int32_t sink,
                             int32_t *sel_chunks, int32_t *prefix_idx, int32_t *prefix_len,
                             uint32_t *df_out, float *idf_out,
                             void *workspace, size_t workspace_bytes,
                             int32_t *device_status, void *stream);

/* ------------------------------------------------------------------------------------------
 * Selection under a chosen chunk score (Appendix C: Eq. 6 TF-IDF, Eq. 7 BM25, Eq. 8 type-token
 * ratio, Eq. 9 Max-IDF).  Blocks, chunks, top-k, tie rule, positional order, prefix list and
 * the first ten arguments' meaning are those of pulsar_maxidf_select; only the score differs:
 *
 *   PULSAR_SCORE_MAX_IDF     max over the chunk's tokens of IDF(t)
 *   PULSAR_SCORE_TF_IDF      (1/|C|) * sum over the chunk's positions of IDF(t_p)
 *   PULSAR_SCORE_BM25        sum over the chunk's distinct tokens of
 *                            ln((B - df + 0.5)/(df + 0.5) + 1) * tf (k1 + 1) / (tf + k1 D),
 *                            k1 = 1.2, b = 0.75, D = (1 - b) + b |C| / mean chunk length (the mean over
 *                            all chunks of the sequence; D = 1 when every chunk has `chunk` tokens),
 *                            tf = occurrences within the chunk
 *   PULSAR_SCORE_TYPE_TOKEN  distinct tokens in the chunk / |C|
 *
 * with IDF(t) = ln(B / max(df(t),1)).  Scores are float64, accumulated left to right over the
 * positions (BM25: over the types in order of first occurrence) with one rounding per add,
 * multiply and divide; chunks whose scores are the same double tie and the lower index wins.
 *
 * Lengths that do not divide are taken as in pulsar_maxidf_select: |C| is the number of tokens a
 * chunk has (the last chunk of a block may be short and is scored on those, as Eq. 6-8 divide by
 * |C|), C = ceil(block_size / chunk) slots per block.
 *
 *   score_out   out [B*C] float64 device, or NULL; -inf for a slot without a chunk
 *
 * Requirements beyond pulsar_maxidf_select's (else PULSAR_ERR_SHAPE): B <= 1024, chunk <= 1024,
 * C <= 4096.  score_mode outside the enum: PULSAR_ERR_INVALID_ARG.
 * ------------------------------------------------------------------------------------------ */
enum {
    PULSAR_SCORE_MAX_IDF = 0,
    PULSAR_SCORE_TF_IDF = 1,
    PULSAR_SCORE_BM25 = 2,
    PULSAR_SCORE_TYPE_TOKEN = 3
};

size_t pulsar_chunk_select_workspace_bytes(int64_t L, int32_t vocab_size, int32_t block_size,
                                           int32_t chunk, int32_t k, int32_t sink, int32_t score_mode);

int32_t pulsar_chunk_select(const uint32_t *token_ids, int64_t L, int32_t vocab_size,
                            int32_t block_size, int32_t chunk, int32_t k, int32_t sink,
                            int32_t score_mode,
                            int32_t *sel_chunks, int32_t *prefix_idx, int32_t *prefix_len,
                            double *score_out,
                            void *workspace, size_t workspace_bytes,
                            int32_t *device_status, void *stream);

/* ------------------------------------------------------------------------------------------
 * Selection for callers that cannot allocate device memory (the paper has no counterpart; this
 * is a packaging variant of pulsar_maxidf_select, same kernels, same results).
 *
 * Some hosts of this library may not call cudaMalloc at all once they are running: a serving
 * process whose device memory is handed out in full to a pool at start-up, a plug-in loaded
 * into an application that owns the GPU's memory budget, code that runs where the CUDA runtime
 * forbids allocation.  Such a caller has nowhere to get the workspace pulsar_maxidf_select asks
 * for.  This entry point takes no workspace: its scratch is a fixed array of
 * pulsar_maxidf_select_noalloc_max_scratch() bytes (4 MiB) that is part of the library image,
 * so every GPU that loads the library holds those bytes until the process exits.  The call
 * itself allocates and frees nothing, on the device or through any library.
 *
 * Arguments, outputs, requirements and status codes are those of pulsar_maxidf_select, minus
 * the workspace pair.  In addition:
 *  - A problem whose workspace (pulsar_maxidf_select_workspace_bytes) exceeds the built-in
 *    scratch is rejected with PULSAR_ERR_WORKSPACE and launches nothing.  The 128K
 *    configuration needs about 0.5 MiB; roughly, B * vocab_size / 8 + 2 * vocab_size +
 *    2 * L / chunk bytes must stay below 4 MiB.
 *  - The first call on each device looks up the device address of the scratch array (one
 *    cudaGetSymbolAddress with that device current).  If the CUDA runtime loads modules lazily,
 *    that look-up is also what makes the runtime place the library's image -- and with it the
 *    4 MiB array -- on the device: the call allocates nothing itself, but the first one can be
 *    the moment those bytes get taken.  Make that first call outside any stream capture; later
 *    calls only enqueue kernels.
 *  - The address is remembered per device for the life of the process.  After a
 *    cudaDeviceReset, or when the device's primary context is destroyed and created again, it
 *    is stale: do not call this entry point again in such a process.
 *  - All calls on a device share the one array.  Nothing in it has to be cleared between calls
 *    (each region is written in full before it is read), but two calls whose kernels may run
 *    at the same time (different streams without an ordering between them) race on it and
 *    corrupt each other's results.  Order them, or use pulsar_maxidf_select with separate
 *    workspaces.
 * ------------------------------------------------------------------------------------------ */
size_t pulsar_maxidf_select_noalloc_max_scratch(void);

int32_t pulsar_maxidf_select_noalloc(const uint32_t *token_ids, int64_t L, int32_t vocab_size,
                                     int32_t block_size, int32_t chunk, int32_t k, int32_t sink,
                                     int32_t *sel_chunks, int32_t *prefix_idx, int32_t *prefix_len,
                                     uint32_t *df_out, float *idf_out,
                                     int32_t *device_status, void *stream);

/* ------------------------------------------------------------------------------------------
 * Phase-1 prefix-block attention (Eq. 1 over the assembled input of Eq. 4; Alg. 1 l.7-8).
 *
 * The L rows form B = ceil(L / block_size) blocks; the last one holds the rows that remain.
 * For block i, row r (global position p = i*block_size + r) and query head h, the keys are
 * rows prefix_idx[0 .. prefix_len[i]) followed by rows i*block_size .. p of K (KV head
 * h / (Hq/Hkv)); the prefix is fully visible, the block causal; a row listed twice counts
 * twice.  O = softmax(q.k * scale) V, LSE = ln sum exp(q.k * scale).  Only block rows are
 * computed; the keys and values of the prefix are read from the given K and V, never
 * produced, so the retained KV of block i (Alg. 1 l.8, Appendix F) is rows
 * [i*block_size, (i+1)*block_size) of K and V themselves; K_ret/V_ret optionally receive a copy.
 * A Star-Attention-style anchor is the same call with prefix_idx = 0..block_size-1 and
 * prefix_len = {0, block_size, block_size, ...}.
 *
 *   Q           in  [L, Hq, d] bf16         K, V   in [L, Hkv, d] bf16
 *   prefix_idx  in  [prefix_total] int32    prefix_len in [B] int32
 *               (entries of prefix_idx that no block's prefix_len reaches are not read)
 *   softmax_scale   <= 0 selects 1/sqrt(d)
 *   O           out [L, Hq, d] bf16         LSE    out [L, Hq] float32 (natural log) or NULL
 *   K_ret,V_ret out [L, Hkv, d] bf16 (block i = rows [i*block_size, ...)) or NULL
 *
 * Requirements (else PULSAR_ERR_SHAPE): d in {64, 128}; Hq % Hkv == 0; B <= 65535;
 * prefix_total >= 0; L < 2^31.  Arithmetic: bf16 operands, fp32 accumulation on the tensor
 * cores, probabilities rounded to bf16 before the PV product, bf16 output.
 * ------------------------------------------------------------------------------------------ */
size_t pulsar_phase1_workspace_bytes(int64_t L, int32_t Hq, int32_t Hkv, int32_t d,
                                     int32_t block_size, int32_t prefix_total);

int32_t pulsar_phase1_attn(const uint16_t *Q, const uint16_t *K, const uint16_t *V,
                           int64_t L, int32_t Hq, int32_t Hkv, int32_t d, int32_t block_size,
                           const int32_t *prefix_idx, const int32_t *prefix_len,
                           int32_t prefix_total, float softmax_scale,
                           uint16_t *O, float *LSE, uint16_t *K_ret, uint16_t *V_ret,
                           void *workspace, size_t workspace_bytes,
                           int32_t *device_status, void *stream);

/* ------------------------------------------------------------------------------------------
 * Phase 1 with the B logical blocks spread over H GPUs by a block-to-host mapping pi (Section 3;
 * Appendix J, Eq. 14-15).  Every GPU holds Q, K, V of its own blocks only, stored back to back
 * in ascending logical order, and runs the selection itself on the replicated token ids (no
 * communication).  The prefix rows a block needs live on other GPUs; they are brought into
 * local memory before the attention kernel, which never reads a peer:
 *
 *   1. pulsar_pack_summary_kv    this GPU's contribution: sink rows and the summary K/V rows of
 *                                each local block, in one fixed-size buffer
 *   2. an all-gather of those buffers (the caller's collective, e.g. NCCL)
 *   3. pulsar_gather_kv_rows     rows of the gathered buffers put into prefix-list order
 *   4. pulsar_phase1_attn_sharded  the Phase-1 attention over the local blocks with that prefix
 *
 * The result equals pulsar_phase1_attn on the whole sequence, row for row.
 *
 * pulsar_pack_summary_kv
 *   K, V        in  [n_local*block_size, Hkv, d] bf16: the local blocks
 *   sel_chunks  in  [n_blocks*k] int32 (pulsar_maxidf_select), for all logical blocks
 *   block_ids   in  [n_local] int32 device: logical index of each local block
 *   K_send, V_send out [sink + n_local*k*chunk, Hkv, d] bf16: rows 0..sink-1 = the first rows of
 *               the first local block (the sink when that is logical block 0, unused otherwise);
 *               then k*chunk rows per local block, chunks ascending
 *   A block id or chunk index out of range sets PULSAR_DEV_BAD_PREFIX.
 *
 * pulsar_gather_kv_rows   K_out[j] = K[idx[j]], V_out[j] = V[idx[j]], j < n_idx
 *   K, V        in  [rows_in, Hkv, d] bf16     idx in [n_idx] int32 device, each in [0, rows_in)
 *   (an index out of range sets PULSAR_DEV_BAD_PREFIX and row 0 is used).  Hkv*d*2 % 16 == 0.
 *
 * pulsar_phase1_attn_sharded
 *   Q           in  [L_local, Hq, d] bf16, K, V in [L_local, Hkv, d] bf16: the local blocks
 *   K_prefix, V_prefix in [prefix_total, Hkv, d] bf16, this GPU's memory, prefix-list order
 *               [sink | Sigma_0 | ... ]; may be NULL when prefix_total == 0
 *   prefix_len_local in [L_local/block_size] int32 device: prefix rows each local block sees
 *               (sink + i*k*chunk for logical block i > 0, 0 for block 0)
 *   O, LSE      out as pulsar_phase1_attn, for the local rows
 *   workspace   256 bytes (the work counter), 256-byte aligned
 * Requirements and status codes otherwise as pulsar_phase1_attn.
 * ------------------------------------------------------------------------------------------ */
int32_t pulsar_pack_summary_kv(const uint16_t *K, const uint16_t *V, int32_t n_local, int32_t block_size,
                               int32_t Hkv, int32_t d, const int32_t *sel_chunks,
                               const int32_t *block_ids, int32_t n_blocks, int32_t chunk, int32_t k,
                               int32_t sink, uint16_t *K_send, uint16_t *V_send,
                               int32_t *device_status, void *stream);

int32_t pulsar_gather_kv_rows(const uint16_t *K, const uint16_t *V, int64_t rows_in, int32_t Hkv,
                              int32_t d, const int32_t *idx, int32_t n_idx,
                              uint16_t *K_out, uint16_t *V_out, int32_t *device_status, void *stream);

int32_t pulsar_phase1_attn_sharded(const uint16_t *Q, const uint16_t *K, const uint16_t *V,
                                   int64_t L_local, int32_t Hq, int32_t Hkv, int32_t d,
                                   int32_t block_size,
                                   const uint16_t *K_prefix, const uint16_t *V_prefix,
                                   int32_t prefix_total, const int32_t *prefix_len_local,
                                   float softmax_scale, uint16_t *O, float *LSE,
                                   void *workspace, size_t workspace_bytes,
                                   int32_t *device_status, void *stream);

/* ------------------------------------------------------------------------------------------
 * Causal attention over assembled inputs (Algorithm 1 line 8 as the paper runs it; Eq. 1, Eq. 4,
 * Appendix F).
 *
 * In the paper every block's assembled input Input_i = [sink | Sigma_0 .. Sigma_{i-1} | B_i]
 * goes through the whole model, so above the first layer the prefix tokens have keys and values
 * of their own per block and are queries as well.  This call is the attention of one layer over
 * such inputs: n_seq independent sequences of different lengths packed back to back, plain
 * causal attention inside each (row p of sequence j sees rows cu_seqlens[j] .. p).  The caller
 * assembles Q, K, V (with pulsar_maxidf_select's prefix list) and afterwards keeps the last
 * block_size key/value rows of each sequence as the retained KV.
 *
 *   Q           in  [total_rows, Hq, d] bf16     K, V in [total_rows, Hkv, d] bf16
 *   cu_seqlens  in  HOST pointer, [n_seq + 1] int32, cu[0] = 0 < cu[1] < ... < cu[n_seq] = total_rows
 *               (read before the call returns)
 *   O           out [total_rows, Hq, d] bf16     LSE out [total_rows, Hq] float32 or NULL
 *   workspace   256 bytes (the work counter)
 *
 * Requirements (else PULSAR_ERR_SHAPE): d in {64,128}; Hq % Hkv == 0; 1 <= n_seq <= 64;
 * total_rows < 2^31.
 * ------------------------------------------------------------------------------------------ */
int32_t pulsar_causal_varlen_attn(const uint16_t *Q, const uint16_t *K, const uint16_t *V,
                                  int64_t total_rows, const int32_t *cu_seqlens /* host */, int32_t n_seq,
                                  int32_t Hq, int32_t Hkv, int32_t d, float softmax_scale,
                                  uint16_t *O, float *LSE,
                                  void *workspace, size_t workspace_bytes,
                                  int32_t *device_status, void *stream);

/* KV discard after the pass over assembled inputs (Section 3.1 "KV discard", Appendix F): the keys
 * and values of the sink and summary tokens are dropped, the last block_size rows of every
 * assembled input -- the block's own -- are kept, so that the retained cache holds every context
 * token exactly once.
 *   K, V        in  [total_rows, Hkv, d] bf16, the inputs packed as for pulsar_causal_varlen_attn
 *   cu_seqlens  in  HOST pointer [n_seq + 1]; every input must be at least block_size rows long
 *   K_ret, V_ret out [n_seq * block_size, Hkv, d] bf16
 * Requirements (else PULSAR_ERR_SHAPE): 1 <= n_seq <= 64, Hkv*d*2 % 16 == 0. */
int32_t pulsar_retain_block_kv(const uint16_t *K, const uint16_t *V, int64_t total_rows,
                               const int32_t *cu_seqlens, int32_t n_seq, int32_t block_size,
                               int32_t Hkv, int32_t d, uint16_t *K_ret, uint16_t *V_ret, void *stream);

/* ------------------------------------------------------------------------------------------
 * Phase-2 query attention over the retained KV of all blocks, merged exactly (Section 3.2;
 * Algorithm 1 lines 12-13; Appendix H).
 *
 * Every query row attends, without mask, to all B*block_size retained keys of its KV head.
 * The KV range is cut into n_splits contiguous parts (each "host" of the paper is a part on
 * this GPU); a split-KV kernel produces per part the normalised output A_j and l_j = ln sum
 * exp(q.k*scale) in fp32, and a merge kernel combines them: l = ln sum_j e^{l_j},
 * O = sum_j e^{l_j - l} A_j, which equals one softmax over the concatenated keys.
 *
 *   Qq          in  [nq, Hq, d] bf16 (a batch of queries is flattened into nq rows)
 *   Kblocks, Vblocks in [B, block_size, Hkv, d] bf16 (the retained rows, i.e. [L, Hkv, d]).
 *               Only the product L = B*block_size matters here (the parts below are the
 *               library's, not the blocks'): the retained KV of a sequence whose last block is
 *               short is passed as B = 1, block_size = L.
 *   n_splits    number of KV parts: 0 = let the library choose, otherwise >= 1.  If n_splits
 *               divides the B*block_size keys, every part has that many keys (n_splits == B
 *               gives the per-block (A_h, l_h) of Algorithm 1 line 12); if not, the parts are
 *               whole 128-key tiles, ceil(tiles / n_splits) each, the last one shorter, and a
 *               count that would leave a part empty is rejected.
 *   O           out [nq, Hq, d] bf16        LSE out [nq, Hq] float32 (natural log), or NULL
 *   part_O      out [n_splits, nq, Hq, d] float32 or NULL (requires n_splits > 0)
 *   part_LSE    out [n_splits, nq, Hq]    float32 or NULL (both or neither)
 *
 *   workspace   pulsar_phase2_workspace_bytes(...) bytes, 256-byte aligned: the partials when the
 *               caller passes none.  Decode shapes (nq * Hq/Hkv <= 32, no caller partials) keep
 *               four partials per part -- each softmax warp works on its own copy of the rows and
 *               a quarter of every key tile -- and therefore need it even with a single part.
 *
 * Requirements (else PULSAR_ERR_SHAPE): d in {64,128}; Hq % Hkv == 0; Hq/Hkv in {1,2,4,8,16};
 * nq >= 1.  pulsar_phase2_choose_splits returns the value used for n_splits == 0.
 * ------------------------------------------------------------------------------------------ */
int32_t pulsar_phase2_choose_splits(int32_t nq, int32_t B, int32_t block_size,
                                    int32_t Hq, int32_t Hkv, int32_t d);

size_t pulsar_phase2_workspace_bytes(int32_t nq, int32_t B, int32_t block_size,
                                     int32_t Hq, int32_t Hkv, int32_t d, int32_t n_splits);

int32_t pulsar_phase2_attn(const uint16_t *Qq, int32_t nq,
                           const uint16_t *Kblocks, const uint16_t *Vblocks,
                           int32_t B, int32_t block_size, int32_t Hq, int32_t Hkv, int32_t d,
                           float softmax_scale, int32_t n_splits,
                           uint16_t *O, float *LSE, float *part_O, float *part_LSE,
                           void *workspace, size_t workspace_bytes,
                           int32_t *device_status, void *stream);

/* ------------------------------------------------------------------------------------------
 * Phase-2 generation step (Algorithm 1 lines 11-16; Section 3.2).
 *
 * The n_new newest tokens (the whole query on the first step, one generated token afterwards)
 * have their keys and values appended to the "designated generation shard" (Alg. 1 l.15) and
 * then attend to (1) all B*block_size retained context keys, without mask, and (2) the
 * generation shard causally: new token u sees shard rows [0, gen_len + u].  The context is cut
 * into n_splits parts as in pulsar_phase2_attn; the generation shard is one more part; all parts
 * are merged exactly through their log-sum-exp (Appendix H), so the result equals one softmax
 * over the concatenation [context | generation shard up to the token].
 *
 *   Qnew        in  [n_new, Hq, d] bf16       Knew, Vnew  in [n_new, Hkv, d] bf16
 *   Kblocks, Vblocks in [B*block_size, Hkv, d] bf16 (retained context KV)
 *   Kgen, Vgen  in/out [gen_capacity, Hkv, d] bf16: rows [0, gen_len) hold the earlier query /
 *               generated tokens; rows [gen_len, gen_len + n_new) are written by this call;
 *               rows from gen_len + n_new on are never read (they may hold anything, NaN included)
 *   n_splits    parts of the context KV: 0 = library's choice, else as in pulsar_phase2_attn
 *   O           out [n_new, Hq, d] bf16       LSE out [n_new, Hq] float32 or NULL
 *
 * Requirements as for pulsar_phase2_attn, plus gen_len >= 0 and gen_len + n_new <= gen_capacity
 * (else PULSAR_ERR_SHAPE).  The workspace (pulsar_phase2_generate_workspace_bytes) is required.
 * The caller advances gen_len by n_new after the call.
 * ------------------------------------------------------------------------------------------ */
size_t pulsar_phase2_generate_workspace_bytes(int32_t n_new, int32_t B, int32_t block_size,
                                              int32_t Hq, int32_t Hkv, int32_t d, int32_t n_splits);

int32_t pulsar_phase2_generate_step(const uint16_t *Qnew, const uint16_t *Knew, const uint16_t *Vnew,
                                    int32_t n_new,
                                    const uint16_t *Kblocks, const uint16_t *Vblocks,
                                    int32_t B, int32_t block_size,
                                    uint16_t *Kgen, uint16_t *Vgen, int32_t gen_len, int32_t gen_capacity,
                                    int32_t Hq, int32_t Hkv, int32_t d, float softmax_scale,
                                    int32_t n_splits, uint16_t *O, float *LSE,
                                    void *workspace, size_t workspace_bytes,
                                    int32_t *device_status, void *stream);

/* ------------------------------------------------------------------------------------------
 * Online-softmax merge (Appendix H, Eq. 12-13), in its order-free closed form:
 *   l = m + ln sum_j e^{l_j - m} (m = max_j l_j),  O = sum_j e^{l_j - l} A_j.
 * A part with l_j = -inf has weight 0.  Also the entry point for merging partials gathered
 * from several GPUs.
 *
 *   part_O   in  [n_parts, rows, d] float32     part_LSE in [n_parts, rows] float32
 *   O        out [rows, d] bf16                 LSE      out [rows] float32, or NULL
 * Requirements: n_parts >= 1, rows >= 0, d % 4 == 0, d <= 1024.
 * ------------------------------------------------------------------------------------------ */
int32_t pulsar_lse_merge(const float *part_O, const float *part_LSE, int32_t n_parts,
                         int64_t rows, int32_t d, uint16_t *O, float *LSE, void *stream);

/* The same merge for partials that are not stored back to back, and optionally with a float32
 * result that can itself be a part of a later merge: the two-level merge of Phase 2 on several
 * GPUs (each GPU merges its own KV parts into one float32 partial, the partials are all-gathered
 * as Appendix H describes, and every GPU merges the gathered set).
 *
 *   part_O   part j starts at part_O + j*part_stride_O floats, [rows, d] float32
 *   part_LSE part j starts at part_LSE + j*part_stride_LSE floats, [rows] float32
 *   O        out [rows, d]: float32 if out_is_f32 != 0 (16-byte aligned), else bf16
 * Requirements as pulsar_lse_merge, plus part_stride_O >= rows*d and a multiple of 4,
 * part_stride_LSE >= rows (else PULSAR_ERR_SHAPE). */
int32_t pulsar_lse_merge_strided(const float *part_O, const float *part_LSE, int32_t n_parts,
                                 int64_t part_stride_O, int64_t part_stride_LSE, int64_t rows,
                                 int32_t d, void *O, int32_t out_is_f32, float *LSE, void *stream);

/* The merge fused with the exchange that precedes it on several GPUs (Appendix H): instead of
 * all-gathering every GPU's partial and merging all rows everywhere, GPU r merges only rows
 * [row_begin, row_begin + rows) and reads that slice of every GPU's partial in place, through
 * peer-mapped addresses, while it merges.  Each GPU then holds 1/H of the merged rows (the caller
 * gathers the bf16 results if every GPU needs them all): H times fewer bytes cross NVLink than
 * with the all-gather of partials.
 *
 *   part_bases  HOST array [n_parts] of DEVICE addresses (this GPU's own memory or peer-mapped
 *               memory of other GPUs), each a buffer [rows_total*d float32 outputs | rows_total
 *               float32 LSE]; n_parts <= 64.  The caller orders the launch after the writers of
 *               those buffers (a barrier across the GPUs) and keeps them unchanged until it ends.
 *   O           out [rows, d] (float32 if out_is_f32, else bf16), LSE out [rows] or NULL: the slice
 * Only plain loads touch the part buffers (no TMA).  Requirements as
 * pulsar_lse_merge_strided; row_begin + rows <= rows_total. */
int32_t pulsar_lse_merge_peers(const float *const *part_bases, int32_t n_parts, int64_t rows_total,
                               int64_t row_begin, int64_t rows, int32_t d,
                               void *O, int32_t out_is_f32, float *LSE, void *stream);

/* ------------------------------------------------------------------------------------------
 * Position ids of the assembled Phase-1 inputs and rotary embedding (Appendix E).
 *
 * pulsar_assemble_positions: Input_i = [first prefix_len[i] entries of the prefix list | block i]
 * (Eq. 4), the B inputs stored back to back (the layout pulsar_causal_varlen_attn takes).
 *   PULSAR_POS_SPARSE      (the paper's default) every token keeps its global position: a prefix
 *                          entry its prefix_idx value, row r of block i the position i*block_size+r
 *   PULSAR_POS_CONTIGUOUS  each input is renumbered 0 .. n_i - 1
 *   pos_out  out [sum_i (prefix_len[i] + block_size)] int32 device; writes beyond pos_capacity
 *            entries are dropped -- which is also how a sequence that ends inside its last block is
 *            given: pos_capacity = sum_i prefix_len[i] + L, the last input then ends with the
 *            sequence.  A prefix_len outside [0, prefix_total] sets PULSAR_DEV_BAD_LENGTH.
 *
 * pulsar_rope_apply: rotary embedding with explicit position ids, rotate-half pairing (element j
 * with element j + d/2), angle = position * theta^(-2j/d):
 *   y[j] = x[j] cos - x[j+d/2] sin,   y[j+d/2] = x[j+d/2] cos + x[j] sin.
 *   X in, Y out [rows, H, d] bf16 device (Y may be X); positions [rows] int32 device, >= 0 (a
 *   negative id sets PULSAR_DEV_BAD_POSITION and counts as 0).  The angle is formed in float64
 *   and reduced before the float32 sine and cosine, products in float32, result rounded to bf16.
 *   Requirements: d % 16 == 0, d <= 256 (else PULSAR_ERR_SHAPE); theta > 0.
 * ------------------------------------------------------------------------------------------ */
enum { PULSAR_POS_SPARSE = 0, PULSAR_POS_CONTIGUOUS = 1 };

int32_t pulsar_assemble_positions(const int32_t *prefix_idx, const int32_t *prefix_len,
                                  int32_t prefix_total, int32_t n_blocks, int32_t block_size,
                                  int32_t mode, int32_t *pos_out, int64_t pos_capacity,
                                  int32_t *device_status, void *stream);

int32_t pulsar_rope_apply(const uint16_t *X, uint16_t *Y, int64_t rows, int32_t H, int32_t d,
                          const int32_t *positions, double theta,
                          int32_t *device_status, void *stream);

/* The same embedding for a query and a key tensor of the same rows in one launch (the rows' sines and
 * cosines are formed once): Q [rows, Hq, d] -> Q_out, K [rows, Hkv, d] -> K_out (each may be in place). */
int32_t pulsar_rope_apply_qk(const uint16_t *Q, uint16_t *Q_out, int32_t Hq,
                             const uint16_t *K, uint16_t *K_out, int32_t Hkv,
                             int64_t rows, int32_t d, const int32_t *positions, double theta,
                             int32_t *device_status, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* PULSAR_H_ */
