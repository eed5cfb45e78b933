/*
 * moda.h -- C ABI of the B200 (sm_100a) Mixture-of-Depths Attention (MoDA) operator.
 *
 * The operator (paper Sec. 2.2, "Mixture-of-Depths Attention"; forward schedule in
 * Alg. 1): for every batch b, head h and position t, the query q_t attends, under ONE
 * softmax, to
 *     - the sequence keys/values of its own layer at positions 0..t (causal mask of
 *       Eq. 2, inclusive of t), and
 *     - the l depth keys/values stored for the SAME position t by the preceding layers
 *       (slots i = 0..l-1; always visible).
 *   s_j = scale <q_t,k_j>, u_i = scale <q_t,kd_i[t]>,
 *   LSE_t = ln( sum_j e^{s_j} + sum_i e^{u_i} ),
 *   O_t = sum_j e^{s_j-LSE_t} v_j + sum_i e^{u_i-LSE_t} vd_i[t].
 * With l = 0 the operator is plain causal attention.
 *
 * Conventions for every call
 *   - All tensor pointers are DEVICE pointers, 16-byte aligned, owned by the caller; the
 *     library allocates no device memory and keeps no per-call state.
 *   - bf16 = IEEE bfloat16 bits.  Q, K, V, O, dO, dQ, dK, dV are contiguous [B][T][H][d].
 *   - `stream` is a cudaStream_t passed as void*.  Calls enqueue work and return; they
 *     never synchronise.  The current CUDA device must be the one that owns the buffers
 *     and must be an sm_100 part.
 *   - Return value: MODA_OK or a negative MODA_ERR_* code.  When an error is returned
 *     nothing has been launched.  No C++ exception crosses the boundary, nothing prints.
 *   - Supported shapes: B, T, H >= 1; d in {64, 128}; 0 <= l <= MODA_MAX_DEPTH.
 *     T need not be a multiple of the 128-row tile.
 *
 * Depth-KV cache layout (chosen so that a warp whose lanes own consecutive query rows
 * reads 512 contiguous bytes per load, and one (slot, b, h, tile, K|V) block is one
 * contiguous 128*d*2-byte run that a bulk copy can move):
 *
 *     cache[slot][b][h][tile][kv][chunk][row][8]      (bf16)
 *       slot  : depth slot 0..l_max-1 (layer index of the K, V that were appended)
 *       tile  : position / 128, 0..ceil(T/128)-1        row : position % 128
 *       kv    : 0 = key, 1 = value                      chunk : feature / 8, 0..d/8-1
 *     rows of the last tile beyond T are zero.  One slot spans
 *     moda_depth_cache_bytes(B,T,H,d,1) bytes, so the layer-l call simply reads the first
 *     l slots of a buffer that grows by one slot per layer ("write" step of Sec. 2.2).
 */
#ifndef MODA_H
#define MODA_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Most depth slots per position.  The paper's models use up to 36 layers and its kernel table up to
 * L = 256; the forward handles the slots in groups of 32 (an online softmax over the groups). */
#define MODA_MAX_DEPTH 256

#define MODA_OK 0
#define MODA_ERR_NULL_POINTER (-1)    /* a required pointer is null */
#define MODA_ERR_MISALIGNED (-2)      /* a tensor pointer is not 16-byte aligned */
#define MODA_ERR_BAD_SHAPE (-3)       /* B, T or H < 1, or a size product overflows */
#define MODA_ERR_BAD_HEAD_DIM (-4)    /* d not in {64, 128} */
#define MODA_ERR_BAD_DEPTH (-5)       /* l outside [0, MODA_MAX_DEPTH] */
#define MODA_ERR_BAD_SLOT (-6)        /* slot outside [0, MODA_MAX_DEPTH) */
#define MODA_ERR_WORKSPACE (-7)       /* workspace null or smaller than required */
#define MODA_ERR_DEVICE (-8)          /* current device is not sm_100 */
#define MODA_ERR_CUDA (-9)            /* a CUDA runtime/driver call failed (see moda_last_cuda_error) */
#define MODA_ERR_DEVICE_TIMEOUT (-10) /* an earlier kernel gave up a bounded wait (see moda_last_status) */
#define MODA_ERR_SCRATCH_LIMIT (-11)  /* problem needs more built-in scratch than moda_attn_bwd_static_scratch holds */
#define MODA_ERR_BAD_GROUP (-12)      /* H_kv does not divide H, or an unsupported number of query heads per group */
#define MODA_ERR_BAD_SCALE (-13)      /* the softmax scale is not finite or below 1e-20 (zero and negative scales are not served) */
#define MODA_MAX_GROUP 32             /* supported group sizes G = H / H_kv: 1 to 8, 16 and 32 */

/* Library version: major * 10000 + minor * 100 + patch. */
int moda_version(void);

/* Static, human-readable text for a MODA_* code. */
const char* moda_strerror(int code);

/* cudaError_t value of the last failing CUDA call seen by this thread (0 if none). */
int moda_last_cuda_error(void);

/*
 * Reads (and optionally clears) the device status word.  Every wait inside the kernels
 * is bounded; a wait that runs out stores (site << 8) | 1 here and the kernel tears
 * down normally, leaving its outputs undefined.  0 means no kernel has reported a
 * problem.  This call synchronises the device.  Returns the status word (>= 0) or a
 * negative MODA_ERR_CUDA.
 *
 * The same code is also written to four bytes of pinned host memory that the library maps
 * into the device on its first launching call on that device (the only memory the library
 * ever allocates: host memory, once per device; make that first call before any stream
 * capture).  Every launching entry point looks at those bytes first, without synchronising:
 * once a kernel has given up a wait, later calls on that device return
 * MODA_ERR_DEVICE_TIMEOUT and launch nothing until moda_last_status(1) has cleared the word.
 * (Kernels that were already queued behind the failed one exit at once and leave their
 * outputs undefined too.)
 */
int moda_last_status(int clear);

/*
 * Self-test of the bounded-wait machinery.  Launches one tiny kernel (one CTA; no TMA, no
 * tensor memory) whose single thread waits on an mbarrier that nobody ever arrives at, with
 * a limit of about 1 ms instead of the production kernels' 1 s.  The wait runs out, the
 * kernel records MODA_SELFTEST_WAIT_STATUS in the status word and returns normally; the GPU
 * context stays healthy.  Afterwards moda_last_status reports that value and launching
 * entry points return MODA_ERR_DEVICE_TIMEOUT until it is cleared.  (No counterpart in the
 * paper: it exercises this library's failure reporting.)
 */
#define MODA_SELFTEST_WAIT_SITE 255
#define MODA_SELFTEST_WAIT_STATUS ((MODA_SELFTEST_WAIT_SITE << 8) | 1)
int moda_selftest_wait_timeout(void* stream);

/* Bytes of a depth-KV cache (or depth-gradient buffer) holding l_max slots. 0 on bad arguments. */
size_t moda_depth_cache_bytes(int B, int T, int H, int d, int l_max);

/*
 * "Write" step of Sec. 2.2: store one layer's keys and values, K_i and V_i (bf16
 * [B][T][H][d]), into slot `slot` of `cache` in the layout above (tail rows zeroed).
 */
int moda_depth_cache_append(void* cache, int B, int T, int H, int d, int slot,
                            const void* K_i, const void* V_i, void* stream);

/* Inverse of append: copy slot `slot` of `cache` back to [B][T][H][d] tensors (either output may be null). */
int moda_depth_cache_unpack(const void* cache, int B, int T, int H, int d, int slot,
                            void* K_i, void* V_i, void* stream);

/*
 * Forward (Sec. 2.2 definition; Alg. 1 computes the same values with an online
 * softmax).  depth_kv holds at least l slots in the cache layout (may be null when
 * l == 0).  Writes O (bf16 [B][T][H][d]) and LSE (fp32 [B][H][T], natural log, taken over
 * the union of sequence and depth keys).  bf16 inputs, fp32 accumulation and softmax.
 * `scale` (every attention call): finite and >= 1e-20; otherwise MODA_ERR_BAD_SCALE.
 */
int moda_attn_fwd(const void* Q, const void* K, const void* V, const void* depth_kv,
                  int B, int T, int H, int d, int l, float scale,
                  void* O, float* LSE, void* stream);

/*
 * Forward with the depth stream's "write" step fused in (Sec. 2.2: after attending, a layer appends
 * its own K, V to the depth stream for the layers above it).  Computes exactly what
 * moda_attn_fwd_gqa computes and, in the same launch, stores K and V (bf16 [B][T][H_kv][d]) into slot
 * `append_slot` of `append_cache` in the cache layout, bit for bit what moda_depth_cache_append(
 * append_cache, B, T, H_kv, d, append_slot, K, V) would store: the depth warps of every CTA copy the
 * K and V rows of the CTA's own positions (which its key loop loads anyway) once they have read the
 * cache, so the separate pass over K and V is gone.  `append_cache` may be the buffer `depth_kv` points to (one
 * growing cache per stack, the layer-l call reads slots < l and writes slot l).  Writing a slot that
 * the same call reads (append_cache == depth_kv and append_slot < l) is allowed with one key/value head
 * per query head (H_kv == H): every position's new K, V replace that slot's old ones after the position's
 * own tile has been attended to with the old ones, which is what a fixed-size slot buffer needs (the
 * bounded depth-KV slots of the paper's Discussion: the caller picks the slot to evict, e.g. the oldest
 * for a sliding window; the order of the slots does not matter to the operator).  With grouped heads it
 * is MODA_ERR_BAD_SLOT (the heads of a group share the blocks).  A backward pass over such a stack needs
 * the slots as they were at each layer's forward: the caller's to keep.
 * Other arguments, validation and errors as for moda_attn_fwd_gqa.
 */
int moda_attn_fwd_append(const void* Q, const void* K, const void* V, const void* depth_kv,
                         int B, int T, int H, int H_kv, int d, int l, float scale,
                         void* O, float* LSE, void* append_cache, int append_slot, void* stream);

/*
 * Bytes of scratch moda_attn_bwd needs: fp32 row terms D_t = <dO_t, O_t> ([B][H][T]) and an fp32
 * accumulator for dQ (B * H * ceil(T/128) * 128 * d values; 4 bytes per dQ element).  Enough for
 * every stage mask of moda_attn_bwd_stages.
 */
size_t moda_bwd_workspace_bytes(int B, int T, int H, int d, int l);

/*
 * Backward of the definition above (the paper prints no backward pass; it is the
 * derivative of Sec. 2.2's operator).  Inputs as for the forward call plus O, LSE as
 * written by it and the upstream gradient dO.  Writes dQ, dK, dV (bf16 [B][T][H][d]) and,
 * when l > 0, slots 0..l-1 of d_depth_kv (bf16, cache layout: kv = 0 holds dKd, kv = 1
 * holds dVd; tail rows zero).  `workspace` is caller-owned scratch of at least
 * moda_bwd_workspace_bytes() bytes; its contents need not be preserved between calls.
 *
 * Three launches.  (1) Everything local to a query row: D_t, the depth gradients dKd_i, dVd_i
 * and the depth share of dQ, which starts the fp32 dQ accumulator.  (2) The sequence part, one
 * CTA per key tile: S and dP are formed once, P = exp(S - LSE) is evaluated once per score, dK
 * and dV accumulate on chip and every dQ tile is ADDED to the accumulator with floating-point
 * atomics in global memory.  (3) dQ = bf16(scale * accumulator).  dK, dV and the depth gradients
 * are bit-reproducible; the last bits of dQ depend on the order in which the CTAs of (2) reach a
 * query tile.  Pass MODA_BWD_DETERMINISTIC to moda_attn_bwd_stages for reproducible bits.
 */
int moda_attn_bwd(const void* Q, const void* K, const void* V, const void* depth_kv,
                  const void* O, const void* dO, const float* LSE,
                  int B, int T, int H, int d, int l, float scale,
                  void* dQ, void* dK, void* dV, void* d_depth_kv,
                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * moda_attn_bwd is three launches; this entry point runs a subset of them so that each can
 * be timed or profiled on its own.  `stages` is a bit mask of the launches in the order above:
 *     MODA_BWD_STAGE_ROWS      (1) row terms, depth gradients, start of the dQ accumulator
 *     MODA_BWD_STAGE_SEQ       (2) dK, dV and the dQ tiles (reads D_t, adds to the accumulator)
 *     MODA_BWD_STAGE_FINISH    (3) dQ from the accumulator
 * moda_attn_bwd(...) is moda_attn_bwd_stages(..., MODA_BWD_ALL_STAGES, stream).
 * MODA_BWD_DETERMINISTIC selects the split form of the backward instead: no floating-point
 * atomics, every output bit-reproducible, at the price of seven contractions for five and two
 * evaluations of every exp (measurably slower; its only scratch is D_t).  Its three launches
 * take the same three bits, under their older names:
 *     MODA_BWD_STAGE_ROWTERMS  D_t = <dO_t, O_t> for every row, into `workspace`
 *     MODA_BWD_STAGE_DQ        dQ and the depth gradients (reads D_t from `workspace`)
 *     MODA_BWD_STAGE_DKDV      dK and dV                  (reads D_t from `workspace`)
 * Grouped-query calls whose depth gradients are formed from per-row factors (see
 * moda_attn_bwd_gqa) always take the split form.
 * One more bit changes how the depth gradients are written:
 *     MODA_BWD_ACCUMULATE_DEPTH  slots [0, l) of d_depth_kv are ADDED TO (bf16 additions,
 *                                one per element per call, so the result does not depend on
 *                                scheduling) instead of overwritten.  In a stack of layers
 *                                K_i, V_i are depth keys of every later layer (Sec. 2.2,
 *                                the depth stream's write step), so one gradient cache,
 *                                zeroed once by the caller, collects d(loss)/d(slot i)
 *                                over the backward calls of all those layers.
 * All arguments are validated as for moda_attn_bwd whatever the mask; a mask with none of the
 * three stage bits, or with bits above MODA_BWD_DETERMINISTIC, is MODA_ERR_BAD_SHAPE.
 */
#define MODA_BWD_STAGE_ROWTERMS 1
#define MODA_BWD_STAGE_DQ 2
#define MODA_BWD_STAGE_DKDV 4
#define MODA_BWD_STAGE_ROWS 1
#define MODA_BWD_STAGE_SEQ 2
#define MODA_BWD_STAGE_FINISH 4
#define MODA_BWD_ALL_STAGES 7
#define MODA_BWD_ACCUMULATE_DEPTH 8
#define MODA_BWD_DETERMINISTIC 16
int moda_attn_bwd_stages(const void* Q, const void* K, const void* V, const void* depth_kv,
                         const void* O, const void* dO, const float* LSE,
                         int B, int T, int H, int d, int l, float scale,
                         void* dQ, void* dK, void* dV, void* d_depth_kv,
                         void* workspace, size_t workspace_bytes, int stages, void* stream);

/*
 * Grouped-query form (Sec. 3, "Group-aware depth KV calculation"; the paper's models use
 * grouped-query attention).  H query heads share H_kv = H / G key/value heads: query head h
 * uses key/value head h / G, i.e. the G heads of a group are adjacent, which is the paper's
 * flattened query row i_q = t G + g with base time floor(i_q / G) = t; a row sees the sequence
 * keys up to its base time and the depth keys stored at its base time.
 *     Q, O, dO, dQ : bf16 [B][T][H][d]          K, V, dK, dV : bf16 [B][T][H_kv][d]
 *     depth_kv, d_depth_kv : cache layout with H_kv heads (moda_depth_cache_bytes(B, T, H_kv, d, l))
 *     LSE : fp32 [B][H][T]                      workspace : moda_bwd_workspace_bytes_gqa(B, T, H, H_kv, d, l)
 * dK, dV and the depth gradients are the sums over the G query heads of a group, taken on chip in a
 * fixed order (bit-reproducible; dQ goes through the fp32 accumulator of the fused form, see
 * moda_attn_bwd).  With G > 1 the backward runs its depth part as a separate kernel that treats
 * the heads of a group as the rows of one small tensor-core product per position (probabilities
 * and their gradients rounded to bf16 for that product, fp32 accumulation, as in the sequence
 * part), and for large groups with many slots the forward does the same; up to 16 heads of a group
 * fill one product, 32 heads run as two groups of 16 whose depth
 * gradients are added one after the other in bf16.  The choice depends only on (d, G, l).  With
 * MODA_BWD_DETERMINISTIC (moda_attn_bwd_gqa_stages) the depth part stays row-local: the workspace then
 * holds two fp32 factors per (row, slot, query head), from which a second kernel forms the depth
 * gradients (fp32 sums over the heads in a fixed order) without reading the depth cache again.  H_kv must divide H
 * and G = H / H_kv must be 1 to 8, 16 or 32 (MODA_ERR_BAD_GROUP otherwise); H_kv == H is exactly
 * moda_attn_fwd / moda_attn_bwd.  Everything else (validation, streams, ownership, errors) is
 * as for those calls.
 */
int moda_attn_fwd_gqa(const void* Q, const void* K, const void* V, const void* depth_kv,
                      int B, int T, int H, int H_kv, int d, int l, float scale,
                      void* O, float* LSE, void* stream);
size_t moda_bwd_workspace_bytes_gqa(int B, int T, int H, int H_kv, int d, int l);
int moda_attn_bwd_gqa(const void* Q, const void* K, const void* V, const void* depth_kv,
                      const void* O, const void* dO, const float* LSE,
                      int B, int T, int H, int H_kv, int d, int l, float scale,
                      void* dQ, void* dK, void* dV, void* d_depth_kv,
                      void* workspace, size_t workspace_bytes, void* stream);
int moda_attn_bwd_gqa_stages(const void* Q, const void* K, const void* V, const void* depth_kv,
                             const void* O, const void* dO, const float* LSE,
                             int B, int T, int H, int H_kv, int d, int l, float scale,
                             void* dQ, void* dK, void* dV, void* d_depth_kv,
                             void* workspace, size_t workspace_bytes, int stages, void* stream);

/*
 * Prefill with a cache (T_q <= T_kv; Table 1's prefilling rows): the T_q newest positions of each
 * sequence attend to the T_kv keys that the layer caches (the T_kv - T_q earlier ones and their own,
 * appended by the caller beforehand) and to the depth pairs of their own positions.  Query row i
 * sits at key position i + (T_kv - T_q); the causal mask is taken at that position.  Forward only.
 *     Q, O     : bf16 [B][T_q][H][d]            K, V : bf16 [B][T_kv][H_kv][d]
 *     depth_kv : cache layout over the T_q positions (moda_depth_cache_bytes(B, T_q, H_kv, d, l))
 *     LSE      : fp32 [B][H][T_q]
 * T_kv == T_q is exactly moda_attn_fwd_gqa; T_kv < T_q is MODA_ERR_BAD_SHAPE.  Any T_kv - T_q is
 * allowed (it need not be a multiple of the 128-row tile).  Same kernels, validation, asynchrony
 * and error codes as moda_attn_fwd_gqa.
 */
int moda_attn_fwd_prefill(const void* Q, const void* K, const void* V, const void* depth_kv,
                          int B, int T_q, int T_kv, int H, int H_kv, int d, int l, float scale,
                          void* O, float* LSE, void* stream);

/*
 * Decode step (T_q = 1; Table 1, "decoding cache" and "decoding FLOPs" rows): the newest token of
 * each of B sequences attends, under one softmax, to the T_kv keys of this layer's KV cache (its
 * own key included: the caller appends before the call) and to its own l depth key/value pairs,
 * the 2 l H_k d values that the decoding cache holds per token.  Forward only.
 *     q, O            : bf16 [B][H][d]
 *     K, V            : bf16 [B][T_cap][H_kv][d]; positions [0, T_kv) are read, T_kv <= T_cap
 *     depth_kv_token  : bf16 [l][B][H_kv][2][d]: slot i holds the key row, then the value row, that
 *                       layer i wrote for this token (may be NULL when l == 0)
 *     LSE             : fp32 [B][H], natural log over the T_kv + l keys
 *     workspace       : at least moda_decode_workspace_bytes(B, H, d) bytes, 16-byte aligned; it
 *                       holds per-split partial softmax states and is overwritten
 * Query head h uses key/value head h / G with G = H / H_kv in 1..8, 16 or 32 (MODA_ERR_BAD_GROUP
 * otherwise; groups of 16 or 32 heads run as two or four groups of 8 that read the same K, V head).
 * Two launches on `stream`: a kernel that streams the KV cache once per key/value head (the key
 * range is split over enough CTAs to fill the device) and a merge kernel that adds the depth pairs.
 * All pointers are device pointers owned by the caller; validation, asynchrony and error codes are
 * as for moda_attn_fwd.  The reduction order depends only on (B, H_kv, T_kv) and the device's SM
 * count, so results are bit-reproducible on one device type.
 */
size_t moda_decode_workspace_bytes(int B, int H, int d);
int moda_attn_decode(const void* q, const void* K, const void* V, const void* depth_kv_token,
                     int B, int T_kv, int T_cap, int H, int H_kv, int d, int l, float scale,
                     void* O, float* LSE, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The decode step for a serving batch: sequences of different lengths, and a paged KV cache.
 * (Beyond the paper, which states the decode step's cache size and FLOPs only; same operator per
 * sequence as moda_attn_decode.)
 *
 * moda_attn_decode_varlen: as moda_attn_decode, but sequence b has seq_lens[b] cached positions
 *     (device int32 [B], 4-byte aligned, each in [1, max_seq_len]; values outside are clamped);
 *     max_seq_len <= T_cap sizes the split of the key range.
 * moda_attn_decode_paged: K and V live in pages,
 *     K_pages, V_pages : bf16 [num_pages][page_size][H_kv][d], page_size a multiple of 64
 *     block_table      : device int32 [B][max_blocks_per_seq]; entry j of row b is the page that holds
 *                        positions [j page_size, (j + 1) page_size) of sequence b; entries past the
 *                        sequence's last block are not read; every entry read must be in [0, num_pages)
 *     seq_lens         : device int32 [B] as above; max_blocks_per_seq * page_size >= max_seq_len
 * Everything else (q, depth_kv_token, O, LSE, workspace, groups, validation, launches) is as for
 * moda_attn_decode.  Positions of a page past the sequence's length may hold anything.
 */
int moda_attn_decode_varlen(const void* q, const void* K, const void* V, const int* seq_lens,
                            const void* depth_kv_token,
                            int B, int max_seq_len, int T_cap, int H, int H_kv, int d, int l, float scale,
                            void* O, float* LSE, void* workspace, size_t workspace_bytes, void* stream);
int moda_attn_decode_paged(const void* q, const void* K_pages, const void* V_pages,
                           const int* block_table, const int* seq_lens, const void* depth_kv_token,
                           int B, int max_seq_len, int page_size, int num_pages, int max_blocks_per_seq,
                           int H, int H_kv, int d, int l, float scale,
                           void* O, float* LSE, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Backward pass for callers that have no scratch buffer to give.  (The paper has no
 * counterpart: this is a deployment convenience of this library, not part of the method.)
 *
 * moda_attn_bwd needs a caller-owned workspace.  Some callers cannot
 * provide one: a plug-in that is only handed its input and output tensors by a host framework,
 * or a serving process that sized all of its device memory at start-up and is not allowed to call
 * cudaMalloc afterwards (the call synchronises the whole device and can fail once memory is
 * fully committed).  This variant computes what moda_attn_bwd_stages computes with
 * MODA_BWD_DETERMINISTIC (the split form of the backward, whose only scratch is the per-row
 * terms D_t), with the same kernels, but keeps D_t in an array that is compiled into the library image
 * (MODA_STATIC_SCRATCH_ROWS fp32 values = 4 MiB, resident on every GPU that loads the library
 * until the process exits).  It calls no cudaMalloc, cudaFree or any other allocating routine.
 *
 *   - Limit: B * H * T <= MODA_STATIC_SCRATCH_ROWS, otherwise MODA_ERR_SCRATCH_LIMIT is
 *     returned and nothing is launched.  Other arguments and errors as for moda_attn_bwd.
 *   - The first call on each device looks up the device address of the built-in array (with
 *     that device current) and remembers it; make that first call before starting any stream
 *     capture.  Later calls on the device only launch kernels.
 *   - Every call on a device uses the same array, and it keeps whatever the previous call left
 *     there.  Nothing in it has to start at zero: the first launch of each call overwrites every
 *     row term the later launches read.  Two calls whose kernels may overlap on the GPU (different
 *     streams, no ordering between them) race on the array and give undefined gradients; order
 *     them, or use moda_attn_bwd with separate workspaces.
 */
#define MODA_STATIC_SCRATCH_ROWS (1 << 20)
int moda_attn_bwd_static_scratch(const void* Q, const void* K, const void* V, const void* depth_kv,
                                 const void* O, const void* dO, const float* LSE,
                                 int B, int T, int H, int d, int l, float scale,
                                 void* dQ, void* dK, void* dV, void* d_depth_kv, void* stream);

/*
 * moda_attn_fwd_e4m3 that also writes the layer's own K, V as slot `append_slot` of an e4m3 cache
 * (the write step of Sec. 2.2 fused into the forward, as moda_attn_fwd_append does for a bf16
 * cache).  The slot receives byte for byte what moda_depth_cache_append_e4m3(append_cache_e4m3, ..., append_slot, K, V)
 * stores.  Rules for writing a slot that the call also reads as in moda_attn_fwd_append.  One launch for T >= 32768; on
 * shorter sequences the quantiser runs as a second launch behind the forward (cheaper there), with the same result.
 */
int moda_attn_fwd_append_e4m3(const void* Q, const void* K, const void* V, const void* depth_kv_e4m3,
                              int B, int T, int H, int H_kv, int d, int l, float scale,
                              void* O, float* LSE, void* append_cache_e4m3, int append_slot, void* stream);

/*
 * ---- Depth cache in e4m3 with one scale per row ----
 *
 * The paper's Discussion names the growing depth-KV cache as the cost to cut next and gives no
 * algorithm.  This library's reading: a slot may be kept in 8 bits per feature.  For every (slot,
 * b, h, position, K or V) row x of d features
 *
 *     scale = max|x| / 448   (1 when the row is all zero),   code_j = e4m3(x_j / scale)
 *
 * with the maximum, the two divisions and the round-to-nearest-even, saturating conversion to e4m3
 * (4 exponent bits, 3 mantissa bits, largest finite value 448) all in fp32.  The operator then sees the
 * keys and values  scale * code_j  (taken as real numbers: the kernels keep the product in fp32, it is never
 * rounded to bf16).  Relative to the bf16 cache a slot shrinks from 4 d to 2 d + 8 bytes per (position, head).
 *
 * Layout: cache8[slot][b][h][tile][kv] = { codes[chunk = d/16][row 128][16 bytes], scales[row 128] fp32 },
 * one contiguous block of 128 d + 512 bytes; rows of a ragged last tile hold code 0, scale 1.
 *
 * moda_depth_cache_e4m3_bytes   bytes of a cache of l_max slots (0 for an unsupported shape).
 * moda_depth_cache_append_e4m3  quantises K_i, V_i (bf16 [B][T][H][d], device) into slot `slot`.
 * moda_attn_fwd_e4m3            moda_attn_fwd_gqa with the depth slots read from such a cache.
 * moda_attn_bwd_e4m3            moda_attn_bwd (one key/value head per query head; the fused form, with its
 *                               workspace of moda_bwd_workspace_bytes) with the depth slots read from such
 *                               a cache.  The depth gradients are those with respect to the dequantised keys
 *                               and values and are written to d_depth_kv in the bf16 cache layout
 *                               (moda_depth_cache_bytes), like moda_attn_bwd's.
 * Other arguments, ownership, validation and error codes as for the bf16 calls they mirror.
 */
size_t moda_depth_cache_e4m3_bytes(int B, int T, int H, int d, int l_max);
int moda_depth_cache_append_e4m3(void* cache, int B, int T, int H, int d, int slot,
                                 const void* K_i, const void* V_i, void* stream);
int moda_attn_fwd_e4m3(const void* Q, const void* K, const void* V, const void* depth_kv_e4m3,
                       int B, int T, int H, int H_kv, int d, int l, float scale,
                       void* O, float* LSE, void* stream);
int moda_attn_bwd_e4m3(const void* Q, const void* K, const void* V, const void* depth_kv_e4m3,
                       const void* O, const void* dO, const float* LSE,
                       int B, int T, int H, int d, int l, float scale,
                       void* dQ, void* dK, void* dV, void* d_depth_kv,
                       void* workspace, size_t workspace_bytes, void* stream);

/*
 * ---- Position-major depth cache for grouped-query calls ----
 *
 * With several query heads per key/value head (Sec. 3, group-aware depth KV) the depth part of a call can run
 * per position: all G heads of a group against the l depth rows of that position, as small dense products.
 * Those kernels consume every row of a few consecutive positions, which the row-interleaved cache layout
 * hands out as 16-byte pieces 2 KiB apart.  This second layout keeps a position's rows together:
 *
 *     cache_pm[slot][b][h_kv][t][kv][d]     bf16; t over whole 128-position tiles, tail rows zero
 *
 * Same size as the row-interleaved cache (moda_depth_cache_bytes); the caller chooses the layout when it
 * appends, and passes the cache to the entry points of that layout only.
 *
 * moda_depth_cache_append_pm / _unpack_pm   as moda_depth_cache_append / _unpack, for this layout.
 * moda_attn_fwd_gqa_pm   moda_attn_fwd_gqa with the depth slots in this layout; needs H_kv < H
 *                        (MODA_ERR_BAD_GROUP otherwise).
 * moda_attn_bwd_gqa_pm   moda_attn_bwd_gqa likewise; d_depth_kv_pm receives the depth gradients in this layout;
 *                        workspace of moda_bwd_workspace_bytes_gqa.
 * Other arguments, ownership, validation and error codes as for the calls they mirror.
 */
int moda_depth_cache_append_pm(void* cache, int B, int T, int H, int d, int slot,
                               const void* K_i, const void* V_i, void* stream);
int moda_depth_cache_unpack_pm(const void* cache, int B, int T, int H, int d, int slot,
                               void* K_i, void* V_i, void* stream);
int moda_attn_fwd_gqa_pm(const void* Q, const void* K, const void* V, const void* depth_kv_pm,
                         int B, int T, int H, int H_kv, int d, int l, float scale,
                         void* O, float* LSE, void* stream);
int moda_attn_bwd_gqa_pm(const void* Q, const void* K, const void* V, const void* depth_kv_pm,
                         const void* O, const void* dO, const float* LSE,
                         int B, int T, int H, int H_kv, int d, int l, float scale,
                         void* dQ, void* dK, void* dV, void* d_depth_kv_pm,
                         void* workspace, size_t workspace_bytes, void* stream);

/*
 * Key / value projection with the depth stream's write step in its epilogue (Sec. 2.1: K = X W_K, V = X W_V;
 * Sec. 2.2, "write": a layer's key-value pair is appended to the depth stream; an FFN layer obtains its pair
 * through a KV projection of its input).
 *
 *     K[b, t, h, :] = X[b, t, :] . Wk[h d + j, :]   (j = 0 .. d-1),   V likewise with Wv
 *
 *     X        : bf16 [B][T][D_model], D_model a multiple of 64 (MODA_ERR_BAD_SHAPE otherwise)
 *     Wk, Wv   : bf16 [H_kv * d][D_model]: one row per output feature, i.e. the transposes of the paper's W_K, W_V
 *     K_out, V_out : bf16 [B][T][H_kv][d], both or neither (an FFN-side projection needs only the slot)
 *     cache, slot  : depth cache in the row-interleaved layout (moda_depth_cache_bytes(B, T, H_kv, d, .)) and the
 *                    slot to write, or cache == NULL for the projection alone
 * bf16 inputs, fp32 accumulation on the tensor cores, one rounding to bf16; the slot receives bit for bit what
 * moda_depth_cache_append(cache, ..., slot, K_out, V_out) would store (tail rows of a ragged last tile are zero),
 * without K and V crossing HBM again.  One launch on `stream`; device pointers owned by the caller; validation,
 * asynchrony and error codes as for the other calls.
 */
int moda_kv_project_append(const void* X, const void* Wk, const void* Wv,
                           int B, int T, int D_model, int H_kv, int d,
                           void* K_out, void* V_out, void* cache, int slot, void* stream);

/*
 * The same projection with the slot written into an e4m3 depth cache (moda_depth_cache_e4m3_bytes(B, T, H_kv, d, .)):
 * codes and one fp32 scale per row, bit for bit what moda_depth_cache_append_e4m3(cache_e4m3, ..., slot, K_out, V_out)
 * would store from the bf16-rounded K and V (row maximum / 448 as the scale, correctly rounded quotients, round to nearest even,
 * saturating; a zero row has scale 1).  K_out, V_out stay bf16 and optional.  Everything else as above.
 */
int moda_kv_project_append_e4m3(const void* X, const void* Wk, const void* Wv,
                                int B, int T, int D_model, int H_kv, int d,
                                void* K_out, void* V_out, void* cache_e4m3, int slot, void* stream);

/*
 * Attention mass on the depth slots (Sec. 2.2: the probabilities of the single softmax; the paper's attention analysis
 * reports the probability that heads give to depth slots, and its bounded slot buffer keeps the entries of highest
 * utility, for which this is the operator's own measure):
 *
 *     mass[b, h, i] = sum_t exp( scale <Q[b,t,h,:], Kd_i[b,t,h / G,:]> - LSE[b,h,t] )      i = 0 .. l-1
 *
 *     Q, LSE       : as passed to / returned by the forward call whose probabilities are meant
 *     depth_kv     : the row-interleaved bf16 cache of H_kv heads that call read (>= l slots)
 *     mass         : fp32 [B][H][l], written (the sum over the slots plus the sequence keys' mass is T per (b, h))
 *     workspace    : moda_depth_slot_mass_workspace_bytes(B, T, H, l) bytes of scratch (partial sums per query tile)
 * fp32 dot products of the bf16 inputs, sums in a fixed order (bit-reproducible).  Two launches on `stream`; l == 0
 * returns MODA_OK without touching anything.  Validation, asynchrony and error codes as for the other calls.
 */
size_t moda_depth_slot_mass_workspace_bytes(int B, int T, int H, int l);
int moda_depth_slot_mass(const void* Q, const void* depth_kv, const float* LSE,
                         int B, int T, int H, int H_kv, int d, int l, float scale,
                         float* mass, void* workspace, size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MODA_H */
