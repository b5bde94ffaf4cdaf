/*
 * fdkv -- FreqDepthKV hot path on one B200 (sm_100a): prefill-time compression of adjacent-layer
 * K/V pairs, the routing probe, and decode attention over the compressed cache.
 *
 * C ABI.  Plain pointers and sizes only.  Unless a parameter says HOST, pointers are DEVICE pointers.
 *
 * Conventions
 *  - Every call returns an fdkv_status.  Argument errors are detected on the host before anything is
 *    enqueued.  No call throws, aborts or traps the device.
 *  - The library never allocates device memory.  The caller owns two device buffers for the lifetime
 *    of the context: an ARENA (packed caches of all sequences, generated-token tails, lookup tables)
 *    and a WORKSPACE (staging of one sequence's compression, histograms, split-K partials).  Sizes come
 *    from fdkv_sizes().  Both must be 256-byte aligned.
 *  - Work is enqueued on the stream the caller passes (a cudaStream_t, given as void*; NULL = the legacy
 *    default stream) and the call returns without waiting, except where stated (fdkv_commit, fdkv_get_*,
 *    the *_host variants).
 *  - Tensors are dense row-major in the storage dtype of the context (float32 or bf16) unless strides
 *    are given.  Device pointers to tensors must be 16-byte aligned; strides are in elements and must be
 *    multiples of 8.
 *  - A "unit" is (sequence, layer pair p = layers 2p and 2p+1, KV head h).  Query head i reads KV head
 *    i / (n_q_heads / n_kv_heads).
 *  - A context is not thread-safe.
 *
 * Notation follows the paper's Method section: T context length, d head dimension, Z0 / Z1 the low /
 * high frequency depth coefficients of Eq. 1 with the 2x2 orthonormal DCT-II, c = 1/sqrt(2).
 */
#ifndef FDKV_H
#define FDKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FDKV_OK = 0,
    FDKV_ERR_INVALID_ARG = 1, /* NULL / misaligned pointer, bad shape, stride, range or order          */
    FDKV_ERR_UNSUPPORTED = 2, /* shape or dtype this build has no kernel for                           */
    FDKV_ERR_ARENA_FULL = 3,  /* the arena cannot hold what fdkv_commit needs; nothing was changed     */
    FDKV_ERR_WORKSPACE = 4,   /* workspace smaller than fdkv_sizes() says                              */
    FDKV_ERR_STATE = 5,       /* call order (probe before compress, decode before commit, tail full)   */
    FDKV_ERR_CUDA = 6,        /* a CUDA runtime call failed; see fdkv_last_cuda_error()                */
    FDKV_ERR_TIMEOUT = 7,     /* a bounded device-side wait gave up (reported by fdkv_device_status)   */
    FDKV_ERR_DEVICE = 8,      /* a device-side consistency check failed (fdkv_device_status)           */
    FDKV_ERR_TOO_LARGE = 9    /* fdkv_compress_unit_noalloc: T * head_dim exceeds FDKV_NOALLOC_MAX_ELEMS */
} fdkv_status;

typedef enum { FDKV_F32 = 0, FDKV_BF16 = 1 } fdkv_dtype;
typedef enum { FDKV_MODE_SHARED = 0, FDKV_MODE_RESIDUAL = 1, FDKV_MODE_EXACT = 2 } fdkv_mode;

typedef struct {
    int32_t n_layers;    /* multiple of the block size B of Eq. 1; block p = layers B p .. B p + B - 1   */
    int32_t n_q_heads;   /* multiple of n_kv_heads; group size n_q_heads / n_kv_heads <= 8             */
    int32_t n_kv_heads;
    int32_t head_dim;    /* 64 or 128                                                                  */
    int32_t max_batch;   /* number of sequence slots                                                   */
    int32_t max_prefill; /* largest T; max_prefill * head_dim < 2^31 (int32 flat indices)              */
    int32_t max_tail;    /* generated tokens kept uncompressed per layer and sequence                  */
    int32_t dtype;       /* fdkv_dtype: storage type of K, V, Q and of the stored coefficients         */
    int32_t keep_num;    /* residual keep fraction: k = floor(T * head_dim * keep_num / keep_den)      */
    int32_t keep_den;    /*   entries per (unit, K or V); 0 <= keep_num <= keep_den                    */
    int32_t residual_rule; /* fdkv_residual_rule: how the sparse high-frequency residual is chosen     */
    int32_t block_size;  /* B of Eq. 1: 2 (also when 0) or 4 layers per depth block                    */
    int32_t max_fold;    /* generated tokens fdkv_fold_tail may move into the compressed form per       */
                         /*   sequence (0: none); fdkv_commit reserves row and list room for them       */
    int32_t row_format;  /* fdkv_row_format: how fdkv_commit stores the dense row streams               */
} fdkv_config;

/*
 * FDKV_ROWS_STORAGE (default): the committed rows (Z0 of shared / residual units, the original rows of exact units)
 *   keep the storage type.
 * FDKV_ROWS_E4M3: they are stored as 8-bit floats (4 exponent bits with bias 7, 3 mantissa bits, no infinities,
 *   largest finite value 448) with one float32 scale per channel of each stored tensor -- the composition with
 *   quantisation that the Method section mentions after Eq. 3; the paper fixes no scheme, this is the build's:
 *       amax_c = max_t |R[t][c]|;  scale_c = amax_c / 448 (float32 division; 1 when amax_c = 0);
 *       code = e4m3(R[t][c] / scale_c)   (float32 division, round to nearest even, saturating);
 *       attention sees decode(code) * scale_c.
 *   Sparse residual values and the generated-token tails keep the storage type.  Halves the bytes a decode call
 *   streams.  bf16 storage, head_dim 128, either block size, either residual rule, group size <= 4; fdkv_fold_tail is
 *   unavailable.  Compression and the probe are unchanged (they see the unquantised coefficients).
 */
typedef enum { FDKV_ROWS_STORAGE = 0, FDKV_ROWS_E4M3 = 1 } fdkv_row_format;

/*
 * Block size 4 (Method, Eq. 1 with the orthonormal DCT-II of size 4; the paper's default for middle layers).
 * Wherever this header says "pair" read "block": pair ranges index blocks, a unit is (block, KV head), modes and
 * scores have one entry per unit.  What is stored per tensor (K or V) of a unit, in float32 arithmetic that is
 * never contracted, rs = rounding to the storage type:
 *     s = (x0 + x1) + (x2 + x3);   Z0 = rs(0.5 s)                the shared coefficient (first DCT row = 1/2 each)
 *     dev_l = rs(x_l - 0.5 Z0),  l = 0..3                         layer l's high-frequency part in layer space:
 *                                                                 sum_{j>=1} F_4[j][l] Z_j = x_l - mean(x)
 *     e = (dev_0^2 + dev_1^2) + (dev_2^2 + dev_3^2)               the position's high-frequency energy (Parseval)
 * The three high-frequency groups share one kept set per tensor (Eq. 3): the k positions of largest e, ties to the
 * lowest flat index; the four values dev_l are kept there (instead of three coefficients), so that a decode call of
 * layer l reads one value per kept position.  Candidates: shared = Z0 / 2, residual = Z0 / 2 + dev_l on the kept
 * positions, exact = x_l.  Eq. 2 averages over the block's four layers; Omega(residual) counts four values and one
 * int32 index per kept position, Omega(exact) four layers.  The mixed schedule of the paper (B = 4 in the middle,
 * B = 2 for the first and last layers) is two contexts, one per block size.  Under FDKV_RESIDUAL_TOKENS (the paper's
 * default pairing: blocks of four with probe-scored tokens) a token's score is the maximum over the block's four layers of
 * | Q_l . dev_l[t,:] |, one token set serves K and V and all four layers, and the kept tokens store the four layers'
 * deviation rows (Omega(residual) counts 2 * 4 * k_tok * d * e + 4 * k_tok bytes).
 */

/*
 * FDKV_RESIDUAL_ENTRIES (default): the k largest-magnitude entries of Z1, K and V independently (chosen in
 *   fdkv_compress_prefill; indices bit-reproducible).
 * FDKV_RESIDUAL_TOKENS: the paper's rule (Method, the unnumbered score between Eq. 2 and Eq. 3): token t of a
 *   unit is scored s_t = max over the pair's two layers, the group's query heads and the probe queries q with
 *   probe_pos[q] >= t of | Q . (c * Z1K[t,:]) |; the k_tok = floor(T * keep_num / keep_den) tokens with the
 *   largest score (ties: lowest t) keep ALL head_dim high-frequency coefficients of K and of V.  The scores
 *   need the probe queries, so the set is chosen inside fdkv_probe (which is then mandatory before commit, even
 *   when modes are overridden); Omega(residual) counts 2*k_tok*d*e + 4*k_tok bytes.  Either storage type, head
 *   dimension and block size (see the note on block size 4 above for the score and the stored rows there); bf16 with
 *   head_dim 128 runs the tensor-core kernels, the rest the float32 score and probe kernels and the portable decode kernel.
 */
typedef enum { FDKV_RESIDUAL_ENTRIES = 0, FDKV_RESIDUAL_TOKENS = 1 } fdkv_residual_rule;

typedef struct fdkv_ctx fdkv_ctx;

/* Bytes the caller must provide.  arena_bytes is the worst case (every unit in exact mode). */
fdkv_status fdkv_sizes(const fdkv_config* cfg /*HOST*/, size_t* arena_bytes /*HOST*/,
                       size_t* workspace_bytes /*HOST*/);

/* Creates the host-side context over caller-owned device memory and zero-initialises the tail counters
 * and the device status word (synchronously, on the legacy default stream).  The context keeps the pointers;
 * the caller frees the buffers only after fdkv_destroy.                                                   */
fdkv_status fdkv_create(const fdkv_config* cfg /*HOST*/, void* arena, size_t arena_bytes, void* workspace,
                        size_t workspace_bytes, fdkv_ctx** out /*HOST*/);
void fdkv_destroy(fdkv_ctx* ctx);
/* Forgets every committed sequence and empties the arena and all tails (synchronous). */
fdkv_status fdkv_reset(fdkv_ctx* ctx);

/*
 * Prefill compression (Method, Eq. 1 and Eq. 3; residual set in entry-magnitude form).
 * For every pair p in [pair_begin, pair_end), every KV head h and for K and V separately:
 *   z0 = rs((x0 + x1) * c32), z1 = rs((x0 - x1) * c32)   one float32 add, one float32 multiply by the
 *        float32 nearest 1/sqrt(2), rs = rounding to the storage dtype (nearest even);
 *   the k entries of z1 with the largest magnitude are kept (ties: lowest flat index t*d + ch) and
 *   emitted in ascending flat index as (int32 index, stored value).
 * k_layers / v_layers: HOST arrays of n_layers DEVICE pointers (only the layers of the pair range are
 *   read); element (t, h, ch) of layer l is at ptr[l] + t*stride_t + h*stride_h + ch.
 * Results are staged in the workspace for sequence slot `seq` (one sequence is staged at a time; a call
 * for another slot discards the previous staging).  The caller keeps K/V alive until fdkv_commit returns.
 */
fdkv_status fdkv_compress_prefill(fdkv_ctx* ctx, int32_t seq, int32_t pair_begin, int32_t pair_end, int32_t T,
                                  const void* const* k_layers /*HOST*/, const void* const* v_layers /*HOST*/,
                                  int64_t stride_t, int64_t stride_h, void* stream);

/*
 * Routing probe (Method, Eq. 2 and the argmin of Eq. 3) for the staged sequence.
 * For every unit of the pair range and mode m in {shared, residual}:
 *   E(m) = mean over (layer of the pair, group query head g, probe query q) of
 *          sum_{j <= probe_pos[q]} ( Q[l][q][h*G+g] . (c * R^(m)[j,:]) / sqrt(d) )^2,
 *   R^(shared) = Z1 of K, R^(residual) = Z1 of K with the kept entries removed; E(exact) = 0.
 *   L(m) = E(m) + lambda * Omega(m), Omega = bytes(m) / bytes(exact) (K and V, int32 indices counted);
 *   mode = argmin, ties to the lowest id.  The same mode applies to K and V.
 * q_layers: HOST array of n_layers DEVICE pointers to [W][n_q_heads][head_dim].
 * probe_pos: HOST int32[W], strictly ascending, each in [0, T).  1 <= W <= 128.
 * modes (may be NULL): DEVICE int32[pair_end-pair_begin][n_kv_heads].
 * scores (may be NULL): DEVICE float[pair_end-pair_begin][n_kv_heads][2] = {E(shared), E(residual)}.
 */
fdkv_status fdkv_probe(fdkv_ctx* ctx, int32_t seq, int32_t pair_begin, int32_t pair_end,
                       const void* const* q_layers /*HOST*/, const int32_t* probe_pos /*HOST*/, int32_t W,
                       double lambda, int32_t* modes, float* scores, void* stream);

/*
 * Budgeted routing (Method: the memory budget is enforced by increasing lambda until the estimated KV footprint fits).
 * Uses the probe errors fdkv_probe left for the staged sequence (every pair must have been probed; waits for the
 * stream) and finds the smallest lambda >= 0 whose routing -- mode = argmin E(m) + lambda * Omega(m) per unit, ties to
 * the lowest id -- has sum over units of Omega(mode) * bytes(exact) <= budget_bytes.  The footprint can only change
 * where two of a unit's loss lines cross, so the candidates are 0 and every crossing, ascending; each is tried at
 * crossing * (1 + 2^-40).  The modes found replace the probe's (as fdkv_set_modes would) and are what fdkv_commit
 * packs.  *lambda_host (HOST, may be NULL) receives lambda; modes_host (HOST int32[n_layers/2][n_kv_heads], may be
 * NULL) the modes.  If even the all-shared routing exceeds the budget: FDKV_ERR_ARENA_FULL, lambda = +inf, all shared.
 * The estimate counts the prefill cache in canonical bytes (as Omega does), not the generated-token tails.
 */
fdkv_status fdkv_route_budget(fdkv_ctx* ctx, int32_t seq, size_t budget_bytes, double* lambda_host /*HOST*/,
                              int32_t* modes_host /*HOST*/, void* stream);

/* Overrides the modes of the staged sequence (forced-mode tests, ablations, benchmark mode mix).
 * modes_host: HOST int32[n_layers/2][n_kv_heads], each 0, 1 or 2.                                        */
fdkv_status fdkv_set_modes(fdkv_ctx* ctx, int32_t seq, const int32_t* modes_host /*HOST*/);

/* Packs the staged sequence into the arena, keeping per unit only what its mode reads at decode time
 * (shared: Z0 of K and V; residual: Z0 plus the two lists; exact: the original rows of both layers).
 * Waits for the stream (it needs the modes on the host), then enqueues the copies and waits again.
 * Every pair of the sequence must have been compressed, and probed or given a mode.                      */
fdkv_status fdkv_commit(fdkv_ctx* ctx, int32_t seq, void* stream);

/*
 * Decode attention for one layer (Method, the paragraph after Eq. 3), split-K over the sequence.
 * For sequence b < batch and query head i (KV head h = i / G), over rows 0..T-1 reconstructed by the
 * unit's mode (shared: c*z0; residual: c*(z0 + s*z1 on kept entries), s = +1 for layer 2p, -1 for 2p+1;
 * exact: the original row) followed by the layer's uncompressed tail rows:
 *   logit = khat . q / sqrt(d);  out = softmax(logit) . vhat      (float32 accumulation)
 * q: [batch][n_q_heads][d].  k_new / v_new: [batch][n_kv_heads][d], appended to the layer's tail before
 * attending, or both NULL (no append).  out: [batch][n_q_heads][d] in out_dtype.
 * Sequence slots 0..batch-1 must be committed.
 * Stream order: q, k_new and v_new are read only after every kernel enqueued earlier on `stream` has completed
 * (the kernels start early under programmatic dependent launch, but wait before their first read of caller data),
 * so the caller's projection kernels may be enqueued directly ahead of this call.  The tail lengths are tracked on
 * the host: a call that would exceed max_tail returns FDKV_ERR_STATE before anything is enqueued.
 * CUDA graphs: the work distribution and the tail lengths are computed on the host and travel in the launch
 * parameters, so a captured call replays exactly the state it was captured in.  Calls on layers without generated
 * tokens and without k_new may be captured and replayed (the benchmark does); a call that appends, or that follows
 * appends made outside the graph, must be issued on the stream.
 */
fdkv_status fdkv_decode_attn(fdkv_ctx* ctx, int32_t layer, int32_t batch, const void* q, const void* k_new,
                             const void* v_new, void* out, int32_t out_dtype, void* stream);

/* Same call with HOST buffers: copies q (and k_new, v_new) to the device, runs the layer, copies out back and
 * waits for the stream.  Buffers should be pinned for the copies to overlap.                              */
fdkv_status fdkv_decode_attn_host(fdkv_ctx* ctx, int32_t layer, int32_t batch, const void* q /*HOST*/,
                                  const void* k_new /*HOST*/, const void* v_new /*HOST*/, void* out /*HOST*/,
                                  int32_t out_dtype, void* stream);

/* All layers of one step with HOST buffers: q and out are [n_layers][batch][n_q_heads][head_dim], k_new / v_new
 * [n_layers][batch][n_kv_heads][head_dim] or both NULL.  One host-to-device copy per input, the n_layers layer calls
 * of fdkv_decode_attn in layer order, one device-to-host copy of all outputs, one wait for the stream.  For callers
 * that know every layer's query up front (attention-only benchmarks, verification of a recorded step); a model that
 * computes layer l+1's query from layer l's output uses the per-layer calls.                                      */
fdkv_status fdkv_decode_step_host(fdkv_ctx* ctx, int32_t batch, const void* q /*HOST*/, const void* k_new /*HOST*/,
                                  const void* v_new /*HOST*/, void* out /*HOST*/, int32_t out_dtype, void* stream);

/* Sets the tail length of every layer of a sequence (0 empties the tails; n <= current length). */
fdkv_status fdkv_set_tail_len(fdkv_ctx* ctx, int32_t seq, int32_t n, void* stream);

/*
 * Periodic refresh (Method, last paragraph: routing is decided once after prefill; the cache may be refreshed every
 * fixed number of tokens).  Moves the first n generated tokens of EVERY layer of a committed sequence out of the
 * exact tails into the compressed form, under each unit's existing mode: the chunk is transformed by Eq. 1, keeps
 * its own k = floor(n * head_dim * keep_num / keep_den) largest-magnitude high-frequency entries per tensor (Eq. 3
 * applied to the chunk; ties to the lowest index) and is appended behind the unit's rows and lists; exact units get
 * the rows themselves.  The remaining tail rows move down; T of the sequence grows by n.  Modes do not change (the
 * originals of shared / residual units no longer exist, so a committed unit cannot be re-routed upwards).
 * Requirements: entry residual rule (either block size; a block of four keeps the chunk's positions of largest
 * high-frequency energy); T and n multiples of 16; every layer's tail holds the same
 * number (>= n) of tokens, i.e. call it between decode steps; the total folded per sequence stays within
 * cfg.max_fold; no other sequence may be staged and uncommitted (the call reuses the staging area and invalidates
 * it).  Synchronous (waits for the stream).  FDKV_ERR_ARENA_FULL when max_fold is exhausted.
 */
fdkv_status fdkv_fold_tail(fdkv_ctx* ctx, int32_t seq, int32_t n, void* stream);

/* FDKV_ROWS_E4M3 only: the 8-bit codes [T][head_dim] and the float32 scales [head_dim] of one committed row stream
 * (layer's K or V rows of a KV head: Z0 for shared / residual units, the layer's own rows for exact ones).  Device
 * buffers, either may be NULL.  Synchronous.                                                                      */
fdkv_status fdkv_get_rows_e4m3(fdkv_ctx* ctx, int32_t seq, int32_t layer, int32_t kv_head, int32_t is_v,
                               uint8_t* codes_out /*DEVICE*/, float* scale_out /*DEVICE*/, void* stream);

/* Introspection of the STAGED sequence (valid from fdkv_compress_prefill until the next one).  Synchronous. */
fdkv_status fdkv_get_shared(fdkv_ctx* ctx, int32_t seq, int32_t pair, int32_t kv_head, int32_t is_v,
                            void* z0_out /*DEVICE [T][d] storage dtype*/, void* stream);
fdkv_status fdkv_get_residual(fdkv_ctx* ctx, int32_t seq, int32_t pair, int32_t kv_head, int32_t is_v,
                              int32_t* idx_out /*DEVICE [k]*/, void* val_out /*DEVICE [k] storage dtype*/,
                              int32_t* count_host /*HOST*/, void* stream);
/* Token rule only: the selected tokens of a staged unit (ascending, DEVICE int32[k_tok], may be NULL), the scores of
 * all T tokens (DEVICE float[T], may be NULL) and the count (HOST).  Valid after fdkv_probe.  Synchronous.          */
fdkv_status fdkv_get_token_set(fdkv_ctx* ctx, int32_t seq, int32_t pair, int32_t kv_head, int32_t* tok_out,
                               float* score_out, int32_t* count_host /*HOST*/, void* stream);
/* Modes of a committed (or mode-overridden) sequence: HOST int32[n_layers/2][n_kv_heads]. */
fdkv_status fdkv_get_modes(fdkv_ctx* ctx, int32_t seq, int32_t* modes_host /*HOST*/);
/* Bytes a committed sequence holds in the arena per mode, and what the uncompressed cache would take. */
fdkv_status fdkv_footprint(fdkv_ctx* ctx, int32_t seq, size_t* bytes_by_mode_host /*HOST [3]*/,
                           size_t* exact_equiv_bytes_host /*HOST*/);
/* Host-only planning call (no GPU is touched; usable without a device): how a decode launch of the tensor-core kernel
 * (bf16 storage, head_dim 128) would cut its work over `n_ctas` thread blocks.  The work list is every (sequence, KV
 * head) unit's prefill tokens in 16-token slices, unit-major; a residual unit's slices weigh more (Method, the
 * paragraph after Eq. 3: decode reconstructs per head mode, so the modes set the cost).  Inputs (HOST): T[batch] prefill
 * lengths, modes[batch * n_kv_heads] of the layer's units.  Outputs (HOST): start_out[n_ctas + 1], block c handles the
 * range [start_out[c], start_out[c+1]) where an entry is unit << 20 | slice and the last one is units << 20;
 * *n_ctas_out <= n_ctas blocks are used; parts_out[batch * n_kv_heads] = split-K parts per unit (blocks whose range
 * holds at least one of its slices).  Errors: FDKV_ERR_INVALID_ARG for null pointers, sizes out of range or more units
 * than the kernel takes (1024).                                                                                      */
fdkv_status fdkv_plan_decode(int32_t batch, int32_t n_kv_heads, const int32_t* T_host, const int32_t* modes_host,
                             int32_t keep_num, int32_t keep_den, int32_t residual_rule, int32_t row_format, int32_t n_ctas,
                             uint32_t* start_out, int32_t* n_ctas_out, int32_t* parts_out);
/* Bytes the decode kernels read from the packed cache for one call of `layer` over `batch` sequences
 * (coefficient or exact rows, residual lists and their tile offsets, tails): the roofline numerator.      */
fdkv_status fdkv_decode_bytes(fdkv_ctx* ctx, int32_t layer, int32_t batch, size_t* bytes_host /*HOST*/);

/*
 * Compression of ONE [T][head_dim] tensor pair without any allocation.  (The paper has no counterpart: this is
 * a packaging of the Eq. 1 / Eq. 3 compression step for callers that cannot allocate.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a serving engine whose memory pool owns
 * every byte of the device, in a plugin that is only handed tensors, or in a latency-critical path where an
 * allocation (an implicit device synchronisation) is not acceptable -- and that has no fdkv context, whose
 * workspace would otherwise provide the scratch.  The scratch this needs (the Z1 temporary, the magnitude
 * histogram, per-tile counts and offsets; about 4.3 MB) is a static array inside the library's device image:
 * every GPU that loads libfdkv holds it until the process exits, whether or not this function is ever called.
 *
 * Computes exactly what fdkv_compress_prefill computes for one unit-tensor: z0_out[T][head_dim] (storage
 * dtype, dense), and the k = floor(T*head_dim*keep_num/keep_den) kept entries of Z1 as ascending flat indices
 * idx_out[k] with their stored values val_out[k] (may be NULL when k == 0).  x0 / x1: rows of layer 2p / 2p+1,
 * row t at x + t*stride_t (elements).  *count_host (HOST, may be NULL) receives k.  All pointers 16-byte aligned.
 *
 * Limits and rules
 *  - T * head_dim <= FDKV_NOALLOC_MAX_ELEMS, else FDKV_ERR_TOO_LARGE and nothing is enqueued.
 *  - Calls cudaMalloc / cudaFree or any allocating routine never; it enqueues a memset and kernels on `stream`.
 *  - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that device
 *    current).  Make that first call outside any stream capture.
 *  - Every call on a device uses the same array, which still holds the previous call's data; the function
 *    clears what has to start at zero itself.  Two calls whose work overlaps on the GPU (different streams
 *    without an ordering between them) race on it: serialise them.
 *  - A device-side count mismatch is not reported here (there is no context to hold a status word the caller
 *    could read); compare *count_host with what you expect to find in idx_out if in doubt.
 */
#define FDKV_NOALLOC_MAX_ELEMS (1 << 20)
fdkv_status fdkv_compress_unit_noalloc(const void* x0, const void* x1, int64_t stride_t, int32_t T, int32_t head_dim,
                                       int32_t dtype, int32_t keep_num, int32_t keep_den, void* z0_out,
                                       int32_t* idx_out, void* val_out, int32_t* count_host /*HOST*/, void* stream);

/* Reads the device status word (synchronises the device): FDKV_OK, FDKV_ERR_TIMEOUT or FDKV_ERR_DEVICE.  */
fdkv_status fdkv_device_status(fdkv_ctx* ctx);
int32_t fdkv_last_cuda_error(void);
const char* fdkv_status_str(fdkv_status s);
/* Kernels launched by this library since it was loaded (all contexts). */
int64_t fdkv_launch_count(void);
/* Which kernel served a call: launches, since the library was loaded, of the kernels that have a portable and an sm_100a
 * form.  bf16 storage with head_dim 128 is always served by the tcgen05 / TMA kernels (the probe of Eq. 2, the token
 * score between Eq. 2 and Eq. 3, decode attention after Eq. 3); float32 storage or head_dim 64 by the portable ones.
 * There is no silent fall-back from one to the other: a configuration the fast kernels cannot take is refused when
 * the context is created.  Returns -1 for an unknown id.                                                            */
typedef enum {
    FDKV_KERNEL_PROBE_TC = 0,       /* probe_tc_kernel: tcgen05 probe error                  */
    FDKV_KERNEL_PROBE_PORTABLE = 1, /* probe_tile_kernel: float32 FMA probe error            */
    FDKV_KERNEL_DECODE_FAST = 2,    /* decode_fast_kernel: TMA + tensor-core decode attention */
    FDKV_KERNEL_DECODE_PORTABLE = 3,/* decode_generic_kernel + combine_kernel                */
    FDKV_KERNEL_TOKEN_SCORE = 4,    /* token_score_kernel: tcgen05 token scores              */
    FDKV_KERNEL_COUNT_ = 5
} fdkv_kernel_id;
int64_t fdkv_kernel_launch_count(int32_t kernel);

#ifdef __cplusplus
}
#endif
#endif /* FDKV_H */
