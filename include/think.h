/*
 * think.h -- C ABI of the ThinK hot path (query-driven key-cache channel pruning)
 * for NVIDIA B200 (sm_100a).
 *
 * Problem statement (paper, Sec. 1 and Sec. 3.1): the key and value caches are
 * tensors K, V in R^{B x S x L x N x D} (batch, tokens, layers, heads, head
 * dimension).  Given a pruning ratio lambda, T = floor((1 - lambda) D) key
 * channels are kept per head (Sec. 3.1, Eq. 2); the channels are chosen by the
 * query-driven score of Sec. 3.2 evaluated with the last S_obs queries
 * ("Observation Window"); the most recent S_recent prompt tokens and all newly
 * decoded tokens keep all D key channels (Sec. 3.3).
 *
 * Call order:   thinK_cache_bytes -> thinK_create -> thinK_score_select -> thinK_compact
 *               (or thinK_prefill for both) -> { thinK_append -> thinK_decode_attn }* -> thinK_destroy
 *
 * Conventions that hold for every entry point
 *  - All tensor pointers are DEVICE pointers unless marked "host".  The caller
 *    allocates and owns every device buffer; the library never allocates device
 *    memory and never frees anything but its own host-side handle.
 *  - `stream` is a cudaStream_t passed as void*.  Calls enqueue work on it and
 *    return without synchronising.  Calls on one handle must be stream-ordered
 *    with respect to each other.
 *  - Errors are return codes.  Arguments are validated on the host before any
 *    launch; an invalid call launches nothing.  Inputs are assumed finite:
 *    NaN/Inf in K or Q sets a bit of the device error word and leaves the
 *    choice among the affected channels unspecified (never an out-of-range write).
 *  - Element type (`dtype`): bf16 or fp32 for K, V, Q, q, k_new, v_new and out.
 */
#ifndef THINK_H_
#define THINK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  THINK_OK = 0,
  THINK_ERR_INVALID_ARG = 1, /* null / misaligned pointer, bad shape, bad layer range */
  THINK_ERR_UNSUPPORTED = 2, /* head dimension, group size or dtype without a kernel */
  THINK_ERR_STATE = 3,       /* call out of order */
  THINK_ERR_CAPACITY = 4,    /* tail full (max_new_tokens) or buffer too small */
  THINK_ERR_CUDA = 5         /* a CUDA runtime call or launch failed */
} thinK_status;

typedef enum { THINK_BF16 = 0, THINK_F32 = 1 } thinK_dtype;

/* Score used to rank the channels of a key head. */
typedef enum {
  THINK_SCORE_QUERY_DRIVEN = 0, /* Sec. 3.2: ||Q[-S_obs:, j] K[:, j]^T||_F                      */
  THINK_SCORE_KEY_L2 = 1,       /* Sec. 3.1, Eq. 1 with p = 2: ||K[:, j]||_2 (paper's baseline) */
  THINK_SCORE_KEY_L1 = 2        /* Sec. 3.1, Eq. 1 with p = 1: ||K[:, j]||_1                    */
} thinK_criterion;

/* Kernel behind the value-channel score of App. D (thinK_score_select_kv). */
typedef enum {
  THINK_VALUE_SCORE_AUTO = 0,     /* tcgen05.mma with accumulators in tensor memory where the shape allows it
                                     (blocks of 128 stacked window rows, D = 128), mma.sync elsewhere */
  THINK_VALUE_SCORE_MMA_SYNC = 1  /* the mma.sync kernel everywhere (same results within the stated tolerance) */
} thinK_value_score_kernel;

typedef struct {
  int32_t B;              /* batch entries */
  int32_t L;              /* layers held by this cache */
  int32_t N_q;            /* query heads; N_q % N_kv == 0, group size G = N_q / N_kv in {1,2,4,8} */
  int32_t N_kv;           /* key/value heads */
  int32_t D;              /* head dimension: 64 or 128 */
  int32_t S_max;          /* rows allocated along S in K and V (>= every seq_len) */
  int32_t S_obs;          /* observation window (Sec. 3.2); seq_len >= S_obs */
  int32_t S_recent;       /* prompt tokens left unpruned (Sec. 3.3, Sec. 4.3 "recent size") */
  int32_t max_new_tokens; /* decode steps the unpruned tail can take */
  int32_t dtype;          /* thinK_dtype */
  int32_t criterion;      /* thinK_criterion */
  int32_t value_score_kernel; /* thinK_value_score_kernel; only read when lambda_v > 0 */
  double lambda;          /* pruning ratio, 0 <= lambda < 1 */
  double lambda_v;        /* pruning ratio of the value channels (App. D); 0 = values untouched (the default path) */
} thinK_config;

/* A strided view of a B x S x L x N x D tensor.  Strides are in ELEMENTS; the D
 * axis is contiguous.  `ptr` and every stride must be multiples of 16 bytes.
 * The paper's layout is stride_b = S*L*N*D, stride_s = L*N*D, stride_l = N*D,
 * stride_n = D; a per-layer cache [B, N, S, D] is expressed by other strides. */
typedef struct {
  void* ptr;
  int64_t stride_b, stride_s, stride_l, stride_n;
} thinK_tensor5;

/* Byte sizes of the caller-allocated device buffers (each 256-byte aligned). */
typedef struct {
  size_t k_thin;    /* pruned prefix keys, library layout (below) */
  size_t tail_k;    /* unpruned keys: recent prompt rows + decoded tokens */
  size_t tail_v;    /* values of the same tokens, [B, L, N_kv, cap, D] */
  size_t idx;       /* kept channels, uint8 [B, L, N_kv, T], ascending */
  size_t scores;    /* channel scores, fp64 [B, L, N_kv, D] */
  size_t workspace; /* reduction partials, split-softmax states, counters */
  /* The paper's accounting of the same cache (Sec. 3.1, Sec. 3.3), in bytes:
   * keys of the pruned prefix at T channels + unpruned keys at D + all values,
   * with the tail at full capacity; and the unpruned cache 2*B*S*L*N*D*e with
   * the same number of tokens. */
  size_t model_think_bytes;
  size_t model_dense_bytes;
  /* Only with lambda_v > 0 (else 0): */
  size_t v_thin;    /* pruned prefix values, bf16 [rows of T_v kept channels padded to a multiple of 16] */
  size_t perm_v;    /* uint8 [B, L, N_kv, D]: kept value channels ascending, then the pruned ones ascending */
} thinK_sizes;

typedef struct thinK_cache thinK_cache; /* opaque, host side */

/* T = floor((1 - lambda) * D) (Sec. 3.1); returns 0 when lambda is outside
 * [0, 1) or T would be 0. */
int32_t thinK_T(double lambda, int32_t D);

const char* thinK_status_string(thinK_status s);

/* Sizes of the buffers thinK_create needs.  `seq_lens` (host, [B]) are the
 * prompt lengths S_b; S_recent <= S_b, S_obs <= S_b <= S_max.
 *
 * Library layout of k_thin and tail_k.  For every (b, l, h) the S_p = S_b - S_recent prefix tokens
 * are cut into tiles of 64 tokens; tile t of head (b, l, h) is tile number
 *   thin_tile_base(b) + (l*N_kv + h)*n_tiles(b) + t,   n_tiles(b) = ceil(S_p(b)/64),
 *   thin_tile_base(b) = sum_{b'<b} L*N_kv*n_tiles(b'),
 * and a tile holds Tp x 64 elements (tokens past S_p are zero).
 *  - fp32: Tp = T; channel-major [T][64], rows of 64 tokens whose 16-byte chunks are XOR-swizzled with
 *    (row & 7): element (token u, channel c) at c*64 + swz(c, u),
 *    swz(c, u) = (((u*4/16) ^ (c & 7)) * 16 + (u*4)%16) / 4.
 *  - bf16: Tp = T rounded up to a multiple of 8 (extra channels are zero); the tile is stored in the
 *    operand order of the tensor-core instruction that consumes it: four 16-token steps of Tp*32
 *    bytes; in a step, for each group s of 16 channels a 512-byte chunk with 16 bytes per lane i
 *    (r = i/4, q = i%4): for jx = 0,1 the channel pairs (16s+2q, +1) and (16s+2q+8, +9) of token
 *    16*step + 8*jx + r; a trailing group of 8 channels is a 256-byte block with 8 bytes per lane
 *    (pair (16*n16+2q, +1) for jx = 0,1).
 * tail_k uses the same tile layout with all D channels: [B, L, N_kv, ceil(cap/64)] tiles of D x 64,
 * cap = S_recent + max_new_tokens.
 * After the n_tiles(b) prompt tiles every head owns ceil(cap/64) more tiles in k_thin, which receive the
 * tail blocks that thinK_reprune_tail thins (so the tile number above uses n_tiles(b) + ceil(cap/64)
 * per head).
 * v_thin (lambda_v > 0): token-major rows of Tvp = T_v rounded up to 16 bf16 elements, row t of head
 * (b, l, h) at element v_base(b) + ((l*N_kv + h)*S_p(b) + t)*Tvp, v_base(b) = sum_{b'<b} L*N_kv*S_p(b')*Tvp;
 * element c < T_v of a row is channel perm_v[b][l][h][c] of the value, the padding is zero.  With
 * lambda_v > 0 the rows of tail_v are stored in the channel order perm_v[b][l][h][0..D). */
thinK_status thinK_cache_bytes(const thinK_config* cfg, const int32_t* seq_lens, thinK_sizes* out);

/* Builds the host-side handle and writes the small device tables (lengths,
 * tile offsets, zeroed counters) into `workspace` with synchronous copies.
 * `sizes` (host) states the bytes the caller actually allocated for each buffer
 * (v_thin and perm_v: for the later thinK_attach_value_cache); a buffer smaller
 * than thinK_cache_bytes reports for this configuration is refused with
 * THINK_ERR_CAPACITY before anything is written.  The buffers stay valid until
 * thinK_destroy.  `scores` may be NULL (scores are then not kept). */
thinK_status thinK_create(const thinK_config* cfg, const int32_t* seq_lens, const thinK_sizes* sizes, void* k_thin,
                          void* tail_k, void* tail_v, void* idx, void* scores, void* workspace, thinK_cache** out);

/* Prefill, Sec. 3.2: channel scores and I = Top_T(Score, T) for layers
 * [layer0, layer0 + nlayers) of every (b, h).
 *   q_obs: [B, S_obs, L, N_q, D] view -- row s of entry b is the query of prompt
 *          token S_b - S_obs + s ("Observation Window"); ignored (may hold a NULL
 *          ptr) for the key-norm criteria of Eq. 1.
 *   k:     [B, S_max, L, N_kv, D] view; rows >= S_b are never read.
 * Score[j] = sqrt(sum_g sum_s q^2 * sum_t k^2): the closed form of the Frobenius
 * norm of the rank-one product, with the G query heads of a group stacked.  All
 * S_b key rows enter the score.  Sums run in fp64 over fp32 partial chains of
 * at most 8 terms (bf16) or directly in fp64 (fp32), in a fixed order: results
 * are deterministic.  Equal scores go to the lower channel.  Writes idx (and
 * scores).  Layer indices address both the views and the cache. */
thinK_status thinK_score_select(thinK_cache* c, thinK_tensor5 q_obs, thinK_tensor5 k, int32_t layer0,
                                int32_t nlayers, void* stream);

/* Value-channel pruning (App. D, "ThinKV"), bf16 caches only.  With cfg.lambda_v > 0 the caller hands
 * over the two extra buffers of thinK_sizes (v_thin, perm_v) right after thinK_create; the path is then
 *   thinK_score_select_kv -> thinK_compact -> { thinK_append -> thinK_decode_attn }*
 * (thinK_prefill takes both steps).  `scores_v` (fp64 [B, L, N_kv, D], thinK_sizes.scores bytes) may be
 * NULL: the value scores are then not kept.  THINK_ERR_STATE if lambda_v == 0. */
thinK_status thinK_attach_value_cache(thinK_cache* c, void* v_thin, void* perm_v, void* scores_v);

/* thinK_score_select plus the value-channel score of App. D, Eqs. 3-4:
 *   Score_v[j] = || softmax(Q[-S_obs:] K^T / sqrt(D)) V[:, j] ||_F,   I_v = Top_T(Score_v, T_v),
 * T_v = floor((1 - lambda_v) D).  All S_b rows of K and V enter, no causal mask inside the window
 * (the formula has none), the G query heads of a group are stacked row-wise as for the key score, ties
 * go to the lower channel.  Both products run on tensor cores in bf16 with fp32 accumulation, the
 * softmax weights as a bf16 pair hi + lo; column norms in fp64.  Against an fp64 evaluation the scores
 * carry a relative error of about 1e-5, so two channels whose scores are closer than that may swap.
 * Writes perm_v (kept channels ascending, then the rest ascending).  `v` as for thinK_compact.
 * Kernels: blocks of 128 stacked window rows at D = 128 run on tcgen05.mma with accumulators in tensor memory,
 * everything else on mma.sync; cfg.value_score_kernel = THINK_VALUE_SCORE_MMA_SYNC keeps the mma.sync kernel
 * everywhere (same results within the tolerance above).
 * The tcgen05 kernel bounds its waits: if one runs out, the device error word gets bit 2 (see
 * thinK_device_error) and the scores of that call are unspecified; the next call starts clean. */
thinK_status thinK_score_select_kv(thinK_cache* c, thinK_tensor5 q_obs, thinK_tensor5 k, thinK_tensor5 v,
                                   int32_t layer0, int32_t nlayers, void* stream);

/* Prefill, Sec. 3.3: builds the two-part key cache for the given layers from
 * the idx thinK_score_select stored: K_T[t][c] = K[t][idx[c]] for t < S_p, and
 * the last S_recent rows of K and V copied unpruned to the tail.  After this
 * call K may be released by the caller; V rows [0, S_p) of `v` stay BORROWED:
 * thinK_decode_attn reads them in place on every step.  One view serves all
 * layers: a call with a different `v` starts a new prompt, i.e. the layers
 * outside its range count as not compacted until they are compacted again.
 * With lambda_v > 0 (after thinK_score_select_kv) the prefix values are thinned too:
 * V_T[t][c] = V[t][perm_v[c]], c < T_v, written to v_thin; the recent rows keep all D channels
 * (declared reading: App. D gives the criterion only; the split mirrors the keys').  `v` is then
 * not borrowed. */
thinK_status thinK_compact(thinK_cache* c, thinK_tensor5 k, thinK_tensor5 v, int32_t layer0, int32_t nlayers,
                           void* stream);

/* Prefill in one call: thinK_score_select followed by thinK_compact for the same layers on the
 * same stream (Sec. 3.2 + 3.3).  Arguments as for those two calls. */
thinK_status thinK_prefill(thinK_cache* c, thinK_tensor5 q_obs, thinK_tensor5 k, thinK_tensor5 v, int32_t layer0,
                           int32_t nlayers, void* stream);

/* Prefill behind a token-eviction method (the setting of the paper's main experiments, Sec. 4.1-4.2:
 * H2O or SnapKV first reduce every head to "KV-size" tokens, then the channels of the surviving keys
 * are pruned).  Instead of gathered K/V tensors the caller passes the method's per-head list of kept
 * tokens; scoring, compaction and the tail seed read the kept rows straight from the prompt tensors.
 *   The cache must have been created with seq_lens[b] = n_b, the number of tokens KEPT for entry b
 *   (the same for every head), and S_max >= max n_b.
 *   tok:        device int32 [B, L, N_kv, tok_stride]; tok[b][l][h][i], i < n_b, is the row of `k`
 *               and `v` that holds kept token i of that head.  The order of the list is the token
 *               order of the compressed cache: its last S_recent entries stay unpruned.  4-byte aligned.
 *   src_tokens: rows of `k` and `v` per entry; every used tok value must lie in [0, src_tokens).
 *               The host cannot see the list: an entry outside the range is read as row 0 and sets
 *               the device error word (thinK_device_error != 0), results are then unspecified.
 *   q_obs:      as for thinK_score_select (the window's queries are not evicted).
 *   v_kept:     device buffer of thinK_v_kept_bytes(c); receives the values of the kept tokens as
 *               dense [B, L, N_kv, S_max, D] and is BORROWED until thinK_destroy (decode reads it);
 *               `k` and `v` themselves may be released after the call.  One buffer for all layers.
 * Score[j] sums the squared keys over the kept rows only; everything downstream is thinK_compact
 * on the gathered tensors.  THINK_ERR_INVALID_ARG if tok_stride < n_b or n_b > src_tokens. */
thinK_status thinK_prefill_evicted(thinK_cache* c, thinK_tensor5 q_obs, thinK_tensor5 k, thinK_tensor5 v,
                                   const int32_t* tok, int64_t tok_stride, int32_t src_tokens, void* v_kept,
                                   int32_t layer0, int32_t nlayers, void* stream);

/* Bytes of the v_kept buffer of thinK_prefill_evicted: B * L * N_kv * S_max * D elements (0 if c is NULL). */
size_t thinK_v_kept_bytes(const thinK_cache* c);

/* Decode, Sec. 3.3: the new token's key and value join the unpruned tail.
 * k_new, v_new: dense [B, nlayers, N_kv, D].  Every layer of the cache must be
 * appended once per step (any split into layer ranges); THINK_ERR_CAPACITY once
 * max_new_tokens have been appended. */
thinK_status thinK_append(thinK_cache* c, const void* k_new, const void* v_new, int32_t layer0, int32_t nlayers,
                          void* stream);

/* Decode, Sec. 3.3 / Fig. 2 with the attention of Sec. 3.2: for each query head
 * the query is gathered to the kept channels and multiplied with the pruned
 * keys, the full query with the unpruned tail keys; the logits are concatenated,
 * scaled by 1/sqrt(D) (original D) and normalised by ONE softmax; the result is
 * the weighted sum of all value rows (prompt V in place + tail).
 *   q, out: dense [B, nlayers, N_q, D] in the cache dtype.
 * bf16: fp32 accumulation; fp32: logits in fp64, fp32 accumulation of p.V.
 * All layers in the range must hold the same number of tail tokens.
 * With lambda_v > 0 a pruned value channel of a prefix token counts as zero: output channel j sums the
 * tail tokens' share always and the prefix tokens' share only if j is kept. */
thinK_status thinK_decode_attn(thinK_cache* c, const void* q, void* out, int32_t layer0, int32_t nlayers,
                               void* stream);

/* One decode step in one call: thinK_append followed by thinK_decode_attn for the same layers (Sec. 3.3),
 * same arguments and results.  The attention kernel is launched as a programmatic dependent of the append
 * kernel: it starts streaming the pruned prefix while the append is still running and waits for it only
 * where it first touches the tail, which takes the append and the launch gap off the step's critical path.
 * bf16 caches; fp32 caches run the two launches back to back. */
thinK_status thinK_append_decode(thinK_cache* c, const void* k_new, const void* v_new, const void* q, void* out,
                                 int32_t layer0, int32_t nlayers, void* stream);

/* Score + select without any caller- or library-side allocation.  (The paper has no counterpart:
 * this is a packaging variant of thinK_score_select, same kernel, same results.)
 *
 * Who needs it: code that may not call cudaMalloc where it runs -- a plugin inside a host
 * application that hands out all device memory itself, a callback running under a memory pool that
 * forbids side allocations, or a process whose memory budget was fixed at start-up.  Such a caller
 * cannot provide the `workspace` that thinK_create asks for, so this call needs no handle and no
 * workspace: its scratch (lengths, ticket counters, fp64 partial sums) is a fixed 8 MiB array
 * compiled into the library.  Every GPU that loads the library holds those 8 MiB until exit.
 *
 *   cfg, seq_lens: as for thinK_cache_bytes (seq_lens on the HOST; copied with the stream).
 *   q_obs, k, layer0, nlayers: as for thinK_score_select.
 *   idx:    device out, uint8 [B, L, N_kv, T]; rows of the given layers are written.
 *   scores: device out, fp64 [B, L, N_kv, D], or NULL.
 *
 * Limit: lengths + counters + 2 * B * nlayers * C * 8 bytes per token split must fit in 8 MiB, where
 * C = N_kv*D when a token's keys are at most 4096 bytes, else N_kv*D rounded up to a whole number of
 * 4096-byte column blocks (2048 bf16 or 1024 fp32 columns each).  The call lowers its token split to
 * fit; if even one split does not fit it launches nothing and returns THINK_ERR_CAPACITY -- pass
 * fewer layers per call.
 * The first call on a device looks up the array's device address (once per device; make that first
 * call outside of any stream capture).  No cudaMalloc/cudaFree is called, here or later.
 * All calls share the one array, which still holds the previous call's contents: the call rewrites
 * the lengths and zeroes the tickets on `stream` before the kernel.  Two calls whose GPU work can
 * overlap (different streams, or different host threads without ordering) race on it: order them. */
thinK_status thinK_score_select_static(const thinK_config* cfg, const int32_t* seq_lens, thinK_tensor5 q_obs,
                                       thinK_tensor5 k, int32_t layer0, int32_t nlayers, uint8_t* idx,
                                       double* scores, void* stream);

/* Periodic re-pruning of the tail (App. C.1 of the paper, without its quantiser): the oldest unpruned
 * keys are thinned with the channels selected at prefill and joined to the pruned part, so the
 * full-width tail stops growing over a long generation.  Moves whole blocks of 64 tokens, oldest
 * first, for as long as at least `keep_recent` tokens stay unpruned; fewer movable tokens than 64 is
 * not an error (nothing happens).  The values of the moved tokens stay where they are (tail_v).
 * Attention afterwards treats those tokens like prefix tokens: gathered query x thinned keys.
 * bf16 caches only (THINK_ERR_UNSUPPORTED otherwise).  All layers of a decode call must have been
 * re-pruned alike.
 * What it saves is HBM traffic per decode step (the moved keys are read at T channels instead of D) and,
 * in the paper's accounting, cache size; it gives no ALLOCATED memory back: tail_k and tail_v stay sized
 * for S_recent + max_new_tokens full-width rows, positions keep counting against that capacity, and
 * k_thin carries ceil(cap/64) spare tiles per head for the moved blocks whether or not they are used.
 * thinK_sizes.model_think_bytes does not account for re-pruning. */
thinK_status thinK_reprune_tail(thinK_cache* c, int32_t keep_recent, int32_t layer0, int32_t nlayers, void* stream);

/* Tokens of the tail buffers of `layer` whose keys have been re-pruned (a multiple of 64), or -1. */
int32_t thinK_repruned_len(const thinK_cache* c, int32_t layer);

/* Tokens in the tail buffers of `layer` (S_recent + appended; re-pruned ones included), or -1. */
int32_t thinK_tail_len(const thinK_cache* c, int32_t layer);

/* Reads the device-side error word (0 = none) with a synchronous copy.  Bits: 1 a kept-token index of
 * thinK_prefill_evicted was out of range; 2 a bounded wait inside a kernel ran out (value-score kernel: that unit's
 * selection is missing; compaction: a tile whose row copies did not complete within about a second is left
 * unwritten -- re-create the cache); 4 a kernel found its shared memory misaligned; 8 a channel score was NaN or infinite (non-finite K or Q: exactly T channels
 * are still selected, NaN scores ranking lowest). */
thinK_status thinK_device_error(thinK_cache* c, int32_t* out_code);

thinK_status thinK_destroy(thinK_cache* c);

#ifdef __cplusplus
}
#endif
#endif /* THINK_H_ */
