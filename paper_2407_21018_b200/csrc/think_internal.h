// Internal declarations shared by the translation units of libthink.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "think.h"

namespace think {

constexpr int kTileTokens = 64;       // tokens per key tile (rows of 64 tokens, channel-major)
constexpr int kSMs = 148;             // B200; used only to size the workspace
constexpr int kScoreThreads = 256;
constexpr int kScoreTargetCtas = kSMs * 8;
constexpr int kMaxDecodeCtas = kSMs * 16;

struct View5 {
  const void* ptr;
  int64_t sb, ss, sl, sn;   // element strides
};

// Optional token-eviction hook: kept token i of unit (b, l, h) is row rows[unit * stride + i] of the
// source views.  rows == nullptr means the identity (row i).  Entries outside [0, src_tokens) set the
// error word and are read as row 0.
struct TokenMap {
  const int32_t* rows;
  int64_t stride;
  int32_t src_tokens;
  uint32_t* error;
};
constexpr uint32_t kErrTokenRange = 1u;   // device error word: a token index was out of range
constexpr uint32_t kErrWaitTimeout = 2u;  // device error word: a bounded wait on an mbarrier ran out
constexpr uint32_t kErrSmemAlign = 4u;    // device error word: dynamic shared memory not on a 1024-byte boundary
constexpr uint32_t kErrNonFinite = 8u;    // device error word: a channel score was NaN or infinite (non-finite K or Q)

struct ScoreParams {
  TokenMap tok;
  View5 k, q;
  const int32_t* seq_len;
  double* partials;
  uint32_t* counters;
  uint8_t* idx;             // [B, L, N_kv, T]
  double* scores;           // [B, L, N_kv, D] or null
  int B, L, N_kv, G, D, T, S_obs;
  int layer0, nlayers;
  int NC;                   // 16-byte chunks per token over all heads
  int CB;                   // chunks per column block
  int ncolblk, nsplit, RP;  // RP = rows in flight per CTA iteration
  int criterion;
  uint32_t* error;          // device error word (may be null)
};

struct CompactParams {
  TokenMap tok;
  View5 k;
  const int32_t* seq_len;
  const int64_t* thin_tile_base;
  const uint8_t* idx;
  void* k_thin;
  int B, L, N_kv, D, T, Tp, R;   // Tp = rows stored per thin tile (T padded to 8 for bf16)
  int re_cap;                    // tiles reserved per head after the prompt's thin tiles (re-pruned tail blocks)
  int layer0, nlayers;
  int max_tiles;                 // longest pruned prefix of the batch, in tiles
  int heads_first;               // CTA order of the bf16 kernel (set by the launcher)
  uint32_t* error;               // device error word (may be null)
};

struct RepruneParams {       // 64-token blocks of the unpruned tail -> thinned tiles (bf16)
  const uint8_t* idx;
  const int64_t* thin_tile_base;
  const int32_t* cum_thin;
  void* k_thin;
  const void* tail_k;
  int B, L, N_kv, D, T, Tp, re_cap, tail_tiles_cap;
  int layer0, nlayers;
  int blk0, nblk;           // tail tiles [blk0, blk0 + nblk)
};

struct GatherRowsParams {    // values of the kept tokens -> dense [B, L, N_kv, S_max, D]
  TokenMap tok;
  View5 v;
  const int32_t* seq_len;
  void* dst;
  int B, L, N_kv, D, S_max;
  int layer0, nlayers;
};

struct ValueScoreParams {    // App. D: Score_v = column norms of the window's attention output
  View5 q, k, v;
  const int32_t* seq_len;
  float* partials;          // per (unit, row block, split): float m[MB] | float l[MB] | float O[MB][D]
  uint32_t* counters;       // per unit of the launch
  uint8_t* perm_v;          // [B, L, N_kv, D]: kept value channels ascending, then the pruned ones ascending
  double* scores_v;         // [B, L, N_kv, D] or null
  int B, L, N_kv, G, D, Tv, S_obs;
  int layer0, nlayers;
  int M;                    // G * S_obs query rows per unit
  int MB;                   // rows per row block (multiple of 16, <= 128)
  int nrb, nsplit;
  int use_tcgen05;          // D = 128 and MB = 128: 1 tcgen05 kernel (accumulators in tensor memory), 0 mma.sync kernel
  uint32_t* error;          // device error word
};

struct CompactValueParams {  // V_T[t][c] = V[t][perm_v[c]], t < S_p; rows of Tvp elements (zero padded)
  View5 v;
  const int32_t* seq_len;
  const int64_t* v_thin_base;   // element offset of entry b's block in v_thin
  const uint8_t* perm_v;
  void* v_thin;
  int B, L, N_kv, D, Tv, Tvp, R;
  int S_pmax;                   // longest pruned prefix over the batch
  int layer0, nlayers;
};

struct TailWriteParams {
  TokenMap tok;             // applies when rows_from_seq_len is set
  const uint8_t* perm_v;    // value-channel pruning: tail values are stored in the order perm_v[unit][0..D) (null: as is)
  View5 k, v;               // sources
  int src_layer_base;       // layer index subtracted before applying sl
  int rows_from_seq_len;    // 1: source row = seq_len[b] - R + r ; 0: source row = r
  const int32_t* seq_len;
  void* tail_k;
  void* tail_v;
  int B, L, N_kv, D, R, cap, tail_tiles_cap;
  int layer0, nlayers;
  int nrows, pos0;          // tail positions [pos0, pos0 + nrows)
};

struct DecodeParams {
  const void* k_thin;
  const void* tail_k;
  const void* tail_v;
  View5 v;                  // prompt values, read in place for tokens < S_p
  const uint8_t* idx;
  const void* q;            // [B, nlayers, N_q, D]
  void* out;
  const int32_t* seq_len;
  const int32_t* cum_thin;
  const int64_t* thin_tile_base;
  uint8_t* records;
  uint32_t* counters;
  int B, L, N_kv, N_q, T, Tp, R, cap, tail_tiles_cap;
  int re_cap;               // tiles reserved per head after the prompt's thin tiles
  int n_re;                 // of which hold re-pruned tail blocks (64 tokens each, values stay in tail_v)
  int n_tail;               // tokens in the tail buffers (re-pruned blocks included)
  int n_tail_tiles;
  // value-channel pruning (App. D): prefix values hold Tvp kept channels per row; tail values and the
  // accumulators use the channel order perm_v[unit][0..D) (kept ascending, then pruned ascending)
  const void* v_thin;
  const int64_t* v_thin_base;
  const uint8_t* perm_v;
  int Tvp;
  int layer0, nlayers;
  long long Ntot;           // tiles over all units of this call
  int grid;
  int dependent_launch;     // host side: launch so that the kernel may start while the preceding kernel of the
                            // stream (the append) is still running; it waits before its first read of the tail
};

// launchers (one per translation unit); return the launch status
cudaError_t launch_score(const ScoreParams& p, int dtype, cudaStream_t s);
int score_ctas_per_sm(int dtype, int criterion);
cudaError_t launch_compact(const CompactParams& p, int dtype, int max_tiles, cudaStream_t s);
cudaError_t launch_tail_write(const TailWriteParams& p, int dtype, cudaStream_t s, bool overlap_previous = false);
cudaError_t launch_reprune(const RepruneParams& p, cudaStream_t s);
cudaError_t launch_score_value(const ValueScoreParams& p, int threads, cudaStream_t s);
cudaError_t score_value_setup(int D);
size_t score_value_record_bytes(int MB, int D);
cudaError_t launch_compact_value(const CompactValueParams& p, cudaStream_t s);
cudaError_t launch_gather_rows(const GatherRowsParams& p, int dtype, cudaStream_t s);
cudaError_t launch_decode(const DecodeParams& p, int dtype, int D, int G, cudaStream_t s);
cudaError_t decode_setup(int dtype, int D, int G);   // one-time per-process kernel attributes
int decode_workers_per_cta(int dtype);
bool decode_supported(int dtype, int D, int G);
int decode_ctas_per_sm(int dtype, int D, int G);
size_t decode_record_bytes(int D, int G);

// Partial softmax state of one (worker, unit): double m[G] | float l[G] | pad to 16 | float o[G][D].
constexpr __host__ __device__ int rec_o_off(int G) { return (G * 12 + 15) & ~15; }
constexpr __host__ __device__ size_t rec_size(int D, int G) { return (size_t)rec_o_off(G) + (size_t)G * D * 4; }

// Rows stored per thin tile: bf16 tiles are laid out in MMA-fragment order and pad T to a
// multiple of 8 (zero rows); fp32 tiles are channel-major with exactly T rows.
inline int padded_T(int T, int dtype) { return dtype == THINK_BF16 ? (T + 7) & ~7 : T; }

// ---- device helpers ------------------------------------------------------
#ifdef __CUDACC__
// bf16 key tile of 64 tokens x Cp channels (Cp % 8 == 0) in MMA-fragment order.  The tile is four
// 16-token steps of Cp*32 bytes.  Inside a step, for every 16-channel group s a 512-byte chunk holds,
// per lane i (r = i/4, q = i%4), the B fragments of mma.m16n8k16 for the two 8-token halves jx:
// [b0(jx=0) b1(jx=0) b0(jx=1) b1(jx=1)], b0 = channels 16s+2q,+1, b1 = channels 16s+2q+8,+9 of token
// 16*step + 8*jx + r.  A trailing group of 8 channels (Cp % 16 == 8) is a 256-byte block with 8 bytes
// per lane: [b(jx=0) b(jx=1)], channels 16*n16+2q,+1 (B fragments of mma.m16n8k8).
// Returns the byte offset of element (token u, channel c).
__host__ __device__ __forceinline__ int frag_elem_byte(int Cp, int c, int u) {
  const int n16 = Cp >> 4;
  const int step = u >> 4, jx = (u >> 3) & 1, r = u & 7;
  const int base = step * Cp * 32;
  if (c < n16 * 16) {
    const int s = c >> 4, w = c & 15, half = w >> 3, q = (w & 7) >> 1, lo = w & 1;
    return base + s * 512 + (r * 4 + q) * 16 + (jx * 2 + half) * 4 + lo * 2;
  }
  const int w = c - n16 * 16, q = w >> 1, lo = w & 1;
  return base + n16 * 512 + (r * 4 + q) * 8 + jx * 4 + lo * 2;
}

// source row of kept token i of `unit`
__device__ __forceinline__ int64_t token_row(const TokenMap& m, int64_t unit, int i) {
  if (!m.rows) return i;
  const int32_t r = __ldg(m.rows + unit * m.stride + i);
  if ((uint32_t)r >= (uint32_t)m.src_tokens) {
    atomicOr(m.error, kErrTokenRange);
    return 0;
  }
  return r;
}

// Rank-count selection of one head by one warp: channel j is kept when fewer than T channels
// beat it, where k beats j if s[k] > s[j] or (s[k] == s[j] and k < j).  out[0..T) = kept channels
// ascending; with `rest`, out[T..D) = the other channels ascending (out is then a permutation).
// A NaN score ranks as -infinity, so the order is total and exactly T channels are kept whatever
// the inputs; a NaN or infinite score raises kErrNonFinite in *error (when given).
// A lane holds the scores of its channels (j = lane, lane + 32, ...; D <= 128) in registers and walks
// all k once, eight broadcast loads at a time, counting for its channels together.
__device__ __forceinline__ void select_head(const double* s, int D, int T, uint8_t* out, int lane, bool rest,
                                            uint32_t* error = nullptr) {
  constexpr int MAXJ = 4;                       // channels per lane: D <= 32 * MAXJ
  double sj[MAXJ];
  int rank[MAXJ];
  bool bad = false;
#pragma unroll
  for (int i = 0; i < MAXJ; ++i) {
    const int j = lane + 32 * i;
    double v = j < D ? s[j] : 0.0;
    bad |= j < D && !(fabs(v) <= 1.7976931348623157e308);
    if (!(v == v)) v = -INFINITY;
    sj[i] = v;
    rank[i] = 0;
  }
  for (int k0 = 0; k0 < D; k0 += 8) {
    double sk[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      sk[u] = s[k0 + u];                        // D is a multiple of 8
      if (!(sk[u] == sk[u])) sk[u] = -INFINITY;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
#pragma unroll
      for (int i = 0; i < MAXJ; ++i) rank[i] += (sk[u] > sj[i]) || (sk[u] == sj[i] && k0 + u < lane + 32 * i);
    }
  }
  int base = 0, base_rest = T;
#pragma unroll
  for (int i = 0; i < MAXJ; ++i) {
    const int j = lane + 32 * i;
    if (32 * i >= D) break;
    const bool keep = j < D && rank[i] < T;
    const unsigned m = __ballot_sync(0xffffffffu, keep);
    const unsigned below = (1u << lane) - 1u;
    if (keep) out[base + __popc(m & below)] = (uint8_t)j;
    base += __popc(m);
    if (rest) {
      const unsigned valid = __ballot_sync(0xffffffffu, j < D);
      const unsigned o = valid & ~m;
      if (j < D && !keep) out[base_rest + __popc(o & below)] = (uint8_t)j;
      base_rest += __popc(o);
    }
  }
  if (error && __any_sync(0xffffffffu, bad) && lane == 0) atomicOr(error, kErrNonFinite);
}

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// byte offset of token u (0..63) inside row c of a channel-major tile, element size e
__device__ __forceinline__ int tile_swz_bytes(int c, int u, int e) {
  int byte = u * e;
  return (((byte >> 4) ^ (c & 7)) << 4) | (byte & 15);
}
#endif

}  // namespace think
