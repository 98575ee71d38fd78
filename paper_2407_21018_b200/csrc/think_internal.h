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
constexpr int kMaxGroup = 8;

struct View5 {
  const void* ptr;
  int64_t sb, ss, sl, sn;   // element strides
};

struct ScoreParams {
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
};

struct CompactParams {
  View5 k;
  const int32_t* seq_len;
  const int64_t* thin_tile_base;
  const uint8_t* idx;
  void* k_thin;
  int B, L, N_kv, D, T, R;
  int layer0, nlayers;
};

struct TailWriteParams {
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
  int B, L, N_kv, N_q, T, R, cap, tail_tiles_cap;
  int n_tail;               // tokens in the tail
  int n_tail_tiles;
  int layer0, nlayers;
  long long Ntot;           // tiles over all units of this call
  int grid;
};

// launchers (one per translation unit); return the launch status
cudaError_t launch_score(const ScoreParams& p, int dtype, cudaStream_t s);
cudaError_t launch_compact(const CompactParams& p, int dtype, int max_tiles, cudaStream_t s);
cudaError_t launch_tail_write(const TailWriteParams& p, int dtype, cudaStream_t s);
cudaError_t launch_decode(const DecodeParams& p, int dtype, int D, int G, cudaStream_t s);
bool decode_supported(int dtype, int D, int G);
int decode_ctas_per_sm(int dtype, int D, int G);
size_t decode_record_bytes(int D, int G);

// ---- device helpers ------------------------------------------------------
#ifdef __CUDACC__
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// byte offset of token u (0..63) inside row c of a channel-major tile, element size e
__device__ __forceinline__ int tile_swz_bytes(int c, int u, int e) {
  int byte = u * e;
  return (((byte >> 4) ^ (c & 7)) << 4) | (byte & 15);
}
#endif

}  // namespace think
