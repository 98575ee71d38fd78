// Host side of the C ABI: validation, buffer sizing, bookkeeping of the tail length, launches.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "think_internal.h"

using namespace think;

namespace {
// NVTX range around an entry point (shows the ABI calls on a profiler's timeline; a no-op without a tool attached)
struct Range {
  explicit Range(const char* name) { nvtxRangePushA(name); }
  ~Range() { nvtxRangePop(); }
};
}  // namespace

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {            // byte offsets inside the workspace
  size_t seq_len, cum_thin, thin_tile_base, error, v_thin_base, score_counters, decode_counters;
  size_t score_partials, decode_records, total;
  size_t value_counters, value_partials;   // value-channel scoring (only with lambda_v > 0)
  size_t header_bytes;     // everything before score_partials (initialised by thinK_create)
};

struct Geometry {
  int B, L, N_q, N_kv, D, G, T, Tp, S_obs, S_max, R, max_new, cap, tail_tiles_cap, E, dtype, criterion;
  int NC, CB, ncolblk, RPmax;
  // value-channel pruning (App. D)
  bool vt;
  int Tv, Tvp;                 // kept value channels, padded to a multiple of 16
  int value_score_kernel;      // thinK_value_score_kernel
  int M, MB, nrb;              // query rows per unit of the value score, rows per row block, row blocks
  int value_slots;             // partial records the workspace holds
  int S_pmax;
  std::vector<int64_t> v_thin_base;   // element offsets per batch entry (+ total)
  int64_t total_thin_tiles;    // over all (b, l, h)
  int max_thin_tiles;          // per (l, h) over b
  std::vector<int32_t> seq_len, cum_thin;
  std::vector<int64_t> thin_tile_base;
};

thinK_status make_geometry(const thinK_config* c, const int32_t* seq_lens, Geometry* g) {
  if (!c || !seq_lens) return THINK_ERR_INVALID_ARG;
  if (c->B < 1 || c->L < 1 || c->N_q < 1 || c->N_kv < 1 || c->S_obs < 1 || c->S_recent < 0 ||
      c->max_new_tokens < 0 || c->S_max < 1)
    return THINK_ERR_INVALID_ARG;
  if (c->N_q % c->N_kv != 0) return THINK_ERR_INVALID_ARG;
  if (c->dtype != THINK_BF16 && c->dtype != THINK_F32) return THINK_ERR_UNSUPPORTED;
  if (c->criterion < THINK_SCORE_QUERY_DRIVEN || c->criterion > THINK_SCORE_KEY_L1) return THINK_ERR_INVALID_ARG;
  if (!decode_supported(c->dtype, c->D, c->N_q / c->N_kv)) return THINK_ERR_UNSUPPORTED;
  const int T = thinK_T(c->lambda, c->D);
  if (T < 1) return THINK_ERR_INVALID_ARG;
  if ((int64_t)c->B * c->L > 65535) return THINK_ERR_UNSUPPORTED;
  g->B = c->B; g->L = c->L; g->N_q = c->N_q; g->N_kv = c->N_kv; g->D = c->D; g->G = c->N_q / c->N_kv;
  g->T = T; g->Tp = padded_T(T, c->dtype); g->S_obs = c->S_obs; g->S_max = c->S_max; g->R = c->S_recent; g->max_new = c->max_new_tokens; g->cap = c->S_recent + c->max_new_tokens;
  if (g->cap < 1) g->cap = 1;
  g->tail_tiles_cap = (g->cap + kTileTokens - 1) / kTileTokens;
  g->dtype = c->dtype; g->E = c->dtype == THINK_BF16 ? 2 : 4; g->criterion = c->criterion;
  if (c->value_score_kernel != THINK_VALUE_SCORE_AUTO && c->value_score_kernel != THINK_VALUE_SCORE_MMA_SYNC)
    return THINK_ERR_INVALID_ARG;
  g->value_score_kernel = c->value_score_kernel;
  const int CH = 16 / g->E;
  g->NC = c->N_kv * c->D / CH;
  g->CB = g->NC < kScoreThreads ? g->NC : kScoreThreads;
  g->ncolblk = (g->NC + g->CB - 1) / g->CB;
  g->RPmax = kScoreThreads / g->CB;
  g->seq_len.assign(seq_lens, seq_lens + c->B);
  g->cum_thin.assign(c->B + 1, 0);
  g->thin_tile_base.assign(c->B + 1, 0);
  g->max_thin_tiles = 0;
  for (int b = 0; b < c->B; ++b) {
    const int S = seq_lens[b];
    if (S < c->S_obs || S < c->S_recent || S > c->S_max || S < 1) return THINK_ERR_INVALID_ARG;
    const int nt = (S - c->S_recent + kTileTokens - 1) / kTileTokens;
    g->cum_thin[b + 1] = g->cum_thin[b] + nt;
    g->thin_tile_base[b + 1] = g->thin_tile_base[b] + (int64_t)c->L * c->N_kv * (nt + g->tail_tiles_cap);
    if (nt > g->max_thin_tiles) g->max_thin_tiles = nt;
  }
  g->total_thin_tiles = g->thin_tile_base[c->B];
  // value channels
  if (!(c->lambda_v >= 0.0 && c->lambda_v < 1.0)) return THINK_ERR_INVALID_ARG;
  g->vt = c->lambda_v > 0.0;
  g->Tv = thinK_T(c->lambda_v, c->D);
  if (g->Tv < 1) return THINK_ERR_INVALID_ARG;
  g->Tvp = (g->Tv + 15) & ~15;
  g->M = g->G * c->S_obs;
  g->MB = g->M < 128 ? (g->M + 15) & ~15 : 128;
  g->nrb = (g->M + g->MB - 1) / g->MB;
  g->value_slots = 0;
  g->S_pmax = 0;
  g->v_thin_base.assign(c->B + 1, 0);
  if (g->vt) {
    if (c->dtype != THINK_BF16) return THINK_ERR_UNSUPPORTED;
    if (g->M > 2048) return THINK_ERR_UNSUPPORTED;
    // partial records of the value score: 48 MB worth, at least one layer's
    const int per_layer = c->B * c->N_kv * g->nrb;
    const size_t by_bytes = ((size_t)48 << 20) / score_value_record_bytes(g->MB, c->D);
    g->value_slots = (size_t)per_layer > by_bytes ? per_layer : (int)by_bytes;
    for (int b = 0; b < c->B; ++b) {
      const int S_p = seq_lens[b] - c->S_recent;
      if (S_p > g->S_pmax) g->S_pmax = S_p;
      g->v_thin_base[b + 1] = g->v_thin_base[b] + (int64_t)c->L * c->N_kv * S_p * g->Tvp;
    }
  }
  return THINK_OK;
}

void make_layout(const Geometry& g, Layout* w) {
  size_t o = 0;
  w->seq_len = o;          o = align_up(o + sizeof(int32_t) * g.B, 256);
  w->cum_thin = o;         o = align_up(o + sizeof(int32_t) * (g.B + 1), 256);
  w->thin_tile_base = o;   o = align_up(o + sizeof(int64_t) * (g.B + 1), 256);
  w->error = o;            o = align_up(o + 256, 256);
  w->v_thin_base = o;      o = align_up(o + sizeof(int64_t) * (g.B + 1), 256);
  w->score_counters = o;   o = align_up(o + sizeof(uint32_t) * (size_t)g.B * g.L * g.ncolblk, 256);
  w->decode_counters = o;  o = align_up(o + sizeof(uint32_t) * (size_t)g.B * g.L * g.N_kv, 256);
  w->value_counters = o;
  if (g.vt) o = align_up(o + sizeof(uint32_t) * (size_t)g.B * g.L * g.N_kv, 256);   // zeroed with the header
  w->header_bytes = o;
  w->score_partials = o;
  // a call splits tokens so that items * nsplit <= target + items
  const size_t slots = (size_t)kScoreTargetCtas + (size_t)g.B * g.L * g.ncolblk;
  o = align_up(o + slots * 2 * (size_t)g.CB * (16 / g.E) * sizeof(double), 256);
  w->decode_records = o;
  o = align_up(o + (size_t)kMaxDecodeCtas * 2 * decode_record_bytes(g.D, g.G), 256);
  w->value_partials = o;
  if (g.vt) o = align_up(o + (size_t)g.value_slots * score_value_record_bytes(g.MB, g.D), 256);
  w->total = o;
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

bool check_view(const thinK_tensor5& t, int E) {
  if (!t.ptr || !aligned16(t.ptr)) return false;
  const int64_t s[4] = {t.stride_b, t.stride_s, t.stride_l, t.stride_n};
  for (int i = 0; i < 4; ++i)
    if (s[i] < 0 || (s[i] * E) % 16 != 0) return false;
  return true;
}

View5 to_view(const thinK_tensor5& t) { return View5{t.ptr, t.stride_b, t.stride_s, t.stride_l, t.stride_n}; }

}  // namespace

struct thinK_cache {
  Geometry g;
  Layout w;
  unsigned char* ws;
  void *k_thin, *tail_k, *tail_v, *idx, *scores;
  void *v_thin, *perm_v, *scores_v;         // value-channel pruning (attached separately)
  std::vector<uint8_t> scored, compacted;   // per layer
  std::vector<uint8_t> scored_v;            // per layer: value channels ranked
  std::vector<int32_t> tail_len;            // per layer, tokens in the tail buffers
  std::vector<int32_t> n_re;                // per layer, 64-token tail blocks already re-pruned
  thinK_tensor5 v;                          // borrowed prompt values (set by thinK_compact)
  bool have_v;
  thinK_sizes have_sizes, need_sizes;       // bytes of the caller's buffers as stated at thinK_create / as required
  int num_sms, decode_grid_max;
  int score_capacity;                       // resident CTAs of the score kernel on this device
  int value_score_tcgen05;                  // 0: the mma.sync value-score kernel everywhere (cfg.value_score_kernel)
};

extern "C" {

int32_t thinK_T(double lambda, int32_t D) {
  if (!(lambda >= 0.0 && lambda < 1.0) || D < 1) return 0;
  const int32_t T = (int32_t)floor((1.0 - lambda) * (double)D + 1e-9);
  return T < 1 ? 0 : (T > D ? D : T);
}

const char* thinK_status_string(thinK_status s) {
  switch (s) {
    case THINK_OK: return "ok";
    case THINK_ERR_INVALID_ARG: return "invalid argument";
    case THINK_ERR_UNSUPPORTED: return "unsupported configuration";
    case THINK_ERR_STATE: return "call out of order";
    case THINK_ERR_CAPACITY: return "capacity exceeded";
    case THINK_ERR_CUDA: return "CUDA error";
  }
  return "unknown status";
}

thinK_status thinK_cache_bytes(const thinK_config* cfg, const int32_t* seq_lens, thinK_sizes* out) {
  if (!out) return THINK_ERR_INVALID_ARG;
  Geometry g;
  thinK_status st = make_geometry(cfg, seq_lens, &g);
  if (st != THINK_OK) return st;
  Layout w;
  make_layout(g, &w);
  const size_t units = (size_t)g.B * g.L * g.N_kv;
  out->k_thin = align_up((size_t)g.total_thin_tiles * g.Tp * kTileTokens * g.E, 256);
  if (out->k_thin == 0) out->k_thin = 256;
  out->tail_k = align_up(units * g.tail_tiles_cap * (size_t)g.D * kTileTokens * g.E, 256);
  out->tail_v = align_up(units * g.cap * (size_t)g.D * g.E, 256);
  out->idx = align_up(units * g.T, 256);
  out->scores = align_up(units * g.D * sizeof(double), 256);
  out->workspace = w.total;
  size_t think_elems = 0, dense_elems = 0;
  const int new_tokens = cfg->max_new_tokens;
  for (int b = 0; b < g.B; ++b) {
    const size_t S = g.seq_len[b], S_p = S - g.R;
    think_elems += S_p * g.T + (size_t)(g.R + new_tokens) * g.D + (S + new_tokens) * g.D;
    dense_elems += 2 * (S + new_tokens) * g.D;
  }
  out->v_thin = out->perm_v = 0;
  if (g.vt) {
    out->v_thin = align_up((size_t)g.v_thin_base[g.B] * g.E, 256);
    if (out->v_thin == 0) out->v_thin = 256;
    out->perm_v = align_up(units * g.D, 256);
    // the prefix values shrink to T_v channels as well
    for (int b = 0; b < g.B; ++b) think_elems -= (size_t)(g.seq_len[b] - g.R) * (g.D - g.Tv);
  }
  out->model_think_bytes = think_elems * g.L * g.N_kv * g.E;
  out->model_dense_bytes = dense_elems * g.L * g.N_kv * g.E;
  return THINK_OK;
}

thinK_status thinK_create(const thinK_config* cfg, const int32_t* seq_lens, const thinK_sizes* sizes, void* k_thin,
                          void* tail_k, void* tail_v, void* idx, void* scores, void* workspace, thinK_cache** out) {
  Range nvtx_range("thinK_create");
  if (!out) return THINK_ERR_INVALID_ARG;
  *out = nullptr;
  if (!sizes || !k_thin || !tail_k || !tail_v || !idx || !workspace) return THINK_ERR_INVALID_ARG;
  thinK_sizes need;
  {
    // the caller states how large its buffers are; anything below what this configuration needs is refused
    thinK_status st = thinK_cache_bytes(cfg, seq_lens, &need);
    if (st != THINK_OK) return st;
    if (sizes->k_thin < need.k_thin || sizes->tail_k < need.tail_k || sizes->tail_v < need.tail_v ||
        sizes->idx < need.idx || sizes->workspace < need.workspace || (scores && sizes->scores < need.scores))
      return THINK_ERR_CAPACITY;
  }
  if (!aligned16(k_thin) || !aligned16(tail_k) || !aligned16(tail_v) || !aligned16(workspace) ||
      (scores && !aligned16(scores)))
    return THINK_ERR_INVALID_ARG;
  thinK_cache* c = new (std::nothrow) thinK_cache();
  if (!c) return THINK_ERR_INVALID_ARG;
  thinK_status st = make_geometry(cfg, seq_lens, &c->g);
  if (st != THINK_OK) { delete c; return st; }
  make_layout(c->g, &c->w);
  c->ws = (unsigned char*)workspace;
  c->k_thin = k_thin; c->tail_k = tail_k; c->tail_v = tail_v; c->idx = idx; c->scores = scores;
  c->v_thin = c->perm_v = c->scores_v = nullptr;
  c->have_sizes = *sizes;
  c->need_sizes = need;
  c->value_score_tcgen05 = c->g.value_score_kernel == THINK_VALUE_SCORE_MMA_SYNC ? 0 : 1;
  c->scored_v.assign(c->g.L, 0);
  c->scored.assign(c->g.L, 0);
  c->compacted.assign(c->g.L, 0);
  c->tail_len.assign(c->g.L, 0);
  c->n_re.assign(c->g.L, 0);
  c->have_v = false;
  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
    delete c;
    return THINK_ERR_CUDA;
  }
  c->num_sms = prop.multiProcessorCount;
  if (decode_setup(c->g.dtype, c->g.D, c->g.G) != cudaSuccess) { delete c; return THINK_ERR_CUDA; }
  if (c->g.vt && score_value_setup(c->g.D) != cudaSuccess) { delete c; return THINK_ERR_CUDA; }
  int occ = decode_ctas_per_sm(c->g.dtype, c->g.D, c->g.G);
  if (occ < 1) { delete c; return THINK_ERR_CUDA; }
  c->decode_grid_max = c->num_sms * occ;
  const int wpc = decode_workers_per_cta(c->g.dtype);
  if (c->decode_grid_max * wpc > kMaxDecodeCtas) c->decode_grid_max = kMaxDecodeCtas / wpc;
  c->score_capacity = c->num_sms * score_ctas_per_sm(c->g.dtype, c->g.criterion);
  if (c->score_capacity < 1) { delete c; return THINK_ERR_CUDA; }
  // device tables
  const Geometry& g = c->g;
  bool ok = cudaMemset(c->ws, 0, c->w.header_bytes) == cudaSuccess;
  ok = ok && cudaMemcpy(c->ws + c->w.seq_len, g.seq_len.data(), sizeof(int32_t) * g.B, cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(c->ws + c->w.cum_thin, g.cum_thin.data(), sizeof(int32_t) * (g.B + 1), cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(c->ws + c->w.thin_tile_base, g.thin_tile_base.data(), sizeof(int64_t) * (g.B + 1), cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(c->ws + c->w.v_thin_base, g.v_thin_base.data(), sizeof(int64_t) * (g.B + 1), cudaMemcpyHostToDevice) == cudaSuccess;
  if (!ok) { delete c; return THINK_ERR_CUDA; }
  *out = c;
  return THINK_OK;
}

static bool layer_range_ok(const thinK_cache* c, int layer0, int nlayers) {
  return layer0 >= 0 && nlayers >= 1 && layer0 + nlayers <= c->g.L;
}

}  // extern "C"

namespace {
const TokenMap kNoTokenMap = {nullptr, 0, 0, nullptr};

thinK_status make_token_map(thinK_cache* c, const int32_t* tok, int64_t tok_stride, int32_t src_tokens, TokenMap* m) {
  if (!tok || ((uintptr_t)tok & 3) != 0 || src_tokens < 1) return THINK_ERR_INVALID_ARG;
  for (int b = 0; b < c->g.B; ++b)
    if (tok_stride < c->g.seq_len[b] || c->g.seq_len[b] > src_tokens) return THINK_ERR_INVALID_ARG;
  m->rows = tok; m->stride = tok_stride; m->src_tokens = src_tokens;
  m->error = (uint32_t*)(c->ws + c->w.error);
  return THINK_OK;
}

thinK_status score_select_impl(thinK_cache* c, thinK_tensor5 q_obs, thinK_tensor5 k, const TokenMap& tok,
                               int32_t layer0, int32_t nlayers, void* stream) {
  if (!c) return THINK_ERR_INVALID_ARG;
  if (!layer_range_ok(c, layer0, nlayers)) return THINK_ERR_INVALID_ARG;
  const Geometry& g = c->g;
  if (!check_view(k, g.E)) return THINK_ERR_INVALID_ARG;
  if (g.criterion == THINK_SCORE_QUERY_DRIVEN && !check_view(q_obs, g.E)) return THINK_ERR_INVALID_ARG;
  ScoreParams p;
  memset(&p, 0, sizeof(p));
  p.tok = tok;
  p.k = to_view(k);
  p.q = to_view(q_obs);
  p.seq_len = (const int32_t*)(c->ws + c->w.seq_len);
  p.partials = (double*)(c->ws + c->w.score_partials);
  p.counters = (uint32_t*)(c->ws + c->w.score_counters);
  p.idx = (uint8_t*)c->idx;
  p.scores = (double*)c->scores;
  p.B = g.B; p.L = g.L; p.N_kv = g.N_kv; p.G = g.G; p.D = g.D; p.T = g.T; p.S_obs = g.S_obs;
  p.layer0 = layer0; p.nlayers = nlayers;
  p.NC = g.NC; p.CB = g.CB; p.ncolblk = g.ncolblk; p.RP = g.RPmax;
  p.criterion = g.criterion;
  p.error = (uint32_t*)(c->ws + c->w.error);
  const int items = g.B * nlayers * g.ncolblk;
  // one wave of CTAs: the token split fills the resident slots without spilling into a second wave
  int nsplit = c->score_capacity / items;
  if (nsplit > (kScoreTargetCtas + items - 1) / items) nsplit = (kScoreTargetCtas + items - 1) / items;
  // keep at least 64 token rows per row lane of a split
  int min_len = g.seq_len[0];
  for (int b = 1; b < g.B; ++b) min_len = g.seq_len[b] < min_len ? g.seq_len[b] : min_len;
  int cap = min_len / (64 * p.RP);
  if (cap < 1) cap = 1;
  if (nsplit > cap) nsplit = cap;
  if (nsplit < 1) nsplit = 1;
  p.nsplit = nsplit;
  if (launch_score(p, g.dtype, (cudaStream_t)stream) != cudaSuccess) return THINK_ERR_CUDA;
  for (int l = layer0; l < layer0 + nlayers; ++l) c->scored[l] = 1;
  return THINK_OK;
}

thinK_status seed_tail(thinK_cache* c, thinK_tensor5 k, thinK_tensor5 v, const TokenMap& tok, thinK_tensor5 v_prefix,
                       int layer0, int nlayers, void* stream);

// `v_prefix`: where decode finds the values of the prefix tokens (the prompt's V itself, or the
// gathered copy when a token map is in use)
thinK_status compact_impl(thinK_cache* c, thinK_tensor5 k, thinK_tensor5 v, const TokenMap& tok, thinK_tensor5 v_prefix,
                          int32_t layer0, int32_t nlayers, void* stream) {
  if (!c) return THINK_ERR_INVALID_ARG;
  if (!layer_range_ok(c, layer0, nlayers)) return THINK_ERR_INVALID_ARG;
  const Geometry& g = c->g;
  if (!check_view(k, g.E) || !check_view(v, g.E)) return THINK_ERR_INVALID_ARG;
  for (int l = layer0; l < layer0 + nlayers; ++l)
    if (!c->scored[l]) return THINK_ERR_STATE;
  if (g.vt) {
    if (tok.rows) return THINK_ERR_UNSUPPORTED;
    if (!c->v_thin) return THINK_ERR_STATE;
    for (int l = layer0; l < layer0 + nlayers; ++l)
      if (!c->scored_v[l]) return THINK_ERR_STATE;
  } else if (c->have_v && memcmp(&c->v, &v_prefix, sizeof(v_prefix)) != 0) {
    // A different V view is a new prompt: decode reads the prefix values of all layers through ONE borrowed
    // view, so the layers outside this call fall back to "not compacted" until they are compacted again.
    for (int l = 0; l < g.L; ++l)
      if (l < layer0 || l >= layer0 + nlayers) c->compacted[l] = 0;
    c->have_v = false;
  }
  CompactParams p;
  memset(&p, 0, sizeof(p));
  p.tok = tok;
  p.k = to_view(k);
  p.seq_len = (const int32_t*)(c->ws + c->w.seq_len);
  p.thin_tile_base = (const int64_t*)(c->ws + c->w.thin_tile_base);
  p.idx = (const uint8_t*)c->idx;
  p.k_thin = c->k_thin;
  p.B = g.B; p.L = g.L; p.N_kv = g.N_kv; p.D = g.D; p.T = g.T; p.Tp = g.Tp; p.R = g.R;
  p.re_cap = g.tail_tiles_cap;
  p.layer0 = layer0; p.nlayers = nlayers;
  p.error = (uint32_t*)(c->ws + c->w.error);
  if (launch_compact(p, g.dtype, g.max_thin_tiles, (cudaStream_t)stream) != cudaSuccess) return THINK_ERR_CUDA;
  if (g.vt) {
    CompactValueParams cv;
    memset(&cv, 0, sizeof(cv));
    cv.v = to_view(v);
    cv.seq_len = (const int32_t*)(c->ws + c->w.seq_len);
    cv.v_thin_base = (const int64_t*)(c->ws + c->w.v_thin_base);
    cv.perm_v = (const uint8_t*)c->perm_v;
    cv.v_thin = c->v_thin;
    cv.B = g.B; cv.L = g.L; cv.N_kv = g.N_kv; cv.D = g.D; cv.Tv = g.Tv; cv.Tvp = g.Tvp; cv.R = g.R;
    cv.S_pmax = g.S_pmax;
    cv.layer0 = layer0; cv.nlayers = nlayers;
    if (launch_compact_value(cv, (cudaStream_t)stream) != cudaSuccess) return THINK_ERR_CUDA;
  }
  return seed_tail(c, k, v, tok, v_prefix, layer0, nlayers, stream);
}

// seeds the unpruned tail with the last S_recent prompt rows (keys and values) and books the layers
thinK_status seed_tail(thinK_cache* c, thinK_tensor5 k, thinK_tensor5 v, const TokenMap& tok, thinK_tensor5 v_prefix,
                       int layer0, int nlayers, void* stream) {
  const Geometry& g = c->g;
  if (g.R > 0) {
    TailWriteParams t;
    memset(&t, 0, sizeof(t));
    t.tok = tok;
    t.perm_v = g.vt ? (const uint8_t*)c->perm_v : nullptr;
    t.k = to_view(k); t.v = to_view(v);
    t.src_layer_base = 0; t.rows_from_seq_len = 1;
    t.seq_len = (const int32_t*)(c->ws + c->w.seq_len);
    t.tail_k = c->tail_k; t.tail_v = c->tail_v;
    t.B = g.B; t.L = g.L; t.N_kv = g.N_kv; t.D = g.D; t.R = g.R; t.cap = g.cap; t.tail_tiles_cap = g.tail_tiles_cap;
    t.layer0 = layer0; t.nlayers = nlayers; t.nrows = g.R; t.pos0 = 0;
    // with value pruning the kernel ahead is the value compaction, which does not let dependents go early
    if (launch_tail_write(t, g.dtype, (cudaStream_t)stream, !g.vt) != cudaSuccess) return THINK_ERR_CUDA;
  }
  c->v = v_prefix;
  c->have_v = true;
  for (int l = layer0; l < layer0 + nlayers; ++l) { c->compacted[l] = 1; c->tail_len[l] = g.R; c->n_re[l] = 0; }
  return THINK_OK;
}
}  // namespace

extern "C" {

thinK_status thinK_score_select(thinK_cache* c, thinK_tensor5 q_obs, thinK_tensor5 k, int32_t layer0,
                                int32_t nlayers, void* stream) {
  Range nvtx_range("thinK_score_select");
  return score_select_impl(c, q_obs, k, kNoTokenMap, layer0, nlayers, stream);
}

thinK_status thinK_compact(thinK_cache* c, thinK_tensor5 k, thinK_tensor5 v, int32_t layer0, int32_t nlayers,
                           void* stream) {
  Range nvtx_range("thinK_compact");
  return compact_impl(c, k, v, kNoTokenMap, v, layer0, nlayers, stream);
}

thinK_status thinK_attach_value_cache(thinK_cache* c, void* v_thin, void* perm_v, void* scores_v) {
  if (c && c->g.vt && (c->have_sizes.v_thin < c->need_sizes.v_thin || c->have_sizes.perm_v < c->need_sizes.perm_v))
    return THINK_ERR_CAPACITY;
  if (!c || !v_thin || !perm_v || !aligned16(v_thin) || !aligned16(perm_v) || (scores_v && !aligned16(scores_v)))
    return THINK_ERR_INVALID_ARG;
  if (!c->g.vt) return THINK_ERR_STATE;
  c->v_thin = v_thin;
  c->perm_v = perm_v;
  c->scores_v = scores_v;
  return THINK_OK;
}

thinK_status thinK_score_select_kv(thinK_cache* c, thinK_tensor5 q_obs, thinK_tensor5 k, thinK_tensor5 v,
                                   int32_t layer0, int32_t nlayers, void* stream) {
  Range nvtx_range("thinK_score_select_kv");
  if (!c) return THINK_ERR_INVALID_ARG;
  if (!layer_range_ok(c, layer0, nlayers)) return THINK_ERR_INVALID_ARG;
  const Geometry& g = c->g;
  if (!g.vt || !c->v_thin) return THINK_ERR_STATE;
  if (!check_view(q_obs, g.E) || !check_view(k, g.E) || !check_view(v, g.E)) return THINK_ERR_INVALID_ARG;
  thinK_status st = score_select_impl(c, q_obs, k, kNoTokenMap, layer0, nlayers, stream);
  if (st != THINK_OK) return st;
  ValueScoreParams p;
  memset(&p, 0, sizeof(p));
  p.q = to_view(q_obs); p.k = to_view(k); p.v = to_view(v);
  p.seq_len = (const int32_t*)(c->ws + c->w.seq_len);
  p.partials = (float*)(c->ws + c->w.value_partials);
  p.counters = (uint32_t*)(c->ws + c->w.value_counters);
  p.perm_v = (uint8_t*)c->perm_v;
  p.scores_v = (double*)c->scores_v;
  p.B = g.B; p.L = g.L; p.N_kv = g.N_kv; p.G = g.G; p.D = g.D; p.Tv = g.Tv; p.S_obs = g.S_obs;
  p.M = g.M; p.MB = g.MB; p.nrb = g.nrb;
  p.use_tcgen05 = c->value_score_tcgen05;
  p.error = (uint32_t*)(c->ws + c->w.error);
  // token splits: at least four 64-token tiles each, the finaliser's weights fit its shared memory,
  // and one launch fills the partial-record slots
  int min_len = g.seq_len[0];
  for (int b = 1; b < g.B; ++b) min_len = g.seq_len[b] < min_len ? g.seq_len[b] : min_len;
  const int per_layer = g.B * g.N_kv * g.nrb;
  int per_launch = g.value_slots / per_layer;             // layers per launch
  if (per_launch > nlayers) per_launch = nlayers;
  if (per_launch < 1) per_launch = 1;
  int max_split = (min_len + kTileTokens - 1) / kTileTokens / 4;
  if (max_split > 4096 / g.M) max_split = 4096 / g.M;
  if (max_split > 8) max_split = 8;
  if (max_split < 1) max_split = 1;
  // the split that wastes least of the last wave of CTAs (ties: the smaller split, less to merge)
  const bool tc = p.use_tcgen05 && g.D == 128 && g.MB == 128;
  const int resident = c->num_sms * (tc ? 2 : (g.MB >= 128 ? 1 : 2));
  int nsplit = 1;
  double best = 0.0;
  for (int s = 1; s <= max_split; ++s) {
    const long long ctas = (long long)per_layer * per_launch * s;
    if (ctas > g.value_slots) break;
    const double waves = (double)ctas / resident, eff = waves / ceil(waves);
    if (eff > best + 1e-9) { best = eff; nsplit = s; }
  }
  p.nsplit = nsplit;
  for (int l0 = layer0; l0 < layer0 + nlayers; l0 += per_launch) {
    p.layer0 = l0;
    p.nlayers = l0 + per_launch <= layer0 + nlayers ? per_launch : layer0 + nlayers - l0;
    // tickets start at zero whatever an earlier launch left behind (a CTA whose bounded wait ran out never takes its ticket)
    if (cudaMemsetAsync(p.counters, 0, sizeof(uint32_t) * (size_t)g.B * p.nlayers * g.N_kv, (cudaStream_t)stream) != cudaSuccess)
      return THINK_ERR_CUDA;
    if (launch_score_value(p, 32 * (g.MB / 16), (cudaStream_t)stream) != cudaSuccess) return THINK_ERR_CUDA;
  }
  for (int l = layer0; l < layer0 + nlayers; ++l) c->scored_v[l] = 1;
  return THINK_OK;
}

size_t thinK_v_kept_bytes(const thinK_cache* c) {
  if (!c) return 0;
  const Geometry& g = c->g;
  return (size_t)g.B * g.L * g.N_kv * g.S_max * g.D * g.E;
}

thinK_status thinK_prefill_evicted(thinK_cache* c, thinK_tensor5 q_obs, thinK_tensor5 k, thinK_tensor5 v,
                                   const int32_t* tok, int64_t tok_stride, int32_t src_tokens, void* v_kept,
                                   int32_t layer0, int32_t nlayers, void* stream) {
  Range nvtx_range("thinK_prefill_evicted");
  if (!c || !v_kept || !aligned16(v_kept)) return THINK_ERR_INVALID_ARG;
  if (!layer_range_ok(c, layer0, nlayers)) return THINK_ERR_INVALID_ARG;
  const Geometry& g = c->g;
  if (g.vt) return THINK_ERR_UNSUPPORTED;
  if (!check_view(v, g.E)) return THINK_ERR_INVALID_ARG;
  TokenMap m;
  thinK_status st = make_token_map(c, tok, tok_stride, src_tokens, &m);
  if (st != THINK_OK) return st;
  st = score_select_impl(c, q_obs, k, m, layer0, nlayers, stream);
  if (st != THINK_OK) return st;
  // values of the kept tokens: dense [B, L, N_kv, S_max, D]
  GatherRowsParams gp;
  memset(&gp, 0, sizeof(gp));
  gp.tok = m; gp.v = to_view(v);
  gp.seq_len = (const int32_t*)(c->ws + c->w.seq_len);
  gp.dst = v_kept;
  gp.B = g.B; gp.L = g.L; gp.N_kv = g.N_kv; gp.D = g.D; gp.S_max = g.S_max;
  gp.layer0 = layer0; gp.nlayers = nlayers;
  if (launch_gather_rows(gp, g.dtype, (cudaStream_t)stream) != cudaSuccess) return THINK_ERR_CUDA;
  thinK_tensor5 vk;
  vk.ptr = v_kept;
  vk.stride_s = g.D; vk.stride_n = (int64_t)g.S_max * g.D; vk.stride_l = (int64_t)g.N_kv * vk.stride_n;
  vk.stride_b = (int64_t)g.L * vk.stride_l;
  return compact_impl(c, k, v, m, vk, layer0, nlayers, stream);
}

thinK_status thinK_prefill(thinK_cache* c, thinK_tensor5 q_obs, thinK_tensor5 k, thinK_tensor5 v, int32_t layer0,
                           int32_t nlayers, void* stream) {
  Range nvtx_range("thinK_prefill");
  if (!c) return THINK_ERR_INVALID_ARG;
  thinK_status st = c->g.vt ? thinK_score_select_kv(c, q_obs, k, v, layer0, nlayers, stream)
                            : thinK_score_select(c, q_obs, k, layer0, nlayers, stream);
  if (st != THINK_OK) return st;
  return thinK_compact(c, k, v, layer0, nlayers, stream);
}

thinK_status thinK_append(thinK_cache* c, const void* k_new, const void* v_new, int32_t layer0, int32_t nlayers,
                          void* stream) {
  Range nvtx_range("thinK_append");
  if (!c || !k_new || !v_new) return THINK_ERR_INVALID_ARG;
  if (!layer_range_ok(c, layer0, nlayers)) return THINK_ERR_INVALID_ARG;
  if (!aligned16(k_new) || !aligned16(v_new)) return THINK_ERR_INVALID_ARG;
  const Geometry& g = c->g;
  const int pos = c->tail_len[layer0];
  for (int l = layer0; l < layer0 + nlayers; ++l) {
    if (!c->compacted[l]) return THINK_ERR_STATE;
    if (c->tail_len[l] != pos) return THINK_ERR_STATE;
  }
  if (pos - g.R >= g.max_new || pos >= g.cap) return THINK_ERR_CAPACITY;
  TailWriteParams t;
  memset(&t, 0, sizeof(t));
  const int64_t sn = g.D, sl = (int64_t)g.N_kv * g.D, sb = (int64_t)nlayers * sl;
  t.perm_v = g.vt ? (const uint8_t*)c->perm_v : nullptr;
  t.k = View5{k_new, sb, 0, sl, sn};
  t.v = View5{v_new, sb, 0, sl, sn};
  t.src_layer_base = layer0; t.rows_from_seq_len = 0;
  t.seq_len = (const int32_t*)(c->ws + c->w.seq_len);
  t.tail_k = c->tail_k; t.tail_v = c->tail_v;
  t.B = g.B; t.L = g.L; t.N_kv = g.N_kv; t.D = g.D; t.R = g.R; t.cap = g.cap; t.tail_tiles_cap = g.tail_tiles_cap;
  t.layer0 = layer0; t.nlayers = nlayers; t.nrows = 1; t.pos0 = pos;
  if (launch_tail_write(t, g.dtype, (cudaStream_t)stream) != cudaSuccess) return THINK_ERR_CUDA;
  for (int l = layer0; l < layer0 + nlayers; ++l) c->tail_len[l] = pos + 1;
  return THINK_OK;
}

static thinK_status decode_impl(thinK_cache* c, const void* q, void* out, int32_t layer0, int32_t nlayers,
                                void* stream, bool dependent_launch) {
  if (!c || !q || !out) return THINK_ERR_INVALID_ARG;
  if (!layer_range_ok(c, layer0, nlayers)) return THINK_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out)) return THINK_ERR_INVALID_ARG;
  const Geometry& g = c->g;
  const int n_tail = c->tail_len[layer0], n_re = c->n_re[layer0];
  for (int l = layer0; l < layer0 + nlayers; ++l) {
    if (!c->compacted[l]) return THINK_ERR_STATE;
    if (c->tail_len[l] != n_tail || c->n_re[l] != n_re) return THINK_ERR_STATE;
  }
  DecodeParams p;
  memset(&p, 0, sizeof(p));
  p.k_thin = c->k_thin; p.tail_k = c->tail_k; p.tail_v = c->tail_v;
  p.v = to_view(c->v);
  p.idx = (const uint8_t*)c->idx;
  p.q = q; p.out = out;
  p.seq_len = (const int32_t*)(c->ws + c->w.seq_len);
  p.cum_thin = (const int32_t*)(c->ws + c->w.cum_thin);
  p.thin_tile_base = (const int64_t*)(c->ws + c->w.thin_tile_base);
  p.records = c->ws + c->w.decode_records;
  p.counters = (uint32_t*)(c->ws + c->w.decode_counters);
  p.B = g.B; p.L = g.L; p.N_kv = g.N_kv; p.N_q = g.N_q; p.T = g.T; p.Tp = g.Tp; p.R = g.R; p.cap = g.cap;
  p.tail_tiles_cap = g.tail_tiles_cap;
  p.re_cap = g.tail_tiles_cap;
  p.n_re = n_re;
  p.n_tail = n_tail;
  p.n_tail_tiles = (n_tail + kTileTokens - 1) / kTileTokens;
  if (g.vt) {
    p.v_thin = c->v_thin;
    p.v_thin_base = (const int64_t*)(c->ws + c->w.v_thin_base);
    p.perm_v = (const uint8_t*)c->perm_v;
    p.Tvp = g.Tvp;
  }
  p.layer0 = layer0; p.nlayers = nlayers;
  p.Ntot = (long long)nlayers * g.N_kv * ((long long)g.cum_thin[g.B] + (long long)g.B * p.n_tail_tiles);
  for (int b = 0; b < g.B; ++b)
    if (g.cum_thin[b + 1] - g.cum_thin[b] + p.n_tail_tiles < 1) return THINK_ERR_STATE;  // nothing to attend to
  p.grid = (int)(p.Ntot < (long long)c->decode_grid_max ? p.Ntot : (long long)c->decode_grid_max);
  p.dependent_launch = dependent_launch && g.dtype == THINK_BF16;
  if (launch_decode(p, g.dtype, g.D, g.G, (cudaStream_t)stream) != cudaSuccess) return THINK_ERR_CUDA;
  return THINK_OK;
}

thinK_status thinK_decode_attn(thinK_cache* c, const void* q, void* out, int32_t layer0, int32_t nlayers,
                               void* stream) {
  Range nvtx_range("thinK_decode_attn");
  return decode_impl(c, q, out, layer0, nlayers, stream, false);
}

thinK_status thinK_append_decode(thinK_cache* c, const void* k_new, const void* v_new, const void* q, void* out,
                                 int32_t layer0, int32_t nlayers, void* stream) {
  Range nvtx_range("thinK_append_decode");
  if (!c || !q || !out || !aligned16(q) || !aligned16(out)) return THINK_ERR_INVALID_ARG;   // nothing launched
  thinK_status st = thinK_append(c, k_new, v_new, layer0, nlayers, stream);
  if (st != THINK_OK) return st;
  return decode_impl(c, q, out, layer0, nlayers, stream, true);
}

thinK_status thinK_reprune_tail(thinK_cache* c, int32_t keep_recent, int32_t layer0, int32_t nlayers, void* stream) {
  Range nvtx_range("thinK_reprune_tail");
  if (!c || keep_recent < 0) return THINK_ERR_INVALID_ARG;
  if (!layer_range_ok(c, layer0, nlayers)) return THINK_ERR_INVALID_ARG;
  const Geometry& g = c->g;
  if (g.dtype != THINK_BF16 || g.vt) return THINK_ERR_UNSUPPORTED;
  const int n_tail = c->tail_len[layer0], n_re = c->n_re[layer0];
  for (int l = layer0; l < layer0 + nlayers; ++l) {
    if (!c->compacted[l]) return THINK_ERR_STATE;
    if (c->tail_len[l] != n_tail || c->n_re[l] != n_re) return THINK_ERR_STATE;
  }
  // whole 64-token tiles, oldest first, as long as keep_recent tokens stay unpruned
  const int movable = n_tail - n_re * kTileTokens - keep_recent;
  const int nblk = movable > 0 ? movable / kTileTokens : 0;
  if (nblk == 0) return THINK_OK;
  RepruneParams p;
  memset(&p, 0, sizeof(p));
  p.idx = (const uint8_t*)c->idx;
  p.thin_tile_base = (const int64_t*)(c->ws + c->w.thin_tile_base);
  p.cum_thin = (const int32_t*)(c->ws + c->w.cum_thin);
  p.k_thin = c->k_thin; p.tail_k = c->tail_k;
  p.B = g.B; p.L = g.L; p.N_kv = g.N_kv; p.D = g.D; p.T = g.T; p.Tp = g.Tp;
  p.re_cap = g.tail_tiles_cap; p.tail_tiles_cap = g.tail_tiles_cap;
  p.layer0 = layer0; p.nlayers = nlayers; p.blk0 = n_re; p.nblk = nblk;
  if (launch_reprune(p, (cudaStream_t)stream) != cudaSuccess) return THINK_ERR_CUDA;
  for (int l = layer0; l < layer0 + nlayers; ++l) c->n_re[l] = n_re + nblk;
  return THINK_OK;
}

int32_t thinK_repruned_len(const thinK_cache* c, int32_t layer) {
  if (!c || layer < 0 || layer >= c->g.L) return -1;
  return c->n_re[layer] * kTileTokens;
}

int32_t thinK_tail_len(const thinK_cache* c, int32_t layer) {
  if (!c || layer < 0 || layer >= c->g.L) return -1;
  return c->tail_len[layer];
}

thinK_status thinK_device_error(thinK_cache* c, int32_t* out_code) {
  if (!c || !out_code) return THINK_ERR_INVALID_ARG;
  uint32_t v = 0;
  if (cudaMemcpy(&v, c->ws + c->w.error, sizeof(v), cudaMemcpyDeviceToHost) != cudaSuccess) return THINK_ERR_CUDA;
  *out_code = (int32_t)v;
  return THINK_OK;
}

thinK_status thinK_destroy(thinK_cache* c) {
  if (!c) return THINK_ERR_INVALID_ARG;
  delete c;
  return THINK_OK;
}

}  // extern "C"
