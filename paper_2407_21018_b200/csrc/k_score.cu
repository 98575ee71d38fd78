// Channel scores and top-T selection (paper Sec. 3.2; Eq. 1 for the key-norm criteria).
//
// Score[j] = ||Q_obs[:, j] K[:, j]^T||_F = sqrt(sum q^2 * sum k^2): one streaming pass over K
// accumulates per-channel energies.  A CTA owns (entry b, layer l, block of columns, token
// range); a thread owns one 16-byte column chunk and walks the token range with independent
// 16-byte loads.  bf16 squares are exact in fp32; fp32 chains of 8 terms are flushed into fp64.
// The CTA that arrives last for its (b, l, column block) -- an atomic ticket, nobody waits --
// adds the partials in split order (deterministic), forms the scores and ranks each head.
#include <string.h>

#include <mutex>

#include "think_internal.h"

namespace think {
namespace {

template <typename Tin>
struct Chunk;
template <>
struct Chunk<__nv_bfloat16> {
  static constexpr int CH = 8;
  __device__ static void unpack(const uint4& v, float (&x)[8]) {
    x[0] = bf16lo(v.x); x[1] = bf16hi(v.x); x[2] = bf16lo(v.y); x[3] = bf16hi(v.y);
    x[4] = bf16lo(v.z); x[5] = bf16hi(v.z); x[6] = bf16lo(v.w); x[7] = bf16hi(v.w);
  }
};
template <>
struct Chunk<float> {
  static constexpr int CH = 4;
  __device__ static void unpack(const uint4& v, float (&x)[4]) {
    x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y);
    x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
  }
};

__device__ __forceinline__ uint4 ldg16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

template <typename Tin, bool L1, bool TOK>
__global__ void __launch_bounds__(kScoreThreads, 3) k_colnorm_score_select(const ScoreParams p) {
  // the compaction kernel behind this launch may be scheduled now; it waits for this grid before it reads idx
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  constexpr int CH = Chunk<Tin>::CH;
  constexpr bool kBf16 = sizeof(Tin) == 2;
  __shared__ double red[kScoreThreads * CH];   // reused: row-lane reduction, then scores
  __shared__ int s_last;

  const int tid = threadIdx.x;
  const int split = blockIdx.x, colblk = blockIdx.y, z = blockIdx.z;
  const int b = z / p.nlayers, l = p.layer0 + z % p.nlayers;
  const int cl = tid % p.CB, rl = tid / p.CB;
  const int chunk = colblk * p.CB + cl;
  const bool active = rl < p.RP && chunk < p.NC;
  const int CPH = p.D / CH;
  const int h = chunk / CPH, j0 = (chunk % CPH) * CH;
  const int S_b = p.seq_len[b];
  const int per = (S_b + p.nsplit - 1) / p.nsplit;
  const int t0 = split * per;
  const int t1 = min(S_b, t0 + per);

  // reduce one accumulator set over the row lanes of this CTA (fixed order) into this CTA's partial
  const int CBE = p.CB * CH;  // elements per column block
  double* my = p.partials + ((int64_t)(z * p.ncolblk + colblk) * p.nsplit + split) * 2 * CBE;
  auto reduce_store = [&](const double (&acc)[CH], int pass) {
    __syncthreads();
#pragma unroll
    for (int i = 0; i < CH; ++i) red[i * kScoreThreads + tid] = acc[i];   // tid = rl * CB + cl
    __syncthreads();
    if (rl == 0) {
#pragma unroll
      for (int i = 0; i < CH; ++i) {
        double s = 0.0;
        for (int r = 0; r < p.RP; ++r) s += red[i * kScoreThreads + r * p.CB + cl];
        my[pass * CBE + cl * CH + i] = s;
      }
    }
  };

  // The window rows of the G query heads that share key head h (stacked).  The first two rows of this thread
  // are fetched now and summed after the key pass, so their latency runs under the key loads.
  const bool with_q = active && p.criterion == THINK_SCORE_QUERY_DRIVEN;
  const int q_rows = p.S_obs * p.G, q_step = p.nsplit * p.RP;
  const Tin* qb = (const Tin*)p.q.ptr + b * p.q.sb + (int64_t)l * p.q.sl + j0;
  auto q_row = [&](int rr) -> uint4 {
    const int s = rr / p.G, g = rr % p.G;
    return ldg16(qb + (int64_t)s * p.q.ss + (int64_t)(h * p.G + g) * p.q.sn);
  };
  uint4 q_early[2];
  {
    const int rr0 = split * p.RP + rl;
#pragma unroll
    for (int u = 0; u < 2; ++u)
      q_early[u] = (with_q && rr0 + u * q_step < q_rows) ? q_row(rr0 + u * q_step) : make_uint4(0, 0, 0, 0);
  }

  double kacc[CH];
#pragma unroll
  for (int i = 0; i < CH; ++i) kacc[i] = 0.0;

  if (active) {
    const Tin* kb = (const Tin*)p.k.ptr + b * p.k.sb + (int64_t)l * p.k.sl + (int64_t)h * p.k.sn + j0;
    const int64_t unit = ((int64_t)b * p.L + l) * p.N_kv + h;
    auto row = [&](int tt) -> int64_t { return TOK ? token_row(p.tok, unit, tt) : (int64_t)tt; };
    int t = t0 + rl;
    const int step = p.RP;
    constexpr int U = 8;
    for (; t + (U - 1) * step < t1; t += U * step) {
      uint4 v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) v[u] = ldg16(kb + row(t + u * step) * p.k.ss);
      if (kBf16) {
        float part[CH];
#pragma unroll
        for (int i = 0; i < CH; ++i) part[i] = 0.f;
#pragma unroll
        for (int u = 0; u < U; ++u) {
          float x[CH];
          Chunk<Tin>::unpack(v[u], x);
#pragma unroll
          for (int i = 0; i < CH; ++i) part[i] = L1 ? part[i] + fabsf(x[i]) : fmaf(x[i], x[i], part[i]);
        }
#pragma unroll
        for (int i = 0; i < CH; ++i) kacc[i] += (double)part[i];
      } else {
#pragma unroll
        for (int u = 0; u < U; ++u) {
          float x[CH];
          Chunk<Tin>::unpack(v[u], x);
#pragma unroll
          for (int i = 0; i < CH; ++i) {
            double d = (double)x[i];
            kacc[i] = L1 ? kacc[i] + fabs(d) : fma(d, d, kacc[i]);
          }
        }
      }
    }
    for (; t < t1; t += step) {
      uint4 v = ldg16(kb + row(t) * p.k.ss);
      float x[CH];
      Chunk<Tin>::unpack(v, x);
#pragma unroll
      for (int i = 0; i < CH; ++i) {
        double d = (double)x[i];
        kacc[i] = L1 ? kacc[i] + fabs(d) : fma(d, d, kacc[i]);
      }
    }
  }
  {
    double qacc[CH];
#pragma unroll
    for (int i = 0; i < CH; ++i) qacc[i] = 0.0;
    auto add_q = [&](const uint4& v) {
      float x[CH];
      Chunk<Tin>::unpack(v, x);
#pragma unroll
      for (int i = 0; i < CH; ++i) {
        const double d = (double)x[i];
        qacc[i] = fma(d, d, qacc[i]);
      }
    };
    if (with_q) {
      add_q(q_early[0]);                               // a row that was not fetched is all zeros
      add_q(q_early[1]);
      for (int rr = split * p.RP + rl + 2 * q_step; rr < q_rows; rr += q_step) add_q(q_row(rr));
    }
    reduce_store(qacc, 1);
  }
  reduce_store(kacc, 0);

  // ticket: the last CTA of this (b, l, column block) finishes the job
  __threadfence();
  __syncthreads();
  uint32_t* ctr = p.counters + (z * p.ncolblk + colblk);
  if (tid == 0) s_last = (atomicAdd(ctr, 1u) == (uint32_t)(p.nsplit - 1));
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  const double* base = p.partials + (int64_t)(z * p.ncolblk + colblk) * p.nsplit * 2 * CBE;
  const int ncols = min(CBE, (p.NC - colblk * p.CB) * CH);
  __syncthreads();
  // Partials are added in split order.  A thread takes two neighbouring columns (one 16-byte load per split and
  // sum) and keeps 8 splits of both sums in flight, so the merge is a few round trips to L2, not one per split.
  for (int c = 2 * tid; c < ncols; c += 2 * kScoreThreads) {
    double kn0 = 0.0, kn1 = 0.0, qn0 = 0.0, qn1 = 0.0;
    for (int s0 = 0; s0 < p.nsplit; s0 += 8) {
      double2 kv[8], qv[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const bool on = s0 + u < p.nsplit;
        const double* row = base + (int64_t)(on ? s0 + u : 0) * 2 * CBE + c;
        kv[u] = on ? __ldcg((const double2*)row) : make_double2(0.0, 0.0);
        qv[u] = on ? __ldcg((const double2*)(row + CBE)) : make_double2(0.0, 0.0);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) { kn0 += kv[u].x; kn1 += kv[u].y; qn0 += qv[u].x; qn1 += qv[u].y; }
    }
    auto score_of = [&](double qn, double kn) -> double {
      if (p.criterion == THINK_SCORE_QUERY_DRIVEN) return sqrt(qn * kn);
      if (p.criterion == THINK_SCORE_KEY_L2) return sqrt(kn);
      return kn;
    };
    red[c] = score_of(qn0, kn0);
    red[c + 1] = score_of(qn1, kn1);
  }
  __syncthreads();
  const int heads = ncols / p.D;
  const int h_first = colblk * p.CB * CH / p.D;
  const int warp = tid >> 5, lane = tid & 31;
  for (int hh = warp; hh < heads; hh += kScoreThreads / 32) {
    const int64_t unit = ((int64_t)b * p.L + l) * p.N_kv + h_first + hh;
    select_head(red + hh * p.D, p.D, p.T, p.idx + unit * p.T, lane, false, p.error);
    if (p.scores)
      for (int j = lane; j < p.D; j += 32) p.scores[unit * p.D + j] = red[hh * p.D + j];
  }
  if (tid == 0) *ctr = 0u;  // ready for the next call
}

}  // namespace

// CTAs of the score kernel that are resident per SM (the grid is sized to one wave)
namespace {
template <typename Tin, bool L1, bool TOK>
cudaError_t occupancy_of(int* n) {
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(n, k_colnorm_score_select<Tin, L1, TOK>, kScoreThreads, 0);
}
template <typename Tin, bool L1>
cudaError_t launch_as(const ScoreParams& p, dim3 grid, cudaStream_t s) {
  if (p.tok.rows) k_colnorm_score_select<Tin, L1, true><<<grid, kScoreThreads, 0, s>>>(p);
  else k_colnorm_score_select<Tin, L1, false><<<grid, kScoreThreads, 0, s>>>(p);
  return cudaGetLastError();
}
}  // namespace

int score_ctas_per_sm(int dtype, int criterion) {
  int n = 0;
  const bool l1 = criterion == THINK_SCORE_KEY_L1;
  cudaError_t e;
  if (dtype == THINK_BF16) e = l1 ? occupancy_of<__nv_bfloat16, true, false>(&n) : occupancy_of<__nv_bfloat16, false, false>(&n);
  else e = l1 ? occupancy_of<float, true, false>(&n) : occupancy_of<float, false, false>(&n);
  return e == cudaSuccess ? n : 0;
}

cudaError_t launch_score(const ScoreParams& p, int dtype, cudaStream_t s) {
  dim3 grid(p.nsplit, p.ncolblk, p.B * p.nlayers);
  const bool l1 = p.criterion == THINK_SCORE_KEY_L1;
  if (dtype == THINK_BF16) return l1 ? launch_as<__nv_bfloat16, true>(p, grid, s) : launch_as<__nv_bfloat16, false>(p, grid, s);
  return l1 ? launch_as<float, true>(p, grid, s) : launch_as<float, false>(p, grid, s);
}

}  // namespace think

// ---------------------------------------------------------------------------------------------
// Score + select for callers that cannot allocate device memory.
//
// The kernel's scratch (per-sequence lengths, ticket counters, fp64 partial sums) lives in a fixed
// array that is part of the library image: every GPU that loads the library holds these bytes until
// the process exits.  Host code cannot use the array's name as an address -- it is only a host-side
// handle of the symbol -- so the device address is looked up once per device with
// cudaGetSymbolAddress and cached.
// ---------------------------------------------------------------------------------------------
#define THINK_STATIC_SCRATCH_BYTES (8u << 20)
static __device__ __align__(256) unsigned char g_think_static_scratch[THINK_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mu;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device (first use on a device resolves it).
cudaError_t static_scratch(unsigned char** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_scratch_mu);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_think_static_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = p;
  }
  *out = (unsigned char*)g_scratch_addr[dev];
  return cudaSuccess;
}

inline size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }
}  // namespace

extern "C" thinK_status thinK_score_select_static(const thinK_config* cfg, const int32_t* seq_lens,
                                                  thinK_tensor5 q_obs, thinK_tensor5 k, int32_t layer0,
                                                  int32_t nlayers, uint8_t* idx, double* scores, void* stream) {
  using namespace think;
  if (!cfg || !seq_lens || !idx || !k.ptr) return THINK_ERR_INVALID_ARG;
  if (cfg->B < 1 || cfg->L < 1 || cfg->N_kv < 1 || cfg->N_q < 1 || cfg->N_q % cfg->N_kv != 0 || cfg->S_obs < 1)
    return THINK_ERR_INVALID_ARG;
  if (cfg->dtype != THINK_BF16 && cfg->dtype != THINK_F32) return THINK_ERR_UNSUPPORTED;
  if (cfg->D != 64 && cfg->D != 128) return THINK_ERR_UNSUPPORTED;
  if (cfg->criterion < THINK_SCORE_QUERY_DRIVEN || cfg->criterion > THINK_SCORE_KEY_L1) return THINK_ERR_INVALID_ARG;
  if (layer0 < 0 || nlayers < 1 || layer0 + nlayers > cfg->L || (int64_t)cfg->B * nlayers > 65535)
    return THINK_ERR_INVALID_ARG;
  if (cfg->criterion == THINK_SCORE_QUERY_DRIVEN && !q_obs.ptr) return THINK_ERR_INVALID_ARG;
  const int T = thinK_T(cfg->lambda, cfg->D);
  if (T < 1) return THINK_ERR_INVALID_ARG;
  const int E = cfg->dtype == THINK_BF16 ? 2 : 4;
  const thinK_tensor5* views[2] = {&k, &q_obs};
  for (int v = 0; v < (cfg->criterion == THINK_SCORE_QUERY_DRIVEN ? 2 : 1); ++v) {
    const int64_t st[4] = {views[v]->stride_b, views[v]->stride_s, views[v]->stride_l, views[v]->stride_n};
    if (((uintptr_t)views[v]->ptr & 15) != 0) return THINK_ERR_INVALID_ARG;
    for (int i = 0; i < 4; ++i)
      if (st[i] < 0 || (st[i] * E) % 16 != 0) return THINK_ERR_INVALID_ARG;
  }
  int min_len = seq_lens[0];
  for (int b = 0; b < cfg->B; ++b) {
    if (seq_lens[b] < cfg->S_obs || seq_lens[b] > cfg->S_max) return THINK_ERR_INVALID_ARG;
    min_len = seq_lens[b] < min_len ? seq_lens[b] : min_len;
  }

  ScoreParams p;
  memset(&p, 0, sizeof(p));
  const int CH = 16 / E;
  p.NC = cfg->N_kv * cfg->D / CH;
  p.CB = p.NC < kScoreThreads ? p.NC : kScoreThreads;
  p.ncolblk = (p.NC + p.CB - 1) / p.CB;
  p.RP = kScoreThreads / p.CB;
  const int items = cfg->B * nlayers * p.ncolblk;
  int nsplit = (kScoreTargetCtas + items - 1) / items;
  int cap = min_len / (64 * p.RP);
  if (cap < 1) cap = 1;
  if (nsplit > cap) nsplit = cap;
  // scratch: lengths | counters | partials; shrink the token split until it fits, else refuse
  const size_t off_cnt = up256(sizeof(int32_t) * (size_t)cfg->B);
  const size_t off_part = off_cnt + up256(sizeof(uint32_t) * (size_t)items);
  const size_t per_split = (size_t)items * 2 * p.CB * CH * sizeof(double);
  while (nsplit > 1 && off_part + per_split * nsplit > THINK_STATIC_SCRATCH_BYTES) --nsplit;
  if (off_part + per_split * nsplit > THINK_STATIC_SCRATCH_BYTES) return THINK_ERR_CAPACITY;
  p.nsplit = nsplit;

  unsigned char* scratch = nullptr;
  if (static_scratch(&scratch) != cudaSuccess) return THINK_ERR_CUDA;
  cudaStream_t s = (cudaStream_t)stream;
  // the array keeps whatever the previous call left: lengths are rewritten, tickets start at zero
  if (cudaMemcpyAsync(scratch, seq_lens, sizeof(int32_t) * (size_t)cfg->B, cudaMemcpyHostToDevice, s) != cudaSuccess)
    return THINK_ERR_CUDA;
  if (cudaMemsetAsync(scratch + off_cnt, 0, sizeof(uint32_t) * (size_t)items, s) != cudaSuccess) return THINK_ERR_CUDA;

  p.k = View5{k.ptr, k.stride_b, k.stride_s, k.stride_l, k.stride_n};
  p.q = View5{q_obs.ptr, q_obs.stride_b, q_obs.stride_s, q_obs.stride_l, q_obs.stride_n};
  p.seq_len = (const int32_t*)scratch;
  p.counters = (uint32_t*)(scratch + off_cnt);
  p.partials = (double*)(scratch + off_part);
  p.idx = idx;
  p.scores = scores;
  p.B = cfg->B; p.L = cfg->L; p.N_kv = cfg->N_kv; p.G = cfg->N_q / cfg->N_kv; p.D = cfg->D; p.T = T;
  p.S_obs = cfg->S_obs; p.layer0 = layer0; p.nlayers = nlayers; p.criterion = cfg->criterion;
  if (launch_score(p, cfg->dtype, s) != cudaSuccess) return THINK_ERR_CUDA;
  return THINK_OK;
}
