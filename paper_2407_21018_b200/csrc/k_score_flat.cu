// Channel scores and top-T selection (paper Sec. 3.2; Eq. 1 for the key-norm criteria): the streaming
// kernel of the regular entry points.
//
// Same arithmetic as k_colnorm_score_select (k_score.cu) -- Score[j] = sqrt(sum q^2 * sum k^2) from one pass
// over K, fp32 chains of 8 squares flushed into fp64, partial sums merged in a fixed order behind an atomic
// ticket on which nobody waits -- with a different split of the work.  All (entry b, layer, column block)
// items are laid end to end, one unit per token row, and that line is cut into EQUAL pieces, one per CTA of
// a grid that fills the GPU exactly once.  A CTA walks its piece and crosses item boundaries as it goes, so
// ragged batches, item counts that do not divide the grid and short prompts all keep every SM streaming
// until the end; with one CTA per (item, token split) the last wave ran partly empty.
// An item that lies inside one piece is ranked by that CTA alone; an item cut over several pieces leaves
// one partial per piece (a piece has at most two cut items, its first and its last: two slots per CTA) and
// the piece that arrives last adds them in piece order.
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

// piece that owns flat position f when F positions are cut into G pieces [F*c/G, F*(c+1)/G)
__device__ __forceinline__ int piece_of(long long f, long long F, int G) { return (int)(((f + 1) * G - 1) / F); }

template <typename Tin, bool L1>
__global__ void __launch_bounds__(kScoreThreads, 3) k_colnorm_flat(const ScoreParams p) {
  // the compaction kernel behind this launch may be scheduled now; it waits for this grid before it reads idx
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  constexpr int CH = Chunk<Tin>::CH;
  constexpr bool kBf16 = sizeof(Tin) == 2;
  __shared__ double red[kScoreThreads * CH];   // reused: row-lane reduction, then scores
  __shared__ int s_last;

  const int tid = threadIdx.x;
  const int cl = tid % p.CB, rl = tid / p.CB;
  const int CPH = p.D / CH;
  const int CBE = p.CB * CH;                   // columns of a column block
  const int G = gridDim.x, c = blockIdx.x;
  const long long F = p.flat_rows;
  const long long f0 = F * c / G, f1 = F * (c + 1) / G;
  const int LC = p.nlayers * p.ncolblk;        // items per batch entry
  double* const slots = p.partials + (size_t)c * 2 * 2 * CBE;

  long long f = f0;
  while (f < f1) {
    // ---- item that owns row f, and the part of it inside this piece
    int lo = 0, hi = p.B - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if ((long long)LC * p.row_cum[mid] <= f) lo = mid; else hi = mid - 1;
    }
    const int b = lo;
    const int S_b = p.seq_len[b];
    const long long rem = f - (long long)LC * p.row_cum[b];
    const int it_in_b = (int)(rem / S_b), t0 = (int)(rem % S_b);
    const int ll = it_in_b / p.ncolblk, colblk = it_in_b % p.ncolblk, l = p.layer0 + ll;
    const long long istart = f - t0, iend = istart + S_b;
    const long long seg_end = f1 < iend ? f1 : iend;
    const int t1 = t0 + (int)(seg_end - f);
    const int c_first = piece_of(istart, F, G), c_last = piece_of(iend - 1, F, G);
    const int n = c_last - c_first + 1, k = c - c_first;        // pieces of this item, this piece's place
    const int item = (b * p.nlayers + ll) * p.ncolblk + colblk;

    const int chunk = colblk * p.CB + cl;
    const bool active = rl < p.RP && chunk < p.NC;
    const int h = chunk / CPH, j0 = (chunk % CPH) * CH;

    double kacc[CH], qacc[CH];
#pragma unroll
    for (int i = 0; i < CH; ++i) kacc[i] = 0.0, qacc[i] = 0.0;
    if (active) {
      const Tin* kb = (const Tin*)p.k.ptr + b * p.k.sb + (int64_t)l * p.k.sl + (int64_t)h * p.k.sn + j0;
      int t = t0 + rl;
      const int step = p.RP;
      constexpr int U = 8;
      for (; t + (U - 1) * step < t1; t += U * step) {
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) v[u] = ldg16(kb + (int64_t)(t + u * step) * p.k.ss);
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
              const double d = (double)x[i];
              kacc[i] = L1 ? kacc[i] + fabs(d) : fma(d, d, kacc[i]);
            }
          }
        }
      }
      for (; t < t1; t += step) {
        float x[CH];
        Chunk<Tin>::unpack(ldg16(kb + (int64_t)t * p.k.ss), x);
#pragma unroll
        for (int i = 0; i < CH; ++i) {
          const double d = (double)x[i];
          kacc[i] = L1 ? kacc[i] + fabs(d) : fma(d, d, kacc[i]);
        }
      }
      // this piece's share of the window rows of the G query heads that share key head h (stacked)
      if (p.criterion == THINK_SCORE_QUERY_DRIVEN) {
        const Tin* qb = (const Tin*)p.q.ptr + b * p.q.sb + (int64_t)l * p.q.sl + j0;
        const int nrows = p.S_obs * p.G;
        for (int rr = k * p.RP + rl; rr < nrows; rr += n * p.RP) {
          const int s = rr / p.G, g = rr % p.G;
          float x[CH];
          Chunk<Tin>::unpack(ldg16(qb + (int64_t)s * p.q.ss + (int64_t)(h * p.G + g) * p.q.sn), x);
#pragma unroll
          for (int i = 0; i < CH; ++i) qacc[i] = fma((double)x[i], (double)x[i], qacc[i]);
        }
      }
    }

    // ---- this piece's partial: sums over the row lanes in a fixed order -> slot (first cut item: 0, last: 1)
    double* const my = slots + (f == f0 ? 0 : 1) * 2 * CBE;
#pragma unroll
    for (int pass = 0; pass < 2; ++pass) {
      __syncthreads();
#pragma unroll
      for (int i = 0; i < CH; ++i) red[i * kScoreThreads + tid] = pass ? qacc[i] : kacc[i];   // tid = rl * CB + cl
      __syncthreads();
      if (rl == 0) {
#pragma unroll
        for (int i = 0; i < CH; ++i) {
          double s = 0.0;
          for (int r = 0; r < p.RP; ++r) s += red[i * kScoreThreads + r * p.CB + cl];
          my[pass * CBE + cl * CH + i] = s;
        }
      }
    }
    __threadfence();
    __syncthreads();
    bool last = true;
    uint32_t* ctr = p.counters + item;
    if (n > 1) {
      if (tid == 0) s_last = (atomicAdd(ctr, 1u) == (uint32_t)(n - 1));
      __syncthreads();
      last = s_last != 0;
      __syncthreads();
    }
    if (last) {
      __threadfence();
      const int ncols = min(CBE, (p.NC - colblk * p.CB) * CH);
      for (int col = tid; col < ncols; col += kScoreThreads) {
        // partials of the item's pieces, added in piece order; loads are batched so their latencies overlap
        double kn = 0.0, qn = 0.0;
        for (int s0 = 0; s0 < n; s0 += 8) {
          double kv[8], qv[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int cc = c_first + s0 + u;
            const bool on = s0 + u < n;
            // a piece's partial of this item sits in its slot 0 when the piece starts inside the item
            const double* src = p.partials + ((size_t)cc * 2 + (F * cc / G >= istart ? 0 : 1)) * 2 * CBE;
            kv[u] = on ? __ldcg(src + col) : 0.0;
            qv[u] = on ? __ldcg(src + CBE + col) : 0.0;
          }
#pragma unroll
          for (int u = 0; u < 8; ++u) { kn += kv[u]; qn += qv[u]; }
        }
        double sc;
        if (p.criterion == THINK_SCORE_QUERY_DRIVEN) sc = sqrt(qn * kn);
        else if (p.criterion == THINK_SCORE_KEY_L2) sc = sqrt(kn);
        else sc = kn;
        red[col] = sc;
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
      if (n > 1 && tid == 0) *ctr = 0u;  // ready for the next call
    }
    f = seg_end;
  }
}

template <typename Tin, bool L1>
cudaError_t occupancy_of(int* n) {
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(n, k_colnorm_flat<Tin, L1>, kScoreThreads, 0);
}

}  // namespace

int score_flat_ctas_per_sm(int dtype, int criterion) {
  int n = 0;
  const bool l1 = criterion == THINK_SCORE_KEY_L1;
  cudaError_t e;
  if (dtype == THINK_BF16) e = l1 ? occupancy_of<__nv_bfloat16, true>(&n) : occupancy_of<__nv_bfloat16, false>(&n);
  else e = l1 ? occupancy_of<float, true>(&n) : occupancy_of<float, false>(&n);
  return e == cudaSuccess ? n : 0;
}

cudaError_t launch_score_flat(const ScoreParams& p, int dtype, int grid, cudaStream_t s) {
  const bool l1 = p.criterion == THINK_SCORE_KEY_L1;
  if (dtype == THINK_BF16) {
    if (l1) k_colnorm_flat<__nv_bfloat16, true><<<grid, kScoreThreads, 0, s>>>(p);
    else k_colnorm_flat<__nv_bfloat16, false><<<grid, kScoreThreads, 0, s>>>(p);
  } else {
    if (l1) k_colnorm_flat<float, true><<<grid, kScoreThreads, 0, s>>>(p);
    else k_colnorm_flat<float, false><<<grid, kScoreThreads, 0, s>>>(p);
  }
  return cudaGetLastError();
}

}  // namespace think
