// Decode attention over the two-part key cache (paper Sec. 3.3 / Fig. 2, attention of Sec. 3.2),
// CUDA-core version.  It serves fp32 caches (logits in fp64); bf16 caches use the tensor-core kernel
// in k_decode_mma.cu, whose key tiles are laid out differently.
//
// Work is the flat list of 64-token tiles of all (b, layer, key head) units: thin tiles [T][64]
// of the pruned prefix first, then tail tiles [D][64] of the unpruned keys.  The grid is
// persistent: CTA i owns tiles [i*N/grid, (i+1)*N/grid), so all SMs stream the same number of
// bytes and a CTA crosses unit boundaries as needed.  Inside a unit segment the four warps take
// tiles round-robin; each warp keeps its own online-softmax state (m, l, o[G][D]) in registers in
// the exp2 domain, a lane owning two tokens for the logits and D/32 channels of the output.
// Segments that do not cover their whole unit leave a partial state in the workspace; the CTA
// that arrives last at the unit's ticket merges the states in token order.  Nobody waits.
#include <math.h>

#include "think_internal.h"

namespace think {
namespace {

constexpr int kDecThreads = 128;
constexpr int kDecWarps = kDecThreads / 32;

template <typename Tin> struct LogitOf { using type = float; };
template <> struct LogitOf<float> { using type = double; };   // fp32 I/O: logits in fp64

__device__ __forceinline__ float ex2(float x) { return exp2f(x); }

template <typename Tin, int N>
__device__ __forceinline__ void load_row(const Tin* p, float (&v)[N]);
template <>
__device__ __forceinline__ void load_row<float, 4>(const float* p, float (&v)[4]) {
  float4 w = __ldg((const float4*)p);
  v[0] = w.x; v[1] = w.y; v[2] = w.z; v[3] = w.w;
}
template <>
__device__ __forceinline__ void load_row<float, 2>(const float* p, float (&v)[2]) {
  float2 w = __ldg((const float2*)p);
  v[0] = w.x; v[1] = w.y;
}

__device__ __forceinline__ void load_pair(const unsigned char* p, float& a, float& b, float*) {
  float2 w = __ldg((const float2*)p);
  a = w.x; b = w.y;
}

__device__ __forceinline__ void store_out(float* p, float v) { *p = v; }

// CTA that owns flat tile f when N tiles are split over `grid` CTAs as [i*N/grid, (i+1)*N/grid)
__device__ __forceinline__ int cta_of(long long f, long long N, int grid) {
  return (int)(((f + 1) * grid - 1) / N);
}

template <typename Tin, int D, int G>
__global__ void __launch_bounds__(kDecThreads) k_decode_generic(const DecodeParams p) {
  using LT = typename LogitOf<Tin>::type;
  constexpr int E = sizeof(Tin);
  constexpr int DPL = D / 32;
  __shared__ __align__(16) LT qs_thin[D * G];   // [channel][g], pre-scaled by log2(e)/sqrt(D)
  __shared__ __align__(16) LT qs_full[D * G];
  __shared__ uint8_t s_idx[D];
  __shared__ float mo[kDecWarps][G][D];
  __shared__ float ml[kDecWarps][G];
  __shared__ double mm[kDecWarps][G];
  __shared__ int s_last;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int cta = blockIdx.x;
  const long long N = p.Ntot;
  const long long f0 = (long long)cta * N / p.grid, f1 = (long long)(cta + 1) * N / p.grid;
  const int LH = p.nlayers * p.N_kv;
  const int ntt = p.n_tail_tiles;
  const size_t rec_bytes = rec_size(D, G);
  const LT scale = (LT)(1.4426950408889634 / sqrt((double)D));

  long long f = f0;
  while (f < f1) {
    // ---- locate the unit that owns tile f
    int lo = 0, hi = p.B - 1;
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      long long cm = (long long)LH * (p.cum_thin[mid] + (long long)mid * ntt);
      if (cm <= f) lo = mid; else hi = mid - 1;
    }
    const int b = lo;
    const int nthin = p.cum_thin[b + 1] - p.cum_thin[b];
    const int tpu = nthin + ntt;
    const long long rem = f - (long long)LH * (p.cum_thin[b] + (long long)b * ntt);
    const int u_in_b = (int)(rem / tpu), j0 = (int)(rem % tpu);
    const int ll = u_in_b / p.N_kv, h = u_in_b % p.N_kv, l = p.layer0 + ll;
    const long long ustart = f - j0, uend = ustart + tpu;
    const long long seg_end = f1 < uend ? f1 : uend;
    const int nseg = (int)(seg_end - f);
    const int S_p = p.seq_len[b] - p.R;
    const int64_t unit_abs = ((int64_t)b * p.L + l) * p.N_kv + h;
    const int unit_call = (b * p.nlayers + ll) * p.N_kv + h;

    // ---- stage the (scaled) queries of the group: gathered for thin tiles, full for tail tiles
    __syncthreads();
    for (int c = tid; c < p.T; c += kDecThreads) s_idx[c] = p.idx[unit_abs * p.T + c];
    __syncthreads();
    const Tin* qg = (const Tin*)p.q + ((int64_t)(b * p.nlayers + ll) * p.N_q + h * G) * D;
    for (int i = tid; i < D * G; i += kDecThreads) {
      int c = i / G, g = i % G;
      qs_full[i] = (LT)(float)qg[g * D + c] * scale;
      if (c < p.T) qs_thin[i] = (LT)(float)qg[g * D + s_idx[c]] * scale;
    }
    __syncthreads();

    // ---- per-warp online softmax over its tiles
    LT m[G];
    float lsum[G], o[G][DPL];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      m[g] = (LT)-INFINITY;
      lsum[g] = 0.f;
#pragma unroll
      for (int d = 0; d < DPL; ++d) o[g][d] = 0.f;
    }
    const int lane_byte = 2 * lane * E, lchunk = lane_byte >> 4, lwithin = lane_byte & 15;

    for (int j = j0 + warp; j < j0 + nseg; j += kDecWarps) {
      const unsigned char* tile;
      const LT* qs;
      const Tin* vrow;
      int64_t vstride;
      int Tc, nvalid;
      if (j < nthin) {
        tile = (const unsigned char*)p.k_thin +
               (p.thin_tile_base[b] + (int64_t)(l * p.N_kv + h) * (nthin + p.re_cap) + j) * (int64_t)p.T * kTileTokens * E;
        qs = qs_thin; Tc = p.T;
        nvalid = min(kTileTokens, S_p - j * kTileTokens);
        vrow = (const Tin*)p.v.ptr + b * p.v.sb + (int64_t)j * kTileTokens * p.v.ss + (int64_t)l * p.v.sl + (int64_t)h * p.v.sn;
        vstride = p.v.ss;
      } else {
        const int jt = j - nthin;
        tile = (const unsigned char*)p.tail_k + (unit_abs * p.tail_tiles_cap + jt) * (int64_t)D * kTileTokens * E;
        qs = qs_full; Tc = D;
        nvalid = min(kTileTokens, p.n_tail - jt * kTileTokens);
        vrow = (const Tin*)p.tail_v + (unit_abs * p.cap + (int64_t)jt * kTileTokens) * D;
        vstride = D;
      }
      // logits of this lane's two tokens for the G query heads
      LT x[G][2];
#pragma unroll
      for (int g = 0; g < G; ++g) x[g][0] = x[g][1] = (LT)0;
#pragma unroll 4
      for (int c = 0; c < Tc; ++c) {
        const unsigned char* row = tile + c * (kTileTokens * E) + (((lchunk ^ (c & 7)) << 4) | lwithin);
        float k0, k1;
        load_pair(row, k0, k1, (Tin*)nullptr);
#pragma unroll
        for (int g = 0; g < G; ++g) {
          LT qv = qs[c * G + g];
          x[g][0] += qv * (LT)k0;
          x[g][1] += qv * (LT)k1;
        }
      }
      const bool v0 = 2 * lane < nvalid, v1 = 2 * lane + 1 < nvalid;
      float pr[G][2];
#pragma unroll
      for (int g = 0; g < G; ++g) {
        LT tmax = v0 ? x[g][0] : (LT)-INFINITY;
        if (v1) tmax = x[g][1] > tmax ? x[g][1] : tmax;
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) {
          LT other = __shfl_xor_sync(0xffffffffu, tmax, s);
          tmax = other > tmax ? other : tmax;
        }
        const LT mnew = m[g] > tmax ? m[g] : tmax;
        const float sc = ex2((float)(m[g] - mnew));
        pr[g][0] = v0 ? ex2((float)(x[g][0] - mnew)) : 0.f;
        pr[g][1] = v1 ? ex2((float)(x[g][1] - mnew)) : 0.f;
        lsum[g] = lsum[g] * sc + pr[g][0] + pr[g][1];
#pragma unroll
        for (int d = 0; d < DPL; ++d) o[g][d] *= sc;
        m[g] = mnew;
      }
      // o += p . V over the valid tokens of the tile
      for (int t0 = 0; t0 < nvalid; t0 += 4) {
        float v[4][DPL];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (t0 + u < nvalid) load_row<Tin, DPL>(vrow + (int64_t)(t0 + u) * vstride + lane * DPL, v[u]);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int tt = t0 + u;
          if (tt < nvalid) {
#pragma unroll
            for (int g = 0; g < G; ++g) {
              const float pg = __shfl_sync(0xffffffffu, (tt & 1) ? pr[g][1] : pr[g][0], tt >> 1);
#pragma unroll
              for (int d = 0; d < DPL; ++d) o[g][d] = fmaf(pg, v[u][d], o[g][d]);
            }
          }
        }
      }
    }

    // ---- merge the warps of this CTA
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float ls = lsum[g];
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, s);
      if (lane == 0) { ml[warp][g] = ls; mm[warp][g] = (double)m[g]; }
#pragma unroll
      for (int d = 0; d < DPL; ++d) mo[warp][g][lane * DPL + d] = o[g][d];
    }
    __syncthreads();

    const bool complete = (f == ustart) && (seg_end == uend);
    uint8_t* rec = p.records + ((size_t)cta * 2 + (f == f0 ? 0 : 1)) * rec_bytes;
    Tin* outp = (Tin*)p.out + ((int64_t)(b * p.nlayers + ll) * p.N_q + h * G) * D;
    for (int i = tid; i < G * D; i += kDecThreads) {
      const int g = i / D, d = i % D;
      double M = mm[0][g];
#pragma unroll
      for (int w = 1; w < kDecWarps; ++w) M = mm[w][g] > M ? mm[w][g] : M;
      float Lsum = 0.f, O = 0.f;
#pragma unroll
      for (int w = 0; w < kDecWarps; ++w) {
        const float sc = ex2((float)(mm[w][g] - M));
        Lsum += ml[w][g] * sc;
        O += mo[w][g][d] * sc;
      }
      if (complete) {
        store_out(outp + g * D + d, O / Lsum);
      } else {
        ((float*)(rec + rec_o_off(G)))[g * D + d] = O;
        if (d == 0) { ((double*)rec)[g] = M; ((float*)(rec + G * 8))[g] = Lsum; }
      }
    }

    if (!complete) {
      // ---- ticket: the last contributor of this unit merges the partial states
      const int c_first = cta_of(ustart, N, p.grid), c_last = cta_of(uend - 1, N, p.grid);
      __threadfence();
      __syncthreads();
      if (tid == 0) s_last = (atomicAdd(p.counters + unit_call, 1u) == (uint32_t)(c_last - c_first));
      __syncthreads();
      if (s_last) {
        __threadfence();
        for (int i = tid; i < G * D; i += kDecThreads) {
          const int g = i / D, d = i % D;
          double M = -INFINITY;
          for (int ci = c_first; ci <= c_last; ++ci) {
            const long long cf0 = (long long)ci * N / p.grid;
            const uint8_t* r = p.records + ((size_t)ci * 2 + (cf0 >= ustart ? 0 : 1)) * rec_bytes;
            const double mi = __ldcg((const double*)r + g);
            M = mi > M ? mi : M;
          }
          float Lsum = 0.f, O = 0.f;
          for (int ci = c_first; ci <= c_last; ++ci) {
            const long long cf0 = (long long)ci * N / p.grid;
            const uint8_t* r = p.records + ((size_t)ci * 2 + (cf0 >= ustart ? 0 : 1)) * rec_bytes;
            const float sc = ex2((float)(__ldcg((const double*)r + g) - M));
            Lsum += __ldcg((const float*)(r + G * 8) + g) * sc;
            O += __ldcg((const float*)(r + rec_o_off(G)) + g * D + d) * sc;
          }
          store_out(outp + g * D + d, O / Lsum);
        }
        if (tid == 0) p.counters[unit_call] = 0u;
      }
    }
    f = seg_end;
  }
}

template <typename Tin, int D, int G>
cudaError_t launch_one(const DecodeParams& p, cudaStream_t s) {
  k_decode_generic<Tin, D, G><<<p.grid, kDecThreads, 0, s>>>(p);
  return cudaGetLastError();
}

template <typename Tin, int D, int G>
int occ_one() {
  int n = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k_decode_generic<Tin, D, G>, kDecThreads, 0) != cudaSuccess) return 0;
  return n;
}

#define THINK_DISPATCH(FN, ...)                                                      \
  do {                                                                               \
    if (D == 128) { switch (G) { case 1: return FN<float, 128, 1>(__VA_ARGS__);       \
                                 case 2: return FN<float, 128, 2>(__VA_ARGS__);       \
                                 case 4: return FN<float, 128, 4>(__VA_ARGS__);       \
                                 case 8: return FN<float, 128, 8>(__VA_ARGS__); } }   \
    if (D == 64)  { switch (G) { case 1: return FN<float, 64, 1>(__VA_ARGS__);        \
                                 case 2: return FN<float, 64, 2>(__VA_ARGS__);        \
                                 case 4: return FN<float, 64, 4>(__VA_ARGS__);        \
                                 case 8: return FN<float, 64, 8>(__VA_ARGS__); } }    \
  } while (0)

cudaError_t launch_f32(const DecodeParams& p, int D, int G, cudaStream_t s) {
  THINK_DISPATCH(launch_one, p, s);
  return cudaErrorInvalidValue;
}
int occ_f32(int D, int G) {
  THINK_DISPATCH(occ_one);
  return 0;
}

}  // namespace

bool decode_supported(int dtype, int D, int G) {
  return (dtype == THINK_BF16 || dtype == THINK_F32) && (D == 64 || D == 128) &&
         (G == 1 || G == 2 || G == 4 || G == 8);
}

cudaError_t launch_decode_bf16(const DecodeParams& p, int D, int G, cudaStream_t s);
cudaError_t decode_setup_bf16(int D, int G);
int decode_warps_bf16();

cudaError_t launch_decode(const DecodeParams& p, int dtype, int D, int G, cudaStream_t s) {
  return dtype == THINK_BF16 ? launch_decode_bf16(p, D, G, s) : launch_f32(p, D, G, s);
}

cudaError_t decode_setup(int dtype, int D, int G) {
  return dtype == THINK_BF16 ? decode_setup_bf16(D, G) : cudaSuccess;
}

// CTAs of the decode kernel that fit on one SM (the bf16 kernel takes the whole shared memory).
int decode_ctas_per_sm(int dtype, int D, int G) { return dtype == THINK_BF16 ? 1 : occ_f32(D, G); }

// Workers per CTA: partial-state records are indexed by worker.
int decode_workers_per_cta(int dtype) { return dtype == THINK_BF16 ? decode_warps_bf16() : 1; }

size_t decode_record_bytes(int D, int G) { return rec_size(D, G); }

}  // namespace think
