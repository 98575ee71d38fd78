// Fused prefill for bf16 caches: channel scores, top-T selection and key compaction (paper Sec. 3.2
// and 3.3) in ONE persistent kernel, so that the keys are read from HBM once.
//
// Scoring must see all tokens of a head before its keys can be compacted, so a two-kernel flow reads
// K twice from DRAM.  Here the unit of work is a head slab (b, layer, key head): S_b rows of D
// channels.  CTAs form teams; a team takes slabs round-robin and its members split a slab's tokens.
// For slab i a member (A) accumulates its share of the column energies and joins a two-level ticket
// reduction -- the member that arrives last ranks the channels, writes idx and raises the slab's flag
// -- and then (B) compacts its share of slab i-1, whose flag was raised one slab ago and whose keys
// are still in L2 (the host sizes the teams so that two slabs per team fit there).  The only wait in
// the kernel is on that flag: it is bounded, and on expiry the kernel records an error and returns.
// The launch is cooperative because the flag wait needs all members of a team to be resident.
#include <cooperative_groups.h>
#include <math.h>

#include "think_internal.h"

namespace think {
namespace {

constexpr int kThreads = 256;
constexpr int kGroup = 16;                 // members per first-level reduction group
constexpr int kSpinLimit = 1 << 18;        // polls of a slab flag before giving up (with nanosleep)

__device__ __forceinline__ uint4 ldg16_nc(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void unpack8(const uint4& v, float (&x)[8]) {
  x[0] = bf16lo(v.x); x[1] = bf16hi(v.x); x[2] = bf16lo(v.y); x[3] = bf16hi(v.y);
  x[4] = bf16lo(v.z); x[5] = bf16hi(v.z); x[6] = bf16lo(v.w); x[7] = bf16hi(v.w);
}

// rank-count selection by one warp (ties to the lower channel), ascending output
__device__ void select_head_w(const double* s, int D, int T, uint8_t* out, int lane) {
  int base = 0;
  for (int j0 = 0; j0 < D; j0 += 32) {
    const int j = j0 + lane;
    bool keep = false;
    if (j < D) {
      const double sj = s[j];
      int rank = 0;
      for (int k = 0; k < D; ++k) {
        const double sk = s[k];
        rank += (sk > sj) || (sk == sj && k < j);
      }
      keep = rank < T;
    }
    const unsigned m = __ballot_sync(0xffffffffu, keep);
    if (keep) out[base + __popc(m & ((1u << lane) - 1u))] = (uint8_t)j;
    base += __popc(m);
  }
}

template <bool L1>
__global__ void __launch_bounds__(kThreads, 2) k_prefill_fused(const PrefillParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int D = p.D, T = p.T, Tp = p.Tp;
  const int pitch = D * 2 + 16;
  unsigned char* s_rows[2] = {smem, smem + kTileTokens * pitch};             // staged key rows (2 buffers)
  double* s_red = (double*)(smem + 2 * kTileTokens * pitch);                 // [kThreads][8] reduction / scores
  uint8_t* s_idx = (uint8_t*)(s_red + kThreads * 8);                         // [Tp]
  __shared__ int s_flag;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int team = blockIdx.x / p.TS, member = blockIdx.x % p.TS;
  const int CPR = D / 8;                      // 16-byte chunks per row
  const int RL = kThreads / CPR;              // row lanes
  const int ck = tid % CPR, rl = tid / CPR;
  const int ngroups = (p.TS + kGroup - 1) / kGroup;
  const int group = member / kGroup;
  const int gsize = min(kGroup, p.TS - group * kGroup);

  auto slab_coords = [&](int s, int& b, int& l, int& h) {
    h = s % p.N_kv;
    const int r = s / p.N_kv;
    l = p.layer0 + r % p.nlayers;
    b = r / p.nlayers;
  };

  // ---------------------------------------------------------------- phase A: energies, ticket, select
  auto phase_a = [&](int s, int parity) {
    int b, l, h;
    slab_coords(s, b, l, h);
    const int S_b = p.seq_len[b];
    const int t0 = (int)((long long)member * S_b / p.TS), t1 = (int)((long long)(member + 1) * S_b / p.TS);
    double kacc[8], qacc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) kacc[i] = 0.0, qacc[i] = 0.0;
    const __nv_bfloat16* kb = (const __nv_bfloat16*)p.k.ptr + b * p.k.sb + (int64_t)l * p.k.sl + (int64_t)h * p.k.sn + ck * 8;
    int t = t0 + rl;
    constexpr int U = 8;
    for (; t + (U - 1) * RL < t1; t += U * RL) {
      uint4 v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) v[u] = ldg16_nc(kb + (int64_t)(t + u * RL) * p.k.ss);
      float part[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) part[i] = 0.f;
#pragma unroll
      for (int u = 0; u < U; ++u) {
        float x[8];
        unpack8(v[u], x);
#pragma unroll
        for (int i = 0; i < 8; ++i) part[i] = L1 ? part[i] + fabsf(x[i]) : fmaf(x[i], x[i], part[i]);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) kacc[i] += (double)part[i];
    }
    for (; t < t1; t += RL) {
      float x[8];
      unpack8(ldg16_nc(kb + (int64_t)t * p.k.ss), x);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const double d = (double)x[i];
        kacc[i] = L1 ? kacc[i] + fabs(d) : fma(d, d, kacc[i]);
      }
    }
    if (p.criterion == THINK_SCORE_QUERY_DRIVEN) {
      const __nv_bfloat16* qb = (const __nv_bfloat16*)p.q.ptr + b * p.q.sb + (int64_t)l * p.q.sl + ck * 8;
      const int nrows = p.S_obs * p.G;
      for (int rr = member * RL + rl; rr < nrows; rr += p.TS * RL) {
        const int sr = rr / p.G, g = rr % p.G;
        float x[8];
        unpack8(ldg16_nc(qb + (int64_t)sr * p.q.ss + (int64_t)(h * p.G + g) * p.q.sn), x);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const double d = (double)x[i];
          qacc[i] = fma(d, d, qacc[i]);
        }
      }
    }
    // CTA reduction over the row lanes (fixed order) -> this member's partial [2][D]
    double* mine = p.partials + (((size_t)team * 2 + parity) * p.TS + member) * 2 * D;
    for (int pass = 0; pass < 2; ++pass) {
      const double* acc = pass ? qacc : kacc;
      __syncthreads();
#pragma unroll
      for (int i = 0; i < 8; ++i) s_red[i * kThreads + tid] = acc[i];
      __syncthreads();
      if (rl == 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          double v = 0.0;
          for (int r = 0; r < RL; ++r) v += s_red[i * kThreads + r * CPR + ck];
          mine[pass * D + ck * 8 + i] = v;
        }
      }
    }
    // level 1: last member of the group adds the group's partials in member order
    __threadfence();
    __syncthreads();
    if (tid == 0) s_flag = atomicAdd(p.tickets + (size_t)s * (ngroups + 1) + group, 1u) == (unsigned)(gsize - 1);
    __syncthreads();
    if (!s_flag) return;
    __threadfence();
    double* gp = p.gpartials + (((size_t)team * 2 + parity) * ngroups + group) * 2 * D;
    const double* first = p.partials + (((size_t)team * 2 + parity) * p.TS + group * kGroup) * 2 * D;
    if (tid < 2 * D) {
      double v[kGroup];
#pragma unroll
      for (int u = 0; u < kGroup; ++u) v[u] = u < gsize ? __ldcg(first + (size_t)u * 2 * D + tid) : 0.0;
      double a = 0.0;
#pragma unroll
      for (int u = 0; u < kGroup; ++u) a += v[u];
      gp[tid] = a;
    }
    if (tid == 0) p.tickets[(size_t)s * (ngroups + 1) + group] = 0u;
    // level 2: last group adds the group sums in group order, ranks the channels, raises the flag
    __threadfence();
    __syncthreads();
    if (tid == 0) s_flag = atomicAdd(p.tickets + (size_t)s * (ngroups + 1) + ngroups, 1u) == (unsigned)(ngroups - 1);
    __syncthreads();
    if (!s_flag) return;
    __threadfence();
    const double* g0 = p.gpartials + ((size_t)team * 2 + parity) * ngroups * 2 * D;
    if (tid < 2 * D) {
      double a = 0.0;
      for (int u0 = 0; u0 < ngroups; u0 += 8) {
        double v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = u0 + u < ngroups ? __ldcg(g0 + (size_t)(u0 + u) * 2 * D + tid) : 0.0;
#pragma unroll
        for (int u = 0; u < 8; ++u) a += v[u];
      }
      s_red[tid] = a;
    }
    __syncthreads();
    if (tid < D) {
      const double kn = s_red[tid], qn = s_red[D + tid];
      double sc;
      if (p.criterion == THINK_SCORE_QUERY_DRIVEN) sc = sqrt(qn * kn);
      else if (p.criterion == THINK_SCORE_KEY_L2) sc = sqrt(kn);
      else sc = kn;
      s_red[2 * D + tid] = sc;
    }
    __syncthreads();
    const int64_t unit = ((int64_t)b * p.L + l) * p.N_kv + h;
    if (warp == 0) select_head_w(s_red + 2 * D, D, T, p.idx + unit * T, lane);
    if (p.scores && tid < D) p.scores[unit * D + tid] = s_red[2 * D + tid];
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      p.tickets[(size_t)s * (ngroups + 1) + ngroups] = 0u;
      atomicExch(p.flags + s, p.epoch);           // idx of this slab is visible to everyone who sees this
    }
  };

  // ---------------------------------------------------------------- phase B: compaction of a scored slab
  auto phase_b = [&](int s) -> bool {
    int b, l, h;
    slab_coords(s, b, l, h);
    if (tid == 0) {
      int ok = 0;
      for (int i = 0; i < kSpinLimit; ++i) {
        if (*(volatile uint32_t*)(p.flags + s) == p.epoch) { ok = 1; break; }
        __nanosleep(64);
      }
      if (!ok) atomicExch(p.error, 1u);
      s_flag = ok;
    }
    __syncthreads();
    if (!s_flag) return false;
    __threadfence();
    const int64_t unit = ((int64_t)b * p.L + l) * p.N_kv + h;
    for (int c = tid; c < Tp; c += kThreads) s_idx[c] = c < T ? __ldcg(p.idx + unit * T + c) : 255;
    const int S_p = p.seq_len[b] - p.R;
    const int ntiles = (S_p + kTileTokens - 1) / kTileTokens;
    const int j0 = (int)((long long)member * ntiles / p.TS), j1 = (int)((long long)(member + 1) * ntiles / p.TS);
    const __nv_bfloat16* src = (const __nv_bfloat16*)p.k.ptr + b * p.k.sb + (int64_t)l * p.k.sl + (int64_t)h * p.k.sn;
    unsigned char* dst0 = (unsigned char*)p.k_thin + (p.thin_tile_base[b] + (int64_t)(l * p.N_kv + h) * ntiles) * (int64_t)Tp * 128;
    auto stage = [&](int j, int buf) {
      const int tok0 = j * kTileTokens;
      const int nvalid = min(kTileTokens, S_p - tok0);
      const uint32_t base = (uint32_t)__cvta_generic_to_shared(s_rows[buf]);
      for (int i = tid; i < kTileTokens * CPR; i += kThreads) {
        const int r = i / CPR, c = i % CPR;
        const bool ok = r < nvalid;
        const void* g = src + (int64_t)(tok0 + (ok ? r : 0)) * p.k.ss + c * 8;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(base + r * pitch + c * 16), "l"(g), "r"(ok ? 16 : 0) : "memory");
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    if (j0 < j1) stage(j0, 0);
    for (int j = j0; j < j1; ++j) {
      const int buf = (j - j0) & 1;
      if (j + 1 < j1) { stage(j + 1, buf ^ 1); asm volatile("cp.async.wait_group 1;" ::: "memory"); }
      else asm volatile("cp.async.wait_group 0;" ::: "memory");
      __syncthreads();
      // 8 warps: warp w builds step (w & 3); the two halves of the warps split the channel groups
      const int step = warp & 3, half = warp >> 2;
      const int r = lane >> 2, q = lane & 3;
      const unsigned char* rowA = s_rows[buf] + (step * 16 + r) * pitch;
      const unsigned char* rowB = rowA + 8 * pitch;
      unsigned char* dst = dst0 + (int64_t)j * Tp * 128 + step * (Tp * 32);
      auto elem = [&](const unsigned char* row, int ch) -> uint32_t {
        return ch == 255 ? 0u : (uint32_t)*(const uint16_t*)(row + ch * 2);
      };
      const int n16 = Tp >> 4;
      for (int g = half; g < n16; g += 2) {
        const int c0 = s_idx[16 * g + 2 * q], c1 = s_idx[16 * g + 2 * q + 1];
        const int c8 = s_idx[16 * g + 2 * q + 8], c9 = s_idx[16 * g + 2 * q + 9];
        uint4 v;
        v.x = elem(rowA, c0) | (elem(rowA, c1) << 16);
        v.y = elem(rowA, c8) | (elem(rowA, c9) << 16);
        v.z = elem(rowB, c0) | (elem(rowB, c1) << 16);
        v.w = elem(rowB, c8) | (elem(rowB, c9) << 16);
        *(uint4*)(dst + g * 512 + lane * 16) = v;
      }
      if ((Tp & 8) && half == (n16 & 1)) {
        const int c0 = s_idx[16 * n16 + 2 * q], c1 = s_idx[16 * n16 + 2 * q + 1];
        uint2 v;
        v.x = elem(rowA, c0) | (elem(rowA, c1) << 16);
        v.y = elem(rowB, c0) | (elem(rowB, c1) << 16);
        *(uint2*)(dst + n16 * 512 + lane * 8) = v;
      }
      __syncthreads();
    }
    return true;
  };

  int prev = -1, it = 0;
  for (int s = team; s < p.nslabs; s += p.NT, ++it) {
    phase_a(s, it & 1);
    if (prev >= 0 && !phase_b(prev)) return;
    prev = s;
  }
  if (prev >= 0) phase_b(prev);
}

}  // namespace

size_t prefill_smem_bytes(int D, int Tp) {
  return (size_t)2 * kTileTokens * (D * 2 + 16) + (size_t)kThreads * 8 * sizeof(double) + ((Tp + 15) & ~15);
}

int prefill_max_ctas_per_sm(int D, int Tp) {
  int n = 0;
  const size_t smem = prefill_smem_bytes(D, Tp);
  if (cudaFuncSetAttribute(k_prefill_fused<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return 0;
  if (cudaFuncSetAttribute(k_prefill_fused<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k_prefill_fused<false>, kThreads, smem) != cudaSuccess) return 0;
  return n > 2 ? 2 : n;
}

int prefill_group_size() { return kGroup; }

cudaError_t launch_prefill_fused(const PrefillParams& p, cudaStream_t s) {
  const size_t smem = prefill_smem_bytes(p.D, p.Tp);
  void* args[] = {(void*)&p};
  const void* fn = p.criterion == THINK_SCORE_KEY_L1 ? (const void*)k_prefill_fused<true> : (const void*)k_prefill_fused<false>;
  return cudaLaunchCooperativeKernel(fn, dim3(p.NT * p.TS), dim3(kThreads), args, smem, s);
}

}  // namespace think
