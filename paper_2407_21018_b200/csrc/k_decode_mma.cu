// Decode attention over the two-part key cache, bf16 (paper Sec. 3.3 / Fig. 2, Sec. 3.2).
//
// The stream of K_T / tail-K / V bytes is what bounds this kernel, so everything is arranged to keep
// many bytes in flight per SM and few instructions per byte:
//  * a WARP is the worker.  The flat list of 64-token tiles of all (b, layer, key head) units is cut
//    evenly over grid x warps workers; a worker walks its contiguous range 16 tokens at a time and
//    crosses unit boundaries as needed.  Warps never wait for each other: no block barriers, no
//    mbarriers, no spinning -- only cp.async groups of the warp itself.
//  * every warp owns a ring of kStages stages in shared memory.  A stage holds one 16-token step:
//    the keys (already in mma B-fragment order in global memory, so the copy is linear and the reads
//    are one conflict-free 16-byte load per lane) and 16 value rows (256 B each, 16-byte chunks
//    XOR-swizzled on the way in so that ldmatrix.trans is conflict-free).
//  * both products run on tensor cores with mma.sync m16n8k16 (bf16 in, fp32 accumulate): the G
//    query heads of the group are the rows of A (rows G..15 are zero), the 16 tokens of the step are
//    the columns of q.K^T and the contraction index of p.V.  The CUDA-core formulation needs about
//    5.5 instructions per key/value element for G = 4, which by itself exceeds the issue slots
//    available in the time HBM needs to deliver the bytes (profiles/k_decode_generic_c2_ncu.md).
//  * online softmax per step in the exp2 domain; partial states of units shared by several workers
//    go to the workspace and the worker that arrives last at the unit's ticket merges them.
#include <math.h>

#include "think_internal.h"

namespace think {
namespace {

constexpr int kWarps = 6;               // workers per CTA
constexpr int kStages = 4;              // ring depth per warp (3 steps in flight)
constexpr int kStepTokens = 16;
constexpr int kKSlot = 4096;            // bytes: keys of one step at D = 128
constexpr int kVSlot = 4096;            // bytes: 16 value rows at D = 128
constexpr int kStage = kKSlot + kVSlot;
constexpr int kSmemBytes = kWarps * kStages * kStage;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  // rows 8..15 of A (registers a1, a3) are zero: the group has at most 8 query heads
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma1688(float (&d)[4], uint32_t a0, uint32_t b0) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(0u), "r"(b0));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *(uint32_t*)&v;
}

__device__ __forceinline__ int worker_of(long long f, long long N, int nworkers) {
  return (int)(((f + 1) * nworkers - 1) / N);
}

// One 16-token step in flight: where its keys and values come from.
struct StepSrc {
  const unsigned char* k;   // Cp*32 contiguous bytes
  const unsigned char* v;   // first value row of the step
  long long vstride;        // bytes between value rows
  int kbytes;               // Cp*32
  int nrows;                // valid tokens in this step (1..16)
};

template <int D, int G>
__global__ void __launch_bounds__(kWarps * 32, 1) k_decode_mma(const DecodeParams p) {
  static_assert(D == 64 || D == 128, "head dimension");
  constexpr int NT = D / 8;              // n-tiles of the output
  constexpr int KS = D / 16;             // 16-channel groups of a full key
  extern __shared__ __align__(128) unsigned char smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int qd = lane & 3, row = lane >> 2;          // fragment coordinates: row = query head
  const uint32_t ring = smem_u32(smem) + warp * (kStages * kStage);
  const long long N = p.Ntot;
  // never more workers than tiles: every worker then owns a non-empty range
  const int nworkers = (int)min((long long)gridDim.x * kWarps, N);
  const int wk = blockIdx.x * kWarps + warp;
  if (wk >= nworkers) return;
  const long long f0 = (long long)wk * N / nworkers, f1 = (long long)(wk + 1) * N / nworkers;
  const int LH = p.nlayers * p.N_kv;
  const int ntt = p.n_tail_tiles;
  const int Tp = p.Tp;
  const int n16_thin = Tp >> 4;
  const bool has8_thin = (Tp & 8) != 0;
  const size_t rec_bytes = rec_size(D, G);
  const float scale = 1.4426950408889634f / sqrtf((float)D);

  long long f = f0;
  while (f < f1) {
    // ---- unit that owns tile f
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
    const int j1 = j0 + (int)(seg_end - f);             // tiles [j0, j1) of this unit
    const int S_p = p.seq_len[b] - p.R;
    const int64_t unit_abs = ((int64_t)b * p.L + l) * p.N_kv + h;
    const int unit_call = (b * p.nlayers + ll) * p.N_kv + h;

    const unsigned char* kthin = (const unsigned char*)p.k_thin +
                                 (p.thin_tile_base[b] + (int64_t)(l * p.N_kv + h) * nthin) * (int64_t)Tp * 128;
    const unsigned char* ktail = (const unsigned char*)p.tail_k + unit_abs * p.tail_tiles_cap * (int64_t)D * 128;
    const unsigned char* vthin = (const unsigned char*)((const __nv_bfloat16*)p.v.ptr + b * p.v.sb +
                                                         (int64_t)l * p.v.sl + (int64_t)h * p.v.sn);
    const unsigned char* vtail = (const unsigned char*)p.tail_v + unit_abs * p.cap * (int64_t)D * 2;

    // tokens valid in tile j of this unit
    auto tile_valid = [&](int j) {
      return j < nthin ? min(kTileTokens, S_p - j * kTileTokens) : min(kTileTokens, p.n_tail - (j - nthin) * kTileTokens);
    };
    // source of step st of tile j
    auto step_src = [&](int j, int st) {
      StepSrc s;
      const int nv = tile_valid(j) - st * kStepTokens;
      s.nrows = nv < kStepTokens ? nv : kStepTokens;
      if (j < nthin) {
        s.kbytes = Tp * 32;
        s.k = kthin + (int64_t)j * Tp * 128 + st * s.kbytes;
        s.vstride = p.v.ss * 2;
        s.v = vthin + (int64_t)(j * kTileTokens + st * kStepTokens) * s.vstride;
      } else {
        const int jt = j - nthin;
        s.kbytes = D * 32;
        s.k = ktail + (int64_t)jt * D * 128 + st * s.kbytes;
        s.vstride = D * 2;
        s.v = vtail + (int64_t)(jt * kTileTokens + st * kStepTokens) * s.vstride;
      }
      return s;
    };
    auto issue = [&](int slot, const StepSrc& s) {
      const uint32_t kdst = ring + slot * kStage, vdst = kdst + kKSlot;
      for (int i = lane; i * 16 < s.kbytes; i += 32) cp_async16(kdst + i * 16, s.k + i * 16, 16);
      constexpr int CPR = D * 2 / 16;                  // 16-byte chunks per value row
#pragma unroll
      for (int it = 0; it < kStepTokens * CPR / 32; ++it) {
        const int r = (it * 32 + lane) / CPR, ck = (it * 32 + lane) % CPR;
        const bool ok = r < s.nrows;                   // rows past the valid tokens are zero-filled
        cp_async16(vdst + r * (D * 2) + ((ck ^ (r & 7)) << 4), ok ? s.v + r * s.vstride + ck * 16 : s.v, ok ? 16 : 0);
      }
    };

    // ---- query fragments (A operand).  qa[s] = channels 16s+2qd,+1 | qa[s+KS] = channels 16s+2qd+8,+9
    const __nv_bfloat16* qg = (const __nv_bfloat16*)p.q + ((int64_t)(b * p.nlayers + ll) * p.N_q + h * G) * D;
    const uint8_t* idx = p.idx + unit_abs * p.T;
    uint32_t qa[KS][2];
    uint32_t qa8 = 0;
    auto q_pair = [&](int c, bool thin) -> uint32_t {   // (q[c], q[c+1]) of this lane's query head
      if (row >= G) return 0u;
      const uint16_t* qr = (const uint16_t*)(qg + row * D);
      uint32_t a = 0, bb = 0;
      if (thin) {
        if (c < p.T) a = qr[idx[c]];
        if (c + 1 < p.T) bb = qr[idx[c + 1]];
      } else {
        a = qr[c]; bb = qr[c + 1];
      }
      return a | (bb << 16);
    };
    auto load_q = [&](bool thin) {
#pragma unroll
      for (int s = 0; s < KS; ++s) {
        const bool on = !thin || s < n16_thin;
        qa[s][0] = on ? q_pair(16 * s + 2 * qd, thin) : 0u;
        qa[s][1] = on ? q_pair(16 * s + 2 * qd + 8, thin) : 0u;
      }
      qa8 = (thin && has8_thin) ? q_pair(16 * n16_thin + 2 * qd, true) : 0u;
    };
    bool q_is_thin = j0 < nthin;
    load_q(q_is_thin);

    // ---- online-softmax state of this worker for the unit (row = query head `row`)
    float m = -INFINITY, lsum = 0.f;
    float o[NT][4];
#pragma unroll
    for (int t = 0; t < NT; ++t) o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f;

    // ---- software pipeline over the steps of tiles [j0, j1)
    int ij = j0, ist = 0, islot = 0;                    // next step to issue
    auto steps_of = [&](int j) { return (tile_valid(j) + kStepTokens - 1) / kStepTokens; };
    int isteps = steps_of(j0);
    auto issue_next = [&]() {
      if (ij < j1) {
        issue(islot, step_src(ij, ist));
        if (++ist == isteps) { ist = 0; ++ij; if (ij < j1) isteps = steps_of(ij); }
      }
      cp_commit();                                      // one group per call, possibly empty
      islot = islot + 1 == kStages ? 0 : islot + 1;
    };
#pragma unroll
    for (int i = 0; i < kStages - 1; ++i) issue_next();

    int cslot = 0;
    for (int cj = j0; cj < j1; ++cj) {
      const bool thin = cj < nthin;
      if (thin != q_is_thin) { load_q(thin); q_is_thin = thin; }
      const int nvalid = tile_valid(cj);
      const int nsteps = (nvalid + kStepTokens - 1) / kStepTokens;
      const int n16 = thin ? n16_thin : KS;
      const bool has8 = thin && has8_thin;
      for (int st = 0; st < nsteps; ++st) {
        cp_wait<kStages - 2>();
        __syncwarp();
        const uint32_t kbase = ring + cslot * kStage, vbase = kbase + kKSlot;
        // S = q . K^T for the two 8-token halves of the step
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int s = 0; s < KS; ++s) {
          if (s < n16) {
            uint4 kb;
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(kb.x), "=r"(kb.y), "=r"(kb.z), "=r"(kb.w) : "r"(kbase + s * 512 + lane * 16));
            mma16816(s0, qa[s][0], qa[s][1], kb.x, kb.y);
            mma16816(s1, qa[s][0], qa[s][1], kb.z, kb.w);
          }
        }
        if (has8) {
          uint2 kb;
          asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(kb.x), "=r"(kb.y) : "r"(kbase + n16 * 512 + lane * 8));
          mma1688(s0, qa8, kb.x);
          mma1688(s1, qa8, kb.y);
        }
        // mask, scale into the exp2 domain, running max of this row over the quad
        const int t0 = st * kStepTokens + 2 * qd;        // token (in tile) of s0[0]
        float x00 = t0 < nvalid ? s0[0] * scale : -INFINITY;
        float x01 = t0 + 1 < nvalid ? s0[1] * scale : -INFINITY;
        float x10 = t0 + 8 < nvalid ? s1[0] * scale : -INFINITY;
        float x11 = t0 + 9 < nvalid ? s1[1] * scale : -INFINITY;
        float mx = fmaxf(fmaxf(x00, x01), fmaxf(x10, x11));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float mnew = fmaxf(m, mx);
        const float sc = exp2f(m - mnew);
        m = mnew;
        const uint32_t pa0 = pack_bf16(exp2f(x00 - mnew), exp2f(x01 - mnew));
        const uint32_t pa2 = pack_bf16(exp2f(x10 - mnew), exp2f(x11 - mnew));
        // the denominator sums the rounded weights, so numerator and denominator agree
        lsum = lsum * sc + (bf16lo(pa0) + bf16hi(pa0)) + (bf16lo(pa2) + bf16hi(pa2));
#pragma unroll
        for (int t = 0; t < NT; ++t) { o[t][0] *= sc; o[t][1] *= sc; }
        // O += P . V : value rows through ldmatrix.trans (tokens become the contraction index)
#pragma unroll
        for (int np = 0; np < NT / 2; ++np) {
          const int mi = lane >> 3;
          const int r = ((mi & 1) << 3) + (lane & 7);
          const int ck = 2 * np + (mi >> 1);
          uint32_t v0, v1, v2, v3;
          ldmatrix_x4_trans(vbase + r * (D * 2) + ((ck ^ (r & 7)) << 4), v0, v1, v2, v3);
          mma16816(o[2 * np], pa0, pa2, v0, v1);
          mma16816(o[2 * np + 1], pa0, pa2, v2, v3);
        }
        __syncwarp();                                   // every lane is done with the slot
        issue_next();
        cslot = cslot + 1 == kStages ? 0 : cslot + 1;
      }
    }
    cp_wait<0>();                                       // nothing of this unit is left in flight

    // ---- finish the segment: complete unit -> output, otherwise partial state + ticket
    lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
    lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
    const bool complete = (f == ustart) && (seg_end == uend);
    __nv_bfloat16* outp = (__nv_bfloat16*)p.out + ((int64_t)(b * p.nlayers + ll) * p.N_q + h * G) * D;
    if (complete) {
      if (row < G) {
        const float inv = 1.f / lsum;
#pragma unroll
        for (int t = 0; t < NT; ++t)
          *(uint32_t*)(outp + row * D + 8 * t + 2 * qd) = pack_bf16(o[t][0] * inv, o[t][1] * inv);
      }
    } else {
      uint8_t* rec = p.records + ((size_t)wk * 2 + (f == f0 ? 0 : 1)) * rec_bytes;
      if (row < G) {
        if (qd == 0) { ((double*)rec)[row] = (double)m; ((float*)(rec + G * 8))[row] = lsum; }
        float* ro = (float*)(rec + rec_o_off(G)) + row * D;
#pragma unroll
        for (int t = 0; t < NT; ++t) *(float2*)(ro + 8 * t + 2 * qd) = make_float2(o[t][0], o[t][1]);
      }
      const int c_first = worker_of(ustart, N, nworkers), c_last = worker_of(uend - 1, N, nworkers);
      __threadfence();
      __syncwarp();
      unsigned last = 0;
      if (lane == 0) last = atomicAdd(p.counters + unit_call, 1u) == (uint32_t)(c_last - c_first);
      last = __shfl_sync(0xffffffffu, last, 0);
      if (last) {
        __threadfence();
        for (int i = lane; i < G * D; i += 32) {
          const int g = i / D, d = i % D;
          float M = -INFINITY;
          for (int ci = c_first; ci <= c_last; ++ci) {
            const long long cf0 = (long long)ci * N / nworkers;
            const uint8_t* r = p.records + ((size_t)ci * 2 + (cf0 >= ustart ? 0 : 1)) * rec_bytes;
            M = fmaxf(M, (float)__ldcg((const double*)r + g));
          }
          float Lsum = 0.f, O = 0.f;
          for (int ci = c_first; ci <= c_last; ++ci) {
            const long long cf0 = (long long)ci * N / nworkers;
            const uint8_t* r = p.records + ((size_t)ci * 2 + (cf0 >= ustart ? 0 : 1)) * rec_bytes;
            const float w = exp2f((float)__ldcg((const double*)r + g) - M);
            Lsum += __ldcg((const float*)(r + G * 8) + g) * w;
            O += __ldcg((const float*)(r + rec_o_off(G)) + g * D + d) * w;
          }
          outp[g * D + d] = __float2bfloat16_rn(O / Lsum);
        }
        __syncwarp();
        if (lane == 0) p.counters[unit_call] = 0u;
      }
    }
    f = seg_end;
  }
}

template <int D, int G>
cudaError_t launch_mma(const DecodeParams& p, cudaStream_t s) {
  k_decode_mma<D, G><<<p.grid, kWarps * 32, kSmemBytes, s>>>(p);
  return cudaGetLastError();
}
template <int D, int G>
cudaError_t setup_mma() {
  return cudaFuncSetAttribute(k_decode_mma<D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
}

#define THINK_MMA_DISPATCH(FN, ...)                                   \
  do {                                                                \
    if (D == 128) switch (G) { case 1: return FN<128, 1>(__VA_ARGS__); \
                               case 2: return FN<128, 2>(__VA_ARGS__); \
                               case 4: return FN<128, 4>(__VA_ARGS__); \
                               case 8: return FN<128, 8>(__VA_ARGS__); } \
    if (D == 64) switch (G) { case 1: return FN<64, 1>(__VA_ARGS__);   \
                              case 2: return FN<64, 2>(__VA_ARGS__);   \
                              case 4: return FN<64, 4>(__VA_ARGS__);   \
                              case 8: return FN<64, 8>(__VA_ARGS__); } \
  } while (0)

}  // namespace

cudaError_t launch_decode_bf16(const DecodeParams& p, int D, int G, cudaStream_t s) {
  THINK_MMA_DISPATCH(launch_mma, p, s);
  return cudaErrorInvalidValue;
}
cudaError_t decode_setup_bf16(int D, int G) {
  THINK_MMA_DISPATCH(setup_mma);
  return cudaErrorInvalidValue;
}
int decode_warps_bf16() { return kWarps; }

}  // namespace think
