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
//    available in the time HBM needs to deliver the bytes (measured: 146.6 M warp instructions per launch of
//    the CUDA-core kernel on the LLaMA-3-8B-shaped workload against 41.5 M here).
//  * online softmax per step in the exp2 domain; partial states of units shared by several workers
//    go to the workspace and the worker that arrives last at the unit's ticket merges them.
#include <math.h>

#include "think_internal.h"

namespace think {
namespace {

#ifndef THINK_DEC_WARPS
#define THINK_DEC_WARPS 8
#endif
#ifndef THINK_DEC_STAGES
#define THINK_DEC_STAGES 3
#endif
constexpr int kWarps = THINK_DEC_WARPS;  // workers per CTA
constexpr int kStages = THINK_DEC_STAGES;  // ring depth per warp (kStages - 1 steps in flight)
constexpr int kStepTokens = 16;
constexpr int kKSlot = 4096;            // bytes: keys of one step at D = 128
constexpr int kVSlot = 4096;            // bytes: 16 value rows at D = 128
constexpr int kStage = kKSlot + kVSlot;
constexpr int kSmemBytes = kWarps * kStages * kStage;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// copies src_bytes (0 or 16) and zero-fills the rest of the 16 bytes
__device__ __forceinline__ void cp_async16_zfill(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  // rows 8..15 of A (registers a1, a3) are zero: the group has at most 8 query heads
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma1688(float (&d)[4], uint32_t a0, uint32_t b0) {
  asm(
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

// A run of consecutive 16-token steps of one kind (thin prefix tiles or unpruned tail tiles):
// keys advance kstep bytes per step, values 16 rows per step.
struct Region {
  const unsigned char* k;   // keys of the first step (fragment order, kstep contiguous bytes per step)
  const unsigned char* v;   // first value row
  long long vstride;        // bytes between value rows
  int kstep;                // Cp * 32
  int ntok;                 // tokens in the region (the last step may be partial)
  int n16;                  // 16-channel groups per key
  bool has8;                // trailing 8-channel group
  bool thin;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// VT: the prefix values are thinned as well (App. D); everything about values then lives in the
// permuted channel order and the output is un-permuted when it is written.
template <int D, int G, bool VT>
__global__ void __launch_bounds__(kWarps * 32, 1) k_decode_mma(const DecodeParams p) {
  static_assert(D == 64 || D == 128, "head dimension");
  constexpr int NT = D / 8;              // n-tiles of the output
  constexpr int KS = D / 16;             // 16-channel groups of a full key
  constexpr int kQScratch = G * D * 2 + 128;          // per warp: the group's query rows + the unit's index list
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
  // per-lane constants of the value path: which 16-byte chunk of which row this lane copies in
  // iteration `it`, where it lands (XOR swizzle), and the ldmatrix row addresses per pair of n-tiles
  constexpr int CPR = D * 2 / 16;          // 16-byte chunks per value row
  constexpr int RPI = 32 / CPR;            // rows per copy iteration
  constexpr int VIT = kStepTokens / RPI;   // copy iterations per step
  const int vlane_row = lane / CPR, vlane_ck = lane % CPR;
  int vdst_off[VIT];
#pragma unroll
  for (int it = 0; it < VIT; ++it) {
    const int r = it * RPI + vlane_row;
    vdst_off[it] = r * (D * 2) + ((vlane_ck ^ (r & 7)) << 4);
  }
  int vld_off[NT / 2];
#pragma unroll
  for (int np = 0; np < NT / 2; ++np) {
    const int mi = lane >> 3, r = ((mi & 1) << 3) + (lane & 7), ck = 2 * np + (mi >> 1);
    vld_off[np] = r * (D * 2) + ((ck ^ (r & 7)) << 4);
  }

  // ---- producer side of the warp's ring.  It walks the worker's whole tile range [f0, f1) on its own,
  // region after region (thin tiles of a unit, then its tail tiles, then the next unit), so the ring stays
  // full across unit boundaries; the consumer below follows the same sequence.
  long long pf = f0;                                  // first tile not yet handed to the producer
  int islot = 0, i_left = 0, i_kstep = 0;
  int i_vck = CPR;                                    // 16-byte chunks per value row of the region
  long long i_vrow = 0;
  const unsigned char* ikl = nullptr;
  const unsigned char* iv = nullptr;
  const unsigned char* i_vsafe = nullptr;
  auto p_next_region = [&]() {                        // load the region that starts at tile pf (pf < f1)
    int lo = 0, hi = p.B - 1;
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      long long cm = (long long)LH * (p.cum_thin[mid] + (long long)mid * ntt);
      if (cm <= pf) lo = mid; else hi = mid - 1;
    }
    const int b = lo;
    const int nthin = p.cum_thin[b + 1] - p.cum_thin[b];
    const int tpu = nthin + ntt;
    const long long rem = pf - (long long)LH * (p.cum_thin[b] + (long long)b * ntt);
    const int u_in_b = (int)(rem / tpu), j0 = (int)(rem % tpu);
    const int l = p.layer0 + u_in_b / p.N_kv, h = u_in_b % p.N_kv;
    const long long uend = pf - j0 + tpu;
    const int j1 = j0 + (int)((f1 < uend ? f1 : uend) - pf);
    const int64_t unit_abs = ((int64_t)b * p.L + l) * p.N_kv + h;
    const unsigned char *k0, *v0;
    int ntiles;
    if (j0 < nthin) {
      const int je = j1 < nthin ? j1 : nthin;
      ntiles = je - j0;
      i_kstep = Tp * 32;
      k0 = (const unsigned char*)p.k_thin + (p.thin_tile_base[b] + (int64_t)(l * p.N_kv + h) * (nthin + p.re_cap) + j0) * (int64_t)Tp * 128;
      if (VT) {
        i_vrow = p.Tvp * 2;
        i_vck = p.Tvp >> 3;
        v0 = (const unsigned char*)p.v_thin +
             (p.v_thin_base[b] + ((int64_t)(l * p.N_kv + h) * (p.seq_len[b] - p.R) + (int64_t)j0 * kTileTokens) * p.Tvp) * 2;
      } else {
        i_vrow = p.v.ss * 2;
        v0 = (const unsigned char*)((const __nv_bfloat16*)p.v.ptr + b * p.v.sb + (int64_t)l * p.v.sl + (int64_t)h * p.v.sn) +
             (int64_t)j0 * kTileTokens * i_vrow;
      }
      i_left = min(p.seq_len[b] - p.R, je * kTileTokens) - j0 * kTileTokens;
    } else if (j0 - nthin < p.n_re) {
      // tail blocks that were re-pruned: keys thinned like the prefix, values still in the tail buffer
      asm volatile("griddepcontrol.wait;" ::: "memory");   // the append ahead of this launch has written the tail
      const int jb = j0 - nthin, je = min(j1 - nthin, p.n_re);
      ntiles = je - jb;
      i_kstep = Tp * 32;
      i_vrow = D * 2;
      if (VT) i_vck = CPR;
      k0 = (const unsigned char*)p.k_thin +
           (p.thin_tile_base[b] + (int64_t)(l * p.N_kv + h) * (nthin + p.re_cap) + nthin + jb) * (int64_t)Tp * 128;
      v0 = (const unsigned char*)p.tail_v + (unit_abs * p.cap + (int64_t)jb * kTileTokens) * D * 2;
      i_left = ntiles * kTileTokens;
    } else {
      asm volatile("griddepcontrol.wait;" ::: "memory");   // the append ahead of this launch has written the tail
      const int jb = j0 - nthin, je = j1 - nthin;
      ntiles = je - jb;
      i_kstep = D * 32;
      i_vrow = D * 2;
      if (VT) i_vck = CPR;
      k0 = (const unsigned char*)p.tail_k + (unit_abs * p.tail_tiles_cap + jb) * (int64_t)D * 128;
      v0 = (const unsigned char*)p.tail_v + (unit_abs * p.cap + (int64_t)jb * kTileTokens) * D * 2;
      i_left = min(p.n_tail, je * kTileTokens) - jb * kTileTokens;
    }
    ikl = k0 + lane * 16;
    iv = v0 + vlane_row * i_vrow + vlane_ck * 16;
    i_vsafe = v0;
    pf += ntiles;
  };
  p_next_region();
  auto issue_next = [&]() {
    if (i_left > 0) {
      const uint32_t sb = ring + islot * kStage;
      const uint32_t kd = sb + lane * 16;
      const int nfull = i_kstep >> 9, krem = i_kstep & 511;       // 512-byte pieces of the key step
#pragma unroll
      for (int n = 0; n < D * 32 / 512; ++n)
        if (n < nfull) cp_async16(kd + n * 512, ikl + n * 512);
      if (lane * 16 < krem) cp_async16(kd + nfull * 512, ikl + nfull * 512);
      const unsigned char* vs = iv;
      const long long rstep = RPI * i_vrow;
      if (!VT || vlane_ck < i_vck) {                  // thinned rows are shorter: the other lanes sit out
        if (i_left >= kStepTokens) {
#pragma unroll
          for (int it = 0; it < VIT; ++it) {
            cp_async16(sb + kKSlot + vdst_off[it], vs);
            vs += rstep;
          }
        } else {                                      // last step of a region: zero-fill missing rows
#pragma unroll
          for (int it = 0; it < VIT; ++it) {
            const bool ok = it * RPI + vlane_row < i_left;
            cp_async16_zfill(sb + kKSlot + vdst_off[it], ok ? vs : i_vsafe, ok ? 16 : 0);
            vs += rstep;
          }
        }
      }
      i_left -= kStepTokens;
      ikl += i_kstep;
      iv += kStepTokens * i_vrow;
      if (i_left <= 0) {
        i_left = 0;
        if (pf < f1) p_next_region();
      }
    }
    cp_commit();                                      // one group per call, possibly empty
    islot = islot + 1 == kStages ? 0 : islot + 1;
  };
#pragma unroll 1
  for (int i = 0; i < kStages - 1; ++i) issue_next();
  int cslot = 0;                                      // consumer's slot, in step with the producer's

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

    // ---- the segment is up to three runs of 16-token steps: thin prefix tiles, re-pruned tail blocks
    // (thin keys as well), unpruned tail tiles.  The consumer only needs their token counts.
    int seg_ntok[3] = {0, 0, 0};
    if (j0 < nthin) seg_ntok[0] = min(S_p, (j1 < nthin ? j1 : nthin) * kTileTokens) - j0 * kTileTokens;
    if (j1 > nthin) {
      const int jb = (j0 > nthin ? j0 : nthin) - nthin, je = j1 - nthin;
      if (jb < p.n_re) seg_ntok[1] = (min(je, p.n_re) - jb) * kTileTokens;
      const int jb2 = jb > p.n_re ? jb : p.n_re;
      if (je > jb2) seg_ntok[2] = min(p.n_tail, je * kTileTokens) - jb2 * kTileTokens;
    }

    // ---- query fragments (A operand): qa[s][0] = channels 16s+2qd,+1 ; qa[s][1] = channels 16s+2qd+8,+9
    // The group's G query rows (contiguous) and the unit's index list go to this warp's scratch in ONE round
    // trip of independent loads; both the gathered and the full query fragments are then read from there, so a
    // segment pays one global latency instead of three (index list -> gathered query -> full query).
    const __nv_bfloat16* qg = (const __nv_bfloat16*)p.q + ((int64_t)(b * p.nlayers + ll) * p.N_q + h * G) * D;
    const uint8_t* idx = p.idx + unit_abs * p.T;
    unsigned char* qs = smem + kSmemBytes + warp * kQScratch;
    {
      constexpr int QV = (G * D / 8 + 31) / 32;        // 16-byte pieces of the query rows per lane
      uint4 qv[QV];
      uint8_t iv[4];
#pragma unroll
      for (int i = 0; i < QV; ++i)
        if (lane + 32 * i < G * D / 8) qv[i] = __ldg((const uint4*)qg + lane + 32 * i);
#pragma unroll
      for (int i = 0; i < 4; ++i) iv[i] = lane + 32 * i < p.T ? idx[lane + 32 * i] : (uint8_t)0;
      __syncwarp();                                     // the previous segment's readers are done
#pragma unroll
      for (int i = 0; i < QV; ++i)
        if (lane + 32 * i < G * D / 8) ((uint4*)qs)[lane + 32 * i] = qv[i];
#pragma unroll
      for (int i = 0; i < 4; ++i) qs[G * D * 2 + lane + 32 * i] = iv[i];
      __syncwarp();
    }
    uint32_t qa[KS][2];
    uint32_t qa8 = 0;
    auto q_pair = [&](int c, bool thin) -> uint32_t {   // (q[c], q[c+1]) of this lane's query head
      if (row >= G) return 0u;
      const unsigned char* qr = qs + row * (D * 2);
      if (!thin) return *(const uint32_t*)(qr + 2 * c);
      const uint8_t* ix = qs + G * D * 2;
      const uint32_t a = c < p.T ? *(const uint16_t*)(qr + 2 * ix[c]) : 0u;
      const uint32_t bb = c + 1 < p.T ? *(const uint16_t*)(qr + 2 * ix[c + 1]) : 0u;
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

    // ---- online-softmax state of this worker for the unit (row = query head `row`), exp2 domain
    float m = -INFINITY, lsum = 0.f;
    float o[NT][4];
#pragma unroll
    for (int t = 0; t < NT; ++t) o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f;

    // ---- consumer side
    int q_kind = -1;                                    // 1: gathered query loaded, 0: full query
#pragma unroll
    for (int cr = 0; cr < 3; ++cr) {
      const int ntok = seg_ntok[cr];
      if (ntok <= 0) continue;
      const bool thin = cr < 2;
      if (q_kind != (int)thin) { load_q(thin); q_kind = thin; }
      const int n16 = thin ? n16_thin : KS;
      const bool has8 = thin && has8_thin;
      const int npv = (VT && cr == 0) ? (p.Tvp >> 4) : NT / 2;   // pairs of n-tiles the region's values fill
      for (int left = ntok; left > 0; left -= kStepTokens) {
        cp_wait<kStages - 2>();
        __syncwarp();       // this step's data has landed; every lane is done with the previous slot
        issue_next();       // refill that slot right away: the loads do not wait for this step's math
        const uint32_t kbase = ring + cslot * kStage + lane * 16, vbase = ring + cslot * kStage + kKSlot;
        // S = q . K^T for the two 8-token halves of the step; even and odd channel groups accumulate
        // separately to halve the chain of dependent MMAs
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
        float u0[4] = {0.f, 0.f, 0.f, 0.f}, u1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int s = 0; s < KS; ++s) {
          if (s < n16) {
            uint4 kb;
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(kb.x), "=r"(kb.y), "=r"(kb.z), "=r"(kb.w) : "r"(kbase + s * 512));
            if (s & 1) {
              mma16816(u0, qa[s][0], qa[s][1], kb.x, kb.y);
              mma16816(u1, qa[s][0], qa[s][1], kb.z, kb.w);
            } else {
              mma16816(s0, qa[s][0], qa[s][1], kb.x, kb.y);
              mma16816(s1, qa[s][0], qa[s][1], kb.z, kb.w);
            }
          }
        }
        if (has8) {
          uint2 kb;
          asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];"
                       : "=r"(kb.x), "=r"(kb.y) : "r"(kbase - lane * 8 + n16 * 512));
          mma1688(u0, qa8, kb.x);
          mma1688(u1, qa8, kb.y);
        }
        s0[0] += u0[0]; s0[1] += u0[1]; s1[0] += u1[0]; s1[1] += u1[1];
        if (left < kStepTokens) {                       // last step of the region: mask the missing tokens
          const int t0 = 2 * qd;
          if (t0 >= left) s0[0] = -INFINITY;
          if (t0 + 1 >= left) s0[1] = -INFINITY;
          if (t0 + 8 >= left) s1[0] = -INFINITY;
          if (t0 + 9 >= left) s1[1] = -INFINITY;
        }
        // running max of this row over the quad, in the exp2 domain
        float mx = fmaxf(fmaxf(s0[0], s0[1]), fmaxf(s1[0], s1[1]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        mx *= scale;
        if (__any_sync(0xffffffffu, mx > m)) {          // some row's maximum grew: rescale the state
          const float mnew = fmaxf(m, mx);
          const float sc = ex2(m - mnew);
          m = mnew;
          lsum *= sc;
#pragma unroll
          for (int t = 0; t < NT; ++t) { o[t][0] *= sc; o[t][1] *= sc; }
        }
        const uint32_t pa0 = pack_bf16(ex2(fmaf(s0[0], scale, -m)), ex2(fmaf(s0[1], scale, -m)));
        const uint32_t pa2 = pack_bf16(ex2(fmaf(s1[0], scale, -m)), ex2(fmaf(s1[1], scale, -m)));
        // the denominator sums the rounded weights, so numerator and denominator agree
        lsum += (bf16lo(pa0) + bf16hi(pa0)) + (bf16lo(pa2) + bf16hi(pa2));
        // O += P . V : value rows through ldmatrix.trans (tokens become the contraction index)
#pragma unroll
        for (int np = 0; np < NT / 2; ++np) {
          if (VT && np >= npv) continue;
          uint32_t v0, v1, v2, v3;
          ldmatrix_x4_trans(vbase + vld_off[np], v0, v1, v2, v3);
          mma16816(o[2 * np], pa0, pa2, v0, v1);
          mma16816(o[2 * np + 1], pa0, pa2, v2, v3);
        }
        cslot = cslot + 1 == kStages ? 0 : cslot + 1;
      }
    }
    // ---- finish the segment: complete unit -> output, otherwise partial state + ticket
    lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
    lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
    const bool complete = (f == ustart) && (seg_end == uend);
    __nv_bfloat16* outp = (__nv_bfloat16*)p.out + ((int64_t)(b * p.nlayers + ll) * p.N_q + h * G) * D;
    const uint8_t* perm = VT ? p.perm_v + unit_abs * D : nullptr;   // accumulator column c is output channel perm[c]
    if (complete) {
      if (row < G) {
        const float inv = 1.f / lsum;
#pragma unroll
        for (int t = 0; t < NT; ++t) {
          if (VT) {
            outp[row * D + perm[8 * t + 2 * qd]] = __float2bfloat16_rn(o[t][0] * inv);
            outp[row * D + perm[8 * t + 2 * qd + 1]] = __float2bfloat16_rn(o[t][1] * inv);
          } else {
            *(uint32_t*)(outp + row * D + 8 * t + 2 * qd) = pack_bf16(o[t][0] * inv, o[t][1] * inv);
          }
        }
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
        // Merge in worker (= token) order.  Lane g < G owns the statistics of query head g; every
        // lane owns G*D/32 output elements.  One round trip per contributor for the maxima, then one
        // per contributor for its weights and all of this lane's output elements at once.
        auto rec_of = [&](int ci) {
          const long long cf0 = (long long)ci * N / nworkers;
          return p.records + ((size_t)ci * 2 + (cf0 >= ustart ? 0 : 1)) * rec_bytes;
        };
        constexpr int EPL = G * D / 32;                  // elements per lane: i = lane + 32 k
        float M = -INFINITY;
        if (lane < G)
          for (int ci = c_first; ci <= c_last; ++ci) M = fmaxf(M, (float)__ldcg((const double*)rec_of(ci) + lane));
        float Lsum = 0.f, acc[EPL];
#pragma unroll
        for (int k = 0; k < EPL; ++k) acc[k] = 0.f;
        // two contributors per trip: both sets of loads are in flight together, sums stay in worker order
        for (int ci = c_first; ci <= c_last; ci += 2) {
          const bool two = ci + 1 <= c_last;
          const uint8_t* r0 = rec_of(ci);
          const uint8_t* r1 = rec_of(two ? ci + 1 : ci);
          float ov0[EPL], ov1[EPL];
#pragma unroll
          for (int k = 0; k < EPL; ++k) ov0[k] = __ldcg((const float*)(r0 + rec_o_off(G)) + lane + 32 * k);
#pragma unroll
          for (int k = 0; k < EPL; ++k) ov1[k] = __ldcg((const float*)(r1 + rec_o_off(G)) + lane + 32 * k);
          float w0 = 0.f, w1 = 0.f;
          if (lane < G) {
            const float m0 = (float)__ldcg((const double*)r0 + lane), m1 = (float)__ldcg((const double*)r1 + lane);
            const float l0 = __ldcg((const float*)(r0 + G * 8) + lane), l1 = __ldcg((const float*)(r1 + G * 8) + lane);
            w0 = exp2f(m0 - M);
            Lsum += l0 * w0;
            if (two) {
              w1 = exp2f(m1 - M);
              Lsum += l1 * w1;
            }
          }
#pragma unroll
          for (int k = 0; k < EPL; ++k) acc[k] = fmaf(ov0[k], __shfl_sync(0xffffffffu, w0, (lane + 32 * k) / D), acc[k]);
#pragma unroll
          for (int k = 0; k < EPL; ++k) acc[k] = fmaf(ov1[k], __shfl_sync(0xffffffffu, w1, (lane + 32 * k) / D), acc[k]);
        }
#pragma unroll
        for (int k = 0; k < EPL; ++k) {
          const int i = lane + 32 * k;
          const int oi = VT ? (i / D) * D + perm[i % D] : i;
          outp[oi] = __float2bfloat16_rn(acc[k] / __shfl_sync(0xffffffffu, Lsum, i / D));
        }
        __syncwarp();
        if (lane == 0) p.counters[unit_call] = 0u;
      }
    }
    f = seg_end;
  }
  cp_wait<0>();
}

template <int D, int G>
cudaError_t launch_mma(const DecodeParams& p, cudaStream_t s) {
  constexpr int smem = kSmemBytes + kWarps * (G * D * 2 + 128);
  if (p.dependent_launch) {
    // programmatic dependent launch: the grid may start while the append kernel ahead of it in the stream is
    // still running; only workers that reach tail tiles wait for it (griddepcontrol.wait in the kernel)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.grid);
    cfg.blockDim = dim3(kWarps * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return p.v_thin ? cudaLaunchKernelEx(&cfg, k_decode_mma<D, G, true>, p) : cudaLaunchKernelEx(&cfg, k_decode_mma<D, G, false>, p);
  }
  if (p.v_thin) k_decode_mma<D, G, true><<<p.grid, kWarps * 32, smem, s>>>(p);
  else k_decode_mma<D, G, false><<<p.grid, kWarps * 32, smem, s>>>(p);
  return cudaGetLastError();
}
template <int D, int G>
cudaError_t setup_mma() {
  constexpr int smem = kSmemBytes + kWarps * (G * D * 2 + 128);
  static_assert(smem <= 227 * 1024, "ring + query scratch exceed the shared memory of a CTA");
  cudaError_t e = cudaFuncSetAttribute(k_decode_mma<D, G, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_decode_mma<D, G, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
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
