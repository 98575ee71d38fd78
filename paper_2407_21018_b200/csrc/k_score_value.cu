// Value-channel scores and their top-T_v (paper App. D, Eqs. 3-4), bf16:
//   Score_v[j] = || softmax(Q[-S_obs:] K^T / sqrt(D)) V[:, j] ||_F ,  I_v = Top_T(Score_v, T_v).
//
// Unlike the key score this has no closed form: it is the attention output of the window's queries
// (the G query heads of the group stacked: M = G * S_obs rows) over the whole prompt, i.e. two dense
// contractions per head, so it runs on tensor cores (mma.sync m16n8k16, bf16 in, fp32 accumulate).
//  * A CTA owns (token split, block of up to 128 query rows, unit (b, l, h)); warp w owns 16 rows.
//    K and V tiles of 64 tokens are staged with cp.async into a two-stage ring shared by the warps
//    (rows XOR-swizzled by 16-byte chunk so that ldmatrix is conflict-free).
//  * Online softmax per row in the exp2 domain.  The weights enter the second product as a bf16
//    pair hi + lo (two MMAs), so their rounding error is 2^-17 instead of 2^-9: the scores then agree
//    with an fp64 evaluation to ~1e-5 and the ranking is stable against it.
//  * Every CTA leaves (m, l, O) of its rows in the workspace; the CTA that takes the unit's last
//    ticket merges the splits in order, forms the column norms in fp64 and ranks the channels.
#include <math.h>

#include "think_internal.h"

namespace think {
namespace {

constexpr int kVTile = 64;        // tokens per staged tile
constexpr int kVStages = 2;
constexpr int kRowGroups = 8;     // row groups of the finaliser's column sums

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16_zfill(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// (lo, hi) -> packed bf16 pair of the values and of what the rounding left over
__device__ __forceinline__ void split_pair(float x0, float x1, uint32_t& hi, uint32_t& lo, float& sum) {
  const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
  const float r0 = x0 - __bfloat162float(h0), r1 = x1 - __bfloat162float(h1);
  const __nv_bfloat16 l0 = __float2bfloat16_rn(r0), l1 = __float2bfloat16_rn(r1);
  hi = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
  lo = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
  sum += (__bfloat162float(h0) + __bfloat162float(l0)) + (__bfloat162float(h1) + __bfloat162float(l1));
}

// the same without the running sum: one packed conversion per pair
__device__ __forceinline__ void split_pair_packed(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
  hi = *(const uint32_t*)&h;
  const __nv_bfloat162 l = __floats2bfloat162_rn(x0 - __uint_as_float(hi << 16), x1 - __uint_as_float(hi & 0xffff0000u));
  lo = *(const uint32_t*)&l;
}

// Ticket + finaliser shared by both kernels: the CTA that arrives last for the unit merges the splits
// row by row (in split order), forms the column norms over all M rows in fp64 and ranks the channels.
// `smem`: scratch of at least nsplit*M*4 + (kRowGroups + 1)*D*8 bytes, free to overwrite; `s_last_slot`: one int of
// shared memory outside that scratch; `arrivals`: token splits this CTA stands for.
template <int D>
__device__ void finish_unit(const ValueScoreParams& p, unsigned char* smem, int* s_last_slot, int ucall, int b, int l, int h,
                            int arrivals = 1) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthreads = blockDim.x;
  const size_t rec_floats = (size_t)p.MB * (2 + D);
  __threadfence();
  __syncthreads();
  if (tid == 0) *s_last_slot = atomicAdd(p.counters + ucall, (uint32_t)arrivals) == (uint32_t)(p.nrb * p.nsplit - arrivals);
  __syncthreads();
  if (!*s_last_slot) return;
  __threadfence();

  float* w = (float*)smem;                                   // [nsplit][M]: weight of a split's row / its denominator
  double* en = (double*)(smem + (((size_t)p.nsplit * p.M * 4 + 15) & ~(size_t)15));   // [kRowGroups][D]
  double* sc = en + kRowGroups * D;                          // [D]
  const float* ubase = p.partials + (size_t)ucall * p.nrb * p.nsplit * rec_floats;
  for (int r = tid; r < p.M; r += nthreads) {
    const float* rrec = ubase + (size_t)(r / p.MB) * p.nsplit * rec_floats;
    const int rl = r % p.MB;
    float mx = -INFINITY;
    for (int sp = 0; sp < p.nsplit; ++sp) mx = fmaxf(mx, __ldcg(rrec + sp * rec_floats + rl));
    float den = 0.f;
    for (int sp = 0; sp < p.nsplit; ++sp)
      den += __ldcg(rrec + sp * rec_floats + p.MB + rl) * exp2f(__ldcg(rrec + sp * rec_floats + rl) - mx);
    for (int sp = 0; sp < p.nsplit; ++sp) w[sp * p.M + r] = exp2f(__ldcg(rrec + sp * rec_floats + rl) - mx) / den;
  }
  __syncthreads();
  for (int item = tid; item < kRowGroups * D; item += nthreads) {
    const int rg = item / D, j = item % D;
    double e = 0.0;
    // four rows at a time so that their loads are in flight together; sums stay in row order
    for (int r0 = rg; r0 < p.M; r0 += 4 * kRowGroups) {
      float x[4] = {0.f, 0.f, 0.f, 0.f};
      const float* rrec[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int r = min(r0 + u * kRowGroups, p.M - 1);
        rrec[u] = ubase + (size_t)(r / p.MB) * p.nsplit * rec_floats + 2 * p.MB + (size_t)(r % p.MB) * D + j;
      }
      for (int sp = 0; sp < p.nsplit; ++sp) {
        float v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = __ldcg(rrec[u] + sp * rec_floats);
#pragma unroll
        for (int u = 0; u < 4; ++u) x[u] = fmaf(v[u], w[sp * p.M + min(r0 + u * kRowGroups, p.M - 1)], x[u]);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (r0 + u * kRowGroups < p.M) e = fma((double)x[u], (double)x[u], e);
    }
    en[rg * D + j] = e;
  }
  __syncthreads();
  for (int j = tid; j < D; j += nthreads) {
    double e = 0.0;
    for (int rg = 0; rg < kRowGroups; ++rg) e += en[rg * D + j];
    sc[j] = sqrt(e);
  }
  __syncthreads();
  const int64_t unit = ((int64_t)b * p.L + l) * p.N_kv + h;
  if (warp == 0) {
    select_head(sc, D, p.Tv, p.perm_v + unit * D, lane, true, p.error);
    if (p.scores_v)
      for (int j = lane; j < D; j += 32) p.scores_v[unit * D + j] = sc[j];
  }
  if (tid == 0) p.counters[ucall] = 0u;   // ready for the next launch
}

template <int D>
__global__ void __launch_bounds__(256, 1) k_score_value(const ValueScoreParams p) {
  constexpr int KS = D / 16, NT = D / 8;
  constexpr int CPR = D * 2 / 16;            // 16-byte chunks per row
  constexpr int ROWB = D * 2;
  constexpr int kTileBytes = kVTile * ROWB;
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthreads = blockDim.x;
  const int qd = lane & 3, frow = lane >> 2;
  const int split = blockIdx.x, rb = blockIdx.y, ucall = blockIdx.z;
  const int h = ucall % p.N_kv, bl = ucall / p.N_kv;
  const int ll = bl % p.nlayers, b = bl / p.nlayers, l = p.layer0 + ll;
  const int S_b = p.seq_len[b];
  const int ntile_all = (S_b + kVTile - 1) / kVTile;
  const int per = (ntile_all + p.nsplit - 1) / p.nsplit;
  const int t0 = min(S_b, split * per * kVTile), t1 = min(S_b, (split + 1) * per * kVTile);
  const int ntl = (t1 - t0 + kVTile - 1) / kVTile;

  // ---- query rows of this warp (A operand).  Row r of the unit = query head h*G + r / S_obs, window row r % S_obs.
  const int rA = rb * p.MB + warp * 16 + frow, rB = rA + 8;
  uint32_t qa[KS][4];
  {
    const __nv_bfloat16* qbase = (const __nv_bfloat16*)p.q.ptr + b * p.q.sb + (int64_t)l * p.q.sl;
    const bool okA = rA < p.M, okB = rB < p.M;
    const __nv_bfloat16* qA = qbase + (int64_t)(okA ? rA % p.S_obs : 0) * p.q.ss + (int64_t)(h * p.G + (okA ? rA / p.S_obs : 0)) * p.q.sn;
    const __nv_bfloat16* qB = qbase + (int64_t)(okB ? rB % p.S_obs : 0) * p.q.ss + (int64_t)(h * p.G + (okB ? rB / p.S_obs : 0)) * p.q.sn;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int c = 16 * ks + 2 * qd;
      qa[ks][0] = okA ? *(const uint32_t*)(qA + c) : 0u;
      qa[ks][1] = okB ? *(const uint32_t*)(qB + c) : 0u;
      qa[ks][2] = okA ? *(const uint32_t*)(qA + c + 8) : 0u;
      qa[ks][3] = okB ? *(const uint32_t*)(qB + c + 8) : 0u;
    }
  }

  const __nv_bfloat16* kg = (const __nv_bfloat16*)p.k.ptr + b * p.k.sb + (int64_t)l * p.k.sl + (int64_t)h * p.k.sn;
  const __nv_bfloat16* vg = (const __nv_bfloat16*)p.v.ptr + b * p.v.sb + (int64_t)l * p.v.sl + (int64_t)h * p.v.sn;
  const uint32_t sbase = smem_u32(smem);
  auto load_tile = [&](int stage, int tok0) {
    const uint32_t kd = sbase + stage * 2 * kTileBytes, vd = kd + kTileBytes;
    for (int i = tid; i < kVTile * CPR; i += nthreads) {
      const int r = i / CPR, ck = i % CPR;
      const bool ok = tok0 + r < t1;                 // rows past the range are zero-filled
      const int64_t t = ok ? tok0 + r : t0;
      const uint32_t off = r * ROWB + ((ck ^ (r & 7)) << 4);
      cp_async16_zfill(kd + off, kg + t * p.k.ss + ck * 8, ok ? 16 : 0);
      cp_async16_zfill(vd + off, vg + t * p.v.ss + ck * 8, ok ? 16 : 0);
    }
  };

  // ---- per-lane ldmatrix offsets inside a tile
  const int mi = lane >> 3;
  // keys (not transposed): matrix mi = (token block mi>>1, channel half mi&1) of a pair of token blocks
  const int k_row = ((mi >> 1) << 3) + (lane & 7);
  // values (transposed): matrix mi = (token half mi&1, n-tile mi>>1) of a pair of n-tiles
  const int v_row = ((mi & 1) << 3) + (lane & 7);

  const float scale = 1.4426950408889634f / sqrtf((float)D);
  float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;
  float o[NT][4];
#pragma unroll
  for (int t = 0; t < NT; ++t) o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f;

  if (ntl > 0) load_tile(0, t0);
  cp_commit();
  for (int it = 0; it < ntl; ++it) {
    if (it + 1 < ntl) load_tile((it + 1) & 1, t0 + (it + 1) * kVTile);
    cp_commit();
    cp_wait<1>();
    __syncthreads();
    const uint32_t kt = sbase + (it & 1) * 2 * kTileBytes, vt = kt + kTileBytes;
    const int nvalid = min(kVTile, t1 - (t0 + it * kVTile));
    // S = Q K^T for the 64 tokens of the tile
    float s[8][4];
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) s[nb][0] = s[nb][1] = s[nb][2] = s[nb][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
      for (int nbp = 0; nbp < 4; ++nbp) {
        const int r = 16 * nbp + k_row, ck = 2 * ks + (mi & 1);
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4(kt + r * ROWB + ((ck ^ (r & 7)) << 4), b0, b1, b2, b3);
        mma16816(s[2 * nbp], qa[ks], b0, b1);
        mma16816(s[2 * nbp + 1], qa[ks], b2, b3);
      }
    }
    // logits in the exp2 domain, masked past the range; row maxima
    float mxA = -INFINITY, mxB = -INFINITY;
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
      const int c = 8 * nb + 2 * qd;
      s[nb][0] = c < nvalid ? s[nb][0] * scale : -INFINITY;
      s[nb][1] = c + 1 < nvalid ? s[nb][1] * scale : -INFINITY;
      s[nb][2] = c < nvalid ? s[nb][2] * scale : -INFINITY;
      s[nb][3] = c + 1 < nvalid ? s[nb][3] * scale : -INFINITY;
      mxA = fmaxf(mxA, fmaxf(s[nb][0], s[nb][1]));
      mxB = fmaxf(mxB, fmaxf(s[nb][2], s[nb][3]));
    }
    mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, 1));
    mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, 2));
    mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, 1));
    mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, 2));
    const float nA = fmaxf(mA, mxA), nB = fmaxf(mB, mxB);     // finite: a tile holds at least one token
    const float cA = ex2(mA - nA), cB = ex2(mB - nB);
    mA = nA; mB = nB;
    lA *= cA; lB *= cB;
#pragma unroll
    for (int t = 0; t < NT; ++t) { o[t][0] *= cA; o[t][1] *= cA; o[t][2] *= cB; o[t][3] *= cB; }
    // O += P V, 16 tokens at a time; P as hi + lo
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t ahi[4], alo[4];
      split_pair(ex2(s[2 * j][0] - mA), ex2(s[2 * j][1] - mA), ahi[0], alo[0], lA);
      split_pair(ex2(s[2 * j][2] - mB), ex2(s[2 * j][3] - mB), ahi[1], alo[1], lB);
      split_pair(ex2(s[2 * j + 1][0] - mA), ex2(s[2 * j + 1][1] - mA), ahi[2], alo[2], lA);
      split_pair(ex2(s[2 * j + 1][2] - mB), ex2(s[2 * j + 1][3] - mB), ahi[3], alo[3], lB);
#pragma unroll
      for (int np = 0; np < NT / 2; ++np) {
        const int r = 16 * j + v_row, ck = 2 * np + (mi >> 1);
        uint32_t v0, v1, v2, v3;
        ldmatrix_x4_trans(vt + r * ROWB + ((ck ^ (r & 7)) << 4), v0, v1, v2, v3);
        mma16816(o[2 * np], ahi, v0, v1);
        mma16816(o[2 * np], alo, v0, v1);
        mma16816(o[2 * np + 1], ahi, v2, v3);
        mma16816(o[2 * np + 1], alo, v2, v3);
      }
    }
    __syncthreads();      // everyone is done with this stage before it is refilled
  }
  cp_wait<0>();

  // ---- partial state of this CTA's rows
  lA += __shfl_xor_sync(0xffffffffu, lA, 1);
  lA += __shfl_xor_sync(0xffffffffu, lA, 2);
  lB += __shfl_xor_sync(0xffffffffu, lB, 1);
  lB += __shfl_xor_sync(0xffffffffu, lB, 2);
  const size_t rec_floats = (size_t)p.MB * (2 + D);
  {
    float* rec = p.partials + ((size_t)(ucall * p.nrb + rb) * p.nsplit + split) * rec_floats;
    const int la = warp * 16 + frow, lb = la + 8;
    if (qd == 0) { rec[la] = mA; rec[lb] = mB; rec[p.MB + la] = lA; rec[p.MB + lb] = lB; }
    float* oa = rec + 2 * p.MB + (size_t)la * D + 2 * qd;
    float* ob = rec + 2 * p.MB + (size_t)lb * D + 2 * qd;
#pragma unroll
    for (int t = 0; t < NT; ++t) {
      *(float2*)(oa + 8 * t) = make_float2(o[t][0], o[t][1]);
      *(float2*)(ob + 8 * t) = make_float2(o[t][2], o[t][3]);
    }
  }
  __shared__ int s_last;
  finish_unit<D>(p, smem, &s_last, ucall, b, l, h);
}

// ---------------------------------------------------------------------------------------------
// The same computation on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor
// memory), for D = 128 and blocks of 128 query rows.  A CTA of 128 threads owns (token split, row
// block, unit); thread t owns query row t = tensor-memory lane t.
//   per tile of 64 tokens:   S = Q K^T      one thread issues 8 MMAs (M128 N64 K16), S in TMEM columns [0, 64) or [64, 128)
//                            softmax        every thread reads its row of S and writes P = hi + lo (bf16) back over it
//                            O += P V       one thread issues 4 + 4 MMAs (M128 N128 K16, A = P from tensor memory), O in columns [128, 256)
// Q, K and V sit in shared memory in the canonical 128-byte-swizzled layouts (rows of 128 bytes, 16-byte
// chunk index XOR row%8, 1024-byte groups of 8 rows): Q and K K-major, V MN-major -- which is exactly
// V's natural [token][channel] order, so no transpose is needed.  The running maximum is only raised when it
// grows by more than 8 (in the exp2 domain): O in tensor memory is then rescaled, otherwise the stale
// maximum stays and numerator and denominator simply carry the same bounded factor.
// K(t+1) is fetched during the softmax of tile t and its first product is issued right behind the second
// product of tile t (into the other S buffer); V(t+1) is fetched during the softmax of tile t+1; two CTAs
// per SM overlap the rest.  Every wait on an mbarrier is bounded: on a
// time-out the CTA raises the error word, releases its tensor memory and leaves without a ticket.
// ---------------------------------------------------------------------------------------------
constexpr int kTcThreads = 128;
constexpr int kTcQ = 0, kTcK = 32768, kTcV = 49152, kTcBytes = 65536;   // Q | K tile | V tile
constexpr int kTcCols = 256;              // allocated tensor-memory columns (power of two): 2 x S 64 + O 128
constexpr uint32_t kTcColS1 = 64, kTcColO = 128;   // S buffers at columns 0 and 64, O at 128
// instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128; N and the majorness of B differ
constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescPV = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

// shared-memory matrix descriptor, 128-byte swizzle: address, leading and stride byte offsets in 16-byte units
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr >> 4) & 0x3fffu) | ((uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t"
      ".reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t"
      "}\n"
      :: "r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
// the same with the A operand in tensor memory (row = lane, K elements packed two per 32-bit column)
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t"
      ".reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t"
      "}\n"
      :: "r"(tmem_d), "r"(tmem_a), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t"
      ".reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t"
      "}\n"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// bounded wait (about a second): false on time-out
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try(bar, parity))
    if (clock64() - t0 > 2000000000LL) return false;
  return true;
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};\n"
      :: "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
         "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
         "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
         "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]),
         "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__global__ void __launch_bounds__(kTcThreads, 2) k_score_value_tc(const ValueScoreParams p) {
  constexpr int D = 128;
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t s_bar[2];
  __shared__ uint32_t s_tmem;
  const uint32_t sraw = smem_u32(smem_raw), sb = (sraw + 1023u) & ~1023u;   // swizzle atoms want 1024-byte alignment
  unsigned char* smem = smem_raw + (sb - sraw);
  const int tid = threadIdx.x, warp = tid >> 5;
  const int split = blockIdx.x, rb = blockIdx.y, ucall = blockIdx.z;
  const int h = ucall % p.N_kv, bl = ucall / p.N_kv;
  const int ll = bl % p.nlayers, b = bl / p.nlayers, l = p.layer0 + ll;
  const int S_b = p.seq_len[b];
  const int ntile_all = (S_b + kVTile - 1) / kVTile;
  const int per = (ntile_all + p.nsplit - 1) / p.nsplit;
  const int t0 = min(S_b, split * per * kVTile), t1 = min(S_b, (split + 1) * per * kVTile);
  const int ntl = (t1 - t0 + kVTile - 1) / kVTile;
  const uint32_t bar_s = smem_u32(&s_bar[0]), bar_o = smem_u32(&s_bar[1]);

  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&s_tmem)), "r"(kTcCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(bar_s) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(bar_o) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }

  // byte offset of 16-byte chunk ck (0..15) of row r inside an operand made of two 64-element blocks
  auto swz = [](int r, int ck, int block_bytes) -> uint32_t {
    return (uint32_t)((ck >> 3) * block_bytes + (r >> 3) * 1024 + (r & 7) * 128 + (((ck & 7) ^ (r & 7)) << 4));
  };
  {
    // query row of this thread: row r of the unit = query head h*G + r / S_obs, window row r % S_obs
    const int r = rb * p.MB + tid;
    const bool ok = r < p.M;
    const __nv_bfloat16* q = (const __nv_bfloat16*)p.q.ptr + b * p.q.sb + (int64_t)l * p.q.sl +
                             (int64_t)(ok ? r % p.S_obs : 0) * p.q.ss + (int64_t)(h * p.G + (ok ? r / p.S_obs : 0)) * p.q.sn;
#pragma unroll
    for (int ck = 0; ck < 16; ++ck) cp_async16_zfill(sb + kTcQ + swz(tid, ck, 16384), q + ck * 8, ok ? 16 : 0);
    cp_commit();
  }
  const __nv_bfloat16* kg = (const __nv_bfloat16*)p.k.ptr + b * p.k.sb + (int64_t)l * p.k.sl + (int64_t)h * p.k.sn;
  const __nv_bfloat16* vg = (const __nv_bfloat16*)p.v.ptr + b * p.v.sb + (int64_t)l * p.v.sl + (int64_t)h * p.v.sn;
  auto load_tile = [&](uint32_t dst, const __nv_bfloat16* g, int64_t stride, int tok0) {
#pragma unroll
    for (int i = 0; i < kVTile * 16 / kTcThreads; ++i) {
      const int idx = tid + i * kTcThreads, r = idx >> 4, ck = idx & 15;
      const bool ok = tok0 + r < t1;               // rows past the range are zero-filled
      cp_async16_zfill(dst + swz(r, ck, 8192), g + (int64_t)(ok ? tok0 + r : t0) * stride + ck * 8, ok ? 16 : 0);
    }
  };
  if (ntl > 0) load_tile(sb + kTcK, kg, p.k.ss, t0);
  cp_commit();
  if (ntl > 0) load_tile(sb + kTcV, vg, p.v.ss, t0);
  cp_commit();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  const uint32_t tlane = tmem + ((uint32_t)(warp * 32) << 16);     // this warp's 32 lanes

  const float scale = 1.4426950408889634f / sqrtf((float)D);
  float m_used = -INFINITY, lsum = 0.f;
  bool ok_all = true;
  // operand descriptors are built once: inside the loops a k-step only adds a constant to the address field
  // (16-byte units)
  const uint64_t dQ = umma_desc(sb + kTcQ, 16, 1024), dK = umma_desc(sb + kTcK, 16, 1024), dV = umma_desc(sb + kTcV, 8192, 1024);
  // first product of tile `t` into S buffer t & 1 (issued by one thread)
  auto issue_qk = [&](int t) {
#pragma unroll
    for (int ks = 0; ks < 8; ++ks)
      umma_bf16(tmem + (uint32_t)(t & 1) * kTcColS1, dQ + (uint64_t)((ks >> 2) * 1024 + (ks & 3) * 2),
                dK + (uint64_t)((ks >> 2) * 512 + (ks & 3) * 2), kIdescQK, ks > 0);
    umma_commit(bar_s);
  };
  if (ntl > 0) {
    cp_wait<1>();                 // Q and K(0) have landed; V(0) may still be in flight
    fence_proxy_async();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      issue_qk(0);
    }
  }
  for (int it = 0; it < ntl; ++it) {
    if (!__syncthreads_and(mbar_wait(bar_s, it & 1))) { ok_all = false; break; }
    tc_fence_after();
    if (it + 1 < ntl) load_tile(sb + kTcK, kg, p.k.ss, t0 + (it + 1) * kVTile);   // the key buffer is free again
    cp_commit();

    // ---- this thread's row of S: logits in the exp2 domain, masked past the range
    uint32_t sr[2][32];
    const uint32_t tS = tlane + (uint32_t)(it & 1) * kTcColS1;
    tmem_ld32(tS, sr[0]);
    tmem_ld32(tS + 32, sr[1]);
    tmem_wait_ld();
    const int nvalid = min(kVTile, t1 - (t0 + it * kVTile));
    if (nvalid < kVTile) {        // last tile of the range: tokens past it get weight zero
#pragma unroll
      for (int j = 0; j < 64; ++j)
        if (j >= nvalid) sr[j >> 5][j & 31] = 0xff800000u;   // -inf
    }
    float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
    for (int j = 0; j < 64; j += 4) {
      mx0 = fmaxf(mx0, __uint_as_float(sr[j >> 5][j & 31]));
      mx1 = fmaxf(mx1, __uint_as_float(sr[(j + 1) >> 5][(j + 1) & 31]));
      mx2 = fmaxf(mx2, __uint_as_float(sr[(j + 2) >> 5][(j + 2) & 31]));
      mx3 = fmaxf(mx3, __uint_as_float(sr[(j + 3) >> 5][(j + 3) & 31]));
    }
    const float m_new = fmaxf(m_used, fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * scale);   // scale > 0
    if (__any_sync(0xffffffffu, m_new > m_used + 8.f)) {
      // raise the maximum: rescale the denominator and this thread's row of O in tensor memory
      const float factor = ex2(m_used - m_new);
      if (it > 0) {
#pragma unroll 1
        for (int c0 = 0; c0 < D; c0 += 32) {
          uint32_t o[32];
          tmem_ld32(tlane + kTcColO + c0, o);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * factor);
          tmem_st32(tlane + kTcColO + c0, o);
        }
        tmem_wait_st();
      }
      lsum *= factor;
      m_used = m_new;
    }
    // ---- P = hi + lo goes back into tensor memory, over the S columns it was computed from: as the A operand
    // of the second product it is read from there (a row per lane, two bf16 per 32-bit column), so the weights
    // never pass through shared memory and the MMA reads only V from it
    const float neg_m = -m_used;
    float ls[4] = {0.f, 0.f, 0.f, 0.f};
    uint32_t hi[32], lo[32];
#pragma unroll
    for (int e = 0; e < 32; ++e) {
      const int j = 2 * e;
      const float p0 = ex2(fmaf(__uint_as_float(sr[j >> 5][j & 31]), scale, neg_m));
      const float p1 = ex2(fmaf(__uint_as_float(sr[(j + 1) >> 5][(j + 1) & 31]), scale, neg_m));
      ls[e & 3] += p0 + p1;        // the denominator takes the weights before the hi + lo split (2^-17 apart)
      split_pair_packed(p0, p1, hi[e], lo[e]);
    }
    tmem_st32(tS, hi);             // columns [0, 32) of this S buffer: P hi, tokens 2c, 2c + 1 in column c
    tmem_st32(tS + 32, lo);        // columns [32, 64): P lo
    tmem_wait_st();
    lsum += (ls[0] + ls[1]) + (ls[2] + ls[3]);
    cp_wait<0>();                 // V(it) and K(it + 1) have landed
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      const uint32_t tP = tmem + (uint32_t)(it & 1) * kTcColS1;      // 16 tokens = 8 columns per MMA
#pragma unroll
      for (int ks = 0; ks < 4; ++ks)
        umma_bf16_ts(tmem + kTcColO, tP + ks * 8, dV + (uint64_t)(ks * 128), kIdescPV, (it > 0 || ks > 0) ? 1u : 0u);
#pragma unroll
      for (int ks = 0; ks < 4; ++ks)
        umma_bf16_ts(tmem + kTcColO, tP + 32 + ks * 8, dV + (uint64_t)(ks * 128), kIdescPV, 1u);
      umma_commit(bar_o);
      // the next tile's first product goes to the other S buffer right behind it: its round trip hides
      // behind this tile's second product instead of adding to it
      if (it + 1 < ntl) issue_qk(it + 1);
    }
    if (!__syncthreads_and(mbar_wait(bar_o, it & 1))) { ok_all = false; break; }
    tc_fence_after();
    if (it + 1 < ntl) load_tile(sb + kTcV, vg, p.v.ss, t0 + (it + 1) * kVTile);   // the value buffer is free again
    cp_commit();
  }
  cp_wait<0>();

  // ---- partial state of this thread's row: (stale maximum, denominator, O row), same record as the other kernel
  if (ok_all) {
    const size_t rec_floats = (size_t)p.MB * (2 + D);
    float* rec = p.partials + ((size_t)(ucall * p.nrb + rb) * p.nsplit + split) * rec_floats;
    rec[tid] = m_used;
    rec[p.MB + tid] = lsum;
    float4* orow = (float4*)(rec + 2 * p.MB + (size_t)tid * D);
#pragma unroll 1
    for (int c0 = 0; c0 < D; c0 += 32) {
      uint32_t o[32];
      if (ntl > 0) {
        tmem_ld32(tlane + kTcColO + c0, o);
        tmem_wait_ld();
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) o[j] = 0u;
      }
#pragma unroll
      for (int j = 0; j < 8; ++j)
        orow[c0 / 4 + j] = make_float4(__uint_as_float(o[4 * j]), __uint_as_float(o[4 * j + 1]), __uint_as_float(o[4 * j + 2]),
                                       __uint_as_float(o[4 * j + 3]));
    }
  } else if (tid == 0 && p.error) {
    atomicOr(p.error, kErrWaitTimeout);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(kTcCols) : "memory");
  if (!ok_all) return;
  __shared__ int s_last_tc;
  finish_unit<D>(p, smem, &s_last_tc, ucall, b, l, h);
}

constexpr int smem_bytes(int D) { return kVStages * 2 * kVTile * D * 2; }

}  // namespace

size_t score_value_record_bytes(int MB, int D) { return (size_t)MB * (2 + D) * sizeof(float); }

cudaError_t score_value_setup(int D) {
  if (D == 128) {
    cudaError_t e = cudaFuncSetAttribute(k_score_value_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcBytes + 1024);
    if (e != cudaSuccess) return e;
  }
  if (D == 128) return cudaFuncSetAttribute(k_score_value<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(128));
  if (D == 64) return cudaFuncSetAttribute(k_score_value<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(64));
  return cudaErrorInvalidValue;
}

// threads = 32 * (MB / 16): one warp per 16 query rows of the row block
cudaError_t launch_score_value(const ValueScoreParams& p, int threads, cudaStream_t s) {
  dim3 grid(p.nsplit, p.nrb, p.B * p.nlayers * p.N_kv);
  if (p.use_tcgen05 && p.D == 128 && p.MB == 128) {
    k_score_value_tc<<<grid, kTcThreads, kTcBytes + 1024, s>>>(p);
    return cudaGetLastError();
  }
  if (p.D == 128) k_score_value<128><<<grid, threads, smem_bytes(128), s>>>(p);
  else if (p.D == 64) k_score_value<64><<<grid, threads, smem_bytes(64), s>>>(p);
  else return cudaErrorInvalidValue;
  return cudaGetLastError();
}

}  // namespace think
