// Key-cache compaction (paper Sec. 3.3): K_T[t][c] = K[t][idx[c]] for the pruned prefix, written
// as 64-token tiles in the layout the decode kernels read (bf16: MMA-fragment order with T padded
// to a multiple of 8 by zero rows; fp32: channel-major [T][64] with XOR-swizzled 16-byte chunks),
// plus the writer of the unpruned tail (recent prompt rows at prefill, the new token at decode).
#include "think_internal.h"

namespace think {
namespace {

// One CTA builds one tile: 64 token rows of one head are staged in shared memory (padded pitch),
// the threads gather the kept channels into the tile image in shared memory, and the finished
// image leaves with coalesced 16-byte stores.
// TOK: rows come from a per-head kept-token list (token-eviction hook) instead of the prompt order.
template <typename Tin, bool TOK>
__global__ void __launch_bounds__(128) k_compact(const CompactParams p) {
  constexpr int E = sizeof(Tin);
  constexpr int CH = 16 / E;             // elements per 16-byte chunk
  extern __shared__ __align__(16) unsigned char smem[];
  const int D = p.D, T = p.T, Tp = p.Tp;
  const int pitch = D * E + 16;          // bytes; odd number of 16-byte chunks per row
  unsigned char* s_in = smem;                                   // [64][pitch]
  unsigned char* s_out = smem + kTileTokens * pitch;            // tile image, Tp*64*E bytes
  uint8_t* s_idx = (uint8_t*)(s_out + Tp * kTileTokens * E);    // [T]

  const int tile = blockIdx.x, h = blockIdx.y;
  const int b = blockIdx.z / p.nlayers, l = p.layer0 + blockIdx.z % p.nlayers;
  const int S_p = p.seq_len[b] - p.R;
  const int ntiles = (S_p + kTileTokens - 1) / kTileTokens;
  if (tile >= ntiles) return;
  const int tok0 = tile * kTileTokens;
  const int nvalid = min(kTileTokens, S_p - tok0);
  const int tid = threadIdx.x;

  const int64_t unit = ((int64_t)b * p.L + l) * p.N_kv + h;
  for (int c = tid; c < T; c += blockDim.x) s_idx[c] = p.idx[unit * T + c];

  const Tin* src = (const Tin*)p.k.ptr + b * p.k.sb + (int64_t)l * p.k.sl + (int64_t)h * p.k.sn;
  const int cpr = D / CH;                // chunks per row
  for (int i = tid; i < kTileTokens * cpr; i += blockDim.x) {
    int r = i / cpr, ck = i % cpr;
    uint4 v = make_uint4(0, 0, 0, 0);    // rows past the prefix become zeros
    if (r < nvalid) {
      const int64_t row = TOK ? token_row(p.tok, unit, tok0 + r) : (int64_t)(tok0 + r);
      v = __ldg((const uint4*)(src + row * p.k.ss + ck * CH));
    }
    *(uint4*)(s_in + r * pitch + ck * 16) = v;
  }
  __syncthreads();

  {
    // item (j, c): tokens [j*CH, (j+1)*CH) of kept channel c; consecutive lanes take consecutive c
    const int nj = kTileTokens / CH;
    for (int item = tid; item < nj * T; item += blockDim.x) {
      int j = item / T, c = item % T;
      int ch = s_idx[c];
      __align__(16) Tin tmp[CH];
#pragma unroll
      for (int i = 0; i < CH; ++i) tmp[i] = *(const Tin*)(s_in + (j * CH + i) * pitch + ch * E);
      *(uint4*)(s_out + c * kTileTokens * E + ((j ^ (c & 7)) << 4)) = *(const uint4*)tmp;
    }
  }
  __syncthreads();

  const int64_t gtile = p.thin_tile_base[b] + (int64_t)(l * p.N_kv + h) * (ntiles + p.re_cap) + tile;
  uint4* dst = (uint4*)((unsigned char*)p.k_thin + gtile * Tp * kTileTokens * E);
  const int n16 = Tp * kTileTokens * E / 16;
  for (int i = tid; i < n16; i += blockDim.x) dst[i] = ((const uint4*)s_out)[i];
}

// bf16 tiles in MMA-fragment order.  The 64 token rows are staged with cp.async (everything in
// flight at once); then warp w builds the four 16-token steps w of the tile: for each group of 16
// kept channels a lane gathers the eight elements of its 16-byte fragment piece (two tokens x four
// channels) and the warp writes the 512-byte chunk straight to global memory.
template <bool TOK>
__global__ void __launch_bounds__(128) k_compact_bf16(const CompactParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  // Launched as a programmatic dependent of the kernel ahead of it (the score pass): the grid is scheduled
  // while that kernel drains, waits here for its results, and only then lets its own dependent (the tail
  // seed, which reads nothing this kernel writes) go.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int D = p.D, T = p.T, Tp = p.Tp;
  const int pitch = D * 2 + 16;
  unsigned char* s_in = smem;                                   // [64][pitch]
  uint16_t* s_off = (uint16_t*)(smem + kTileTokens * pitch);    // [Tp]: byte offset of kept channel c inside a staged row;
                                                                // padding channels point at the 16 zero bytes behind the row
  // Which CTAs run side by side.  heads_first: the same 64 tokens of neighbouring heads and layers -- in the
  // paper's B x S x L x N x D layout those rows are one contiguous stretch (L*N*D elements per token), which
  // pays when that stretch is short (grouped-query shapes).  Otherwise: consecutive tiles of one head, whose
  // thinned tiles are contiguous in k_thin, which pays when a token's keys span many heads (MHA).
  int tile_i, h, l;
  if (p.heads_first) {
    h = blockIdx.x % p.N_kv;
    l = p.layer0 + blockIdx.x / p.N_kv;
    tile_i = blockIdx.y;
  } else {
    tile_i = blockIdx.x % p.max_tiles;
    h = blockIdx.x / p.max_tiles;
    l = p.layer0 + blockIdx.y;
  }
  const int b = blockIdx.z;
  const int S_p = p.seq_len[b] - p.R;
  const int ntiles = (S_p + kTileTokens - 1) / kTileTokens;
  if (tile_i >= ntiles) return;
  const int tile = tile_i;
  const int tok0 = tile * kTileTokens;
  const int nvalid = min(kTileTokens, S_p - tok0);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  const int64_t unit = ((int64_t)b * p.L + l) * p.N_kv + h;
  for (int c = tid; c < Tp; c += 128) s_off[c] = (uint16_t)(c < T ? 2 * p.idx[unit * T + c] : 2 * D);
  const __nv_bfloat16* src = (const __nv_bfloat16*)p.k.ptr + b * p.k.sb + (int64_t)l * p.k.sl + (int64_t)h * p.k.sn;
  // The tile's rows arrive by bulk copies: one instruction per 2 * D-byte row (threads 0..nvalid-1 issue one each),
  // all completing on one mbarrier; rows past the prefix are zeroed with plain stores.
  __shared__ __align__(8) uint64_t s_bar;
  const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&s_bar);
  const uint32_t s_in_addr = (uint32_t)__cvta_generic_to_shared(s_in);
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < kTileTokens) *(uint4*)(s_in + tid * pitch + 2 * D) = make_uint4(0, 0, 0, 0);
  for (int i = tid; i < (kTileTokens - nvalid) * (D / 8); i += 128)
    *(uint4*)(s_in + (nvalid + i / (D / 8)) * pitch + (i % (D / 8)) * 16) = make_uint4(0, 0, 0, 0);
  __syncthreads();
  if (tid == 0) asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(nvalid * D * 2) : "memory");
  if (tid < nvalid) {
    const int64_t row = TOK ? token_row(p.tok, unit, tok0 + tid) : (int64_t)(tok0 + tid);
    const void* g = src + row * p.k.ss;
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(s_in_addr + tid * pitch), "l"(g), "r"(D * 2), "r"(bar) : "memory");
  }
  {
    // bounded wait (about a second at most): on expiry the error word is raised and the tile is left unwritten
    uint32_t done = 0;
    const long long t_start = clock64();
    while (!done) {
      asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                   : "=r"(done) : "r"(bar) : "memory");
      if (!done && clock64() - t_start > 2000000000LL) break;
    }
    if (!done) {
      if (tid == 0 && p.error) atomicOr(p.error, kErrWaitTimeout);
      return;
    }
  }

  const int64_t gtile = p.thin_tile_base[b] + (int64_t)(l * p.N_kv + h) * (ntiles + p.re_cap) + tile;
  unsigned char* dst = (unsigned char*)p.k_thin + gtile * Tp * 128 + warp * (Tp * 32);   // step = warp
  // a lane's four source channels of a group come as two 32-bit loads of byte offsets (pairs are neighbours in s_off)
  const int r = lane >> 2, q = lane & 3;
  const unsigned char* rowA = s_in + (warp * 16 + r) * pitch;
  const unsigned char* rowB = rowA + 8 * pitch;
  auto pair = [](const unsigned char* row, uint32_t oo) -> uint32_t {      // elements at byte offsets oo & 0xffff, oo >> 16
    return (uint32_t)*(const uint16_t*)(row + (oo & 0xffffu)) | ((uint32_t)*(const uint16_t*)(row + (oo >> 16)) << 16);
  };
  const int n16 = Tp >> 4;
  for (int s = 0; s < n16; ++s) {
    const uint32_t o01 = *(const uint32_t*)(s_off + 16 * s + 2 * q), o89 = *(const uint32_t*)(s_off + 16 * s + 2 * q + 8);
    uint4 v;
    v.x = pair(rowA, o01);
    v.y = pair(rowA, o89);
    v.z = pair(rowB, o01);
    v.w = pair(rowB, o89);
    *(uint4*)(dst + s * 512 + lane * 16) = v;
  }
  if (Tp & 8) {
    const uint32_t o01 = *(const uint32_t*)(s_off + 16 * n16 + 2 * q);
    uint2 v;
    v.x = pair(rowA, o01);
    v.y = pair(rowB, o01);
    *(uint2*)(dst + n16 * 512 + lane * 8) = v;
  }
}

// Re-pruning of tail blocks (paper App. C.1: once enough new keys have gathered they are pruned and
// joined to the pruned part).  One CTA turns one full 64-token tile of the unpruned tail ([D] channels,
// fragment order) into a thinned tile (the kept channels of idx, fragment order); warp w builds step w.
__global__ void __launch_bounds__(128) k_reprune_bf16(const RepruneParams p) {
  const int jt = p.blk0 + blockIdx.x, h = blockIdx.y;
  const int b = blockIdx.z / p.nlayers, l = p.layer0 + blockIdx.z % p.nlayers;
  const int lane = threadIdx.x & 31, step = threadIdx.x >> 5;
  const int D = p.D, T = p.T, Tp = p.Tp;
  const int64_t unit = ((int64_t)b * p.L + l) * p.N_kv + h;
  const int nthin = p.cum_thin[b + 1] - p.cum_thin[b];
  const unsigned char* src = (const unsigned char*)p.tail_k + (unit * p.tail_tiles_cap + jt) * (int64_t)D * 128;
  unsigned char* dst = (unsigned char*)p.k_thin +
                       (p.thin_tile_base[b] + (int64_t)(l * p.N_kv + h) * (nthin + p.re_cap) + nthin + jt) * (int64_t)Tp * 128 +
                       step * (Tp * 32);
  const uint8_t* ix = p.idx + unit * T;
  const int r = lane >> 2, q = lane & 3;
  const int uA = step * 16 + r, uB = uA + 8;
  auto elem = [&](int u, int c) -> uint32_t {       // kept channel c of token u; channels >= T are padding
    return c < T ? (uint32_t)*(const uint16_t*)(src + frag_elem_byte(D, ix[c], u)) : 0u;
  };
  const int n16 = Tp >> 4;
  for (int g = 0; g < n16; ++g) {
    const int c = 16 * g + 2 * q;
    uint4 v;
    v.x = elem(uA, c) | (elem(uA, c + 1) << 16);
    v.y = elem(uA, c + 8) | (elem(uA, c + 9) << 16);
    v.z = elem(uB, c) | (elem(uB, c + 1) << 16);
    v.w = elem(uB, c + 8) | (elem(uB, c + 9) << 16);
    *(uint4*)(dst + g * 512 + lane * 16) = v;
  }
  if (Tp & 8) {
    const int c = 16 * n16 + 2 * q;
    uint2 v;
    v.x = elem(uA, c) | (elem(uA, c + 1) << 16);
    v.y = elem(uB, c) | (elem(uB, c + 1) << 16);
    *(uint2*)(dst + n16 * 512 + lane * 8) = v;
  }
}

// Rows of unpruned keys and their values into the tail.  One thread moves one 16-byte chunk of
// one row: the value chunk is copied as is, the key chunk is scattered into the channel-major tile.
template <typename Tin>
__global__ void __launch_bounds__(256) k_tail_write(const TailWriteParams p) {
  // a kernel launched behind this one as a programmatic dependent may start now (it synchronises on this
  // grid's completion itself before it reads what is written here); without such a launch this is a no-op
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  constexpr int E = sizeof(Tin);
  constexpr int CH = 16 / E;
  const int cpr = p.D / CH;
  const int64_t total = (int64_t)p.B * p.nlayers * p.N_kv * p.nrows * cpr;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    int ck = i % cpr;
    int64_t r1 = i / cpr;
    int r = r1 % p.nrows; r1 /= p.nrows;
    int h = r1 % p.N_kv; r1 /= p.N_kv;
    int ll = r1 % p.nlayers;
    int b = r1 / p.nlayers;
    int l = p.layer0 + ll;
    const int64_t unit = ((int64_t)b * p.L + l) * p.N_kv + h;
    int64_t srow = p.rows_from_seq_len ? token_row(p.tok, unit, p.seq_len[b] - p.R + r) : r;
    int sl = l - p.src_layer_base;
    const Tin* ks = (const Tin*)p.k.ptr + b * p.k.sb + srow * p.k.ss + (int64_t)sl * p.k.sl + (int64_t)h * p.k.sn + ck * CH;
    const Tin* vs = (const Tin*)p.v.ptr + b * p.v.sb + srow * p.v.ss + (int64_t)sl * p.v.sl + (int64_t)h * p.v.sn + ck * CH;
    uint4 kv = __ldg((const uint4*)ks);
    uint4 vv;
    if (p.perm_v) {                                 // channel c of the stored row = channel perm_v[c] of the source
      const uint8_t* pm = p.perm_v + unit * p.D + ck * CH;
      Tin* e = (Tin*)&vv;
#pragma unroll
      for (int j = 0; j < CH; ++j) e[j] = vs[(int)pm[j] - ck * CH];
    } else {
      vv = __ldg((const uint4*)vs);
    }
    const int u = p.pos0 + r;                       // position in the tail
    *(uint4*)((Tin*)p.tail_v + (unit * p.cap + u) * p.D + ck * CH) = vv;
    unsigned char* tile = (unsigned char*)p.tail_k + (unit * p.tail_tiles_cap + u / kTileTokens) * (int64_t)p.D * kTileTokens * E;
    const Tin* kk = (const Tin*)&kv;
    const int uu = u % kTileTokens;
    if (E == 2) {
      // channels 2q, 2q + 1 of a token are neighbours in the fragment order: one 4-byte store per pair
      const uint32_t* kw = (const uint32_t*)&kv;
#pragma unroll
      for (int q = 0; q < 4; ++q) *(uint32_t*)(tile + frag_elem_byte(p.D, ck * 8 + 2 * q, uu)) = kw[q];
    } else {
#pragma unroll
      for (int j = 0; j < CH; ++j) {
        int c = ck * CH + j;
        *(Tin*)(tile + c * kTileTokens * E + tile_swz_bytes(c, uu, E)) = kk[j];
      }
    }
  }
  // When this grid was launched as a programmatic dependent (the tail seed beside the compaction kernel) it must
  // not complete before the grid ahead of it: the next kernel in the stream waits for THIS grid only.  Without
  // such a launch the instruction returns at once.
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Seed of the unpruned tail at prefill (paper Sec. 3.3: the most recent prompt tokens keep every channel), bf16,
// prompt order, values stored as they are.  One CTA moves up to 64 recent rows of one head: the key rows are staged
// in shared memory and leave as whole 16-token steps of the fragment-order tail tile -- a lane builds one 16-byte
// piece, a warp writes 512 contiguous bytes -- instead of one scattered 4-byte store per channel pair; the value
// rows are copied 16 bytes per thread.  Rows of the last step beyond S_recent are written as zeros (the appends
// that follow overwrite them one token at a time).
__global__ void __launch_bounds__(128) k_tail_seed_bf16(const TailWriteParams p) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  extern __shared__ __align__(16) unsigned char smem[];
  const int D = p.D, pitch = D * 2 + 16, cpr = D / 8;
  const int chunk = blockIdx.x, h = blockIdx.y;
  const int b = blockIdx.z / p.nlayers, l = p.layer0 + blockIdx.z % p.nlayers;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t unit = ((int64_t)b * p.L + l) * p.N_kv + h;
  const int row0 = chunk * kTileTokens;                       // first tail position of this CTA
  const int nrows = min(kTileTokens, p.R - row0);
  const int64_t srow0 = (int64_t)p.seq_len[b] - p.R + row0;   // its source row
  const __nv_bfloat16* ks = (const __nv_bfloat16*)p.k.ptr + b * p.k.sb + (int64_t)l * p.k.sl + (int64_t)h * p.k.sn;
  const __nv_bfloat16* vs = (const __nv_bfloat16*)p.v.ptr + b * p.v.sb + (int64_t)l * p.v.sl + (int64_t)h * p.v.sn;
  const uint32_t s_addr = (uint32_t)__cvta_generic_to_shared(smem);
  const int nsteps = (nrows + 15) >> 4;
  for (int i = tid; i < nsteps * 16 * cpr; i += 128) {
    const int r = i / cpr, ck = i % cpr;
    const bool ok = r < nrows;
    const void* g = ks + (srow0 + (ok ? r : 0)) * p.k.ss + ck * 8;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(s_addr + r * pitch + ck * 16), "l"(g), "r"(ok ? 16 : 0) : "memory");
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
  for (int i = tid; i < nrows * cpr; i += 128) {
    const int r = i / cpr, ck = i % cpr;
    const uint4 v = __ldg((const uint4*)(vs + (srow0 + r) * p.v.ss + ck * 8));
    *(uint4*)((__nv_bfloat16*)p.tail_v + (unit * p.cap + row0 + r) * D + ck * 8) = v;
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();
  unsigned char* tile = (unsigned char*)p.tail_k + (unit * p.tail_tiles_cap + chunk) * (int64_t)D * 128;
  const int r8 = lane >> 2, q = lane & 3, ng = D >> 4;
  for (int item = warp; item < nsteps * ng; item += 4) {
    const int step = item / ng, s = item % ng;
    const unsigned char* rowA = smem + (step * 16 + r8) * pitch + (16 * s + 2 * q) * 2;
    const unsigned char* rowB = rowA + 8 * pitch;
    uint4 v;
    v.x = *(const uint32_t*)rowA;            // channels 16s + 2q, + 1 of token 16 * step + r8
    v.y = *(const uint32_t*)(rowA + 16);     // channels 16s + 2q + 8, + 9
    v.z = *(const uint32_t*)rowB;            // the same of token + 8
    v.w = *(const uint32_t*)(rowB + 16);
    *(uint4*)(tile + step * (D * 32) + s * 512 + lane * 16) = v;
  }
  // as in k_tail_write: launched beside the compaction kernel, this grid must not complete before the grid ahead of it
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Value-channel pruning (paper App. D): V_T[t][c] = V[t][perm_v[c]] for c < T_v, rows of Tvp elements
// (zero padded), t < S_p.  A CTA stages 64 value rows of one head in shared memory (cp.async, padded
// pitch); a thread then owns one 16-byte piece of the thinned rows -- its eight source channels stay in
// registers -- and walks down the rows, so consecutive threads write consecutive bytes of v_thin.
__global__ void __launch_bounds__(128) k_compact_value(const CompactValueParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int D = p.D, Tvp = p.Tvp;
  const int pitch = D * 2 + 16;
  const int h = blockIdx.y;
  const int b = blockIdx.z / p.nlayers, l = p.layer0 + blockIdx.z % p.nlayers;
  const int S_p = p.seq_len[b] - p.R;
  const int tok0 = blockIdx.x * kTileTokens;
  if (tok0 >= S_p) return;
  const int nvalid = min(kTileTokens, S_p - tok0);
  const int tid = threadIdx.x;
  const int64_t unit = ((int64_t)b * p.L + l) * p.N_kv + h;
  const __nv_bfloat16* src = (const __nv_bfloat16*)p.v.ptr + b * p.v.sb + (int64_t)l * p.v.sl + (int64_t)h * p.v.sn;
  const int cpr = D / 8;
  const uint32_t s_addr = (uint32_t)__cvta_generic_to_shared(smem);
  for (int i = tid; i < nvalid * cpr; i += 128) {
    const int r = i / cpr, ck = i % cpr;
    const void* g = src + (int64_t)(tok0 + r) * p.v.ss + ck * 8;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s_addr + r * pitch + ck * 16), "l"(g) : "memory");
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
  // this thread's piece and its source channels (byte offsets inside a staged row; 0xffff = padding)
  const int cpo = Tvp / 8;                     // pieces per thinned row
  const int rpp = 128 / cpo;                   // rows per pass
  const int ck = tid % cpo, r0 = tid / cpo;
  uint32_t off[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int c = ck * 8 + j;
    off[j] = c < p.Tv ? 2u * p.perm_v[unit * D + c] : 0xffffu;
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();
  if (r0 >= rpp) return;
  unsigned char* dst = (unsigned char*)p.v_thin +
                       (p.v_thin_base[b] + ((int64_t)(l * p.N_kv + h) * S_p + tok0) * Tvp) * 2 + ck * 16;
  for (int r = r0; r < nvalid; r += rpp) {
    const unsigned char* row = smem + r * pitch;
    uint32_t w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t lo = off[2 * j] == 0xffffu ? 0u : *(const uint16_t*)(row + off[2 * j]);
      const uint32_t hi = off[2 * j + 1] == 0xffffu ? 0u : *(const uint16_t*)(row + off[2 * j + 1]);
      w[j] = lo | (hi << 16);
    }
    *(uint4*)(dst + (int64_t)r * Tvp * 2) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// Values of the kept tokens, gathered into a dense [B, L, N_kv, S_max, D] buffer (token-eviction
// hook: the decode kernels then read the prefix values from that buffer).  One thread moves 16 bytes.
template <int E>
__global__ void __launch_bounds__(256) k_gather_rows(const GatherRowsParams p) {
  const int cpr = p.D * E / 16;
  const int64_t total = (int64_t)p.B * p.nlayers * p.N_kv * p.S_max * cpr;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int ck = i % cpr;
    int64_t r1 = i / cpr;
    const int t = r1 % p.S_max; r1 /= p.S_max;
    const int h = r1 % p.N_kv; r1 /= p.N_kv;
    const int l = p.layer0 + (int)(r1 % p.nlayers);
    const int b = (int)(r1 / p.nlayers);
    if (t >= p.seq_len[b]) continue;
    const int64_t unit = ((int64_t)b * p.L + l) * p.N_kv + h;
    const unsigned char* src = (const unsigned char*)p.v.ptr +
        (b * p.v.sb + token_row(p.tok, unit, t) * p.v.ss + (int64_t)l * p.v.sl + (int64_t)h * p.v.sn) * E + ck * 16;
    *(uint4*)((unsigned char*)p.dst + ((unit * p.S_max + t) * (int64_t)p.D) * E + ck * 16) = __ldg((const uint4*)src);
  }
}

}  // namespace

cudaError_t launch_compact_value(const CompactValueParams& p, cudaStream_t s) {
  const int ntiles = (p.S_pmax + kTileTokens - 1) / kTileTokens;
  if (ntiles <= 0) return cudaSuccess;
  const size_t smem = (size_t)kTileTokens * (p.D * 2 + 16);
  k_compact_value<<<dim3(ntiles, p.N_kv, p.B * p.nlayers), 128, smem, s>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_gather_rows(const GatherRowsParams& p, int dtype, cudaStream_t s) {
  const int E = dtype == THINK_BF16 ? 2 : 4;
  const int64_t total = (int64_t)p.B * p.nlayers * p.N_kv * p.S_max * (p.D * E / 16);
  if (total <= 0) return cudaSuccess;
  int blocks = (int)((total + 255) / 256 < (int64_t)kSMs * 16 ? (total + 255) / 256 : (int64_t)kSMs * 16);
  if (E == 2) k_gather_rows<2><<<blocks, 256, 0, s>>>(p);
  else k_gather_rows<4><<<blocks, 256, 0, s>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_compact(const CompactParams& p_in, int dtype, int max_tiles, cudaStream_t s) {
  if (max_tiles <= 0) return cudaSuccess;
  CompactParams p = p_in;
  p.max_tiles = max_tiles;
  dim3 grid(max_tiles, p.N_kv, p.B * p.nlayers);
  const int E = dtype == THINK_BF16 ? 2 : 4;
  size_t smem = (size_t)kTileTokens * (p.D * E + 16) + (size_t)p.Tp * kTileTokens * E + ((p.T + 15) & ~15);
  cudaError_t e;
  if (dtype == THINK_BF16) {
    smem = (size_t)kTileTokens * (p.D * 2 + 16) + 2 * (size_t)((p.Tp + 15) & ~15);
    cudaLaunchConfig_t cfg = {};
    if (p.B > 65535 || p.nlayers > 65535) return cudaErrorInvalidValue;
    p.heads_first = p.N_kv * p.nlayers <= 256 && max_tiles <= 65535;
    cfg.gridDim = p.heads_first ? dim3(p.N_kv * p.nlayers, max_tiles, p.B) : dim3(p.N_kv * max_tiles, p.nlayers, p.B);
    cfg.blockDim = dim3(128);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return p.tok.rows ? cudaLaunchKernelEx(&cfg, k_compact_bf16<true>, p) : cudaLaunchKernelEx(&cfg, k_compact_bf16<false>, p);
  } else if (p.tok.rows) {
    e = cudaFuncSetAttribute(k_compact<float, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k_compact<float, true><<<grid, 128, smem, s>>>(p);
  } else {
    e = cudaFuncSetAttribute(k_compact<float, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k_compact<float, false><<<grid, 128, smem, s>>>(p);
  }
  return cudaGetLastError();
}

cudaError_t launch_reprune(const RepruneParams& p, cudaStream_t s) {
  if (p.nblk <= 0) return cudaSuccess;
  k_reprune_bf16<<<dim3(p.nblk, p.N_kv, p.B * p.nlayers), 128, 0, s>>>(p);
  return cudaGetLastError();
}

// `overlap_previous`: the kernel ahead in the stream writes nothing this launch reads or writes and has itself
// waited for everything before it (the compaction kernel at prefill), so the two may run side by side.
cudaError_t launch_tail_write(const TailWriteParams& p, int dtype, cudaStream_t s, bool overlap_previous) {
  const int E = dtype == THINK_BF16 ? 2 : 4;
  const int64_t total = (int64_t)p.B * p.nlayers * p.N_kv * p.nrows * (p.D * E / 16);
  if (total <= 0) return cudaSuccess;
  int blocks = (int)((total + 255) / 256);
  if (blocks > kSMs * 16) blocks = kSMs * 16;
  if (dtype == THINK_BF16 && p.rows_from_seq_len && !p.tok.rows && !p.perm_v && p.pos0 == 0 && p.nrows == p.R &&
      p.B * p.nlayers <= 65535 && p.N_kv <= 65535) {
    // the prefill seed in prompt order: whole fragment-order steps per CTA
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((p.R + kTileTokens - 1) / kTileTokens, p.N_kv, p.B * p.nlayers);
    cfg.blockDim = dim3(128);
    cfg.dynamicSmemBytes = (size_t)kTileTokens * (p.D * 2 + 16);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_previous ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, k_tail_seed_bf16, p);
  }
  if (overlap_previous && dtype == THINK_BF16) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks);
    cfg.blockDim = dim3(256);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_tail_write<__nv_bfloat16>, p);
  }
  if (dtype == THINK_BF16) k_tail_write<__nv_bfloat16><<<blocks, 256, 0, s>>>(p);
  else k_tail_write<float><<<blocks, 256, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace think
