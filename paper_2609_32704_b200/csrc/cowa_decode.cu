// Split-KV single-token decode for CoWindow Attention (Sec. 2.3 "Decoding"): the forward
// with N_q = 1, delta = N_k - 1 - i_k, windows recomputed from the current key length of each
// sequence; the visible rows of a head are divided over split programs whose partial
// online-softmax states are merged afterwards.
//
// HBM-bound: every visible K and V row is read exactly once, with 128-bit loads, straight
// into registers.  Per (sequence, KV head, split) one 128-thread block, 5 blocks per SM:
//   1. scores:  each warp takes 16 visible rows at a time; K rows are loaded as the A
//      fragment of mma.sync m16n8k16 (bf16, fp32 accumulate), the group's query vectors are
//      the B fragment.  The contraction index is permuted identically on both operands so
//      that every thread's loads are 16-byte vectors.  Scores (log2 units) go to shared memory.
//   2. block-wide max / exp2 / sum per QO head (no running rescale: the split's scores are
//      all in shared memory before any V row is touched).
//   3. values:  again mma.sync m16n8k16, O^T += V^T P^T with 16 visible rows per instruction; V rows are
//      loaded with 16-byte vectors and neighbouring rows are paired with byte permutes (the d index is
//      permuted inside the fragment and restored on output); the four warps' partial sums meet in shared
//      memory; un-normalised partial (o, m, l) written to the workspace.
// A second kernel merges the splits (log-sum-exp combine with warp shuffles).
#include <cuda_bf16.h>

#include "cowa_common.h"

namespace {

constexpr int kThreads = 128;
constexpr int kChunkCap = 1024;  // max visible rows per split (scores of a split live in shared memory)
constexpr int kScStride = kChunkCap + 8;  // row stride of the score array: heads land in different banks

// Scratch of cowa_decode_static: lives in the library's device image, so every GPU that loads the
// library keeps these bytes reserved until the process exits.
constexpr size_t kStaticScratchBytes = 8u << 20;
static __device__ __align__(256) unsigned char g_decode_static_scratch[kStaticScratchBytes];

// Device address of the scratch array on the current device.  The array's name is only a
// host-side handle here; the address the kernels need comes from cudaGetSymbolAddress, looked
// up once per device with that device current.
void* static_scratch_ptr(cudaError_t* err) {
  static void* cache[64] = {nullptr};
  int dev = 0;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return nullptr;
  if (dev < 0 || dev >= 64) { *err = cudaErrorInvalidDevice; return nullptr; }
  if (!cache[dev]) {
    void* ptr = nullptr;
    *err = cudaGetSymbolAddress(&ptr, g_decode_static_scratch);
    if (*err != cudaSuccess) return nullptr;
    cache[dev] = ptr;
  }
  return cache[dev];
}

struct DecodeArgs {
  const __nv_bfloat16* q;
  const __nv_bfloat16* kc;
  const __nv_bfloat16* vc;
  const int32_t* lens;
  float* ws_o;  // [B, Hq, S, D]
  float* ws_m;  // [B, Hq, S]
  float* ws_l;  // [B, Hq, S]
  int B, Tmax, Hq, Hkv, S;
  CowaStrides sk, sv;  // element strides (batch, head, token) of the contiguous-row cache
  int sink, near, hkv_global, hkv_offset, full_attn;
  float scale_log2;
  // extended kernel only: several newest tokens per sequence and / or a paged cache
  const int32_t* block_table;  // [B, max_pages] page of every page_size-row stretch of a sequence, or nullptr
  int NQ;                      // query tokens per sequence, at key positions lens[b] - NQ .. lens[b] - 1
  int tpg, ngroups;            // tokens per block (columns = tpg * Hq / Hkv <= 8), blocks per (sequence, KV head)
  int page_size, max_pages, page_shift;  // page_shift = log2(page_size) when that is a power of two, else -1
};

// Position of the v-th visible row (v in the concatenation of the head's ranges).
struct VisMap {
  int lo0, n0, lo1, n1, lo2;
  __device__ __forceinline__ int token(int v) const {
    return v < n0 ? lo0 + v : (v < n0 + n1 ? lo1 + (v - n0) : lo2 + (v - n0 - n1));
  }
};

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 ldg128(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

// G = columns of the mma n-tile in use.  Plain kernel (EXT = false): the G query heads of the group, one
// token.  Extended kernel: (token, head) pairs of up to a.tpg of the a.NQ newest tokens, token-major; every
// column masks the keys its own token must not see; rows may come from a paged cache.
template <int D, int G, bool EXT>
// 5 blocks per SM (up to 102 registers, no spills) measured best: fewer, longer splits than at 7 per SM
__global__ void __launch_bounds__(kThreads, 5) cowa_decode_split_kernel(const DecodeArgs a) {
  static_assert(D == 64 || D == 128, "head dim");
  static_assert(G >= 1 && G <= 8, "group size per mma n-tile");
  constexpr int KC = D / 32;          // 32-wide d chunks (two k16 steps each)

  __shared__ __align__(16) float sc[G * kScStride];  // scores, later the value-phase reduction buffer
  __shared__ float m_s[G], l_s[G];

  // The merge kernel is launched with programmatic stream serialisation: once every block of this grid has
  // started, its blocks may be scheduled and wait (griddepcontrol.wait) for this grid's results.
  asm volatile("griddepcontrol.launch_dependents;");
  const int split = blockIdx.x, hk = blockIdx.y;
  const int b = EXT ? blockIdx.z / a.ngroups : blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int Nk = a.lens[b];

  // visible ranges of this head for the current key length
  CowaWin w;
  if (a.full_attn) { w.s = 0; w.n = Nk; w.g = 0; w.l = 0; }
  else w = cowa_default_window(Nk, a.hkv_global, a.hkv_offset + hk, a.sink, a.near);
  CowaRange rg[3];
  // extended: this block's tokens tq0 .. tq1 sit at key positions Nk - NQ + tq
  const int gsz = EXT ? a.Hq / a.Hkv : G;
  const int tq0 = EXT ? (blockIdx.z % a.ngroups) * a.tpg : 0;
  const int tq1 = EXT ? min(tq0 + a.tpg, a.NQ) - 1 : 0;
  const int pos0 = EXT ? Nk - a.NQ : Nk - 1;  // key position of token 0
  const int nr = EXT ? cowa_decode_ranges_span(w, pos0 + tq0, pos0 + tq1, rg) : cowa_decode_ranges(w, Nk, rg);
  // index of column c in q, o, lse and the split states ([B, NQ, Hq] order)
  auto col = [&](int c) -> size_t {
    if constexpr (EXT) return ((size_t)b * a.NQ + tq0 + c / gsz) * a.Hq + (size_t)hk * gsz + c % gsz;
    else return (size_t)b * a.Hq + (size_t)hk * G + c;
  };
  auto col_valid = [&](int c) -> bool { return EXT ? (c < G && tq0 + c / gsz <= tq1) : (c < G); };
  // address of cache row `tok` of this (sequence, KV head)
  auto row_ptr = [&](const __nv_bfloat16* base, const CowaStrides& cs, int tok) -> const __nv_bfloat16* {
    if constexpr (EXT) {
      if (a.block_table) {
        // page sizes are almost always powers of two: shift and mask instead of a runtime division
        const int pi = a.page_shift >= 0 ? tok >> a.page_shift : tok / a.page_size;
        const int po = a.page_shift >= 0 ? tok & (a.page_size - 1) : tok % a.page_size;
        const int pg = a.block_table[(size_t)b * a.max_pages + pi];
        return base + (((size_t)pg * a.Hkv + hk) * a.page_size + po) * D;
      }
    }
    return base + (size_t)b * cs.b + (size_t)hk * cs.h + (size_t)tok * cs.t;
  };
  VisMap vm;
  vm.lo0 = rg[0].lo; vm.n0 = nr > 0 ? rg[0].hi - rg[0].lo + 1 : 0;
  vm.lo1 = nr > 1 ? rg[1].lo : 0; vm.n1 = nr > 1 ? rg[1].hi - rg[1].lo + 1 : 0;
  vm.lo2 = nr > 2 ? rg[2].lo : 0;
  const int n2 = nr > 2 ? rg[2].hi - rg[2].lo + 1 : 0;
  const int V = vm.n0 + vm.n1 + n2;

  int chunk = (V + a.S - 1) / a.S;
  chunk = (chunk + 15) & ~15;
  const int c0 = split * chunk;
  const int clen = min(chunk, V - c0);  // <= kChunkCap by the host's choice of S

  if (clen <= 0) {  // empty split: neutral partial state
    for (int i = tid; i < G * D; i += kThreads)
      if (col_valid(i / D)) a.ws_o[(col(i / D) * a.S + split) * D + (i % D)] = 0.f;
    if (tid < G && col_valid(tid)) {
      a.ws_m[col(tid) * a.S + split] = -INFINITY;
      a.ws_l[col(tid) * a.S + split] = 0.f;
    }
    return;
  }

  // ---------------- phase 1: scores ----------------
  {
    const int g = lane >> 2, t = lane & 3;
    // B fragments: query head g (zero beyond the group), permuted contraction index
    uint32_t bq[KC][4];
#pragma unroll
    for (int cc = 0; cc < KC; ++cc) {
      uint4 x = make_uint4(0, 0, 0, 0);
      if (col_valid(g)) x = *reinterpret_cast<const uint4*>(a.q + col(g) * D + cc * 32 + t * 8);
      bq[cc][0] = x.x; bq[cc][1] = x.y; bq[cc][2] = x.z; bq[cc][3] = x.w;
    }
    const int nblk = (clen + 15) >> 4;
    for (int blk = warp; blk < nblk; blk += kThreads / 32) {
      const int rA = blk * 16 + g, rB = rA + 8;
      const int tokA = vm.token(c0 + min(rA, clen - 1));
      const int tokB = vm.token(c0 + min(rB, clen - 1));
      const __nv_bfloat16* pa = row_ptr(a.kc, a.sk, tokA) + t * 8;
      const __nv_bfloat16* pb = row_ptr(a.kc, a.sk, tokB) + t * 8;
      uint4 ka[KC], kb[KC];
#pragma unroll
      for (int cc = 0; cc < KC; ++cc) { ka[cc] = ldg128(pa + cc * 32); kb[cc] = ldg128(pb + cc * 32); }
      float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int cc = 0; cc < KC; ++cc) {
        mma_bf16_16816(c, ka[cc].x, kb[cc].x, ka[cc].y, kb[cc].y, bq[cc][0], bq[cc][1]);
        mma_bf16_16816(c, ka[cc].z, kb[cc].z, ka[cc].w, kb[cc].w, bq[cc][2], bq[cc][3]);
      }
      // c[0],c[1]: row rA, heads 2t, 2t+1;  c[2],c[3]: row rB
      const int h0 = 2 * t, h1 = 2 * t + 1;
      if constexpr (EXT) {  // a column only sees what its own token sees (Eq. fwa_support at that token's distance)
        const int p0_ = pos0 + tq0 + h0 / gsz, p1_ = pos0 + tq0 + h1 / gsz;
        if (!col_valid(h0) || !cowa_visible(w, p0_ - tokA, tokA)) c[0] = -INFINITY;
        if (!col_valid(h1) || !cowa_visible(w, p1_ - tokA, tokA)) c[1] = -INFINITY;
        if (!col_valid(h0) || !cowa_visible(w, p0_ - tokB, tokB)) c[2] = -INFINITY;
        if (!col_valid(h1) || !cowa_visible(w, p1_ - tokB, tokB)) c[3] = -INFINITY;
      }
      if (rA < clen) {
        if (h0 < G) sc[h0 * kScStride + rA] = c[0] * a.scale_log2;
        if (h1 < G) sc[h1 * kScStride + rA] = c[1] * a.scale_log2;
      }
      if (rB < clen) {
        if (h0 < G) sc[h0 * kScStride + rB] = c[2] * a.scale_log2;
        if (h1 < G) sc[h1 * kScStride + rB] = c[3] * a.scale_log2;
      }
    }
  }
  __syncthreads();

  // ---------------- phase 2: max, exp2, sum per head ----------------
  for (int h = warp; h < G; h += kThreads / 32) {
    float* s = sc + h * kScStride;
    float m = -INFINITY;
    for (int r = lane; r < clen; r += 32) m = fmaxf(m, s[r]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float l = 0.f;
    const float msub = (EXT && m == -INFINITY) ? 0.f : m;  // a token that sees none of this split's rows
    for (int r = lane; r < clen; r += 32) {
      float p = exp2f(s[r] - msub);
      s[r] = p;
      l += p;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    if (lane == 0) { m_s[h] = m; l_s[h] = l; }
  }
  __syncthreads();

  // ---------------- phase 3: values, O^T[d, h] += V^T[d, rows] P^T[rows, h] on the tensor cores ----------------
  // 16 visible rows per mma.  A = V^T: thread (g, t) loads 16 bytes (8 consecutive d) of rows 2t, 2t+1, 2t+8,
  // 2t+9 and pairs equal d of neighbouring rows with byte permutes; the row index of an m-tile is a
  // permutation of d (row g <-> d = 8g + 2i, row g+8 <-> d = 8g + 2i + 1 for m-tile i), undone when the
  // accumulators are written out.  B = P^T (bf16), head g of the group in column g.
  {
    const int g = lane >> 2, t = lane & 3;
    constexpr int NB = D / 64;
    float acc[NB][4][4];
#pragma unroll
    for (int bb = 0; bb < NB; ++bb)
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[bb][i][c] = 0.f;
    const int nblk = (clen + 15) >> 4;
    for (int blk = warp; blk < nblk; blk += kThreads / 32) {
      const int r0 = blk * 16 + 2 * t;
      const int rr[4] = {r0, r0 + 1, r0 + 8, r0 + 9};
      uint4 vv[4][NB];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const __nv_bfloat16* src = row_ptr(a.vc, a.sv, vm.token(c0 + min(rr[k], clen - 1))) + g * 8;
#pragma unroll
        for (int bb = 0; bb < NB; ++bb) vv[k][bb] = ldg128(src + bb * 64);
      }
      float pr[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) pr[k] = (g < G && rr[k] < clen) ? sc[g * kScStride + rr[k]] : 0.f;
      uint32_t b0, b1;
      asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(b0) : "f"(pr[1]), "f"(pr[0]));
      asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(b1) : "f"(pr[3]), "f"(pr[2]));
#pragma unroll
      for (int bb = 0; bb < NB; ++bb) {
        const uint32_t x0[4] = {vv[0][bb].x, vv[0][bb].y, vv[0][bb].z, vv[0][bb].w};
        const uint32_t x1[4] = {vv[1][bb].x, vv[1][bb].y, vv[1][bb].z, vv[1][bb].w};
        const uint32_t x2[4] = {vv[2][bb].x, vv[2][bb].y, vv[2][bb].z, vv[2][bb].w};
        const uint32_t x3[4] = {vv[3][bb].x, vv[3][bb].y, vv[3][bb].z, vv[3][bb].w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
          mma_bf16_16816(acc[bb][i], __byte_perm(x0[i], x1[i], 0x5410), __byte_perm(x0[i], x1[i], 0x7632),
                         __byte_perm(x2[i], x3[i], 0x5410), __byte_perm(x2[i], x3[i], 0x7632), b0, b1);
      }
    }
    __syncthreads();  // scores no longer needed: reuse their space as red[warp][h][d]
    static_assert((kThreads / 32) * D <= kChunkCap, "reduction buffer fits the score buffer");
#pragma unroll
    for (int bb = 0; bb < NB; ++bb)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int d = bb * 64 + 8 * g + 2 * i;
        const int h0 = 2 * t, h1 = 2 * t + 1;
        if (h0 < G) *reinterpret_cast<float2*>(sc + ((size_t)(warp * G + h0) * D + d)) = make_float2(acc[bb][i][0], acc[bb][i][2]);
        if (h1 < G) *reinterpret_cast<float2*>(sc + ((size_t)(warp * G + h1) * D + d)) = make_float2(acc[bb][i][1], acc[bb][i][3]);
      }
  }
  __syncthreads();
  for (int i = tid; i < G * D; i += kThreads) {
    float s = 0.f;
#pragma unroll
    for (int r = 0; r < kThreads / 32; ++r) s += sc[r * G * D + i];
    if (col_valid(i / D)) a.ws_o[(col(i / D) * a.S + split) * D + (i % D)] = s;
  }
  if (tid < G && col_valid(tid)) {
    a.ws_m[col(tid) * a.S + split] = m_s[tid];
    a.ws_l[col(tid) * a.S + split] = l_s[tid];
  }
}

// Merge of the split states: M = max m_s, L = sum l_s 2^(m_s - M), o = sum o_s 2^(m_s - M) / L,
// lse = ln2 * (M + log2 L).  One block of 4 warps per (sequence, QO head): every warp reduces M and L
// with shuffles, takes every fourth split with D/32 columns per lane (several loads in flight), and the
// four partial sums meet in shared memory.
template <int D>
__global__ void __launch_bounds__(128) cowa_decode_combine_kernel(const float* __restrict__ ws_o,
                                                                  const float* __restrict__ ws_m,
                                                                  const float* __restrict__ ws_l,
                                                                  __nv_bfloat16* __restrict__ o,
                                                                  float* __restrict__ lse, int S) {
  constexpr int V = D / 32;  // columns per lane
  __shared__ float part[4][D];
  const size_t bh = blockIdx.x;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the split kernel's states are complete and visible
  const float* m = ws_m + bh * S;
  const float* l = ws_l + bh * S;
  const float* po = ws_o + bh * S * D + lane * V;
  float acc[V];
#pragma unroll
  for (int i = 0; i < V; ++i) acc[i] = 0.f;
  float mx = -INFINITY, L = 0.f;
  constexpr int U = 8;
  if (S <= 32) {
    // one round trip: every load is issued before the first use
    const float ms = lane < S ? m[lane] : -INFINITY;
    const float ls = lane < S ? l[lane] : 0.f;
    float x[U][V];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int s = warp + 4 * u;
#pragma unroll
      for (int i = 0; i < V; ++i) x[u][i] = s < S ? po[(size_t)s * D + i] : 0.f;
    }
    mx = ms;
#pragma unroll
    for (int o_ = 16; o_ > 0; o_ >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o_));
    const float wl = exp2f(ms - mx);  // empty splits: m = -inf -> weight 0
    L = ls * wl;
#pragma unroll
    for (int o_ = 16; o_ > 0; o_ >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o_);
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const float wgt = __shfl_sync(0xffffffffu, wl, (warp + 4 * u) & 31);
#pragma unroll
      for (int i = 0; i < V; ++i) acc[i] = fmaf(x[u][i], wgt, acc[i]);
    }
  } else {
    for (int s = lane; s < S; s += 32) mx = fmaxf(mx, m[s]);
#pragma unroll
    for (int o_ = 16; o_ > 0; o_ >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o_));
    for (int s = lane; s < S; s += 32) L += l[s] * exp2f(m[s] - mx);
#pragma unroll
    for (int o_ = 16; o_ > 0; o_ >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o_);
    for (int s0 = warp; s0 < S; s0 += 4 * U) {
      float x[U][V], wgt[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int s = s0 + 4 * u;
        const bool in = s < S;
        wgt[u] = in ? exp2f(m[s] - mx) : 0.f;
#pragma unroll
        for (int i = 0; i < V; ++i) x[u][i] = in ? po[(size_t)s * D + i] : 0.f;
      }
#pragma unroll
      for (int u = 0; u < U; ++u)
#pragma unroll
        for (int i = 0; i < V; ++i) acc[i] = fmaf(x[u][i], wgt[u], acc[i]);
    }
  }
#pragma unroll
  for (int i = 0; i < V; ++i) part[warp][lane * V + i] = acc[i];
  __syncthreads();
  if (tid < D) {
    const float v = (part[0][tid] + part[1][tid]) + (part[2][tid] + part[3][tid]);
    o[bh * D + tid] = __float2bfloat16_rn(v / L);
  }
  if (lse && tid == 0) lse[bh] = 0.6931471805599453f * (mx + log2f(L));
}

// Upper bound of visible rows per head for any key length <= Tmax.
int max_visible(int Tmax, int hg, const cowa_params_t* p) {
  if (p->full_attn) return Tmax;
  long long shared = (long long)p->sink + p->local;
  if (shared >= Tmax) return Tmax;
  long long band = ((long long)Tmax - shared + hg - 1) / hg;  // widest band, ceil(L / Hk)
  long long v = shared + band;
  return (int)(v < Tmax ? v : Tmax);
}

// Blocks of the split kernel that fit the current device at once (SM count x resident blocks per SM).
// Falls back to 148 x 5 (B200, up to 102 registers per thread) when no device can be queried.
template <int D, int G, bool EXT>
int resident_blocks_of() {
  int dev = 0, sms = 0, occ = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, cowa_decode_split_kernel<D, G, EXT>, kThreads, 0) !=
      cudaSuccess)
    return 0;
  return sms * occ;
}

template <bool EXT>
int resident_blocks(int D, int G) {
  static int cache[2][4] = {{0, 0, 0, 0}, {0, 0, 0, 0}};
  const int di = D == 128 ? 1 : 0, gi = G == 1 ? 0 : G == 2 ? 1 : G == 4 ? 2 : 3;
  if (cache[di][gi] == 0) {
    int r = 0;
    if (D == 128) r = G == 1 ? resident_blocks_of<128, 1, EXT>() : G == 2 ? resident_blocks_of<128, 2, EXT>()
                    : G == 4 ? resident_blocks_of<128, 4, EXT>() : resident_blocks_of<128, 8, EXT>();
    else r = G == 1 ? resident_blocks_of<64, 1, EXT>() : G == 2 ? resident_blocks_of<64, 2, EXT>()
             : G == 4 ? resident_blocks_of<64, 4, EXT>() : resident_blocks_of<64, 8, EXT>();
    if (r <= 0) { cudaGetLastError(); return 148 * 5; }
    cache[di][gi] = r;
  }
  return cache[di][gi];
}

// Splits per (sequence, KV head[, token group]): the grid should be a whole number of waves of resident
// blocks, each split at most kChunkCap rows (its scores live in shared memory) and not much shorter than
// 128 rows.  `vmax` bounds the visible rows of a block, `units` counts the blocks per split index.
int splits_for(int vmax, int units, int slots) {
  const int by_cap = (vmax + (kChunkCap - 16) - 1) / (kChunkCap - 16);
  const int by_len = (vmax + 127) / 128;
  int s = by_cap;
  for (int waves = 1; waves <= 64; ++waves) {
    s = (int)(((long long)waves * slots) / units);
    if (s >= by_cap && s >= 1) break;
  }
  if (s > by_len) s = by_len;
  if (s < by_cap) s = by_cap;
  return s < 1 ? 1 : s;
}

int pick_splits(int B, int Tmax, int Hq, int Hkv, int D, const cowa_params_t* p) {
  const int hg = p->hkv_global > 0 ? p->hkv_global : Hkv;
  return splits_for(max_visible(Tmax, hg, p), B * Hkv, resident_blocks<false>(D, Hq / Hkv));
}

// Extended kernel: tokens per block and blocks per (sequence, KV head) for NQ tokens and group size gsz.
void token_groups(int NQ, int gsz, int* tpg, int* ngroups, int* cols) {
  int t = 1;
  while (t * 2 * gsz <= 8 && t < NQ) t *= 2;
  *tpg = t; *ngroups = (NQ + t - 1) / t; *cols = t * gsz;
}

int pick_splits_ext(int B, int NQ, int Tmax, int Hq, int Hkv, int D, const cowa_params_t* p) {
  const int hg = p->hkv_global > 0 ? p->hkv_global : Hkv;
  int tpg, ngroups, cols;
  token_groups(NQ, Hq / Hkv, &tpg, &ngroups, &cols);
  long long vmax = (long long)max_visible(Tmax, hg, p) + 3ll * (tpg - 1);  // each range grows by the token span
  if (vmax > Tmax) vmax = Tmax;
  return splits_for((int)vmax, B * Hkv * ngroups, resident_blocks<true>(D, cols));
}

// Launch of the merge kernel right behind the split kernel, allowed to start before that one has drained.
template <int D>
cudaError_t launch_combine(unsigned rows, const float* ws_o, const float* ws_m, const float* ws_l, __nv_bfloat16* o,
                           float* lse, int S, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(rows); cfg.blockDim = dim3(128); cfg.dynamicSmemBytes = 0; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, cowa_decode_combine_kernel<D>, ws_o, ws_m, ws_l, o, lse, S);
}

template <int D, int G, bool EXT>
cudaError_t launch_split(const DecodeArgs& a, cudaStream_t st) {
  dim3 grid(a.S, a.Hkv, EXT ? a.B * a.ngroups : a.B);
  cowa_decode_split_kernel<D, G, EXT><<<grid, kThreads, 0, st>>>(a);
  return cudaGetLastError();
}

template <int D, bool EXT>
cudaError_t dispatch_split(int G, const DecodeArgs& a, cudaStream_t st) {
  switch (G) {
    case 1: return launch_split<D, 1, EXT>(a, st);
    case 2: return launch_split<D, 2, EXT>(a, st);
    case 4: return launch_split<D, 4, EXT>(a, st);
    case 8: return launch_split<D, 8, EXT>(a, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

namespace cowa {

// Validates a decode call; on success fills S (number of splits).
int decode_validate(const void* q, const void* kc, const void* vc, const int32_t* lens, void* o, int B,
                    int Tmax, int Hq, int Hkv, int D, const cowa_params_t* p, int* S) {
  if (!q || !kc || !vc || !lens || !o || !p) return COWA_ERR_INVALID_ARG;
  if (B <= 0 || Tmax <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0) return COWA_ERR_INVALID_ARG;
  if (!p->full_attn && (p->sink < 0 || p->local < 1)) return COWA_ERR_INVALID_ARG;
  const int hg = p->hkv_global > 0 ? p->hkv_global : Hkv;
  if (p->hkv_offset < 0 || p->hkv_offset + Hkv > hg) return COWA_ERR_INVALID_ARG;
  if (D != 64 && D != 128) return COWA_ERR_UNSUPPORTED;
  const int G = Hq / Hkv;
  if (G != 1 && G != 2 && G != 4 && G != 8) return COWA_ERR_UNSUPPORTED;
  if (B > 65535 || Hkv > 65535) return COWA_ERR_UNSUPPORTED;
  if (!(p->softmax_scale > 0.f)) return COWA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(kc) || !aligned16(vc) || !aligned16(o)) return COWA_ERR_MISALIGNED;
  for (int i = 0; i < 3; ++i)
    if (p->q_strides[i] || p->o_strides[i]) return COWA_ERR_UNSUPPORTED;  // q and o of a decode step are [B, Hq, D]
  *S = pick_splits(B, Tmax, Hq, Hkv, D, p);
  return COWA_OK;
}

size_t decode_ws_bytes(int B, int Hq, int D, int S) {
  return (size_t)B * Hq * S * (D + 2) * sizeof(float);
}

// Enqueues the split and combine kernels using `ws` (>= decode_ws_bytes) as scratch.
int decode_launch(const void* q, const void* kc, const void* vc, const int32_t* lens, void* o, float* lse,
                  int B, int Tmax, int Hq, int Hkv, int D, const cowa_params_t* p, int S, void* ws,
                  cudaStream_t st) {
  DecodeArgs a;
  a.q = static_cast<const __nv_bfloat16*>(q);
  a.kc = static_cast<const __nv_bfloat16*>(kc);
  a.vc = static_cast<const __nv_bfloat16*>(vc);
  a.lens = lens;
  a.ws_o = static_cast<float*>(ws);
  a.ws_m = a.ws_o + (size_t)B * Hq * S * D;
  a.ws_l = a.ws_m + (size_t)B * Hq * S;
  a.B = B; a.Tmax = Tmax; a.Hq = Hq; a.Hkv = Hkv; a.S = S;
  int rc;
  if ((rc = resolve_strides(p->k_strides, Hkv, Tmax, D, &a.sk))) return rc;
  if ((rc = resolve_strides(p->v_strides, Hkv, Tmax, D, &a.sv))) return rc;
  a.sink = p->sink; a.near = p->local;
  a.hkv_global = p->hkv_global > 0 ? p->hkv_global : Hkv;
  a.hkv_offset = p->hkv_offset;
  a.full_attn = p->full_attn;
  a.scale_log2 = p->softmax_scale * 1.4426950408889634f;
  a.block_table = nullptr; a.NQ = 1; a.tpg = 1; a.ngroups = 1; a.page_size = 0; a.max_pages = 0; a.page_shift = -1;
  const int G = Hq / Hkv;
  cudaError_t e = (D == 128) ? dispatch_split<128, false>(G, a, st) : dispatch_split<64, false>(G, a, st);
  if (e != cudaSuccess) return record_cuda_error(e);
  e = (D == 128) ? launch_combine<128>((unsigned)(B * Hq), a.ws_o, a.ws_m, a.ws_l, static_cast<__nv_bfloat16*>(o), lse, S, st)
                 : launch_combine<64>((unsigned)(B * Hq), a.ws_o, a.ws_m, a.ws_l, static_cast<__nv_bfloat16*>(o), lse, S, st);
  if (e != cudaSuccess) return record_cuda_error(e);
  return COWA_OK;
}

// Multi-token and / or paged decode: q, o [B, NQ, Hq, D], lse [B, NQ, Hq]; block_table == nullptr means a
// contiguous cache [B, Hkv, Tmax, D], otherwise pages [num_pages, Hkv, page_size, D] and Tmax = max_pages * page_size.
int decode_ext_launch(const void* q, const void* kc, const void* vc, const int32_t* block_table, const int32_t* lens,
                      void* o, float* lse, int B, int NQ, int Tmax, int page_size, int max_pages, int Hq, int Hkv,
                      int D, const cowa_params_t* p, int S, void* ws, cudaStream_t st) {
  DecodeArgs a;
  a.q = static_cast<const __nv_bfloat16*>(q);
  a.kc = static_cast<const __nv_bfloat16*>(kc);
  a.vc = static_cast<const __nv_bfloat16*>(vc);
  a.lens = lens;
  const size_t rows = (size_t)B * NQ * Hq;
  a.ws_o = static_cast<float*>(ws);
  a.ws_m = a.ws_o + rows * S * D;
  a.ws_l = a.ws_m + rows * S;
  a.B = B; a.Tmax = Tmax; a.Hq = Hq; a.Hkv = Hkv; a.S = S;
  const int64_t none[3] = {0, 0, 0};
  resolve_strides(none, Hkv, Tmax, D, &a.sk);  // contiguous [B, Hkv, Tmax, D] (paged: rows are addressed through the table)
  a.sv = a.sk;
  a.sink = p->sink; a.near = p->local;
  a.hkv_global = p->hkv_global > 0 ? p->hkv_global : Hkv;
  a.hkv_offset = p->hkv_offset;
  a.full_attn = p->full_attn;
  a.scale_log2 = p->softmax_scale * 1.4426950408889634f;
  a.block_table = block_table; a.NQ = NQ; a.page_size = page_size; a.max_pages = max_pages;
  a.page_shift = -1;
  if (page_size > 0 && (page_size & (page_size - 1)) == 0)
    for (int sft = 0; sft < 31; ++sft)
      if ((1 << sft) == page_size) a.page_shift = sft;
  int cols;
  token_groups(NQ, Hq / Hkv, &a.tpg, &a.ngroups, &cols);
  cudaError_t e = (D == 128) ? dispatch_split<128, true>(cols, a, st) : dispatch_split<64, true>(cols, a, st);
  if (e != cudaSuccess) return record_cuda_error(e);
  e = (D == 128) ? launch_combine<128>((unsigned)rows, a.ws_o, a.ws_m, a.ws_l, static_cast<__nv_bfloat16*>(o), lse, S, st)
                 : launch_combine<64>((unsigned)rows, a.ws_o, a.ws_m, a.ws_l, static_cast<__nv_bfloat16*>(o), lse, S, st);
  if (e != cudaSuccess) return record_cuda_error(e);
  return COWA_OK;
}

}  // namespace cowa

extern "C" {

size_t cowa_decode_multi_workspace_bytes(int B, int Nq, int Tmax, int Hq, int Hkv, int D, const cowa_params_t* p) {
  if (!p || B <= 0 || Nq <= 0 || Tmax <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || (D != 64 && D != 128)) return 0;
  return cowa::decode_ws_bytes(B * Nq, Hq, D, pick_splits_ext(B, Nq, Tmax, Hq, Hkv, D, p));
}

static int decode_ext(const void* q, const void* kc, const void* vc, const int32_t* block_table, const int32_t* lens,
                      void* o, float* lse, int B, int Nq, int Tmax, int page_size, int max_pages, int Hq, int Hkv,
                      int D, const cowa_params_t* p, void* workspace, size_t workspace_bytes, void* stream) {
  int S = 0;
  int st = cowa::decode_validate(q, kc, vc, lens, o, B, Tmax, Hq, Hkv, D, p, &S);
  if (st != COWA_OK) return st;
  if (Nq <= 0 || Nq > 64 || !workspace) return COWA_ERR_INVALID_ARG;
  if (cowa::any_stride_set(p)) return COWA_ERR_UNSUPPORTED;
  if ((long long)B * ((Nq + 7) / 8 * 8) > 65535) return COWA_ERR_UNSUPPORTED;
  if (!cowa::aligned16(workspace)) return COWA_ERR_MISALIGNED;
  S = pick_splits_ext(B, Nq, Tmax, Hq, Hkv, D, p);
  if (workspace_bytes < cowa::decode_ws_bytes(B * Nq, Hq, D, S)) return COWA_ERR_WORKSPACE_TOO_SMALL;
  return cowa::decode_ext_launch(q, kc, vc, block_table, lens, o, lse, B, Nq, Tmax, page_size, max_pages, Hq, Hkv, D,
                                 p, S, workspace, static_cast<cudaStream_t>(stream));
}

int cowa_decode_multi(const void* q, const void* kcache, const void* vcache, const int32_t* lens, void* o,
                      float* lse, int B, int Nq, int Tmax, int Hq, int Hkv, int D, const cowa_params_t* p,
                      void* workspace, size_t workspace_bytes, void* stream) {
  return decode_ext(q, kcache, vcache, nullptr, lens, o, lse, B, Nq, Tmax, 0, 0, Hq, Hkv, D, p, workspace,
                    workspace_bytes, stream);
}

int cowa_decode_paged(const void* q, const void* kpages, const void* vpages, const int32_t* block_table,
                      const int32_t* lens, void* o, float* lse, int B, int Nq, int max_pages, int page_size,
                      int Hq, int Hkv, int D, const cowa_params_t* p, void* workspace, size_t workspace_bytes,
                      void* stream) {
  if (!block_table || max_pages <= 0 || page_size <= 0 || page_size % 16 != 0) return COWA_ERR_INVALID_ARG;
  if ((long long)max_pages * page_size > 0x7FFFFFFFll) return COWA_ERR_UNSUPPORTED;
  return decode_ext(q, kpages, vpages, block_table, lens, o, lse, B, Nq, max_pages * page_size, page_size, max_pages,
                    Hq, Hkv, D, p, workspace, workspace_bytes, stream);
}

size_t cowa_decode_workspace_bytes(int B, int Tmax, int Hq, int Hkv, int D, const cowa_params_t* p) {
  if (!p || B <= 0 || Tmax <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || (D != 64 && D != 128)) return 0;
  return cowa::decode_ws_bytes(B, Hq, D, pick_splits(B, Tmax, Hq, Hkv, D, p));
}

int cowa_decode(const void* q, const void* kcache, const void* vcache, const int32_t* lens, void* o,
                float* lse, int B, int Tmax, int Hq, int Hkv, int D, const cowa_params_t* p,
                void* workspace, size_t workspace_bytes, void* stream) {
  int S = 0;
  int st = cowa::decode_validate(q, kcache, vcache, lens, o, B, Tmax, Hq, Hkv, D, p, &S);
  if (st != COWA_OK) return st;
  if (!workspace) return COWA_ERR_INVALID_ARG;
  if (!cowa::aligned16(workspace)) return COWA_ERR_MISALIGNED;
  if (workspace_bytes < cowa::decode_ws_bytes(B, Hq, D, S)) return COWA_ERR_WORKSPACE_TOO_SMALL;
  return cowa::decode_launch(q, kcache, vcache, lens, o, lse, B, Tmax, Hq, Hkv, D, p, S, workspace,
                             static_cast<cudaStream_t>(stream));
}

size_t cowa_decode_static_capacity(void) { return kStaticScratchBytes; }

int cowa_decode_static(const void* q, const void* kcache, const void* vcache, const int32_t* lens, void* o,
                       float* lse, int B, int Tmax, int Hq, int Hkv, int D, const cowa_params_t* p,
                       void* stream) {
  int S = 0;
  int st = cowa::decode_validate(q, kcache, vcache, lens, o, B, Tmax, Hq, Hkv, D, p, &S);
  if (st != COWA_OK) return st;
  if (cowa::decode_ws_bytes(B, Hq, D, S) > kStaticScratchBytes) return COWA_ERR_STATIC_SCRATCH_EXCEEDED;
  cudaError_t e = cudaSuccess;
  void* scratch = static_scratch_ptr(&e);
  if (!scratch) return cowa::record_cuda_error(e);
  // Every slot of the split states that the merge kernel reads is written by the split kernel of
  // the same call, so nothing left over from an earlier call needs clearing.
  return cowa::decode_launch(q, kcache, vcache, lens, o, lse, B, Tmax, Hq, Hkv, D, p, S, scratch,
                             static_cast<cudaStream_t>(stream));
}

}  // extern "C"
