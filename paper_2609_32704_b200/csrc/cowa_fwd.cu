// CoWindow Attention forward (Algorithm 1) for sm_100a.
//
// One thread block = one (batch, QO head, 128-row QO tile); it walks the tile's visited KV tiles
// J_h(i) (analytic scheduler, descending order) in steps of 64 keys.  Five warps:
//   warps 0-3  softmax: one query row per thread.  tcgen05.ld of S, (boundary tiles only) the
//              window/causal mask from a per-row bit mask, online softmax in base 2 with the
//              scale folded in, P written back to TMEM as bf16 over S's columns.
//   warp 4     control (one lane): TMA loads of K and V (128B swizzle, two buffers each) and all
//              tcgen05.mma issue: S = Q K^T into one of two TMEM buffers, O += P V with P as the
//              TMEM operand.  S of step t+1 is issued before the softmax of step t starts, so the
//              softmax threads never wait for the tensor pipe in steady state.
// The running max is only advanced when the row max grows by more than 2^8 (the accumulator is
// rescaled in TMEM only then); the final normalisation uses the same reference max, so the
// result is the exact softmax.  Two blocks fit per SM (96 KB shared memory, 256 TMEM columns
// each).  The QO heads of a GQA group at the same tile are adjacent in launch order and share
// K/V through L2.
// The same kernel serves N_q <= N_k (queries bottom-right aligned) and, with VARLEN, packed batches
// [H, total, D] whose sequences have their own N_q <= N_k: a block then finds its (sequence, tile) by a
// warp scan of the offset arrays and stores a sequence's last, partial tile row by row.
#include <cuda_bf16.h>

#include "cowa_common.h"
#include "cowa_ptx.cuh"
#include "cowa_tma.h"

using namespace cowa_ptx;

namespace {

constexpr int BQ = 128, BK = 64;
constexpr int kFwdThreads = 160;

struct FwdArgs {
  float* lse;
  unsigned int* status;
  int B, Nq, Nk, Hq, Hkv, G;  // packed batches: Nq, Nk unused
  float scale_log2;
  CowaHeadWindows wins;
  // packed (variable-length) batches only
  const int* cu_q;   // [B+1] row offsets of the sequences in q / o / lse
  const int* cu_k;   // [B+1] row offsets in k / v
  __nv_bfloat16* o;  // raw output pointer for the last, partial tile of a sequence
  int total_q, total_k;
  int sink, local, hkv_global, hkv_offset, full_attn, explicit_windows;
};

// bits [lo, hi] of the 32-bit word covering columns [base, base+32)
__device__ __forceinline__ uint32_t interval_bits(int a, int b, int base) {
  int lo = max(a - base, 0), hi = min(b - base, 31);
  if (lo > hi) return 0u;
  return (0xFFFFFFFFu >> (31 - (hi - lo))) << lo;
}

template <int D>
struct FwdSmem {
  static constexpr int kQ = BQ * D * 2;   // Q tile (later the O staging tile)
  static constexpr int kKV = BK * D * 2;  // one K or V step tile
  static constexpr int oQ = 0, oK = kQ, oV = kQ + 2 * kKV, oBar = kQ + 4 * kKV;
  static constexpr int kBytes = oBar + 128 + 1024;  // + barriers + alignment slack
};

template <int D, bool VARLEN>
__global__ void __launch_bounds__(kFwdThreads, 2)
cowa_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                const __grid_constant__ FwdArgs a) {
  using SM = FwdSmem<D>;
  constexpr int NSLAB = D / 64;          // 64-element (128-byte) slabs along D
  constexpr int SLAB_Q = BQ * 128;       // bytes of one slab of a 128-row tile
  constexpr int SLAB_K = BK * 128;       // ... of a 64-row tile
  constexpr uint32_t TMEM_COLS = 256;    // S/P buffers: [0,64), [64,128); O: [128, 128+D)
  constexpr uint32_t cO = 128;
  constexpr uint32_t IDESC_S = idesc_bf16(128, BK, 0, 0);
  constexpr uint32_t IDESC_O = idesc_bf16(128, D, 0, 1);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem + SM::oQ;
  uint8_t* sK = smem + SM::oK;  // [2][kKV]
  uint8_t* sV = smem + SM::oV;  // [2][kKV]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::oBar);
  uint64_t* bar_q = bars + 0;
  uint64_t* bar_k = bars + 1;   // [2] K step tile landed
  uint64_t* bar_v = bars + 3;   // [2] V step tile landed
  uint64_t* bar_s = bars + 5;   // [2] S of a step is in TMEM buffer b
  uint64_t* bar_p = bars + 7;   // [2] count 128: P written over S
  uint64_t* bar_pv = bars + 9;  //     O += P V of a step has completed
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 10);

  const int tid = threadIdx.x;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);  // warp-uniform by construction

  // ---- work item (heaviest QO tiles first; the group's heads adjacent) ----
  int idx = blockIdx.x;
  const int g = idx % a.G; idx /= a.G;
  const int hk = idx % a.Hkv; idx /= a.Hkv;
  int b, i;
  if constexpr (!VARLEN) {
    b = idx % a.B; idx /= a.B;
    i = (a.Nq + BQ - 1) / BQ - 1 - idx;
  } else {
    // idx counts the QO tiles of the packed batch, sequence after sequence, each sequence's heaviest
    // (last) tile first.  Every warp finds its (sequence, tile) by a cooperative scan of the offsets.
    int lt, nts, pb;
    if (!varlen_locate(a.cu_q, a.B, idx, BQ, 0, &b, &lt, &nts, &pb)) return;  // the grid is an upper bound
    i = nts - 1 - lt;
  }
  const int h = hk * a.G + g;
  // Sequence geometry.  Packed batches: every sequence has its own N_q <= N_k, its rows start at
  // cu_q[b] / cu_k[b] of a [H, total, D] tensor, and its windows follow from its own N_k.
  int Nq = a.Nq, Nk = a.Nk, qbase = 0, kbase = 0;
  int bt = b;  // batch coordinate of the tensor maps (packed tensors have none)
  CowaWin w = a.wins.w[hk];
  if constexpr (VARLEN) {
    qbase = a.cu_q[b]; Nq = a.cu_q[b + 1] - qbase;
    kbase = a.cu_k[b]; Nk = a.cu_k[b + 1] - kbase;
    bt = 0;
    if (Nq > Nk || qbase < 0 || kbase < 0 || qbase + Nq > a.total_q || kbase + Nk > a.total_k) {
      // malformed offsets: report, touch nothing
      if (threadIdx.x == 0) atomicOr(a.status, (unsigned)COWA_DEV_BAD_SEQLENS);
      return;
    }
    if (a.full_attn) { w.s = 0; w.n = Nk; w.g = 0; w.l = 0; }
    else if (!a.explicit_windows) w = cowa_default_window(Nk, a.hkv_global, a.hkv_offset + hk, a.sink, a.local);
  }
  const int off = Nk - Nq;
  const int q0 = i * BQ, q1 = min(q0 + BQ, Nq) - 1;
  CowaRange rg[3];
  cowa_fwd_ranges(w, q0, q1, off, Nk, BK, rg);
  const int nt = cowa_range_len(rg[0]) + cowa_range_len(rg[1]) + cowa_range_len(rg[2]);

  // ---- set-up ----
  if (tid == 0) {
    mbar_init(bar_q, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar_k + s, 1); mbar_init(bar_v + s, 1); mbar_init(bar_s + s, 1); mbar_init(bar_p + s, 128);
    }
    mbar_init(bar_pv, 1);
    fence_mbar_init();
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(tmem_holder, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  bool ok = true;  // false once a bounded wait ran out; every role then falls through to the teardown

  if (warp == 4) {
    // ======================= control: TMA loads and MMA issue =======================
    // The whole warp runs the loop (uniform control flow keeps descriptors and counters in uniform
    // registers); only the elected lane executes the TMA and tcgen05 instructions.
    if (nt > 0) {
      const bool lead = elect_one();
      const uint32_t tb = tmem_base;
      const uint64_t dQ = smem_desc_sw128(smem_u32(sQ), 16, 1024);                 // Q, K-major (A of S)
      const uint64_t dK0 = smem_desc_sw128(smem_u32(sK), 16, 1024);                // K buffer 0, K-major (B of S)
      const uint64_t dV0 = smem_desc_sw128(smem_u32(sV), SLAB_K, 1024);            // V buffer 0, MN-major (B of O)
      constexpr uint32_t kKV16 = SM::kKV >> 4;
      auto load_k = [&](int t) {
        if (lead) {
          const int j = cowa_fwd_tile_at(rg, t);
          uint8_t* dst = sK + (t & 1) * SM::kKV;
          mbar_expect_tx(bar_k + (t & 1), SM::kKV);
          for (int s = 0; s < NSLAB; ++s) tma_load_4d(dst + s * SLAB_K, &tmK, bar_k + (t & 1), s * 64, kbase + j * BK, hk, bt);
        }
      };
      auto load_v = [&](int t) {
        if (lead) {
          const int j = cowa_fwd_tile_at(rg, t);
          uint8_t* dst = sV + (t & 1) * SM::kKV;
          mbar_expect_tx(bar_v + (t & 1), SM::kKV);
          for (int s = 0; s < NSLAB; ++s) tma_load_4d(dst + s * SLAB_K, &tmV, bar_v + (t & 1), s * 64, kbase + j * BK, hk, bt);
        }
      };
      auto issue_s = [&](int buf) {  // S = Q K^T into TMEM buffer buf from K buffer buf
        if (lead) {
          const uint64_t dK = dK0 + buf * kKV16;
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk)
            mma_ss(tb + buf * 64, dQ + (((kk / 4) * SLAB_Q + (kk % 4) * 32) >> 4),
                   dK + (((kk / 4) * SLAB_K + (kk % 4) * 32) >> 4), IDESC_S, kk > 0);
          mma_commit(bar_s + buf);
        }
      };
      if (lead) {
        prefetch_tmap(&tmQ); prefetch_tmap(&tmK); prefetch_tmap(&tmV);
        mbar_expect_tx(bar_q, SM::kQ);
        for (int s = 0; s < NSLAB; ++s) tma_load_4d(sQ + s * SLAB_Q, &tmQ, bar_q, s * 64, qbase + q0, h, bt);
      }
      load_k(0);
      if (nt > 1) load_k(1);
      load_v(0);
      ok = mbar_wait(bar_q, 0, a.status) && mbar_wait(bar_k, 0, a.status);
      if (ok) { tc_fence_after(); issue_s(0); }
      uint32_t par = 0;  // (t >> 1) & 1
      for (int t = 0; t < nt && ok; ++t) {
        const int b_ = t & 1;
        if (t + 1 < nt) {  // S(t+1): its buffer last held P(t-1), whose product was issued before this one
          ok = mbar_wait(bar_k + (b_ ^ 1), b_ ? (par ^ 1) : par, a.status);
          if (!ok) break;
          tc_fence_after();
          issue_s(b_ ^ 1);
        }
        if (t + 2 < nt) {  // K(t+2) over K(t), once S(t) has been computed
          ok = mbar_wait(bar_s + b_, par, a.status);
          if (!ok) break;
          load_k(t + 2);
        }
        if (t + 1 < nt) {  // V(t+1) over V(t-1), once O += P V of step t-1 has completed
          if (t >= 1) ok = mbar_wait(bar_pv, (t - 1) & 1, a.status);
          if (!ok) break;
          load_v(t + 1);
        }
        ok = mbar_wait(bar_p + b_, par, a.status) && mbar_wait(bar_v + b_, par, a.status);
        if (!ok) break;
        tc_fence_after();
        if (lead) {
          const uint64_t dV = dV0 + b_ * kKV16;
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk)
            mma_ts(tb + cO, tb + b_ * 64 + kk * 8, dV + ((kk * 2048) >> 4), IDESC_O, (t > 0 || kk > 0) ? 1u : 0u);
          mma_commit(bar_pv);
        }
        if (b_) par ^= 1;
      }
    }
  } else {
    // ======================= softmax: one query row per thread =======================
    const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16);  // this warp's 32 lanes
    const uint32_t t_O = t_lane + cO;
    const int row = q0 + tid;
    const bool row_valid = row < Nq;
    // Last, partial tile of a packed sequence: the rows after it belong to the next sequence, so the
    // tile is written row by row instead of by one bulk store.
    const bool tail_rows = VARLEN && (q0 + BQ > Nq);
    const int rowpos = row + off;  // position of this query on the key axis
    float m_ref = -INFINITY, l_sum = 0.f;
    const float2 sc2 = make_float2(a.scale_log2, a.scale_log2);

    // Which visited tiles need no mask?  Inside each of the three ranges these form one interval of tile
    // indices, found once here; the loop then only compares.  The intervals are conservative (a tile that
    // straddles two windows, or sink and non-sink columns, is treated as a boundary tile and masked, which
    // is always correct).  With d = (row position) - (key index): every pair of tile j is causal iff
    // 64 j + 63 <= q0 + off; it lies in the near window iff q1 + off - 64 j < n; in the long window iff also
    // q0 + off - (64 j + 63) >= n + g and q1 + off - 64 j < n + g + l; in the sink iff 64 j + 63 < s.
    int f_lo[3] = {1, 1, 1}, f_hi[3] = {0, 0, 0};
    if (q0 + BQ <= Nq) {
      auto fdiv = [](long long x) -> int { return (int)(x >= 0 ? x / BK : -((-x + BK - 1) / BK)); };
      const long long p0 = (long long)q0 + off, p1 = p0 + BQ - 1;
      const int causal_hi = fdiv(p0 - (BK - 1));
      f_lo[0] = fdiv(p1 - w.n) + 1; f_hi[0] = causal_hi;
      if (w.l > 0) {
        f_lo[1] = fdiv(p1 - ((long long)w.n + w.g + w.l)) + 1;
        f_hi[1] = min(causal_hi, fdiv(p0 - ((long long)w.n + w.g) - (BK - 1)));
      }
      f_lo[2] = 0; f_hi[2] = min(causal_hi, w.s >= BK ? (w.s - BK) / BK : -1);
    }
    // walk of the ranges: tile j steps down to j_last, then the next non-empty range is entered; the
    // current range's bounds live in registers (selects, no indexed local arrays)
    int rr = -1, j = 0, j_last = 0, fl = 1, fh = 0;
    auto next_range = [&]() {
#pragma unroll
      for (int c = 0; c < 3; ++c) {
        if (rr < c && rg[c].hi >= rg[c].lo) {
          rr = c; j = rg[c].hi; j_last = rg[c].lo; fl = f_lo[c]; fh = f_hi[c];
          return;
        }
      }
      rr = 3;
    };
    next_range();

    for (int t = 0; t < nt && ok; ++t) {
      const int b_ = t & 1;
      const int k0 = j * BK;
      const bool full = j >= fl && j <= fh;
      const uint32_t t_S = t_lane + b_ * 64;

      ok = mbar_wait(bar_s + b_, (t >> 1) & 1, a.status);
      if (!ok) break;
      tc_fence_after();
      uint32_t sr[2][32];
      tmem_ld32(t_S, sr[0]);
      tmem_ld32(t_S + 32, sr[1]);
      tmem_wait_ld();

      if (!full) {
        const int kend = min(rowpos, Nk - 1);  // last causal key of this row
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const int base = k0 + c * 32;
          uint32_t mk = interval_bits(rowpos - w.n + 1, kend, base) | interval_bits(0, min(w.s - 1, kend), base);
          if (w.l > 0) mk |= interval_bits(rowpos - (w.n + w.g + w.l) + 1, min(rowpos - (w.n + w.g), kend), base);
          if (!row_valid) mk = 0u;
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (!((mk >> e) & 1u)) sr[c][e] = 0xFF800000u;  // -inf
        }
      }
      // row max: four independent chains of 3-input max
      float mxa[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int c = 0; c < 2; ++c)
#pragma unroll
        for (int e = 0; e < 32; e += 2)
          mxa[(e >> 1) & 3] = max3(mxa[(e >> 1) & 3], __uint_as_float(sr[c][e]), __uint_as_float(sr[c][e + 1]));
      const float mx = fmaxf(fmaxf(mxa[0], mxa[1]), fmaxf(mxa[2], mxa[3])) * a.scale_log2;
      float m_new = m_ref;
      if (mx > m_ref + 8.f) m_new = mx;
      const float alpha = (m_new == m_ref) ? 1.f : ex2(m_ref - m_new);
      const float sub = (m_new == -INFINITY) ? 0.f : m_new;
      m_ref = m_new;

      // p = 2^(s * scale - m): packed fp32 pairs for the multiply-add and the row sum
      const float2 nsub2 = make_float2(-sub, -sub);
      float2 rsa[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
      uint32_t pk[32];
#pragma unroll
      for (int c = 0; c < 2; ++c)
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          const float2 x = fma2(make_float2(__uint_as_float(sr[c][e]), __uint_as_float(sr[c][e + 1])), sc2, nsub2);
          const float2 pp = make_float2(ex2(x.x), ex2(x.y));
          rsa[(e >> 1) & 3] = add2(rsa[(e >> 1) & 3], pp);
          pk[c * 16 + e / 2] = pack_bf16(pp.x, pp.y);
        }
      const float2 rs2 = add2(add2(rsa[0], rsa[1]), add2(rsa[2], rsa[3]));
      l_sum = l_sum * alpha + (rs2.x + rs2.y);

      // Every step waits for the product of the step before (normally long finished): the accumulator
      // may then be rescaled safely, and no thread ever falls two phases behind on this barrier, which
      // its parity wait could not tell apart.
      if (t > 0) {
        ok = mbar_wait(bar_pv, (t - 1) & 1, a.status);
        if (!ok) break;
        tc_fence_after();
      }
      // rescale the accumulator when some row of this warp moved its reference max
      if (t > 0 && __any_sync(0xFFFFFFFFu, alpha != 1.f)) {
        const float2 al2 = make_float2(alpha, alpha);
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t ov[32];
          tmem_ld32(t_O + c * 32, ov);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const float2 y = mul2(make_float2(__uint_as_float(ov[e]), __uint_as_float(ov[e + 1])), al2);
            ov[e] = __float_as_uint(y.x); ov[e + 1] = __float_as_uint(y.y);
          }
          tmem_st32(t_O + c * 32, ov);
        }
      }
      tmem_st32(t_S, pk);  // P over the first 32 columns of this S buffer
      tmem_wait_st();
      if constexpr (VARLEN) {
        // Last key tile of a packed sequence: the rows after it in shared memory belong to the next sequence.
        // Their P entries are exactly zero, but 0 x (Inf or NaN) in the product would still poison this
        // sequence, so those V rows are cleared before the product may start.
        const int vrows = Nk - j * BK;  // valid rows of this 64-row tile
        if (vrows < BK) {
          ok = mbar_wait(bar_v + b_, (t >> 1) & 1, a.status);
          if (!ok) break;
          uint8_t* vt = sV + b_ * SM::kKV;
          const int nchunk = (BK - vrows) * 8;  // 16-byte chunks per slab
          for (int s_ = 0; s_ < NSLAB; ++s_)
            for (int c_ = tid; c_ < nchunk; c_ += 128)
              *reinterpret_cast<uint4*>(vt + s_ * SLAB_K + vrows * 128 + c_ * 16) = make_uint4(0u, 0u, 0u, 0u);
          fence_proxy_async_smem();
        }
      }
      tc_fence_before();
      mbar_arrive(bar_p + b_);
      if (j > j_last) --j; else next_range();
    }

    // ---- epilogue: O / l, LSE ----
    if (nt > 0) ok = mbar_wait(bar_pv, (nt - 1) & 1, a.status) && ok;
    if (ok && nt > 0) {
      tc_fence_after();
      const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t ov[32];
        tmem_ld32(t_O + c * 32, ov);
        tmem_wait_ld();
        // 32 columns = 4 chunks of 8 elements (16 B); slab = (c*32)/64, chunk index within slab
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint4 v;
          v.x = pack_bf16(__uint_as_float(ov[q * 8 + 0]) * inv, __uint_as_float(ov[q * 8 + 1]) * inv);
          v.y = pack_bf16(__uint_as_float(ov[q * 8 + 2]) * inv, __uint_as_float(ov[q * 8 + 3]) * inv);
          v.z = pack_bf16(__uint_as_float(ov[q * 8 + 4]) * inv, __uint_as_float(ov[q * 8 + 5]) * inv);
          v.w = pack_bf16(__uint_as_float(ov[q * 8 + 6]) * inv, __uint_as_float(ov[q * 8 + 7]) * inv);
          const int d0 = c * 32 + q * 8;
          const int slab = d0 / 64, chunk = (d0 % 64) / 8;
          if (!tail_rows)
            *reinterpret_cast<uint4*>(sQ + slab * SLAB_Q + tid * 128 + ((chunk ^ (tid & 7)) << 4)) = v;
          else if (row_valid)
            *reinterpret_cast<uint4*>(a.o + ((size_t)h * a.total_q + qbase + row) * D + d0) = v;
        }
      }
      if (row_valid) {
        const size_t li = VARLEN ? (size_t)h * a.total_q + qbase + row : ((size_t)b * a.Hq + h) * Nq + row;
        a.lse[li] = 0.6931471805599453f * (m_ref + log2f(l_sum));
      }
      fence_proxy_async_smem();
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");  // the four softmax warps
    if (tid == 0 && ok && nt > 0 && !tail_rows) {
      for (int s = 0; s < NSLAB; ++s) tma_store_4d(&tmO, sQ + s * SLAB_Q, s * 64, qbase + q0, h, bt);
      tma_commit_group();
      tma_wait_group<0>();
    }
  }

  // ---- teardown ----
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    __syncwarp();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// One launch for both layouts.  Batched: cu_q == nullptr, tensors [B,H,N,D].  Packed: tensors
// [H,total,D]; the grid is sized from total_q / BQ + B, an upper bound of the batch's tile count.
template <int D, bool VARLEN>
int launch_fwd(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Nq, int Nk, int Hq,
               int Hkv, const cowa_params_t* p, const CowaHeadWindows& hw, const int* cu_q, const int* cu_k,
               int total_q, int total_k, cudaStream_t st) {
  CUtensorMap mq, mk, mv, mo;
  int rc;
  const int rows_q = VARLEN ? total_q : Nq, rows_k = VARLEN ? total_k : Nk;
  const int nb = VARLEN ? 1 : B;  // packed tensors are [H, total, D]
  CowaStrides sq, sk, sv, so;
  if (VARLEN && cowa::any_stride_set(p)) return COWA_ERR_UNSUPPORTED;
  if ((rc = cowa::resolve_strides(p->q_strides, Hq, rows_q, D, &sq))) return rc;
  if ((rc = cowa::resolve_strides(p->k_strides, Hkv, rows_k, D, &sk))) return rc;
  if ((rc = cowa::resolve_strides(p->v_strides, Hkv, rows_k, D, &sv))) return rc;
  if ((rc = cowa::resolve_strides(p->o_strides, Hq, rows_q, D, &so))) return rc;
  if ((rc = cowa::make_tensor_map(&mq, q, cowa::MapType::BF16, D, rows_q, Hq, nb, sq, 64, BQ))) return rc;
  if ((rc = cowa::make_tensor_map(&mk, k, cowa::MapType::BF16, D, rows_k, Hkv, nb, sk, 64, BK))) return rc;
  if ((rc = cowa::make_tensor_map(&mv, v, cowa::MapType::BF16, D, rows_k, Hkv, nb, sv, 64, BK))) return rc;
  if ((rc = cowa::make_tensor_map(&mo, o, cowa::MapType::BF16, D, rows_q, Hq, nb, so, 64, BQ))) return rc;
  FwdArgs a;
  a.lse = lse;
  a.status = cowa::device_status_word();
  if (!a.status) return COWA_ERR_CUDA;
  a.B = B; a.Nq = Nq; a.Nk = Nk; a.Hq = Hq; a.Hkv = Hkv; a.G = Hq / Hkv;
  a.scale_log2 = p->softmax_scale * 1.4426950408889634f;
  a.wins = hw;
  a.cu_q = cu_q; a.cu_k = cu_k; a.o = static_cast<__nv_bfloat16*>(o); a.total_q = total_q; a.total_k = total_k;
  a.sink = p->sink; a.local = p->local;
  a.hkv_global = p->hkv_global > 0 ? p->hkv_global : Hkv;
  a.hkv_offset = p->hkv_offset; a.full_attn = p->full_attn; a.explicit_windows = p->windows != nullptr;
  COWA_CUDA_TRY(cudaFuncSetAttribute(cowa_fwd_kernel<D, VARLEN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     FwdSmem<D>::kBytes));
  const long long nblocks = VARLEN ? ((long long)total_q / BQ + B) * Hq : (long long)((Nq + BQ - 1) / BQ) * B * Hq;
  if (nblocks > 0x7FFFFFFFll) return COWA_ERR_UNSUPPORTED;
  cowa_fwd_kernel<D, VARLEN><<<(unsigned)nblocks, kFwdThreads, FwdSmem<D>::kBytes, st>>>(mq, mk, mv, mo, a);
  COWA_CUDA_TRY(cudaGetLastError());
  return COWA_OK;
}

}  // namespace

extern "C" {

int cowa_prefill(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Nq, int Nk, int Hq,
                 int Hkv, int D, const cowa_params_t* p, void* stream) {
  if (!q || !k || !v || !o || !lse || !p) return COWA_ERR_INVALID_ARG;
  if (B <= 0 || Nq <= 0 || Nk < Nq || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0) return COWA_ERR_INVALID_ARG;
  if (!(p->softmax_scale > 0.f)) return COWA_ERR_INVALID_ARG;
  if (D != 64 && D != 128) return COWA_ERR_UNSUPPORTED;
  if (!cowa::aligned16(q) || !cowa::aligned16(k) || !cowa::aligned16(v) || !cowa::aligned16(o))
    return COWA_ERR_MISALIGNED;
  CowaHeadWindows hw;
  int rc = cowa::resolve_windows(Nk, Hkv, p, &hw);
  if (rc != COWA_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return D == 128 ? launch_fwd<128, false>(q, k, v, o, lse, B, Nq, Nk, Hq, Hkv, p, hw, nullptr, nullptr, 0, 0, st)
                  : launch_fwd<64, false>(q, k, v, o, lse, B, Nq, Nk, Hq, Hkv, p, hw, nullptr, nullptr, 0, 0, st);
}

int cowa_prefill_varlen(const void* q, const void* k, const void* v, void* o, float* lse, const int32_t* cu_seqlens_q,
                        const int32_t* cu_seqlens_k, int B, int total_q, int total_k, int Hq, int Hkv, int D,
                        const cowa_params_t* p, void* stream) {
  if (!q || !k || !v || !o || !lse || !p || !cu_seqlens_q || !cu_seqlens_k) return COWA_ERR_INVALID_ARG;
  if (B <= 0 || total_q <= 0 || total_k < total_q || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0)
    return COWA_ERR_INVALID_ARG;
  if (!(p->softmax_scale > 0.f)) return COWA_ERR_INVALID_ARG;
  if (D != 64 && D != 128) return COWA_ERR_UNSUPPORTED;
  if (!cowa::aligned16(q) || !cowa::aligned16(k) || !cowa::aligned16(v) || !cowa::aligned16(o))
    return COWA_ERR_MISALIGNED;
  // Explicit tuples are validated and copied here; the default rule is evaluated per sequence on the
  // device (any positive N_k passes the same checks on sink / local / head offsets).
  CowaHeadWindows hw;
  int rc = cowa::resolve_windows(total_k, Hkv, p, &hw);
  if (rc != COWA_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return D == 128 ? launch_fwd<128, true>(q, k, v, o, lse, B, 0, 0, Hq, Hkv, p, hw, cu_seqlens_q,
                                          cu_seqlens_k, total_q, total_k, st)
                  : launch_fwd<64, true>(q, k, v, o, lse, B, 0, 0, Hq, Hkv, p, hw, cu_seqlens_q,
                                         cu_seqlens_k, total_q, total_k, st);
}

int cowa_fwd(const void* q, const void* k, const void* v, void* o, float* lse, int B, int T, int Hq, int Hkv, int D,
             const cowa_params_t* p, void* stream) {
  return cowa_prefill(q, k, v, o, lse, B, T, T, Hq, Hkv, D, p, stream);
}

}  // extern "C"
