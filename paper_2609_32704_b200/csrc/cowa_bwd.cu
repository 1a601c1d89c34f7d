// CoWindow Attention backward (Algorithm 2) for sm_100a.
//
// Three launches on the caller's stream:
//   1. preprocess   Delta = rowsum(O * dO) (Algorithm 2 line 13) and LSE * log2(e), fp32 row vectors
//                   padded to a multiple of 64 rows (padding: LSE = +inf, so that P = 0 there);
//                   the fp32 dQ accumulator is zeroed by a memset before it.
//   2. main kernel  one thread block per (batch, KV head, 128-row KV tile), KV-stationary as in
//                   Algorithm 2, looping over the G QO heads of the group and over the 64-row QO
//                   tiles of I_h(j) (analytic scheduler, ascending).  Per step five tcgen05 MMAs:
//                     S^T  = K Q^T            (TMEM, 128 kv x 64 q)
//                     dP^T = V dO^T           (TMEM)
//                     dV  += P^T dO           (P^T as the TMEM operand)
//                     dK  += dS^T Q           (dS^T as the TMEM operand)
//                     dQ^T = K^T dS^T         (dS^T from shared memory; 128 d x 64 q in TMEM)
//                   dK and dV stay in TMEM for the whole loop, all G heads included, so they need no
//                   atomics (Algorithm 2 line 17 needs them only because it gives each QO head its
//                   own program).  dQ^T is drained by a separate warpgroup through shared memory and
//                   added to the fp32 accumulator with bulk add-reductions of contiguous 32-row ranges (Algorithm 2 line 15).
//                   Warp roles: TMA producer / MMA issuer / two compute warpgroups (P, dS; each takes 32
//                   of the 64 query columns of every step, which halves the latency between S^T and
//                   dS^T) / dQ drain warpgroup, connected by mbarriers; S^T is double buffered so that the
//                   MMAs of steps n+1, n+2 overlap the element-wise work of
//                   step n.  Blocks are ordered sink tiles first (they meet every query tile), then
//                   head by head with ascending KV tile, so that the blocks in flight sweep the same
//                   dQ rows at nearly the same time and the reductions hit in L2.
//   3. convert      dQ accumulator (already scaled) -> bf16.
// Two variations of the main kernel's work split:
//   - `parts` > 1: the G heads of a group are spread over several blocks per KV tile (few tiles, or sink
//     tiles that would be the critical path); each block writes fp32 partial dK, dV to its own slot and a
//     fourth kernel adds the slots in order (bwd_parts, cowa_bwd_reduce_dkv_kernel).
//   - VARLEN: packed batch [H, total, D]; a block finds (sequence, KV tile) by a warp scan of the offsets,
//     windows follow from the sequence's own length, the accumulator and the row vectors use a row space
//     in which every sequence is padded to 64 rows, and a sequence's last, partial KV tile is stored row
//     by row (cowa_bwd_varlen and its own preprocess / convert kernels).
#include <cuda_bf16.h>

#include <algorithm>
#include <type_traits>

#include "cowa_common.h"
#include "cowa_ptx.cuh"
#include "cowa_tma.h"

using namespace cowa_ptx;

namespace {

constexpr int BKV = 128;  // KV rows per block (MMA M)
constexpr int BQS = 64;   // QO rows per step (MMA N of S^T / dP^T)
constexpr int NST = 3;    // Q / dO stages
constexpr float kDqFixedOne = 262144.f;  // 2^18: one unit of dQ in the fixed-point accumulation mode

struct BwdArgs {
  const float* lse2;   // [B*Hq, Tpad]  LSE * log2(e)
  const float* delta;  // [B*Hq, Tpad]
  float* dq_acc;       // [B*Hq, Tpad, D] fp32
  unsigned int* status;
  int B, Nq, Nk, Hq, Hkv, G, Tpad;
  int sink_tiles;      // KV tiles per head that hold sink columns (launched first)
  int dq_fixed;        // 1: dQ partial sums travel as 32-bit fixed point (order-independent addition)
  int parts;           // blocks per KV tile: each takes G / parts heads of the group (1: the whole group)
  float* dkv_part;     // parts > 1: fp32 partial dK, dV [B*Hkv, nKV, parts, 2, BKV, D], summed by a last kernel
  // packed (variable-length) batches only: tensors are [H, total, D], sequence b owns rows cu[b] .. cu[b+1]
  const int* cu;       // [B+1] device
  __nv_bfloat16* dk;   // raw outputs for the last, partial KV tile of a sequence
  __nv_bfloat16* dv;
  int total, tiles_bound;  // rows of the packed tensors; grid tiles per KV head (upper bound of the real count)
  int sink, local, hkv_global, hkv_offset, full_attn, explicit_windows;
  float scale, scale_log2;
  CowaHeadWindows wins;
};

template <int D>
struct BwdSmem {
  static constexpr int kKV = BKV * D * 2;      // K or V tile
  static constexpr int kQS = BQS * D * 2;      // Q or dO step tile
  static constexpr int kStage = 2 * kQS;       // Q + dO
  static constexpr int kDS = BKV * BQS * 2;    // dS^T tile (bf16)
  static constexpr int oK = 0, oV = kKV, oStage = 2 * kKV, oDS = oStage + NST * kStage;
  static constexpr int oVec = oDS + 2 * kDS;   // per stage: 64 floats lse2, 64 floats delta
  static constexpr int oDQ = oVec + NST * 512;  // dQ staging: two tiles of 32 query rows x D fp32
  static constexpr int kDQ = 32 * D * 4;
  static constexpr int oBar = oDQ + 2 * kDQ;
  static constexpr int kBytes = oBar + 256 + 1024;  // barriers + alignment slack; 232192 B at D = 128 (limit 232448)
};

__device__ __forceinline__ void bulk_load_1d(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

__device__ __forceinline__ uint32_t interval_bits32(long long a, long long b, long long base) {
  long long lo = a - base, hi = b - base;
  if (lo < 0) lo = 0;
  if (hi > 31) hi = 31;
  if (lo > hi) return 0u;
  return (0xFFFFFFFFu >> (31 - (int)(hi - lo))) << (int)lo;
}

// named barrier for one 128-thread warpgroup
__device__ __forceinline__ void wg_sync(int id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }

template <int D, bool VARLEN>
__global__ void __launch_bounds__(512, 1)
cowa_bwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmdO,
                const __grid_constant__ CUtensorMap tmdK, const __grid_constant__ CUtensorMap tmdV,
                const __grid_constant__ BwdArgs a) {
  using SM = BwdSmem<D>;
  constexpr int NSLAB = D / 64;
  constexpr int SLAB_KV = BKV * 128;  // bytes of one 64-wide slab of a 128-row tile
  constexpr int SLAB_QS = BQS * 128;  // ... of a 64-row tile
  // TMEM columns
  constexpr uint32_t cS0 = 0, cDP0 = 128, cDK = 256, cDV = 384, TMEM_COLS = 512;  // S^T x2, dP^T/dQ^T x2, dK, dV
  constexpr uint32_t ID_ST = idesc_bf16(128, BQS, 0, 0);   // S^T, dP^T
  constexpr uint32_t ID_ACC = idesc_bf16(128, D, 0, 1);    // dV, dK (B = dO / Q, MN-major)
  constexpr uint32_t ID_DQ = idesc_bf16(128, BQS, 1, 1);   // dQ^T (A = K^T, B = dS^T, both MN-major)

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sK = smem + SM::oK;
  uint8_t* sV = smem + SM::oV;
  uint8_t* sStage = smem + SM::oStage;
  uint8_t* sDS = smem + SM::oDS;
  float* sVec = reinterpret_cast<float*>(smem + SM::oVec);
  float* sDQ = reinterpret_cast<float*>(smem + SM::oDQ);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::oBar);
  uint64_t* bar_kv = bars + 0;
  uint64_t* bar_ld_full = bars + 1;             // [NST]  Q/dO/LSE/Delta of a step have landed
  uint64_t* bar_ld_empty = bars + 1 + NST;      // [NST]  the step's products have consumed the stage
  uint64_t* bar_s_full = bars + 1 + 2 * NST;    // [2]    S^T of a step is in TMEM buffer b
  uint64_t* bar_dp_full = bars + 3 + 2 * NST;   // [2]    dP^T ...
  uint64_t* bar_p_ready = bars + 5 + 2 * NST;   // [2]    count 256: P^T written over S^T
  uint64_t* bar_ds_ready = bars + 7 + 2 * NST;  // [2]    count 256: dS^T in TMEM and shared memory, dP^T consumed
  uint64_t* bar_dq_full = bars + 9 + 2 * NST;   // [2]    dQ^T is in the columns dP^T left
  uint64_t* bar_dq_free = bars + 11 + 2 * NST;  // [2]    count 128: dQ^T drained
  uint64_t* bar_done = bars + 13 + 2 * NST;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 14 + 2 * NST);

  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);  // warp-uniform by construction (helps the compiler)

  // ---- work item: sink tiles of every head first, then head-major with ascending KV tile ----
  int hk, b, j;
  const int part = VARLEN ? 0 : blockIdx.x % a.parts;
  // Sequence geometry.  Packed batches: N_q = N_k = the sequence's length, rows start at cu[b]; the fp32
  // dQ accumulator and the LSE / Delta vectors are laid out with every sequence padded to 64 rows (pbase).
  int Nq = a.Nq, Nk = a.Nk, rbase = 0, pbase = 0;
  CowaWin w;
  if constexpr (!VARLEN) {
    int idx = blockIdx.x / a.parts;
    const int nKV = (a.Nk + BKV - 1) / BKV, nsk = a.sink_tiles, nhead = a.B * a.Hkv;
    if (idx < nsk * nhead) {
      j = idx / nhead; idx %= nhead;
    } else {
      idx -= nsk * nhead;
      j = nsk + idx % (nKV - nsk); idx /= (nKV - nsk);
    }
    hk = idx % a.Hkv; b = idx / a.Hkv;
    w = a.wins.w[hk];
  } else {
    // The sink tiles of every (sequence, head) first (they meet every query tile of their sequence and are
    // the longest blocks); then head-major: consecutive blocks are consecutive KV tiles of one head (their
    // dQ rows overlap in L2).
    const int nsk = a.sink_tiles, nhead = a.B * a.Hkv;
    int nts;
    if ((int)blockIdx.x < nsk * nhead) {
      j = blockIdx.x / nhead;
      b = (blockIdx.x % nhead) / a.Hkv; hk = blockIdx.x % a.Hkv;
      varlen_seq_info(a.cu, b, BKV, BQS, &nts, &pbase);
      if (j >= nts) return;  // the sequence is shorter than its sink
    } else {
      const int rest = blockIdx.x - nsk * nhead;
      hk = rest / a.tiles_bound;
      if (!varlen_locate(a.cu, a.B, rest % a.tiles_bound, BKV, BQS, &b, &j, &nts, &pbase, nsk)) return;
    }
    rbase = a.cu[b];
    Nq = Nk = a.cu[b + 1] - rbase;
    if (rbase < 0 || rbase + Nk > a.total) {  // malformed offsets: report, touch nothing
      if (threadIdx.x == 0) atomicOr(a.status, (unsigned)COWA_DEV_BAD_SEQLENS);
      return;
    }
    w = a.wins.w[hk];
    if (a.full_attn) { w.s = 0; w.n = Nk; w.g = 0; w.l = 0; }
    else if (!a.explicit_windows) w = cowa_default_window(Nk, a.hkv_global, a.hkv_offset + hk, a.sink, a.local);
  }
  const int off = Nk - Nq;
  const int k0 = j * BKV, k1 = min(k0 + BKV, Nk) - 1;
  CowaRange rg[2];
  cowa_bwd_ranges(w, k0, k1, off, Nq, BQS, rg);
  const int cnt = cowa_range_len(rg[0]) + cowa_range_len(rg[1]);  // QO steps per head
  const int gs = a.G / a.parts;          // heads of the group handled by this block
  const int N = cnt * gs;
  const int bt = VARLEN ? 0 : b;                                                    // batch coordinate of the tensor maps
  const int bhk = VARLEN ? hk : b * a.Hkv + hk;                                     // (batch, KV head) row of the partial dK, dV slots
  const int hq0 = hk * a.G + part * gs;                                             // first QO head of this block
  const int bhq0 = (VARLEN ? 0 : b * a.Hq) + hq0;                                   // ... as a row of lse2 / delta / dq_acc
  const size_t vec_stride = (size_t)a.Tpad;                                         // rows per head in lse2 / delta / dq_acc
  const bool tail_kv = VARLEN && (k0 + BKV > Nk);  // rows after the tile's last valid one belong to the next sequence

  if (tid == 0) {
    mbar_init(bar_kv, 1);
    for (int s = 0; s < NST; ++s) { mbar_init(bar_ld_full + s, 1); mbar_init(bar_ld_empty + s, 1); }
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar_s_full + s, 1); mbar_init(bar_dp_full + s, 1);
      mbar_init(bar_p_ready + s, 256); mbar_init(bar_ds_ready + s, 256);
      mbar_init(bar_dq_full + s, 1); mbar_init(bar_dq_free + s, 128);
    }
    mbar_init(bar_done, 1);
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

  bool ok = true;

  // dK (first compute warpgroup) and dV (drain warpgroup): TMEM -> bf16 -> shared -> TMA store.  Called from
  // inside the role branches so that it is compiled under that role's register budget.
  auto store_grad = [&](bool is_dk) {
    const int r = (warp & 3) * 32 + lane;
    const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    if (N > 0) ok = mbar_wait(bar_done, 0, a.status) && ok;
    tc_fence_after();
    uint8_t* sOut = sStage + (is_dk ? 0 : SM::kKV);
    const float mul = is_dk ? a.scale : 1.f;
    if (tail_kv) {
      // last, partial KV tile of a packed sequence: row by row, straight from registers
      __nv_bfloat16* dst = (is_dk ? a.dk : a.dv) + ((size_t)hk * a.total + rbase + k0 + r) * D;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t ov[32];
        if (N > 0 && ok) {
          tmem_ld32(t_lane + (is_dk ? cDK : cDV) + c * 32, ov);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) ov[e] = 0u;
        }
        if (k0 + r < Nk) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint4 v;
            v.x = pack_bf16(__uint_as_float(ov[q * 8 + 0]) * mul, __uint_as_float(ov[q * 8 + 1]) * mul);
            v.y = pack_bf16(__uint_as_float(ov[q * 8 + 2]) * mul, __uint_as_float(ov[q * 8 + 3]) * mul);
            v.z = pack_bf16(__uint_as_float(ov[q * 8 + 4]) * mul, __uint_as_float(ov[q * 8 + 5]) * mul);
            v.w = pack_bf16(__uint_as_float(ov[q * 8 + 6]) * mul, __uint_as_float(ov[q * 8 + 7]) * mul);
            *reinterpret_cast<uint4*>(dst + c * 32 + q * 8) = v;
          }
        }
      }
      return;
    }
    if (a.parts > 1) {
      // The group's heads are spread over several blocks: this block's share goes out in fp32, one slot
      // per block, and a last kernel adds the slots in a fixed order.
      const int nKV = (a.Nk + BKV - 1) / BKV;
      float* dst = a.dkv_part + ((((size_t)bhk * nKV + j) * a.parts + part) * 2 + (is_dk ? 0 : 1)) * (size_t)(BKV * D) +
                   (size_t)r * D;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t ov[32];
        if (N > 0 && ok) {
          tmem_ld32(t_lane + (is_dk ? cDK : cDV) + c * 32, ov);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) ov[e] = 0u;
        }
#pragma unroll
        for (int q = 0; q < 8; ++q)
          *reinterpret_cast<float4*>(dst + c * 32 + q * 4) =
              make_float4(__uint_as_float(ov[q * 4]) * mul, __uint_as_float(ov[q * 4 + 1]) * mul,
                          __uint_as_float(ov[q * 4 + 2]) * mul, __uint_as_float(ov[q * 4 + 3]) * mul);
      }
      return;
    }
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
      uint32_t ov[32];
      if (N > 0 && ok) {
        tmem_ld32(t_lane + (is_dk ? cDK : cDV) + c * 32, ov);
        tmem_wait_ld();
      } else {
#pragma unroll
        for (int e = 0; e < 32; ++e) ov[e] = 0u;
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint4 v;
        v.x = pack_bf16(__uint_as_float(ov[q * 8 + 0]) * mul, __uint_as_float(ov[q * 8 + 1]) * mul);
        v.y = pack_bf16(__uint_as_float(ov[q * 8 + 2]) * mul, __uint_as_float(ov[q * 8 + 3]) * mul);
        v.z = pack_bf16(__uint_as_float(ov[q * 8 + 4]) * mul, __uint_as_float(ov[q * 8 + 5]) * mul);
        v.w = pack_bf16(__uint_as_float(ov[q * 8 + 6]) * mul, __uint_as_float(ov[q * 8 + 7]) * mul);
        const int d0 = c * 32 + q * 8;
        const int slab = d0 / 64, chunk = (d0 % 64) / 8;
        *reinterpret_cast<uint4*>(sOut + slab * SLAB_KV + r * 128 + ((chunk ^ (r & 7)) << 4)) = v;
      }
    }
    fence_proxy_async_smem();
    wg_sync(is_dk ? 1 : 2);
    if (r == 0 && ok) {
      for (int s = 0; s < NSLAB; ++s) tma_store_4d(is_dk ? &tmdK : &tmdV, sOut + s * SLAB_KV, s * 64, rbase + k0, hk, bt);
      tma_commit_group();
      tma_wait_group<0>();
    }
  };

  // Register budget per role: 128 per thread at launch (512 threads), moved to where the work is.  Each
  // setmaxnreg sits at the top of its own branch so that the code below it is compiled for that budget.
  if (warp < 4) {
    setmaxnreg_dec<64>();
    if (warp == 0) {
      // ================= TMA producer =================
      if (lane == 0 && N > 0) {
        prefetch_tmap(&tmQ); prefetch_tmap(&tmdO); prefetch_tmap(&tmK); prefetch_tmap(&tmV);
        mbar_expect_tx(bar_kv, 2 * SM::kKV);
        for (int s = 0; s < NSLAB; ++s) {
          tma_load_4d(sK + s * SLAB_KV, &tmK, bar_kv, s * 64, rbase + k0, hk, bt);
          tma_load_4d(sV + s * SLAB_KV, &tmV, bar_kv, s * 64, rbase + k0, hk, bt);
        }
        int st = 0, g = 0, t_in = 0;   // stage, head of the group, position in I_h(j): kept incrementally
        uint32_t ph_e = 0;             // parity of the "stage empty" wait (the first NST steps need none)
        for (int n = 0; n < N && ok; ++n) {
          if (n >= NST) ok = mbar_wait(bar_ld_empty + st, ph_e, a.status);
          if (!ok) break;
          const int i = cowa_bwd_tile_at(rg, t_in);
          const int bhq = bhq0 + g, q0 = i * BQS;
          uint8_t* sQ = sStage + st * SM::kStage;
          uint8_t* sdO = sQ + SM::kQS;
          mbar_expect_tx(bar_ld_full + st, SM::kStage + 512);
          for (int s = 0; s < NSLAB; ++s) {
            tma_load_4d(sQ + s * SLAB_QS, &tmQ, bar_ld_full + st, s * 64, rbase + q0, hq0 + g, bt);
            tma_load_4d(sdO + s * SLAB_QS, &tmdO, bar_ld_full + st, s * 64, rbase + q0, hq0 + g, bt);
          }
          bulk_load_1d(sVec + st * 128, a.lse2 + (size_t)bhq * vec_stride + pbase + q0, 256, bar_ld_full + st);
          bulk_load_1d(sVec + st * 128 + 64, a.delta + (size_t)bhq * vec_stride + pbase + q0, 256, bar_ld_full + st);
          if (++t_in == cnt) { t_in = 0; ++g; }
          if (++st == NST) { st = 0; if (n >= NST) ph_e ^= 1; }
        }
      }
    } else if (warp == 1) {
      // ================= MMA issuer =================
      // The whole warp runs this loop (uniform control flow, so that descriptors and counters stay in
      // uniform registers); only the elected lane executes the tcgen05 instructions.  Everything that
      // can be computed once is: descriptor of every operand base, stage and parity bookkeeping is
      // incremental, and the loop body is instantiated for both TMEM buffers.
      if (N > 0) {
        const bool lead = elect_one();
        const uint32_t tb = tmem_base;
        // Descriptors: a byte offset o inside a tile is added as o >> 4 to the address field (bits 0-13);
        // no tile crosses the field's range, so the 64-bit add never carries out of it.
        const uint64_t dK_k = smem_desc_sw128(smem_u32(sK), 16, 1024);                       // K, K-major (A of S^T)
        const uint64_t dV_k = smem_desc_sw128(smem_u32(sV), 16, 1024);                       // V, K-major (A of dP^T)
        const uint64_t dK_mn = smem_desc_sw128(smem_u32(sK), D == 128 ? SLAB_KV : 0, 1024);  // K^T, MN-major (A of dQ^T)
        const uint64_t dQ_k0 = smem_desc_sw128(smem_u32(sStage), 16, 1024);                  // Q of stage 0, K-major (B of S^T)
        const uint64_t dO_k0 = smem_desc_sw128(smem_u32(sStage) + SM::kQS, 16, 1024);        // dO of stage 0, K-major (B of dP^T)
        const uint64_t dQ_mn0 = smem_desc_sw128(smem_u32(sStage), SLAB_QS, 1024);            // Q, MN-major (B of dK)
        const uint64_t dO_mn0 = smem_desc_sw128(smem_u32(sStage) + SM::kQS, SLAB_QS, 1024);  // dO, MN-major (B of dV)
        const uint64_t dDS0 = smem_desc_sw128(smem_u32(sDS), 0, 1024);                       // dS^T, MN-major (B of dQ^T)
        constexpr uint32_t kStage16 = SM::kStage >> 4, kDS16 = SM::kDS >> 4;

        auto gemm_st = [&](uint32_t d_col, uint64_t dA, uint64_t dB) {  // [128 x 64] = A[128 x D] B[64 x D]^T
          if (lead) {
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk)
              mma_ss(tb + d_col, dA + (((kk / 4) * SLAB_KV + (kk % 4) * 32) >> 4),
                     dB + (((kk / 4) * SLAB_QS + (kk % 4) * 32) >> 4), ID_ST, kk > 0);
          }
        };
        auto gemm_acc = [&](uint32_t d_col, uint32_t a_col, uint64_t dB, uint32_t acc_first) {  // [128 x D] += A(TMEM) B
          if (lead) {
#pragma unroll
            for (int kk = 0; kk < BQS / 16; ++kk)
              mma_ts(tb + d_col, tb + a_col + (kk >> 1) * 32 + (kk & 1) * 8, dB + ((kk * 2048) >> 4), ID_ACC, kk > 0 ? 1u : acc_first);
          }
        };
        auto gemm_dq = [&](uint32_t d_col, uint64_t dB) {  // dQ^T[D x 64] = K^T dS^T
          if (lead) {
#pragma unroll
            for (int kk = 0; kk < BKV / 16; ++kk)
              mma_ss(tb + d_col, dK_mn + ((kk * 2048) >> 4), dB + ((kk * 2048) >> 4), ID_DQ, kk > 0);
          }
        };
        auto commit = [&](uint64_t* bar) {
          if (lead) mma_commit(bar);
        };

        // Packed batches: rows of a tile that lie past the end of the sequence belong to the next one.  Every
        // product they enter is multiplied by an exact zero, but 0 x (Inf or NaN) would still poison this
        // sequence, so they are cleared in shared memory (whole 128-byte rows, by this warp) before use.
        auto clear_rows = [&](uint8_t* tile, int first, int rows, int slab_bytes) {
          const int nchunk = (rows - first) * 8;  // 16-byte chunks per slab
          for (int s_ = 0; s_ < NSLAB; ++s_)
            for (int c_ = lane; c_ < nchunk; c_ += 32)
              *reinterpret_cast<uint4*>(tile + s_ * slab_bytes + first * 128 + c_ * 16) = make_uint4(0u, 0u, 0u, 0u);
        };
        int t_clr = 0;  // position in I_h(j) of the next step whose Q / dO stage is checked (packed batches only)
        auto clear_stage_tail = [&](int stage) {
          if constexpr (VARLEN) {
            const int q0_ = cowa_bwd_tile_at(rg, t_clr) * BQS;
            if (++t_clr == cnt) t_clr = 0;
            if (q0_ + BQS > Nq) {
              uint8_t* sQ_ = sStage + stage * SM::kStage;
              clear_rows(sQ_, Nq - q0_, BQS, SLAB_QS);
              clear_rows(sQ_ + SM::kQS, Nq - q0_, BQS, SLAB_QS);
              fence_proxy_async_smem();
              __syncwarp();
            }
          }
        };
        ok = mbar_wait(bar_kv, 0, a.status);
        if (ok && tail_kv) {
          clear_rows(sK, Nk - k0, BKV, SLAB_KV);
          clear_rows(sV, Nk - k0, BKV, SLAB_KV);
          fence_proxy_async_smem();
          __syncwarp();
        }
        // prologue: S^T(0), dP^T(0), S^T(1)
        ok = ok && mbar_wait(bar_ld_full + 0, 0, a.status);
        if (ok) {
          clear_stage_tail(0);
          tc_fence_after();
          gemm_st(cS0, dK_k, dQ_k0);
          commit(bar_s_full + 0);
          gemm_st(cDP0, dV_k, dO_k0);
          commit(bar_dp_full + 0);
        }
        if (ok && N > 1) {
          ok = mbar_wait(bar_ld_full + 1, 0, a.status);
          if (ok) {
            clear_stage_tail(1);
            tc_fence_after();
            gemm_st(cS0 + 64, dK_k, dQ_k0 + kStage16);
            commit(bar_s_full + 1);
          }
        }
        // Step n uses TMEM buffer b = n & 1 (the two compute warpgroups alternate steps).  Issue order:
        //   dV(n) | dP^T(n+1) | dK(n) | S^T(n+2) | dQ^T(n)
        // so that every wait below is for something produced about one step earlier.
        int st = 0, st1 = (N > 1) ? 1 : 0, st2 = 2 % NST;    // stages of steps n, n+1, n+2
        uint32_t ph2 = (2 / NST) & 1;                        // parity of the load that fills stage st2 for step n+2
        uint32_t par = 0;                                    // (n >> 1) & 1
        auto body = [&](int n, auto B_) {
          constexpr int b_ = decltype(B_)::value;
          constexpr uint32_t sbuf = cS0 + b_ * 64, dpbuf = cDP0 + b_ * 64, dpother = cDP0 + (b_ ^ 1) * 64;
          ok = mbar_wait(bar_p_ready + b_, par, a.status);
          if (!ok) return;
          tc_fence_after();
          gemm_acc(cDV, sbuf, dO_mn0 + st * kStage16, n > 0 ? 1u : 0u);     // dV += P^T dO
          if (n + 1 < N) {                                                  // dP^T(n+1), once dQ^T(n-1) has left its buffer
            if (n >= 1) {
              ok = mbar_wait(bar_dq_free + (b_ ^ 1), ((n - 1) >> 1) & 1, a.status);
              if (!ok) return;
              tc_fence_after();
            }
            gemm_st(dpother, dV_k, dO_k0 + st1 * kStage16);
            commit(bar_dp_full + (b_ ^ 1));
          }
          ok = mbar_wait(bar_ds_ready + b_, par, a.status);
          if (!ok) return;
          tc_fence_after();
          gemm_acc(cDK, sbuf + 16, dQ_mn0 + st * kStage16, n > 0 ? 1u : 0u);  // dK += dS^T Q
          commit(bar_ld_empty + st);
          if (n + 2 < N) {                                                  // S^T(n+2) into the buffer P^T(n), dS^T(n) just left:
            ok = mbar_wait(bar_ld_full + st2, ph2, a.status);               // it heads the next step's dependency chain, so it
            if (!ok) return;                                                // goes ahead of dQ^T(n), which only feeds the drain
            clear_stage_tail(st2);
            tc_fence_after();
            gemm_st(sbuf, dK_k, dQ_k0 + st2 * kStage16);
            commit(bar_s_full + b_);
          }
          gemm_dq(dpbuf, dDS0 + b_ * kDS16);                                // dQ^T = K^T dS^T over the consumed dP^T(n)
          commit(bar_dq_full + b_);
          // advance the bookkeeping to step n+1
          st = st1; st1 = st2;
          if (++st2 == NST) { st2 = 0; ph2 ^= 1; }
          if (b_ == 1) par ^= 1;
        };
        for (int n = 0; n < N && ok; n += 2) {
          body(n, std::integral_constant<int, 0>{});
          if (n + 1 < N && ok) body(n + 1, std::integral_constant<int, 1>{});
        }
        commit(bar_done);
      }
    }
  } else if (warp < 12) {
    setmaxnreg_inc<176>();
    {
      // ======== two compute warpgroups, each takes 32 of the 64 query columns of every step: P^T and dS^T, one
      // KV row per thread.  Inside the 64-column S^T buffer a warpgroup only ever writes into the 32 columns
      // it reads: P^T (bf16 pairs) into the first 16 of them, dS^T into the last 16.
      const int wg = (warp - 4) >> 2;        // query columns [32 wg, 32 wg + 32) of every step
      const int r = (warp & 3) * 32 + lane;  // KV row = TMEM lane
      const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
      const int kcol = k0 + r;               // key index of this thread
      const long long kpos = (long long)kcol - off;  // first causal query of this key
      const float2 sc2 = make_float2(a.scale_log2, a.scale_log2);
      int st = 0, t_in = 0;                  // stage and position in I_h(j) of the next step
      uint32_t ph_l = 0, par = 0;
      for (int n = 0; n < N && ok; ++n) {
        const int b_ = n & 1;
        const uint32_t sbuf = t_lane + cS0 + b_ * 64 + wg * 32, dpbuf = t_lane + cDP0 + b_ * 64 + wg * 32;
        uint8_t* ds_row = sDS + b_ * SM::kDS + r * 128;
        const int i = cowa_bwd_tile_at(rg, t_in);
        const int q0 = i * BQS;
        const bool full = cowa_tile_full(w, q0, BQS, k0, BKV, off, Nq, Nk);
        uint32_t mk = 0xFFFFFFFFu;
        if (!full) {
          const long long qend = Nq - 1;
          const long long base = q0 + wg * 32;
          uint32_t m = interval_bits32(kpos, min(kpos + w.n - 1, qend), base);
          if (w.l > 0)
            m |= interval_bits32(kpos + w.n + w.g, min(kpos + (long long)w.n + w.g + w.l - 1, qend), base);
          if (kcol < w.s) m |= interval_bits32(kpos, qend, base);
          mk = kcol < Nk ? m : 0u;
        }
        const float* lse2 = sVec + st * 128 + wg * 32;
        const float* dlt = lse2 + 64;
        ok = mbar_wait(bar_ld_full + st, ph_l, a.status);
        ok = ok && mbar_wait(bar_s_full + b_, par, a.status);
        if (!ok) break;
        tc_fence_after();
        float p[32];
        {
          uint32_t sr[32], pk[16];
          tmem_ld32(sbuf, sr);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const float2 x = fma2(make_float2(__uint_as_float(sr[e]), __uint_as_float(sr[e + 1])), sc2,
                                  make_float2(-lse2[e], -lse2[e + 1]));
            p[e] = ex2(x.x);
            p[e + 1] = ex2(x.y);
          }
          if (!full) {
#pragma unroll
            for (int e = 0; e < 32; ++e)
              if (!((mk >> e) & 1u)) p[e] = 0.f;
          }
#pragma unroll
          for (int e = 0; e < 32; e += 2) pk[e / 2] = pack_bf16(p[e], p[e + 1]);
          tmem_st16(sbuf, pk);  // P^T: this warpgroup's 32 queries as 16 bf16 pairs
        }
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar_p_ready + b_);

        ok = mbar_wait(bar_dp_full + b_, par, a.status);
        if (!ok) break;
        tc_fence_after();
        {
          uint32_t dr[32], dsp[16];
          tmem_ld32(dpbuf, dr);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const float2 y = add2(make_float2(__uint_as_float(dr[e]), __uint_as_float(dr[e + 1])),
                                  make_float2(-dlt[e], -dlt[e + 1]));
            const float2 z = mul2(make_float2(p[e], p[e + 1]), y);
            dsp[e / 2] = pack_bf16(z.x, z.y);
          }
          tmem_st16(sbuf + 16, dsp);  // dS^T beside P^T
          // dS^T also to shared memory (row r = 128 B = 8 chunks, 128B swizzle) for the dQ^T product
#pragma unroll
          for (int ch = 0; ch < 4; ++ch)
            *reinterpret_cast<uint4*>(ds_row + (((wg * 4 + ch) ^ (r & 7)) << 4)) =
                make_uint4(dsp[ch * 4], dsp[ch * 4 + 1], dsp[ch * 4 + 2], dsp[ch * 4 + 3]);
        }
        tmem_wait_st();
        tc_fence_before();
        fence_proxy_async_smem();
        mbar_arrive(bar_ds_ready + b_);
        if (b_) par ^= 1;
        if (++st == NST) { st = 0; ph_l ^= 1; }
        if (++t_in == cnt) t_in = 0;
      }
      if (wg == 0) store_grad(true);
    }
  } else {
    setmaxnreg_dec<96>();
    {
      // ======== dQ drain warpgroup: one d column of dQ^T per thread; TMEM -> shared -> bulk reduce-add ========
      const int d = (warp & 3) * 32 + lane;
      const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
      const bool issuer = (d == 0);
      int g = 0, t_in = 0;
      for (int n = 0; n < N && ok; ++n) {
        const int i = cowa_bwd_tile_at(rg, t_in);
        const int bhq = bhq0 + g, q0 = i * BQS;
        if (++t_in == cnt) { t_in = 0; ++g; }
        ok = mbar_wait(bar_dq_full + (n & 1), (n >> 1) & 1, a.status);
        if (!ok) break;
        tc_fence_after();
        uint32_t v[2][32];
        tmem_ld32(t_lane + cDP0 + (n & 1) * 64, v[0]);
        tmem_ld32(t_lane + cDP0 + (n & 1) * 64 + 32, v[1]);
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive(bar_dq_free + (n & 1));
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          float* stage = sDQ + hf * (SM::kDQ / 4);
          if (issuer) tma_wait_group_read<1>();  // the reduction issued from this tile one step ago has read it
          wg_sync(3);
          if (d < D) {
            if (a.dq_fixed) {
              const float fx = a.scale * kDqFixedOne;
              bool out_of_range = false;
#pragma unroll
              for (int c = 0; c < 32; ++c) {
                const float x = __uint_as_float(v[hf][c]) * fx;
                out_of_range |= !(fabsf(x) < 2147483520.f);  // the conversion would saturate (or x is not a number)
                reinterpret_cast<int*>(stage)[c * D + d] = __float2int_rn(x);
              }
              if (out_of_range) atomicOr(a.status, (unsigned)COWA_DEV_DQ_RANGE);
            } else {
#pragma unroll
              for (int c = 0; c < 32; ++c) stage[c * D + d] = __uint_as_float(v[hf][c]) * a.scale;
            }
          }
          fence_proxy_async_smem();
          wg_sync(3);
          if (issuer) {
            // 32 query rows of the accumulator are one contiguous range (rows are D floats, padded row space)
            void* gdst = a.dq_acc + (((size_t)bhq * vec_stride + pbase + q0 + hf * 32) * D);
            if (a.dq_fixed) bulk_reduce_add_s32(gdst, stage, 32 * D * 4);
            else bulk_reduce_add_f32(gdst, stage, 32 * D * 4);
            tma_commit_group();
          }
        }
      }
      if (issuer) tma_wait_group<0>();
      store_grad(false);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    __syncwarp();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// Delta = rowsum(O * dO), lse2 = LSE * log2(e); rows in [T, Tpad) get lse2 = +inf, Delta = 0.
template <int D>
__global__ void cowa_bwd_preprocess_kernel(const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ d_o,
                                           const float* __restrict__ lse, float* __restrict__ lse2,
                                           float* __restrict__ delta, int T, int Tpad, long long BH, int H,
                                           CowaStrides so) {
  constexpr int TPR = D / 8;  // threads per row (16 bytes each)
  const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long row = gid / TPR;
  const int part = (int)(gid % TPR);
  if (row >= BH * Tpad) return;
  const long long bh = row / Tpad;
  const int t = (int)(row % Tpad);
  float s = 0.f;
  if (t < T) {
    const size_t base = (size_t)(bh / H) * so.b + (size_t)(bh % H) * so.h + (size_t)t * so.t + part * 8;
    const uint4 x = *reinterpret_cast<const uint4*>(o + base);
    const uint4 y = *reinterpret_cast<const uint4*>(d_o + base);
    const uint32_t xs[4] = {x.x, x.y, x.z, x.w}, ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      s = fmaf(__uint_as_float(xs[i] << 16), __uint_as_float(ys[i] << 16), s);
      s = fmaf(__uint_as_float(xs[i] & 0xffff0000u), __uint_as_float(ys[i] & 0xffff0000u), s);
    }
  }
#pragma unroll
  for (int o_ = TPR / 2; o_ > 0; o_ >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o_);
  if (part == 0) {
    delta[row] = s;
    lse2[row] = t < T ? lse[(size_t)bh * T + t] * 1.4426950408889634f : INFINITY;
  }
}

template <int D>
__global__ void cowa_bwd_convert_dq_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ dq, int T,
                                           int Tpad, long long BH, int fixed, int H, CowaStrides sq,
                                           unsigned int* status) {
  const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;  // one thread per 8 elements
  const long long total = BH * T * (D / 8);
  if (gid >= total) return;
  const long long row = gid / (D / 8);
  const int part = (int)(gid % (D / 8));
  const long long bh = row / T;
  const int t = (int)(row % T);
  const float4* src = reinterpret_cast<const float4*>(acc + ((size_t)bh * Tpad + t) * D + part * 8);
  float4 x = src[0], y = src[1];
  if (fixed) {  // the accumulator holds 32-bit integers in units of 2^-18
    const float u = 1.f / kDqFixedOne;
    x = make_float4(__float_as_int(x.x) * u, __float_as_int(x.y) * u, __float_as_int(x.z) * u, __float_as_int(x.w) * u);
    y = make_float4(__float_as_int(y.x) * u, __float_as_int(y.y) * u, __float_as_int(y.z) * u, __float_as_int(y.w) * u);
    // half of the representable range: a total that wrapped around lands out here in most cases
    const float big = fmaxf(fmaxf(fmaxf(fabsf(x.x), fabsf(x.y)), fmaxf(fabsf(x.z), fabsf(x.w))),
                            fmaxf(fmaxf(fabsf(y.x), fabsf(y.y)), fmaxf(fabsf(y.z), fabsf(y.w))));
    if (big >= 4096.f) atomicOr(status, (unsigned)COWA_DEV_DQ_RANGE);
  }
  uint4 v;
  v.x = pack_bf16(x.x, x.y); v.y = pack_bf16(x.z, x.w); v.z = pack_bf16(y.x, y.y); v.w = pack_bf16(y.z, y.w);
  *reinterpret_cast<uint4*>(dq + (size_t)(bh / H) * sq.b + (size_t)(bh % H) * sq.h + (size_t)t * sq.t + part * 8) = v;
}

// Packed batches.  One block per (64-row chunk of the padded row space, QO head): Delta and LSE * log2(e)
// of the chunk's rows (padding rows: +inf, 0), read from the packed tensors.
template <int D>
__global__ void cowa_bwd_preprocess_varlen_kernel(const __nv_bfloat16* __restrict__ o,
                                                  const __nv_bfloat16* __restrict__ d_o,
                                                  const float* __restrict__ lse, float* __restrict__ lse2,
                                                  float* __restrict__ delta, const int* __restrict__ cu, int B,
                                                  int total, int Tpad) {
  constexpr int TPR = D / 8;  // threads per row (16 bytes each)
  const int chunk = blockIdx.x, h = blockIdx.y;
  const int r = threadIdx.x / TPR, part = threadIdx.x % TPR;
  int b, lc, nch, pb;
  const bool in = varlen_locate(cu, B, chunk, BQS, BQS, &b, &lc, &nch, &pb);
  const int t = lc * BQS + r;  // row inside the sequence
  const int rbase = in ? cu[b] : 0;
  const bool valid = in && t < cu[b + 1] - rbase && rbase >= 0 && rbase + t < total;
  float s = 0.f;
  if (valid) {
    const size_t base = ((size_t)h * total + rbase + t) * D + part * 8;
    const uint4 x = *reinterpret_cast<const uint4*>(o + base);
    const uint4 y = *reinterpret_cast<const uint4*>(d_o + base);
    const uint32_t xs[4] = {x.x, x.y, x.z, x.w}, ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      s = fmaf(__uint_as_float(xs[i] << 16), __uint_as_float(ys[i] << 16), s);
      s = fmaf(__uint_as_float(xs[i] & 0xffff0000u), __uint_as_float(ys[i] & 0xffff0000u), s);
    }
  }
#pragma unroll
  for (int o_ = TPR / 2; o_ > 0; o_ >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o_);
  if (part == 0) {
    const size_t row = (size_t)h * Tpad + (size_t)chunk * BQS + r;  // chunks are laid out in order: pb == chunk * BQS
    delta[row] = s;
    lse2[row] = valid ? lse[(size_t)h * total + rbase + t] * 1.4426950408889634f : INFINITY;
  }
}

// Packed batches: fp32 (or fixed-point) dQ accumulator in the padded row space -> bf16 dq in the packed one.
template <int D>
__global__ void cowa_bwd_convert_dq_varlen_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ dq,
                                                  const int* __restrict__ cu, int B, int total, int Tpad, int fixed,
                                                  unsigned int* status) {
  constexpr int TPR = D / 8;
  const int chunk = blockIdx.x, h = blockIdx.y;
  const int r = threadIdx.x / TPR, part = threadIdx.x % TPR;
  int b, lc, nch, pb;
  if (!varlen_locate(cu, B, chunk, BQS, BQS, &b, &lc, &nch, &pb)) return;
  const int t = lc * BQS + r;
  const int rbase = cu[b];
  if (t >= cu[b + 1] - rbase || rbase < 0 || rbase + t >= total) return;
  const float4* src = reinterpret_cast<const float4*>(acc + ((size_t)h * Tpad + (size_t)chunk * BQS + r) * D + part * 8);
  float4 x = src[0], y = src[1];
  if (fixed) {
    const float u = 1.f / kDqFixedOne;
    x = make_float4(__float_as_int(x.x) * u, __float_as_int(x.y) * u, __float_as_int(x.z) * u, __float_as_int(x.w) * u);
    y = make_float4(__float_as_int(y.x) * u, __float_as_int(y.y) * u, __float_as_int(y.z) * u, __float_as_int(y.w) * u);
    const float big = fmaxf(fmaxf(fmaxf(fabsf(x.x), fabsf(x.y)), fmaxf(fabsf(x.z), fabsf(x.w))),
                            fmaxf(fmaxf(fabsf(y.x), fabsf(y.y)), fmaxf(fabsf(y.z), fabsf(y.w))));
    if (big >= 4096.f) atomicOr(status, (unsigned)COWA_DEV_DQ_RANGE);
  }
  uint4 v;
  v.x = pack_bf16(x.x, x.y); v.y = pack_bf16(x.z, x.w); v.z = pack_bf16(y.x, y.y); v.w = pack_bf16(y.z, y.w);
  *reinterpret_cast<uint4*>(dq + ((size_t)h * total + rbase + t) * D + part * 8) = v;
}

// Sum of the per-block partial dK, dV (heads of a group spread over `parts` blocks), in slot order, to bf16.
template <int D>
__global__ void cowa_bwd_reduce_dkv_kernel(const float* __restrict__ part, __nv_bfloat16* __restrict__ dk,
                                           __nv_bfloat16* __restrict__ dv, int T, int nKV, int parts, long long BHk,
                                           int H, CowaStrides sk, CowaStrides sv) {
  const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;  // one thread per 8 elements of dK and dV
  const long long total = BHk * nKV * BKV * (D / 8);
  if (gid >= total) return;
  const int ch = (int)(gid % (D / 8));
  const int r = (int)((gid / (D / 8)) % BKV);
  const long long tile = gid / ((D / 8) * BKV);  // bhk * nKV + j
  const int j = (int)(tile % nKV);
  const long long bhk = tile / nKV;
  const int t = j * BKV + r;
  if (t >= T) return;
  float acc[2][8];
#pragma unroll
  for (int m = 0; m < 2; ++m)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[m][e] = 0.f;
  for (int pi = 0; pi < parts; ++pi)
#pragma unroll
    for (int m = 0; m < 2; ++m) {
      const float4* src = reinterpret_cast<const float4*>(part + (((size_t)tile * parts + pi) * 2 + m) * (size_t)(BKV * D) +
                                                          (size_t)r * D + ch * 8);
      const float4 x = src[0], y = src[1];
      acc[m][0] += x.x; acc[m][1] += x.y; acc[m][2] += x.z; acc[m][3] += x.w;
      acc[m][4] += y.x; acc[m][5] += y.y; acc[m][6] += y.z; acc[m][7] += y.w;
    }
#pragma unroll
  for (int m = 0; m < 2; ++m) {
    uint4 v;
    v.x = pack_bf16(acc[m][0], acc[m][1]); v.y = pack_bf16(acc[m][2], acc[m][3]);
    v.z = pack_bf16(acc[m][4], acc[m][5]); v.w = pack_bf16(acc[m][6], acc[m][7]);
    const CowaStrides& sg = m == 0 ? sk : sv;
    *reinterpret_cast<uint4*>((m == 0 ? dk : dv) + (size_t)(bhk / H) * sg.b + (size_t)(bhk % H) * sg.h + (size_t)t * sg.t + ch * 8) = v;
  }
}

// Blocks per KV tile.  A block normally takes the whole GQA group of its KV tile (dK, dV then never leave
// TMEM).  That starves the GPU when B * Hkv * tiles is small, and it makes the sink tiles -- visited by
// every query tile of every head -- the critical path when Hkv is small; in both cases the group's heads
// are spread over `parts` blocks (a divisor of G), chosen as the smallest that gives two waves of
// blocks and keeps the longest block under 3/4 of an even share of the work.
int sm_count() {
  static int cached = 0;
  if (cached == 0) {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess &&
        n > 0)
      cached = n;
    else {
      cudaGetLastError();
      return 148;  // B200; used when no device can be queried (workspace sizing on a machine without a GPU)
    }
  }
  return cached;
}

int bwd_parts(int B, int Nq, int Nk, int Hkv, int G, const CowaHeadWindows& hw) {
  const int nKV = (Nk + BKV - 1) / BKV;
  long long total = 0, longest = 0;
  for (int h = 0; h < Hkv; ++h)
    for (int j = 0; j < nKV; ++j) {
      CowaRange rg[2];
      const int k0 = j * BKV, k1 = std::min(k0 + BKV, Nk) - 1;
      cowa_bwd_ranges(hw.w[h], k0, k1, Nk - Nq, Nq, BQS, rg);
      const long long cnt = cowa_range_len(rg[0]) + cowa_range_len(rg[1]);
      total += cnt;
      longest = std::max(longest, cnt);
    }
  total *= (long long)B * G;
  longest *= G;
  const long long blocks = (long long)B * Hkv * nKV;
  const int kSMs = sm_count();
  for (int p = 1; p < G; ++p) {
    if (G % p) continue;
    if (blocks * p >= 2 * kSMs && longest * 4 * kSMs <= 3 * total * p) return p;
  }
  return G;
}

size_t part_bytes(int B, int Nk, int Hkv, int D, int parts) {
  if (parts <= 1) return 0;
  return (size_t)B * Hkv * ((Nk + BKV - 1) / BKV) * parts * 2 * BKV * D * sizeof(float);
}

size_t ws_bytes(int B, int Nq, int Nk, int Hq, int Hkv, int D, int parts) {
  const size_t Tpad = ((size_t)Nq + BQS - 1) / BQS * BQS;
  return (size_t)B * Hq * Tpad * ((size_t)D + 2) * sizeof(float) + part_bytes(B, Nk, Hkv, D, parts);
}

// Contiguous [H, T, D] (x batch) strides.
CowaStrides packed_strides(int H, long long T, int D) {
  CowaStrides st;
  st.t = D; st.h = T * D; st.b = (long long)H * T * D;
  return st;
}

template <int D>
int launch_bwd(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o,
               void* dq, void* dk, void* dv, int B, int Nq, int Nk, int Hq, int Hkv, const cowa_params_t* p,
               const CowaHeadWindows& hw, int parts, void* ws, cudaStream_t st) {
  const int T = Nq;  // rows of q, o, d_o, dq, lse
  const int Tpad = (T + BQS - 1) / BQS * BQS;
  const long long BH = (long long)B * Hq;
  float* dq_acc = static_cast<float*>(ws);
  float* lse2 = dq_acc + (size_t)BH * Tpad * D;
  float* delta = lse2 + (size_t)BH * Tpad;
  float* dkv_part = delta + (size_t)BH * Tpad;
  // Everything that can fail is done before the first launch: strides, tensor maps, the status word.
  int rc;
  CowaStrides sq, sk, sv, so;
  if ((rc = cowa::resolve_strides(p->q_strides, Hq, Nq, D, &sq))) return rc;
  if ((rc = cowa::resolve_strides(p->k_strides, Hkv, Nk, D, &sk))) return rc;
  if ((rc = cowa::resolve_strides(p->v_strides, Hkv, Nk, D, &sv))) return rc;
  if ((rc = cowa::resolve_strides(p->o_strides, Hq, Nq, D, &so))) return rc;
  if (BH > 0x7FFFFFFFll) return COWA_ERR_UNSUPPORTED;
  CUtensorMap mq, mk, mv, mdo, mdk, mdv;
  if ((rc = cowa::make_tensor_map(&mq, q, cowa::MapType::BF16, D, T, Hq, B, sq, 64, BQS))) return rc;
  if ((rc = cowa::make_tensor_map(&mdo, d_o, cowa::MapType::BF16, D, T, Hq, B, so, 64, BQS))) return rc;
  if ((rc = cowa::make_tensor_map(&mk, k, cowa::MapType::BF16, D, Nk, Hkv, B, sk, 64, BKV))) return rc;
  if ((rc = cowa::make_tensor_map(&mv, v, cowa::MapType::BF16, D, Nk, Hkv, B, sv, 64, BKV))) return rc;
  if ((rc = cowa::make_tensor_map(&mdk, dk, cowa::MapType::BF16, D, Nk, Hkv, B, sk, 64, BKV))) return rc;
  if ((rc = cowa::make_tensor_map(&mdv, dv, cowa::MapType::BF16, D, Nk, Hkv, B, sv, 64, BKV))) return rc;
  BwdArgs a;
  a.lse2 = lse2; a.delta = delta; a.dq_acc = dq_acc;
  a.status = cowa::device_status_word();
  if (!a.status) return COWA_ERR_CUDA;
  a.B = B; a.Nq = Nq; a.Nk = Nk; a.Hq = Hq; a.Hkv = Hkv; a.G = Hq / Hkv; a.Tpad = Tpad;
  a.scale = p->softmax_scale;
  a.scale_log2 = p->softmax_scale * 1.4426950408889634f;
  a.wins = hw;
  a.sink_tiles = 0;
  a.dq_fixed = p->deterministic ? 1 : 0;
  a.parts = parts; a.dkv_part = dkv_part;
  a.cu = nullptr; a.dk = nullptr; a.dv = nullptr; a.total = 0; a.tiles_bound = 0;
  a.sink = 0; a.local = 0; a.hkv_global = 0; a.hkv_offset = 0; a.full_attn = 0; a.explicit_windows = 0;
  for (int h = 0; h < Hkv; ++h) {
    const int sk_ = hw.w[h].s < Nk ? hw.w[h].s : Nk;
    a.sink_tiles = std::max(a.sink_tiles, (sk_ + BKV - 1) / BKV);
  }
  const long long nblocks = (long long)((Nk + BKV - 1) / BKV) * B * Hkv * parts;
  if (nblocks > 0x7FFFFFFFll) return COWA_ERR_UNSUPPORTED;
  COWA_CUDA_TRY(cudaFuncSetAttribute(cowa_bwd_kernel<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     BwdSmem<D>::kBytes));
  COWA_CUDA_TRY(cudaMemsetAsync(dq_acc, 0, (size_t)BH * Tpad * D * sizeof(float), st));
  {
    const long long threads = BH * Tpad * (D / 8);
    cowa_bwd_preprocess_kernel<D><<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(
        static_cast<const __nv_bfloat16*>(o), static_cast<const __nv_bfloat16*>(d_o), lse, lse2, delta, T, Tpad, BH, Hq, so);
    COWA_CUDA_TRY(cudaGetLastError());
  }
  if (p->bwd_main_start_event) COWA_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(p->bwd_main_start_event), st));
  cowa_bwd_kernel<D, false><<<(unsigned)nblocks, 512, BwdSmem<D>::kBytes, st>>>(mq, mk, mv, mdo, mdk, mdv, a);
  COWA_CUDA_TRY(cudaGetLastError());
  if (p->bwd_main_stop_event) COWA_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(p->bwd_main_stop_event), st));
  {
    const long long threads = BH * T * (D / 8);
    cowa_bwd_convert_dq_kernel<D><<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(
        dq_acc, static_cast<__nv_bfloat16*>(dq), T, Tpad, BH, p->deterministic ? 1 : 0, Hq, sq, a.status);
    COWA_CUDA_TRY(cudaGetLastError());
  }
  if (parts > 1) {
    const int nKV = (Nk + BKV - 1) / BKV;
    const long long threads = (long long)B * Hkv * nKV * BKV * (D / 8);
    cowa_bwd_reduce_dkv_kernel<D><<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(
        dkv_part, static_cast<__nv_bfloat16*>(dk), static_cast<__nv_bfloat16*>(dv), Nk, nKV, parts, (long long)B * Hkv,
        Hkv, sk, sv);
    COWA_CUDA_TRY(cudaGetLastError());
  }
  return COWA_OK;
}

// Padded row space of a packed batch: every sequence rounded up to 64 rows; the bound needs no lengths.
int varlen_tpad(int B, int total) { return (total / BQS + B) * BQS; }

size_t ws_bytes_varlen(int B, int total, int Hq, int D) {
  return (size_t)Hq * varlen_tpad(B, total) * ((size_t)D + 2) * sizeof(float);
}

template <int D>
int launch_bwd_varlen(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o,
                      void* dq, void* dk, void* dv, const int* cu, int B, int total, int Hq, int Hkv,
                      const cowa_params_t* p, const CowaHeadWindows& hw, void* ws, cudaStream_t st) {
  const int Tpad = varlen_tpad(B, total);
  float* dq_acc = static_cast<float*>(ws);
  float* lse2 = dq_acc + (size_t)Hq * Tpad * D;
  float* delta = lse2 + (size_t)Hq * Tpad;
  if (cowa::any_stride_set(p)) return COWA_ERR_UNSUPPORTED;  // packed tensors are contiguous [H, total, D]
  CUtensorMap mq, mk, mv, mdo, mdk, mdv;
  int rc;
  const CowaStrides sq = packed_strides(Hq, total, D), sk = packed_strides(Hkv, total, D);
  if ((rc = cowa::make_tensor_map(&mq, q, cowa::MapType::BF16, D, total, Hq, 1, sq, 64, BQS))) return rc;
  if ((rc = cowa::make_tensor_map(&mdo, d_o, cowa::MapType::BF16, D, total, Hq, 1, sq, 64, BQS))) return rc;
  if ((rc = cowa::make_tensor_map(&mk, k, cowa::MapType::BF16, D, total, Hkv, 1, sk, 64, BKV))) return rc;
  if ((rc = cowa::make_tensor_map(&mv, v, cowa::MapType::BF16, D, total, Hkv, 1, sk, 64, BKV))) return rc;
  if ((rc = cowa::make_tensor_map(&mdk, dk, cowa::MapType::BF16, D, total, Hkv, 1, sk, 64, BKV))) return rc;
  if ((rc = cowa::make_tensor_map(&mdv, dv, cowa::MapType::BF16, D, total, Hkv, 1, sk, 64, BKV))) return rc;
  BwdArgs a;
  a.lse2 = lse2; a.delta = delta; a.dq_acc = dq_acc;
  a.status = cowa::device_status_word();
  if (!a.status) return COWA_ERR_CUDA;
  a.B = B; a.Nq = 0; a.Nk = 0; a.Hq = Hq; a.Hkv = Hkv; a.G = Hq / Hkv; a.Tpad = Tpad;
  a.scale = p->softmax_scale;
  a.scale_log2 = p->softmax_scale * 1.4426950408889634f;
  a.wins = hw;
  a.sink_tiles = 0;  // KV tiles per sequence that hold sink columns (launched first)
  if (!p->full_attn)
    for (int h = 0; h < Hkv; ++h) {
      const int sk_ = std::min(p->windows ? hw.w[h].s : p->sink, total);
      a.sink_tiles = std::max(a.sink_tiles, (sk_ + BKV - 1) / BKV);
    }
  a.dq_fixed = p->deterministic ? 1 : 0;
  a.parts = 1; a.dkv_part = nullptr;
  a.cu = cu; a.dk = static_cast<__nv_bfloat16*>(dk); a.dv = static_cast<__nv_bfloat16*>(dv);
  a.total = total; a.tiles_bound = total / BKV + B;
  a.sink = p->sink; a.local = p->local;
  a.hkv_global = p->hkv_global > 0 ? p->hkv_global : Hkv;
  a.hkv_offset = p->hkv_offset; a.full_attn = p->full_attn; a.explicit_windows = p->windows != nullptr;
  const long long nblocks = (long long)a.tiles_bound * Hkv + (long long)a.sink_tiles * B * Hkv;
  if (nblocks > 0x7FFFFFFFll) return COWA_ERR_UNSUPPORTED;
  COWA_CUDA_TRY(cudaFuncSetAttribute(cowa_bwd_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     BwdSmem<D>::kBytes));
  COWA_CUDA_TRY(cudaMemsetAsync(dq_acc, 0, (size_t)Hq * Tpad * D * sizeof(float), st));
  const dim3 chunks(Tpad / BQS, Hq);
  cowa_bwd_preprocess_varlen_kernel<D><<<chunks, BQS * (D / 8), 0, st>>>(
      static_cast<const __nv_bfloat16*>(o), static_cast<const __nv_bfloat16*>(d_o), lse, lse2, delta, cu, B, total, Tpad);
  COWA_CUDA_TRY(cudaGetLastError());
  if (p->bwd_main_start_event) COWA_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(p->bwd_main_start_event), st));
  cowa_bwd_kernel<D, true><<<(unsigned)nblocks, 512, BwdSmem<D>::kBytes, st>>>(mq, mk, mv, mdo, mdk, mdv, a);
  COWA_CUDA_TRY(cudaGetLastError());
  if (p->bwd_main_stop_event) COWA_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(p->bwd_main_stop_event), st));
  cowa_bwd_convert_dq_varlen_kernel<D><<<chunks, BQS * (D / 8), 0, st>>>(dq_acc, static_cast<__nv_bfloat16*>(dq), cu, B,
                                                                        total, Tpad, p->deterministic ? 1 : 0, a.status);
  COWA_CUDA_TRY(cudaGetLastError());
  return COWA_OK;
}

}  // namespace

extern "C" {

size_t cowa_bwd_varlen_workspace_bytes(int B, int total, int Hq, int Hkv, int D, const cowa_params_t* p) {
  (void)p;
  if (B <= 0 || total <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || (D != 64 && D != 128)) return 0;
  return ws_bytes_varlen(B, total, Hq, D);
}

int cowa_bwd_varlen(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o,
                    void* dq, void* dk, void* dv, const int32_t* cu_seqlens, int B, int total, int Hq, int Hkv, int D,
                    const cowa_params_t* p, void* workspace, size_t workspace_bytes, void* stream) {
  if (!q || !k || !v || !o || !lse || !d_o || !dq || !dk || !dv || !p || !workspace || !cu_seqlens)
    return COWA_ERR_INVALID_ARG;
  if (B <= 0 || total <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0) return COWA_ERR_INVALID_ARG;
  if (!(p->softmax_scale > 0.f)) return COWA_ERR_INVALID_ARG;
  if (D != 64 && D != 128) return COWA_ERR_UNSUPPORTED;
  const void* ptrs[] = {q, k, v, o, d_o, dq, dk, dv, workspace};
  for (const void* x : ptrs)
    if (!cowa::aligned16(x)) return COWA_ERR_MISALIGNED;
  if (workspace_bytes < ws_bytes_varlen(B, total, Hq, D)) return COWA_ERR_WORKSPACE_TOO_SMALL;
  CowaHeadWindows hw;
  int rc = cowa::resolve_windows(total, Hkv, p, &hw);  // validates; explicit tuples are copied, the default rule runs per sequence
  if (rc != COWA_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return D == 128 ? launch_bwd_varlen<128>(q, k, v, o, lse, d_o, dq, dk, dv, cu_seqlens, B, total, Hq, Hkv, p, hw,
                                           workspace, st)
                  : launch_bwd_varlen<64>(q, k, v, o, lse, d_o, dq, dk, dv, cu_seqlens, B, total, Hq, Hkv, p, hw,
                                          workspace, st);
}

size_t cowa_bwd_prefill_workspace_bytes(int B, int Nq, int Nk, int Hq, int Hkv, int D, const cowa_params_t* p) {
  if (B <= 0 || Nq <= 0 || Nk < Nq || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || D <= 0 || !p) return 0;
  CowaHeadWindows hw;
  if (cowa::resolve_windows(Nk, Hkv, p, &hw) != COWA_OK) return 0;
  return ws_bytes(B, Nq, Nk, Hq, Hkv, D, bwd_parts(B, Nq, Nk, Hkv, Hq / Hkv, hw));
}

size_t cowa_bwd_workspace_bytes(int B, int T, int Hq, int Hkv, int D, const cowa_params_t* p) {
  return cowa_bwd_prefill_workspace_bytes(B, T, T, Hq, Hkv, D, p);
}

int cowa_bwd_prefill(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o,
                     void* dq, void* dk, void* dv, int B, int Nq, int Nk, int Hq, int Hkv, int D,
                     const cowa_params_t* p, void* workspace, size_t workspace_bytes, void* stream) {
  if (!q || !k || !v || !o || !lse || !d_o || !dq || !dk || !dv || !p || !workspace) return COWA_ERR_INVALID_ARG;
  if (B <= 0 || Nq <= 0 || Nk < Nq || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0) return COWA_ERR_INVALID_ARG;
  if (!(p->softmax_scale > 0.f)) return COWA_ERR_INVALID_ARG;
  if (D != 64 && D != 128) return COWA_ERR_UNSUPPORTED;
  const void* ptrs[] = {q, k, v, o, d_o, dq, dk, dv, workspace};
  for (const void* x : ptrs)
    if (!cowa::aligned16(x)) return COWA_ERR_MISALIGNED;
  CowaHeadWindows hw;
  int rc = cowa::resolve_windows(Nk, Hkv, p, &hw);
  if (rc != COWA_OK) return rc;
  const int parts = bwd_parts(B, Nq, Nk, Hkv, Hq / Hkv, hw);
  if (workspace_bytes < ws_bytes(B, Nq, Nk, Hq, Hkv, D, parts)) return COWA_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return D == 128 ? launch_bwd<128>(q, k, v, o, lse, d_o, dq, dk, dv, B, Nq, Nk, Hq, Hkv, p, hw, parts, workspace, st)
                  : launch_bwd<64>(q, k, v, o, lse, d_o, dq, dk, dv, B, Nq, Nk, Hq, Hkv, p, hw, parts, workspace, st);
}

int cowa_bwd(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o,
             void* dq, void* dk, void* dv, int B, int T, int Hq, int Hkv, int D, const cowa_params_t* p,
             void* workspace, size_t workspace_bytes, void* stream) {
  return cowa_bwd_prefill(q, k, v, o, lse, d_o, dq, dk, dv, B, T, T, Hq, Hkv, D, p, workspace, workspace_bytes, stream);
}

}  // extern "C"
