// Host-side pieces of the C ABI that launch nothing: window resolution, the schedule dump,
// tile counts, status reporting.
#include <string.h>

#include <algorithm>
#include <vector>
#include "cowa_common.h"
#include "cowa_ptx.cuh"

namespace {
thread_local int g_last_cuda_error = 0;
__device__ unsigned int g_cowa_status_word = 0;

// One warp-free block: thread 0 waits on a barrier that has no arrivals until the bounded wait gives up.
__global__ void cowa_selftest_wait_kernel(unsigned int* status, long long limit) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    cowa_ptx::mbar_init(&bar, 1);
    cowa_ptx::fence_mbar_init();
    cowa_ptx::mbar_wait(&bar, 0, status, limit);
  }
}
}  // namespace

namespace cowa {

int record_cuda_error(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return COWA_ERR_CUDA;
}

unsigned int* device_status_word() {
  // One address per device; looked up once per device with that device current.
  static unsigned int* cache[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!cache[dev]) {
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_cowa_status_word);
    if (e != cudaSuccess) { record_cuda_error(e); return nullptr; }
    cache[dev] = static_cast<unsigned int*>(ptr);
  }
  return cache[dev];
}

int resolve_strides(const int64_t s[3], int H, long long T, int D, CowaStrides* out) {
  if (s[0] == 0 && s[1] == 0 && s[2] == 0) {
    out->t = D; out->h = (long long)T * D; out->b = (long long)H * T * D;
    return COWA_OK;
  }
  if (s[0] < 0 || s[1] < 0 || s[2] < D) return COWA_ERR_INVALID_ARG;
  if ((s[0] | s[1] | s[2]) & 7) return COWA_ERR_MISALIGNED;
  out->b = s[0]; out->h = s[1]; out->t = s[2];
  return COWA_OK;
}

bool any_stride_set(const cowa_params_t* p) {
  for (int i = 0; i < 3; ++i)
    if (p->q_strides[i] || p->k_strides[i] || p->v_strides[i] || p->o_strides[i]) return true;
  return false;
}

int resolve_windows(int Nk, int Hkv, const cowa_params_t* p, CowaHeadWindows* out) {
  if (!p || Hkv <= 0 || Nk <= 0) return COWA_ERR_INVALID_ARG;
  if (Hkv > COWA_MAX_HKV) return COWA_ERR_UNSUPPORTED;
  const int hg = p->hkv_global > 0 ? p->hkv_global : Hkv;
  if (p->hkv_offset < 0 || p->hkv_offset + Hkv > hg) return COWA_ERR_INVALID_ARG;
  for (int h = 0; h < Hkv; ++h) {
    CowaWin w;
    if (p->full_attn) {
      w.s = 0; w.n = Nk; w.g = 0; w.l = 0;  // near window spans the whole prefix
    } else if (p->windows) {
      const cowa_window_t& t = p->windows[h];
      if (t.sink < 0 || t.near < 1 || t.gap < 0 || t.len < 0) return COWA_ERR_INVALID_ARG;
      // no key lies further than Nk away: widths beyond Nk mean the same as Nk, and clamping them keeps the
      // sums near + gap + len inside 32 bits everywhere
      w.s = std::min(t.sink, Nk); w.n = std::min(t.near, Nk); w.g = std::min(t.gap, Nk); w.l = std::min(t.len, Nk);
    } else {
      if (p->sink < 0 || p->local < 1) return COWA_ERR_INVALID_ARG;
      w = cowa_default_window(Nk, hg, p->hkv_offset + h, p->sink, p->local);
    }
    out->w[h] = w;
  }
  return COWA_OK;
}

}  // namespace cowa

extern "C" {

int cowa_default_windows(int Nk, int Hkv_global, int hkv_offset, int Hkv_local, int sink, int local,
                         cowa_window_t* out) {
  if (!out || Nk <= 0 || Hkv_global <= 0 || Hkv_local <= 0 || hkv_offset < 0 ||
      hkv_offset + Hkv_local > Hkv_global || sink < 0 || local < 1)
    return COWA_ERR_INVALID_ARG;
  for (int h = 0; h < Hkv_local; ++h) {
    CowaWin w = cowa_default_window(Nk, Hkv_global, hkv_offset + h, sink, local);
    out[h].sink = w.s; out[h].near = w.n; out[h].gap = w.g; out[h].len = w.l;
  }
  return COWA_OK;
}

int cowa_equal_area_windows(int Nq, int Nk, int Hkv_global, int hkv_offset, int Hkv_local, int sink, int local,
                            cowa_window_t* out) {
  if (!out || Nq <= 0 || Nk < Nq || Hkv_global <= 0 || Hkv_local <= 0 || hkv_offset < 0 ||
      hkv_offset + Hkv_local > Hkv_global || sink < 0 || local < 1)
    return COWA_ERR_INVALID_ARG;
  const long long L = std::max((long long)Nk - sink - local, 0ll);
  const long long off = (long long)Nk - Nq;
  // queries that reach a key outside the sink at band offset x (distance local + x)
  auto weight = [&](long long x) {
    const long long first = std::max(local + x + sink - off, 0ll);
    return std::min(std::max((long long)Nq - first, 0ll), (long long)Nq);
  };
  unsigned __int128 total = 0;
  for (long long x = 0; x < L; ++x) total += (unsigned long long)weight(x);
  // one sweep: b_h = first b whose cumulative weight, times H, reaches h * total
  std::vector<long long> b(Hkv_global + 1, L);
  unsigned __int128 cum = 0;
  long long x = 0;
  for (int h = 0; h <= Hkv_global; ++h) {
    while ((unsigned __int128)Hkv_global * cum < (unsigned __int128)h * total) cum += (unsigned long long)weight(x++);
    b[h] = x;
  }
  for (int h = 0; h < Hkv_local; ++h) {
    const int g = hkv_offset + h;
    out[h].sink = sink; out[h].near = local;
    out[h].gap = (int32_t)b[g]; out[h].len = (int32_t)(b[g + 1] - b[g]);
  }
  return COWA_OK;
}

int cowa_schedule_dump(int which, int Nq, int Nk, int Hkv, const cowa_params_t* p, int32_t* out,
                       size_t out_cap, size_t* out_len) {
  if (!p || !out_len || Nq <= 0 || Nk <= 0 || Nq > Nk || Hkv <= 0) return COWA_ERR_INVALID_ARG;
  if (p->block_q <= 0 || p->block_k <= 0) return COWA_ERR_INVALID_ARG;
  if (Hkv > COWA_MAX_HKV) return COWA_ERR_UNSUPPORTED;
  CowaHeadWindows hw;
  int st = cowa::resolve_windows(Nk, Hkv, p, &hw);
  if (st != COWA_OK) return st;
  const int Bq = p->block_q, Bk = p->block_k, off = Nk - Nq;
  const int Tq = (Nq + Bq - 1) / Bq, Tk = (Nk + Bk - 1) / Bk;
  size_t n = 0;
  auto put = [&](int32_t x) {
    if (out && n < out_cap) out[n] = x;
    ++n;
  };
  for (int h = 0; h < Hkv; ++h) {
    const CowaWin& w = hw.w[h];
    if (which == COWA_SCHED_FWD) {
      for (int i = 0; i < Tq; ++i) {
        const int q0 = i * Bq, q1 = cowa_imin(q0 + Bq, Nq) - 1;
        CowaRange r[3];
        cowa_fwd_ranges(w, q0, q1, off, Nk, Bk, r);
        const int tot = cowa_range_len(r[0]) + cowa_range_len(r[1]) + cowa_range_len(r[2]);
        put(h); put(i); put(tot);
        for (int t = 0; t < tot; ++t) {
          const int j = cowa_fwd_tile_at(r, t);
          put(j);
          put(cowa_tile_full(w, q0, Bq, j * Bk, Bk, off, Nq, Nk) ? 1 : 0);
        }
      }
    } else if (which == COWA_SCHED_BWD) {
      for (int j = 0; j < Tk; ++j) {
        const int k0 = j * Bk, k1 = cowa_imin(k0 + Bk, Nk) - 1;
        CowaRange r[2];
        cowa_bwd_ranges(w, k0, k1, off, Nq, Bq, r);
        const int tot = cowa_range_len(r[0]) + cowa_range_len(r[1]);
        put(h); put(j); put(tot);
        for (int t = 0; t < tot; ++t) {
          const int i = cowa_bwd_tile_at(r, t);
          put(i);
          put(cowa_tile_full(w, i * Bq, Bq, k0, Bk, off, Nq, Nk) ? 1 : 0);
        }
      }
    } else if (which == COWA_SCHED_DECODE) {
      CowaRange r[3];
      const int nr = Nq == 1 ? cowa_decode_ranges(w, Nk, r) : cowa_decode_ranges_span(w, Nk - Nq, Nk - 1, r);
      put(h); put(nr);
      for (int t = 0; t < nr; ++t) { put(r[t].lo); put(r[t].hi + 1); }
      // visited blocks: the blocks touched by the ranges, each once
      size_t cnt_at = n;
      put(0);
      int32_t cnt = 0;
      int last = -1;
      for (int t = 0; t < nr; ++t) {
        for (int b = cowa_imax(r[t].lo / Bk, last + 1); b <= r[t].hi / Bk; ++b) { put(b); ++cnt; last = b; }
      }
      if (out && cnt_at < out_cap) out[cnt_at] = cnt;
    } else {
      return COWA_ERR_INVALID_ARG;
    }
  }
  *out_len = n;
  return (out && n <= out_cap) ? COWA_OK : COWA_ERR_WORKSPACE_TOO_SMALL;
}

int cowa_tile_counts(int Nq, int Nk, int Hkv, const cowa_params_t* p, int64_t out[3]) {
  if (!p || !out || Nq <= 0 || Nk <= 0 || Nq > Nk || Hkv <= 0) return COWA_ERR_INVALID_ARG;
  CowaHeadWindows hw;
  int st = cowa::resolve_windows(Nk, Hkv, p, &hw);
  if (st != COWA_OK) return st;
  const int B = 128, off = Nk - Nq, Tq = (Nq + B - 1) / B;
  int64_t visited = 0, full = 0, causal = 0;
  for (int h = 0; h < Hkv; ++h) {
    for (int i = 0; i < Tq; ++i) {
      const int q0 = i * B, q1 = cowa_imin(q0 + B, Nq) - 1;
      CowaRange r[3];
      cowa_fwd_ranges(hw.w[h], q0, q1, off, Nk, B, r);
      const int tot = cowa_range_len(r[0]) + cowa_range_len(r[1]) + cowa_range_len(r[2]);
      visited += tot;
      for (int t = 0; t < tot; ++t)
        full += cowa_tile_full(hw.w[h], q0, B, cowa_fwd_tile_at(r, t) * B, B, off, Nq, Nk) ? 1 : 0;
      causal += cowa_imin(q1 + off, Nk - 1) / B + 1;
    }
  }
  out[0] = visited; out[1] = full; out[2] = causal;
  return COWA_OK;
}

int cowa_check_device_status(void* stream) {
  unsigned int* word = cowa::device_status_word();
  if (!word) return COWA_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  unsigned int host = 0;
  COWA_CUDA_TRY(cudaMemcpyAsync(&host, word, sizeof(host), cudaMemcpyDeviceToHost, s));
  COWA_CUDA_TRY(cudaStreamSynchronize(s));
  if (host != 0) {
    COWA_CUDA_TRY(cudaMemsetAsync(word, 0, sizeof(host), s));
    COWA_CUDA_TRY(cudaStreamSynchronize(s));
    if (host & COWA_DEV_TIMEOUT) return COWA_ERR_DEVICE_TIMEOUT;
    if (host & COWA_DEV_BAD_SEQLENS) return COWA_ERR_DEVICE_BAD_SEQLENS;
    return COWA_ERR_DEVICE_DQ_RANGE;
  }
  return COWA_OK;
}

int cowa_selftest_bounded_wait(long long limit_clocks, void* stream) {
  unsigned int* word = cowa::device_status_word();
  if (!word) return COWA_ERR_CUDA;
  const long long limit = std::min(std::max(limit_clocks, 1ll << 10), 1ll << 24);
  cowa_selftest_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(word, limit);
  COWA_CUDA_TRY(cudaGetLastError());
  return COWA_OK;
}

const char* cowa_status_string(int status) {
  switch (status) {
    case COWA_OK: return "ok";
    case COWA_ERR_INVALID_ARG: return "invalid argument";
    case COWA_ERR_UNSUPPORTED: return "unsupported configuration";
    case COWA_ERR_MISALIGNED: return "pointer not 16-byte aligned";
    case COWA_ERR_WORKSPACE_TOO_SMALL: return "workspace or output buffer too small";
    case COWA_ERR_CUDA: return "CUDA call failed";
    case COWA_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    case COWA_ERR_STATIC_SCRATCH_EXCEEDED:
      return "cowa_decode_static: the call needs more scratch than the library's built-in array holds";
    case COWA_ERR_DEVICE_BAD_SEQLENS:
      return "cowa_prefill_varlen: a sequence with N_q > N_k was skipped";
    case COWA_ERR_DEVICE_DQ_RANGE:
      return "deterministic backward: a dQ value left the fixed-point range";
    default: return "unknown status";
  }
}

int cowa_last_cuda_error(void) { return g_last_cuda_error; }

}  // extern "C"
