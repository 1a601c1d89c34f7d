// Analytic tile scheduler for CoWindow Attention: every visited-tile list is derived
// from positions and the head's 4-tuple alone, in O(1) integer work per tile row/column
// (Sec. 2.3: J_h(i) = KV blocks with at least one legal pair with QO block i, I_h(j) the
// inverse relation; blocks outside are skipped, only blocks crossing a causal, window or
// sequence boundary are masked element-wise).  The same functions run on the host
// (cowa_schedule_dump, FLOP accounting) and inside the kernels.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define COWA_HD __host__ __device__ __forceinline__
#else
#define COWA_HD inline
#endif

struct CowaWin {
  int s, n, g, l;  // sink width, near width, gap after near, long width
};

// Inclusive range of tile (or token) indices; empty when lo > hi.
struct CowaRange {
  int lo, hi;
};

COWA_HD int cowa_imin(int a, int b) { return a < b ? a : b; }
COWA_HD int cowa_imax(int a, int b) { return a > b ? a : b; }

// Default pattern, Eq. (fwa_long_range_span): L = max(Nk - s - n, 0), b_h = floor(h L / Hk),
// tuple of global head h = (s, n, b_h, b_{h+1} - b_h).
COWA_HD CowaWin cowa_default_window(int Nk, int Hk_global, int h_global, int s, int n) {
  long long L = (long long)Nk - s - n;
  if (L < 0) L = 0;
  int b0 = (int)(((long long)h_global * L) / Hk_global);
  int b1 = (int)(((long long)(h_global + 1) * L) / Hk_global);
  CowaWin w;
  w.s = s; w.n = n; w.g = b0; w.l = b1 - b0;
  return w;
}

// Element predicate, Eq. (fwa_support) with delta from Eq. (fwa_distance).
COWA_HD bool cowa_visible(const CowaWin& w, int delta, int ik) {
  return delta >= 0 && (delta < w.n || ik < w.s || (delta >= w.n + w.g && delta < w.n + w.g + w.l));
}

// ---------------------------------------------------------------------------------------
// Forward: KV tiles visited by the QO tile with rows [q0, q1] (q1 already clipped to Nq-1).
// off = Nk - Nq.  Result: up to three disjoint tile ranges, r[0] = near part, r[1] = long
// part, r[2] = sink part, each to be walked from hi down to lo; r[0] > r[1] > r[2] in
// position, so walking r[0], r[1], r[2] visits tiles in descending order exactly once.
// ---------------------------------------------------------------------------------------
COWA_HD void cowa_fwd_ranges(const CowaWin& w, int q0, int q1, int off, int Nk, int Bk, CowaRange r[3]) {
  const int kmax = cowa_imin(q1 + off, Nk - 1);  // last causal key of the tile
  r[0].lo = 0; r[0].hi = -1; r[1] = r[0]; r[2] = r[0];
  if (kmax < 0) return;
  // near part: keys [q0+off-n+1, kmax]; everything else lies in tiles below `floor`
  int floor_tile = kmax / Bk + 1;
  if (w.n > 0) {
    const int klo = cowa_imax(q0 + off - w.n + 1, 0);
    r[0].lo = klo / Bk; r[0].hi = kmax / Bk;
    floor_tile = r[0].lo;
  }
  // sink part: tiles [0, x]
  int x = -1;
  if (w.s > 0) x = cowa_imin(cowa_imin(w.s - 1, kmax) / Bk, floor_tile - 1);
  r[2].lo = 0; r[2].hi = x;
  // long part: keys [q0+off-(n+g+l)+1, q1+off-(n+g)], minus what near and sink already list
  if (w.l > 0) {
    long long lo_ll = (long long)q0 + off - ((long long)w.n + w.g + w.l) + 1;
    const int klo = lo_ll < 0 ? 0 : (int)lo_ll;
    long long hi_ll = (long long)q1 + off - ((long long)w.n + w.g);
    if (hi_ll > kmax) hi_ll = kmax;
    if (hi_ll >= klo) {
      const int y = cowa_imin((int)hi_ll / Bk, floor_tile - 1);
      if (y > x) { r[1].lo = cowa_imax(klo / Bk, x + 1); r[1].hi = y; }
    }
  }
}

COWA_HD int cowa_range_len(const CowaRange& r) { return r.hi >= r.lo ? r.hi - r.lo + 1 : 0; }

// t-th visited tile in descending order, t in [0, total).
COWA_HD int cowa_fwd_tile_at(const CowaRange r[3], int t) {
  int n0 = cowa_range_len(r[0]);
  if (t < n0) return r[0].hi - t;
  t -= n0;
  int n1 = cowa_range_len(r[1]);
  if (t < n1) return r[1].hi - t;
  t -= n1;
  return r[2].hi - t;
}

// Is every pair of the nominal tile rows [q0, q0+Bq) x cols [k0, k0+Bk) legal?
// Tiles clipped by a sequence end are never full.
COWA_HD bool cowa_tile_full(const CowaWin& w, int q0, int Bq, int k0, int Bk, int off, int Nq, int Nk) {
  const int q1 = q0 + Bq - 1, k1 = k0 + Bk - 1;
  if (q1 > Nq - 1 || k1 > Nk - 1) return false;
  const long long dmin = (long long)q0 + off - k1;
  if (dmin < 0) return false;
  const int k0p = cowa_imax(k0, w.s);  // first column that is not a sink column
  if (k0p > k1) return true;           // all sink columns, all causal
  const long long dmaxp = (long long)q1 + off - k0p;
  const long long far_end = (long long)w.n + w.g + w.l;
  if (w.l <= 0) return dmaxp < w.n;
  if (dmaxp >= far_end) return false;
  return w.g == 0 || dmaxp < w.n || dmin >= (long long)w.n + w.g;
}

// Does the tile hold at least one legal pair?  (Used by the dump and by tests; the
// kernels enumerate ranges instead.)  q1, k1 are clipped to the sequence ends.
COWA_HD bool cowa_tile_visited(const CowaWin& w, int q0, int q1, int k0, int k1, int off) {
  const long long dmin = (long long)q0 + off - k1, dmax = (long long)q1 + off - k0;
  if (dmax < 0) return false;
  const long long lo = dmin < 0 ? 0 : dmin;
  if (lo <= (dmax < w.n - 1 ? dmax : (long long)w.n - 1)) return true;
  if (k0 < w.s) return true;
  if (w.l > 0) {
    const long long a = (long long)w.n + w.g, b = a + w.l - 1;
    if ((lo > a ? lo : a) <= (dmax < b ? dmax : b)) return true;
  }
  return false;
}

// ---------------------------------------------------------------------------------------
// Backward: QO tiles visited by the KV tile with columns [k0, k1] (k1 clipped to Nk-1).
// Up to two disjoint ascending ranges r[0] < r[1]; walk r[0] then r[1], lo to hi.
// ---------------------------------------------------------------------------------------
COWA_HD void cowa_bwd_ranges(const CowaWin& w, int k0, int k1, int off, int Nq, int Bq, CowaRange r[2]) {
  r[0].lo = 0; r[0].hi = -1; r[1] = r[0];
  long long qlo = (long long)k0 - off;  // first causal query of column k0
  if (qlo < 0) qlo = 0;
  if (qlo > Nq - 1) return;
  if (k0 < w.s) {  // a sink column is seen by every causal query
    r[0].lo = (int)qlo / Bq; r[0].hi = (Nq - 1) / Bq;
    return;
  }
  int cursor = -1;  // highest tile already listed
  if (w.n > 0) {
    long long qhi = (long long)k1 - off + w.n - 1;
    if (qhi > Nq - 1) qhi = Nq - 1;
    if (qhi >= qlo) {
      r[0].lo = (int)qlo / Bq; r[0].hi = (int)qhi / Bq;
      cursor = r[0].hi;
    }
  }
  if (w.l > 0) {
    long long a = (long long)k0 - off + w.n + w.g;
    long long b = (long long)k1 - off + (long long)w.n + w.g + w.l - 1;
    if (a < 0) a = 0;
    if (b > Nq - 1) b = Nq - 1;
    if (b >= a) {
      r[1].lo = cowa_imax((int)a / Bq, cursor + 1); r[1].hi = (int)b / Bq;
    }
  }
}

COWA_HD int cowa_bwd_tile_at(const CowaRange r[2], int t) {
  int n0 = cowa_range_len(r[0]);
  if (t < n0) return r[0].lo + t;
  return r[1].lo + (t - n0);
}

// ---------------------------------------------------------------------------------------
// Decode (N_q = 1, delta = Nk - 1 - i_k): visible keys as up to three disjoint, maximal,
// ascending token ranges [lo, hi] (inclusive).  Returns the number of ranges.
// ---------------------------------------------------------------------------------------
COWA_HD int cowa_decode_ranges(const CowaWin& w, int Nk, CowaRange out[3]) {
  CowaRange c[3];
  int nc = 0;
  if (w.s > 0) { c[nc].lo = 0; c[nc].hi = cowa_imin(w.s, Nk) - 1; nc++; }
  if (w.l > 0) {
    long long lo = (long long)Nk - w.n - w.g - w.l, hi = (long long)Nk - 1 - w.n - w.g;
    if (lo < 0) lo = 0;
    if (hi >= lo) { c[nc].lo = (int)lo; c[nc].hi = (int)hi; nc++; }
  }
  if (w.n > 0) { c[nc].lo = cowa_imax(Nk - w.n, 0); c[nc].hi = Nk - 1; nc++; }
  // candidates are ascending in lo; merge the ones that overlap or abut
  int n = 0;
  for (int i = 0; i < nc; ++i) {
    if (n > 0 && c[i].lo <= out[n - 1].hi + 1) {
      out[n - 1].hi = cowa_imax(out[n - 1].hi, c[i].hi);
    } else {
      out[n++] = c[i];
    }
  }
  return n;
}

// Several queries at once (multi-token decode): queries at key positions p0 .. p1 (p1 = Nk - 1 for the
// newest token); the union of their visible keys, same form as cowa_decode_ranges.  Which query sees
// which key inside the union is decided per element with cowa_visible.
COWA_HD int cowa_decode_ranges_span(const CowaWin& w, int p0, int p1, CowaRange out[3]) {
  CowaRange c[3];
  int nc = 0;
  if (w.s > 0) { c[nc].lo = 0; c[nc].hi = cowa_imin(w.s - 1, p1); nc++; }
  if (w.l > 0) {
    long long lo = (long long)p0 - w.n - w.g - w.l + 1, hi = (long long)p1 - w.n - w.g;
    if (lo < 0) lo = 0;
    if (hi >= lo) { c[nc].lo = (int)lo; c[nc].hi = (int)hi; nc++; }
  }
  if (w.n > 0) { c[nc].lo = cowa_imax(p0 - w.n + 1, 0); c[nc].hi = p1; nc++; }
  int n = 0;
  for (int i = 0; i < nc; ++i) {
    if (n > 0 && c[i].lo <= out[n - 1].hi + 1) {
      out[n - 1].hi = cowa_imax(out[n - 1].hi, c[i].hi);
    } else {
      out[n++] = c[i];
    }
  }
  return n;
}
