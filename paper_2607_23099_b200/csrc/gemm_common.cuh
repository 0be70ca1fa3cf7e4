// Work-item decoding and small device helpers shared by the bf16 and fp8 grouped GEMMs.
#pragma once
#include "common.cuh"

namespace damoe {

struct Item {
  int e, m_tile, q0, valid;
};

__device__ __forceinline__ Item decode_item(int w, const int* s_pref, const int* s_off, int E, int MT) {
  int lo = 0, hi = E - 1;
  while (lo < hi) {  // largest e with s_pref[e] * MT <= w
    const int mid = (lo + hi + 1) >> 1;
    if (s_pref[mid] * MT <= w) lo = mid;
    else hi = mid - 1;
  }
  Item it;
  it.e = lo;
  const int nt = s_pref[lo + 1] - s_pref[lo];  // ceil(t_e / N_v) token tiles
  const int local = w - s_pref[lo] * MT;
  it.m_tile = local / nt;
  const int n_tile = local - it.m_tile * nt;
  // The expert's tokens are split evenly over its tiles (sizes differ by at most one) instead of
  // N_v, N_v, ..., remainder: tiles of one expert then take the same time, so the CTAs that work on
  // them side by side stay in step and share the expert's weights through L2, and no tile is
  // nearly empty.  The MMA width follows the tile's size (multiples of 16).
  const int off = s_off[lo];
  const int n_e = s_off[lo + 1] - off;
  const int base = n_e / nt, rem = n_e - base * nt;
  it.q0 = off + n_tile * base + (n_tile < rem ? n_tile : rem);
  it.valid = base + (n_tile < rem ? 1 : 0);
  return it;
}

__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.0f + __expf(-g)) * u; }

}  // namespace damoe
