// Work-item decoding and small device helpers shared by the bf16 and fp8 grouped GEMMs.
#pragma once
#include "common.cuh"

namespace damoe {

struct Item {
  int e, m_tile, q0, valid;
};

__device__ __forceinline__ Item decode_item(int w, const int* s_pref, const int* s_off, int E, int MT, int BN) {
  int lo = 0, hi = E - 1;
  while (lo < hi) {  // largest e with s_pref[e] * MT <= w
    const int mid = (lo + hi + 1) >> 1;
    if (s_pref[mid] * MT <= w) lo = mid;
    else hi = mid - 1;
  }
  Item it;
  it.e = lo;
  const int nt = s_pref[lo + 1] - s_pref[lo];
  const int local = w - s_pref[lo] * MT;
  it.m_tile = local / nt;
  const int n_tile = local - it.m_tile * nt;
  const int off = s_off[lo];
  it.q0 = off + n_tile * BN;
  const int left = s_off[lo + 1] - it.q0;
  it.valid = left < BN ? left : BN;
  return it;
}

__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.0f + __expf(-g)) * u; }

}  // namespace damoe
