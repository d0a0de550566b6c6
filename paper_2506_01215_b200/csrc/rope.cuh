// Rotary position embedding at consecutive position ids (Sec. 3.1: after each
// compression the cache rows are re-assigned consecutive ids, so the cache
// keeps un-rotated keys and row r of [cache ; chunk] is rotated by position
// pos_begin + r when the step's operands are prepared).  HBM-bound: one read
// and one write of the rotated rows.  The angle depends on (row, pair) only,
// so a thread evaluates cos/sin once and reuses them for every batch entry and
// head of that row.  Positions reach 10^6, where an fp32 angle would be off by
// 1e-2 rad, so the angle is reduced in fp64: the host passes each pair's
// frequency in turns per position (fp64), the product with the position is
// reduced to [-1/2, 1/2] turns in fp64, and only the reduced angle -- as an
// fp32 value plus its fp32 remainder -- goes through the fp32 sincospi.
#pragma once

#include "common.cuh"

namespace reform {

constexpr int kRopeMaxPairs = 256;  // head dimensions up to 512
struct RopeFreq {
  double turns[kRopeMaxPairs];  // theta_base^(-2 i / d) / (2 pi)
};

// Thread = (row, group of NP consecutive pairs); block = 256 threads.
//   half layout (interleaved == 0): pair i = (x[i], x[i + d/2]); a thread loads NP consecutive
//     elements from each half.
//   interleaved: pair i = (x[2i], x[2i+1]); a thread loads 2*NP consecutive elements.
template <typename T, bool INTERLEAVED>
__global__ void __launch_bounds__(256)
rope_kernel(const T* __restrict__ src, T* __restrict__ dst, int BH, int d, long long cap,
            long long row_begin, long long rows, long long pos_begin, const __grid_constant__ RopeFreq freq) {
  constexpr int NP = 16 / (int)sizeof(T) / (INTERLEAVED ? 2 : 1);  // pairs per thread: one or two 16-byte vectors
  const int groups = (d / 2) / NP;                                  // thread groups per row
  const long long items = rows * groups;
  for (long long it = (long long)blockIdx.x * blockDim.x + threadIdx.x; it < items;
       it += (long long)gridDim.x * blockDim.x) {
    const long long r = it / groups;
    const int p0 = (int)(it % groups) * NP;  // first pair of this thread
    const double pos = (double)(pos_begin + r);
    float c[NP], s[NP];
#pragma unroll
    for (int i = 0; i < NP; ++i) {
      const double t = pos * freq.turns[p0 + i];
      const double fr = t - rint(t);           // [-1/2, 1/2] turns, exact
      const float hi = (float)fr;
      const float lo = (float)(fr - (double)hi) * 6.2831853071795865f;  // radians left over
      float sn, cs;
      sincospif(2.0f * hi, &sn, &cs);
      c[i] = fmaf(-lo, sn, cs);                // first-order correction for the remainder
      s[i] = fmaf(lo, cs, sn);
    }
#pragma unroll 4
    for (int bh = 0; bh < BH; ++bh) {
      const long long off = ((long long)bh * cap + row_begin + r) * d;
      if (INTERLEAVED) {
        uint4 v = *reinterpret_cast<const uint4*>(src + off + 2 * p0);
        T* e = reinterpret_cast<T*>(&v);
#pragma unroll
        for (int i = 0; i < NP; ++i) {
          const float a = to_float(e[2 * i]), b = to_float(e[2 * i + 1]);
          e[2 * i] = from_float<T>(a * c[i] - b * s[i]);
          e[2 * i + 1] = from_float<T>(b * c[i] + a * s[i]);
        }
        *reinterpret_cast<uint4*>(dst + off + 2 * p0) = v;
      } else {
        uint4 lo = *reinterpret_cast<const uint4*>(src + off + p0);
        uint4 hi = *reinterpret_cast<const uint4*>(src + off + d / 2 + p0);
        T* a = reinterpret_cast<T*>(&lo);
        T* b = reinterpret_cast<T*>(&hi);
#pragma unroll
        for (int i = 0; i < NP; ++i) {
          const float x = to_float(a[i]), y = to_float(b[i]);
          a[i] = from_float<T>(x * c[i] - y * s[i]);
          b[i] = from_float<T>(y * c[i] + x * s[i]);
        }
        *reinterpret_cast<uint4*>(dst + off + p0) = lo;
        *reinterpret_cast<uint4*>(dst + off + d / 2 + p0) = hi;
      }
    }
  }
}

template <typename T>
inline int launch_rope(const void* src, void* dst, int BH, int d, long long cap, long long row_begin,
                       long long rows, long long pos_begin, double base, bool interleaved,
                       cudaStream_t st) {
  if (rows == 0 || BH == 0) return REFORM_OK;
  const int np = 16 / (int)sizeof(T) / (interleaved ? 2 : 1);
  const long long items = rows * ((d / 2) / np);
  long long blocks = (items + 255) / 256;
  const long long cap_blocks = (long long)num_sms() * 16;
  const int grid = (int)(blocks < cap_blocks ? blocks : cap_blocks);
  RopeFreq freq;
  for (int i = 0; i < d / 2; ++i) freq.turns[i] = pow(base, -2.0 * i / d) / 6.283185307179586476925;
  if (interleaved)
    rope_kernel<T, true><<<grid, 256, 0, st>>>((const T*)src, (T*)dst, BH, d, cap, row_begin, rows, pos_begin, freq);
  else
    rope_kernel<T, false><<<grid, 256, 0, st>>>((const T*)src, (T*)dst, BH, d, cap, row_begin, rows, pos_begin, freq);
  count_launch();
  return check_launch();
}

}  // namespace reform
