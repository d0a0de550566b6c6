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

// cos and sin of pos * turns (turns = frequency in turns per position): the product is reduced to
// [-1/2, 1/2] turns in fp64, and only the reduced angle, as an fp32 value plus its fp32 remainder,
// goes through the fp32 sincospi.
__device__ __forceinline__ void rope_cos_sin(double pos, double turns, float& c, float& s) {
  const double t = pos * turns;
  const double fr = t - rint(t);           // [-1/2, 1/2] turns, exact
  const float hi = (float)fr;
  const float lo = (float)(fr - (double)hi) * 6.2831853071795865f;  // radians left over
  float sn, cs;
  sincospif(2.0f * hi, &sn, &cs);
  c = fmaf(-lo, sn, cs);                   // first-order correction for the remainder
  s = fmaf(lo, cs, sn);
}

// Table of (cos, sin) for rows positions pos_begin .. pos_begin + rows - 1 and every pair:
// tab[r * pairs + i].  Read by the chunk-step kernel that rotates its query tiles at load.
__global__ void __launch_bounds__(256)
rope_table_kernel(float2* __restrict__ tab, long long rows, int pairs, long long pos_begin,
                  const __grid_constant__ RopeFreq freq) {
  const long long items = rows * pairs;
  for (long long it = (long long)blockIdx.x * blockDim.x + threadIdx.x; it < items;
       it += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(it % pairs);
    float c, s;
    rope_cos_sin((double)(pos_begin + it / pairs), freq.turns[i], c, s);
    tab[it] = make_float2(c, s);
  }
}

// The rotation itself, with the roundings spelled out so that every kernel that rotates (this
// file's and the chunk step's rotation at load) produces the same bits:
//   a' = fma(a, cos, -(b * sin)),   b' = fma(b, cos, a * sin)
__device__ __forceinline__ void rope_rotate(float a, float b, float c, float s, float& ra, float& rb) {
  ra = __fmaf_rn(a, c, -__fmul_rn(b, s));
  rb = __fmaf_rn(b, c, __fmul_rn(a, s));
}

// Thread = (row, group of NP consecutive pairs); block = 256 threads.
//   half layout (interleaved == 0): pair i = (x[i], x[i + d/2]); a thread loads NP consecutive
//     elements from each half.
//   interleaved: pair i = (x[2i], x[2i+1]); a thread loads 2*NP consecutive elements.
template <typename T, bool INTERLEAVED>
__global__ void __launch_bounds__(256)
rope_kernel(const T* __restrict__ src, T* __restrict__ dst, int BH, int d, long long cap,
            long long row_begin, long long rows, long long pos_begin, long long dst_cap, long long dst_row_begin,
            const __grid_constant__ RopeFreq freq) {
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
    for (int i = 0; i < NP; ++i) rope_cos_sin(pos, freq.turns[p0 + i], c[i], s[i]);
    // blockIdx.y splits the (batch, head) range when there are too few rows to fill the device
    const int bh_per = (BH + (int)gridDim.y - 1) / (int)gridDim.y;
    const int bh_begin = (int)blockIdx.y * bh_per, bh_end = min(BH, bh_begin + bh_per);
#pragma unroll 4
    for (int bh = bh_begin; bh < bh_end; ++bh) {
      const long long off = ((long long)bh * cap + row_begin + r) * d;
      const long long dof = ((long long)bh * dst_cap + dst_row_begin + r) * d;
      if (INTERLEAVED) {
        uint4 v = *reinterpret_cast<const uint4*>(src + off + 2 * p0);
        T* e = reinterpret_cast<T*>(&v);
#pragma unroll
        for (int i = 0; i < NP; ++i) {
          float ra, rb;
          rope_rotate(to_float(e[2 * i]), to_float(e[2 * i + 1]), c[i], s[i], ra, rb);
          e[2 * i] = from_float<T>(ra);
          e[2 * i + 1] = from_float<T>(rb);
        }
        *reinterpret_cast<uint4*>(dst + dof + 2 * p0) = v;
      } else {
        uint4 lo = *reinterpret_cast<const uint4*>(src + off + p0);
        uint4 hi = *reinterpret_cast<const uint4*>(src + off + d / 2 + p0);
        T* a = reinterpret_cast<T*>(&lo);
        T* b = reinterpret_cast<T*>(&hi);
#pragma unroll
        for (int i = 0; i < NP; ++i) {
          float ra, rb;
          rope_rotate(to_float(a[i]), to_float(b[i]), c[i], s[i], ra, rb);
          a[i] = from_float<T>(ra);
          b[i] = from_float<T>(rb);
        }
        *reinterpret_cast<uint4*>(dst + dof + p0) = lo;
        *reinterpret_cast<uint4*>(dst + dof + d / 2 + p0) = hi;
      }
    }
  }
}

inline RopeFreq rope_freq(int d, double base) {
  RopeFreq freq;
  for (int i = 0; i < d / 2; ++i) freq.turns[i] = pow(base, -2.0 * i / d) / 6.283185307179586476925;
  return freq;
}

inline int launch_rope_table(float2* tab, long long rows, int d, long long pos_begin, double base, cudaStream_t st) {
  if (rows == 0) return REFORM_OK;
  const long long items = rows * (d / 2);
  long long blocks = (items + 255) / 256;
  const long long cap_blocks = (long long)num_sms() * 16;
  rope_table_kernel<<<(int)(blocks < cap_blocks ? blocks : cap_blocks), 256, 0, st>>>(tab, rows, d / 2, pos_begin,
                                                                                       rope_freq(d, base));
  count_launch();
  return check_launch();
}

// dst_cap / dst_row_begin: row capacity per (batch, head) of dst and the row of dst that receives
// the first rotated row (negative dst_cap: same layout as src).
template <typename T>
inline int launch_rope(const void* src, void* dst, int BH, int d, long long cap, long long row_begin,
                       long long rows, long long pos_begin, double base, bool interleaved,
                       cudaStream_t st, long long dst_cap = -1, long long dst_row_begin = 0) {
  if (rows == 0 || BH == 0) return REFORM_OK;
  if (dst_cap < 0) { dst_cap = cap; dst_row_begin = row_begin; }
  const int np = 16 / (int)sizeof(T) / (interleaved ? 2 : 1);
  const long long items = rows * ((d / 2) / np);
  long long blocks = (items + 255) / 256;
  const long long cap_blocks = (long long)num_sms() * 16;
  const int grid_x = (int)(blocks < cap_blocks ? blocks : cap_blocks);
  // few rows (a score window, a decode step): spread the (batch, head) loop over blockIdx.y as well
  int grid_y = 1;
  while (grid_x * grid_y < 2 * num_sms() && grid_y < BH) grid_y *= 2;
  if (grid_y > BH) grid_y = BH;
  const dim3 grid(grid_x, grid_y);
  const RopeFreq freq = rope_freq(d, base);
  if (interleaved)
    rope_kernel<T, true><<<grid, 256, 0, st>>>((const T*)src, (T*)dst, BH, d, cap, row_begin, rows, pos_begin,
                                               dst_cap, dst_row_begin, freq);
  else
    rope_kernel<T, false><<<grid, 256, 0, st>>>((const T*)src, (T*)dst, BH, d, cap, row_begin, rows, pos_begin,
                                                dst_cap, dst_row_begin, freq);
  count_launch();
  return check_launch();
}

}  // namespace reform
