// Context-embedding append (Sec. 3.2, "Combining multiple heads"): every
// selected head state of a token is divided by its L2 norm and stored in its
// slot of the token's bank row.  HBM-bound: one read of the selected states,
// one write of the bank rows.  One warp owns one (token, slot) vector; the
// warps of a block cover neighbouring slots of the same token so a block
// writes whole bank rows.
#pragma once

#include "common.cuh"

namespace reform {

struct EmbedSel {
  const void* src[REFORM_MAX_SEL];  // base of the [B,H,Lc,d] state tensor of that kind
  int H[REFORM_MAX_SEL];
  int head[REFORM_MAX_SEL];
  int slot[REFORM_MAX_SEL];
  int n_sel;
};

constexpr int kEmbedMaxVec = 4;  // vectors of 4 elements per lane: d <= 32 * 4 * 4 = 512

template <typename T>
struct Vec4;
template <>
struct Vec4<float> {
  using type = float4;
  __device__ static void load(const float* p, float (&x)[4]) {
    float4 v = *reinterpret_cast<const float4*>(p);
    x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
  }
  __device__ static void store(float* p, const float (&x)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
  }
};
template <>
struct Vec4<__nv_bfloat16> {
  __device__ static void load(const __nv_bfloat16* p, float (&x)[4]) {
    uint2 v = *reinterpret_cast<const uint2*>(p);
    __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&v.x);
    __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&v.y);
    x[0] = __low2float(a); x[1] = __high2float(a); x[2] = __low2float(b); x[3] = __high2float(b);
  }
  __device__ static void store(__nv_bfloat16* p, const float (&x)[4]) {
    __nv_bfloat162 a = __floats2bfloat162_rn(x[0], x[1]);
    __nv_bfloat162 b = __floats2bfloat162_rn(x[2], x[3]);
    uint2 v;
    v.x = *reinterpret_cast<uint32_t*>(&a);
    v.y = *reinterpret_cast<uint32_t*>(&b);
    *reinterpret_cast<uint2*>(p) = v;
  }
};

// Arithmetic type of the norm and the quotient.  A bf16 bank takes fp32 (its 8-bit significand
// hides fp32 rounding: the result is within one bf16 unit of the exact quotient).  An fp32 bank
// takes fp64, so that the single rounding to fp32 is the only error (within one fp32 unit).
template <typename T>
struct EmbedAcc { using type = float; };
template <>
struct EmbedAcc<float> { using type = double; };

__device__ __forceinline__ float embed_norm(float ss, float eps) { return fmaxf(sqrtf(ss), eps); }
__device__ __forceinline__ double embed_norm(double ss, float eps) { return fmax(sqrt(ss), (double)eps); }

template <typename T>
__global__ void __launch_bounds__(256)
embed_append_kernel(EmbedSel sel, T* __restrict__ bank, int B, int Lc, int d, int E,
                    long long N_cap, long long token_offset, float eps) {
  using Acc = typename EmbedAcc<T>::type;
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long n_warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const long long items = (long long)B * Lc * sel.n_sel;
  const int nvec = d >> 2;
  for (long long it = warp; it < items; it += n_warps) {
    int s = (int)(it % sel.n_sel);
    long long bt = it / sel.n_sel;
    int t = (int)(bt % Lc);
    int b = (int)(bt / Lc);
    const T* x = reinterpret_cast<const T*>(sel.src[s]) +
                 (((long long)b * sel.H[s] + sel.head[s]) * Lc + t) * d;
    float v[kEmbedMaxVec][4];
    Acc ss = 0;
#pragma unroll
    for (int c = 0; c < kEmbedMaxVec; ++c) {
      int vi = lane + 32 * c;
      if (vi < nvec) {
        Vec4<T>::load(x + 4 * vi, v[c]);
#pragma unroll
        for (int i = 0; i < 4; ++i) ss += (Acc)v[c][i] * (Acc)v[c][i];
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    const Acc nrm = embed_norm(ss, eps);
    T* y = bank + ((long long)b * N_cap + token_offset + t) * E + (long long)sel.slot[s] * d;
#pragma unroll
    for (int c = 0; c < kEmbedMaxVec; ++c) {
      int vi = lane + 32 * c;
      if (vi < nvec) {
        float o[4] = {(float)((Acc)v[c][0] / nrm), (float)((Acc)v[c][1] / nrm), (float)((Acc)v[c][2] / nrm),
                      (float)((Acc)v[c][3] / nrm)};
        Vec4<T>::store(y + 4 * vi, o);
      }
    }
  }
}


// Fast path for vectors of 4, 8, 16 or 32 sixteen-byte chunks (bf16 d = 32..256,
// fp32 d = 16..128): LP lanes own one vector, a warp works on 32/LP vectors at
// a time and keeps four such groups in flight.
template <typename T, int LP>
__global__ void __launch_bounds__(256)
embed_append_vec_kernel(EmbedSel sel, T* __restrict__ bank, int B, int Lc, int d, int E,
                        long long N_cap, long long token_offset, float eps) {
  using Acc = typename EmbedAcc<T>::type;
  constexpr int VPW = 32 / LP, U = 4, EPC = 16 / (int)sizeof(T);
  const int lane = threadIdx.x & 31;
  const int sub = lane % LP, which = lane / LP;
  const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint32_t n_warps = (gridDim.x * blockDim.x) >> 5;
  const uint32_t n_sel = (uint32_t)sel.n_sel;
  const uint32_t items = (uint32_t)B * (uint32_t)Lc * n_sel;  // < 2^31, checked by the launcher
  for (uint32_t it0 = warp * (VPW * U); it0 < items; it0 += n_warps * (VPW * U)) {
    uint4 x[U];
    T* y[U];
    bool ok[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t it = it0 + u * VPW + which;
      ok[u] = it < items;
      x[u] = make_uint4(0, 0, 0, 0);
      y[u] = nullptr;
      if (ok[u]) {
        const uint32_t bt = it / n_sel, s = it - bt * n_sel;
        const uint32_t b = bt / (uint32_t)Lc, t = bt - b * (uint32_t)Lc;
        const T* src = reinterpret_cast<const T*>(sel.src[s]) +
                       (((long long)b * sel.H[s] + sel.head[s]) * Lc + t) * d;
        x[u] = __ldcs(reinterpret_cast<const uint4*>(src) + sub);
        y[u] = bank + ((long long)b * N_cap + token_offset + t) * E + (long long)sel.slot[s] * d + sub * EPC;
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float f[EPC];
      const T* e = reinterpret_cast<const T*>(&x[u]);
      Acc ss = 0;
#pragma unroll
      for (int i = 0; i < EPC; ++i) {
        f[i] = to_float(e[i]);
        ss += (Acc)f[i] * (Acc)f[i];
      }
#pragma unroll
      for (int o = LP / 2; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      uint4 w;
      T* o4 = reinterpret_cast<T*>(&w);
      if (sizeof(T) == 4) {  // fp32 bank: fp64 quotient, one rounding
        const Acc nrm = embed_norm(ss, eps);
#pragma unroll
        for (int i = 0; i < EPC; ++i) o4[i] = from_float<T>((float)((Acc)f[i] / nrm));
      } else {
        const float inv = 1.0f / embed_norm((float)ss, eps);
#pragma unroll
        for (int i = 0; i < EPC; ++i) o4[i] = from_float<T>(f[i] * inv);
      }
      if (ok[u]) __stcs(reinterpret_cast<uint4*>(y[u]), w);
    }
  }
}

template <typename T>
inline int launch_embed(const EmbedSel& sel, void* bank, int B, int Lc, int d, int E,
                        long long N_cap, long long token_offset, float eps, cudaStream_t st) {
  long long items = (long long)B * Lc * sel.n_sel;
  if (items == 0) return REFORM_OK;
  const int chunks = d * (int)sizeof(T) / 16;
  const bool vec_ok = (d * sizeof(T)) % 16 == 0 && items < (1LL << 31) &&
                      (chunks == 4 || chunks == 8 || chunks == 16 || chunks == 32);
  if (vec_ok) {
    long long per_warp = (32 / chunks) * 4;
    long long blocks = (items + 8 * per_warp - 1) / (8 * per_warp);
    long long cap = (long long)num_sms() * 8;
    int grid = (int)(blocks < cap ? blocks : cap);
#define REFORM_EMBED_CASE(LP)                                                                          \
  case LP:                                                                                             \
    embed_append_vec_kernel<T, LP><<<grid, 256, 0, st>>>(sel, (T*)bank, B, Lc, d, E, N_cap,           \
                                                         token_offset, eps);                           \
    break;
    switch (chunks) {
      REFORM_EMBED_CASE(4)
      REFORM_EMBED_CASE(8)
      REFORM_EMBED_CASE(16)
      REFORM_EMBED_CASE(32)
    }
#undef REFORM_EMBED_CASE
    count_launch();
    return check_launch();
  }
  long long blocks = (items + 7) / 8;  // 8 warps per block
  long long cap = (long long)num_sms() * 16;
  int grid = (int)(blocks < cap ? blocks : cap);
  embed_append_kernel<T><<<grid, 256, 0, st>>>(sel, (T*)bank, B, Lc, d, E, N_cap, token_offset, eps);
  count_launch();
  return check_launch();
}

}  // namespace reform
