// Microbenchmark of the tcgen05.mma issue path on sm_100a (a stand-alone
// program, not part of libreform.so): what one issuing thread can feed the
// tensor pipe, which is what bounds the chunk-step attention and the
// similarity scan.  One block per SM; the issuing thread times itself with
// clock64.  Build and run: python -m paper_2506_01215_b200.mma_issue_bench
//
//   rate   cycles per MMA instruction (M = 128, K = 16, bf16), back to back,
//          against N and the operand form
//   ahead  thread time to issue n MMAs into an idle pipe, and until their
//          commit arrives: how far the thread can run ahead of the pipe
//   extra  the same loop with a satisfied mbarrier wait, a commit or a tcgen05
//          fence between groups of eight, and with eight busy neighbour warps
#include <cstdio>
#include <cstdlib>
#include <cuda_runtime.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

using namespace reform;

constexpr uint32_t kTile = 128 * 128 * 2;

struct Shared {
  uint8_t* smem;
  uint64_t* bar;        // [4]
  uint32_t* slot;
  volatile int* flags;  // [0] abort, [1] done
};

__device__ __forceinline__ Shared carve(uint8_t* raw, uint32_t operand_bytes) {
  Shared s;
  s.smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
  s.bar = reinterpret_cast<uint64_t*>(s.smem + operand_bytes);
  s.slot = reinterpret_cast<uint32_t*>(s.bar + 4);
  s.flags = reinterpret_cast<volatile int*>(s.slot + 1);
  return s;
}

// operands: seeded bf16 values in about [-2, 2) (zeros give the same timings)
__device__ __forceinline__ uint32_t setup(const Shared& s, uint32_t operand_bytes) {
  for (uint32_t i = threadIdx.x; i < operand_bytes / 4; i += blockDim.x) {
    uint32_t h = (i + 1) * 2654435761u;
    h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
    reinterpret_cast<uint32_t*>(s.smem)[i] = (h & 0x807F807Fu) | 0x3F003F00u;
  }
  if (threadIdx.x == 0) {
    for (int i = 0; i < 4; ++i) ptx::mbar_init(s.bar + i, 1);
    s.flags[0] = 0;
    s.flags[1] = 0;
    ptx::fence_barrier_init();
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (threadIdx.x < 32) { ptx::tmem_alloc(s.slot, 512); ptx::tmem_relinquish(); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  return *s.slot;
}

__device__ __forceinline__ void teardown(uint32_t tm) {
  ptx::tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) { ptx::tc_fence_after(); ptx::tmem_dealloc(tm, 512); }
}

// FORM 0: SS, both K-major (the Q K^T form)   1: SS, B MN-major   2: TS (A from TMEM), B K-major
//      3: TS, B MN-major (the P V form)
template <int N, int FORM>
__global__ void __launch_bounds__(128, 1) rate_kernel(int rounds, long long* out) {
  extern __shared__ uint8_t raw[];
  constexpr uint32_t kB = N * 128 * 2;
  Shared s = carve(raw, kTile + kB);
  const uint32_t tm = setup(s, kTile + kB);
  if (threadIdx.x == 0) {
    const uint32_t aA = ptx::smem_u32(s.smem), aB = aA + kTile;
    constexpr uint32_t idesc = ptx::idesc_bf16(128, N, false, FORM == 1 || FORM == 3);
    constexpr int nacc = N <= 128 ? 2 : 1;
    const uint32_t ap = tm + 384;
    uint32_t a_lo[8], b_lo[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      a_lo[k] = ptx::smem_desc_lo(aA + (k >> 2) * (kTile / 2) + (k & 3) * 32, 16);
      b_lo[k] = (FORM == 0 || FORM == 2) ? ptx::smem_desc_lo(aB + (k >> 2) * (kB / 2) + (k & 3) * 32, 16)
                                         : ptx::smem_desc_lo(aB + k * 2048, kB / 2);
    }
    const long long t0 = clock64();
#pragma unroll 1
    for (int r = 0; r < rounds; r += 2) {
#pragma unroll
      for (int rr = 0; rr < 2; ++rr) {
        const uint32_t d = tm + (nacc == 2 ? N * rr : 0);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          if (FORM < 2) ptx::mma_ss_c<1>(d, a_lo[k], b_lo[k], ptx::kDescHiSw128, idesc);
          else ptx::mma_ts_c<1>(d, ap + 8 * k, b_lo[k], ptx::kDescHiSw128, idesc);
        }
      }
    }
    ptx::mma_commit(s.bar);
    ptx::mbar_wait(s.bar, 0, s.flags);
    if (blockIdx.x == 0) out[0] = clock64() - t0;
  }
  teardown(tm);
}

template <int NMMA>
__global__ void __launch_bounds__(128, 1) ahead_kernel(long long* out) {
  extern __shared__ uint8_t raw[];
  Shared s = carve(raw, 2 * kTile);
  const uint32_t tm = setup(s, 2 * kTile);
  if (threadIdx.x == 0) {
    const uint32_t aA = ptx::smem_u32(s.smem), aB = aA + kTile;
    constexpr uint32_t idesc = ptx::idesc_bf16(128, 128, false, false);
    uint32_t a_lo[8], b_lo[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      a_lo[k] = ptx::smem_desc_lo(aA + (k >> 2) * (kTile / 2) + (k & 3) * 32, 16);
      b_lo[k] = ptx::smem_desc_lo(aB + (k >> 2) * (kTile / 2) + (k & 3) * 32, 16);
    }
    long long issue = 0, total = 0;
    for (int rep = 0; rep < 64; ++rep) {
      const long long t0 = clock64();
#pragma unroll
      for (int i = 0; i < NMMA; ++i)
        ptx::mma_ss_c<1>(tm + 128 * ((i >> 3) & 1), a_lo[i & 7], b_lo[i & 7], ptx::kDescHiSw128, idesc);
      const long long t1 = clock64();
      ptx::mma_commit(s.bar);
      ptx::mbar_wait(s.bar, rep & 1, s.flags);
      const long long t2 = clock64();
      issue += t1 - t0;
      total += t2 - t0;
    }
    if (blockIdx.x == 0) { out[0] = issue / 64; out[1] = total / 64; }
  }
  teardown(tm);
}

// EXTRA 0: nothing between groups of eight MMAs   1: tcgen05.fence::after_thread_sync   2: a commit
//       3: an arrival on an mbarrier and the (then satisfied) wait for it
// busy: warps 1..busy run a loop of ex2 and FMAs until the issuing thread is done
template <int EXTRA>
__global__ void __launch_bounds__(384, 1) extra_kernel(int rounds, int busy, long long* out) {
  extern __shared__ uint8_t raw[];
  Shared s = carve(raw, 3 * kTile);
  const uint32_t tm = setup(s, 3 * kTile);
  if (threadIdx.x >= 32 && threadIdx.x < 32 + 32 * busy) {
    float acc = threadIdx.x, x = 0.5f;
    while (!s.flags[1]) {
#pragma unroll
      for (int i = 0; i < 64; ++i) { acc = fmaf(acc, 0.999f, ptx::ex2(x)); x = fmaf(x, 0.5f, 0.25f); }
    }
    if (acc == 123.f) out[7] = 1;
  }
  if (threadIdx.x == 0) {
    const uint32_t aA = ptx::smem_u32(s.smem), aB = aA + kTile;
    constexpr uint32_t idesc = ptx::idesc_bf16(128, 128, false, false);
    const uint32_t a_lo = ptx::smem_desc_lo(aA, 16);
    const long long t0 = clock64();
#pragma unroll 1
    for (int r = 0; r < rounds; ++r) {
      const int st = r & 1;  // stage offset from the loop counter, as the attention kernel has it
      const uint32_t b_lo = ptx::smem_desc_lo(aB + st * kTile, 16);
      const uint32_t d = tm + 128 * st;
      if (EXTRA == 1) ptx::tc_fence_after();
      if (EXTRA == 2) ptx::mma_commit(s.bar + 2 + st);
      if (EXTRA == 3) { ptx::mbar_arrive(s.bar + 1); if (!ptx::mbar_wait(s.bar + 1, r & 1, s.flags)) break; }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const uint32_t off = (k >> 2) * (kTile >> 5) + (k & 3) * 2;
        ptx::mma_ss_c<1>(d, a_lo + off, b_lo + off, ptx::kDescHiSw128, idesc);
      }
    }
    ptx::mma_commit(s.bar);
    ptx::mbar_wait(s.bar, 0, s.flags);
    if (blockIdx.x == 0) out[0] = clock64() - t0;
    s.flags[1] = 1;
  }
  teardown(tm);
}

static void check(const char* what) {
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) { printf("%s: %s\n", what, cudaGetErrorString(e)); exit(1); }
}

template <int N, int FORM>
static void run_rate(long long* out) {
  const int smem = kTile + N * 128 * 2 + 2048;
  cudaFuncSetAttribute(rate_kernel<N, FORM>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  rate_kernel<N, FORM><<<148, 128, smem>>>(2000, out);
  check("rate");
  static const char* names[] = {"SS K-major", "SS, B MN-major", "TS, B K-major", "TS, B MN-major"};
  printf("rate   N %3d  %-15s  %6.1f cycles per MMA (ideal %d)\n", N, names[FORM], (double)out[0] / 2000 / 8, N / 2);
}

template <int NMMA>
static void run_ahead(long long* out) {
  const int smem = 2 * kTile + 2048;
  cudaFuncSetAttribute(ahead_kernel<NMMA>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  ahead_kernel<NMMA><<<148, 128, smem>>>(out);
  check("ahead");
  printf("ahead  %2d MMAs: issued after %4lld cycles, complete after %4lld\n", NMMA, out[0], out[1]);
}

template <int EXTRA>
static void run_extra(long long* out, int busy) {
  const int smem = 3 * kTile + 2048;
  cudaFuncSetAttribute(extra_kernel<EXTRA>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  extra_kernel<EXTRA><<<148, 384, smem>>>(2000, busy, out);
  check("extra");
  static const char* names[] = {"nothing", "tcgen05 fence", "commit", "arrive + satisfied wait"};
  printf("extra  %-24s per 8 MMAs, %2d busy warps: %6.1f cycles per MMA\n", names[EXTRA], busy,
         (double)out[0] / 2000 / 8);
}

int main() {
  long long* out;
  if (cudaMallocManaged(&out, 8 * sizeof(long long)) != cudaSuccess) { printf("no device memory\n"); return 1; }
  run_rate<64, 0>(out); run_rate<64, 2>(out);
  run_rate<128, 0>(out); run_rate<128, 1>(out); run_rate<128, 2>(out); run_rate<128, 3>(out);
  run_rate<256, 0>(out); run_rate<256, 2>(out);
  run_ahead<1>(out); run_ahead<2>(out); run_ahead<4>(out); run_ahead<8>(out); run_ahead<16>(out); run_ahead<32>(out);
  for (int busy : {0, 8}) { run_extra<0>(out, busy); run_extra<1>(out, busy); run_extra<2>(out, busy); run_extra<3>(out, busy); }
  return 0;
}
