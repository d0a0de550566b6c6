// Tensor-core similarity scan (Sec. 3.3) for bf16 banks whose row width is a
// multiple of 64: the bank is streamed once from HBM by TMA into a deep
// shared-memory ring (128 tokens x 64 columns per stage, 128-byte swizzle) and
// multiplied against the query embeddings, which stay resident in shared
// memory for the whole kernel, by tcgen05 MMAs (M = 128 tokens, N = padded
// query count, fp32 accumulators in tensor memory, two buffers).  Each of 128
// epilogue threads owns one token (one TMEM lane), takes the maximum over the
// queries and writes ts[token].  The arithmetic (nq flop per byte) never shows:
// the kernel is a pure HBM stream for any nq up to 64.
//
// Persistent blocks, one per SM: warp 0 = TMA producer, warp 1 = MMA issuer
// and TMEM owner, warps 2..5 = epilogue.  All waits are bounded.
#pragma once

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace reform {

constexpr int kScanThreads = 192;
constexpr int kScanTileTokens = 128;
constexpr uint32_t kScanStageBytes = 128 * 128;   // 128 tokens x 64 bf16
constexpr uint32_t kScanTmemCols = 128;           // two accumulators of up to 64 columns
constexpr size_t kScanSmemLimit = 226 * 1024;  // dynamic shared memory this kernel may ask for

__device__ __forceinline__ void tmem_ld16_sync(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}

__global__ void __launch_bounds__(kScanThreads, 1)
scan_sm100_kernel(const __grid_constant__ CUtensorMap tmBank, const __grid_constant__ CUtensorMap tmQ,
                  float* __restrict__ ts, long long N, int E, int nq, int n_pad, int n_stages, float scale,
                  int tiles_per_seq, int32_t* dev_status) {
  extern __shared__ uint8_t smem_raw[];
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // a dependent selection may be placed as SMs free up
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int KB = E / 64;
  const uint32_t q_box_bytes = (uint32_t)n_pad * 128;
  uint8_t* sQ = smem;                                  // [KB] boxes of n_pad rows x 128 B
  uint8_t* sA = smem + (size_t)KB * q_box_bytes;       // [n_stages] stages of 16 KB
  uint64_t* bars = reinterpret_cast<uint64_t*>(sA + (size_t)n_stages * kScanStageBytes);
  uint64_t* q_full = bars;
  uint64_t* a_full = bars + 1;                 // [n_stages]
  uint64_t* a_empty = a_full + n_stages;       // [n_stages]
  uint64_t* acc_full = a_empty + n_stages;     // [2]
  uint64_t* acc_empty = acc_full + 2;          // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.y;

  if (threadIdx.x == 0) {
    ptx::mbar_init(q_full, 1);
    for (int s = 0; s < n_stages; ++s) {
      ptx::mbar_init(a_full + s, 1);
      ptx::mbar_init(a_empty + s, 1);
    }
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(acc_full + s, 1);
      ptx::mbar_init(acc_empty + s, 128);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, kScanTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      ptx::prefetch_tmap(&tmBank);
      ptx::prefetch_tmap(&tmQ);
      ptx::mbar_expect_tx(q_full, (uint32_t)KB * q_box_bytes);
      for (int kb = 0; kb < KB; ++kb) ptx::tma_load_3d(sQ + (size_t)kb * q_box_bytes, &tmQ, q_full, 64 * kb, 0, b);
      uint32_t it = 0, s = 0, ph = 0;  // stage uses so far; stage and phase of the next one
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < tiles_per_seq; tile += gridDim.x) {
        for (int kb = 0; kb < KB; ++kb, ++it) {
          if (!ptx::mbar_wait(a_empty + s, ph ^ 1, abort_flag)) { ok = false; break; }
          ptx::mbar_expect_tx(a_full + s, kScanStageBytes);
          ptx::tma_load_3d(sA + (size_t)s * kScanStageBytes, &tmBank, a_full + s, 64 * kb, tile * kScanTileTokens, b);
          if (++s == (uint32_t)n_stages) { s = 0; ph ^= 1; }
        }
      }
      if (*abort_flag) {  // let copies in flight land before shared memory is released
        volatile int ignore = 0;
        ptx::mbar_wait(q_full, 0, &ignore);
        for (uint32_t u = 1; u <= (uint32_t)n_stages && u <= it; ++u) {
          const uint32_t last = it - u;
          ptx::mbar_wait(a_full + last % n_stages, (last / n_stages) & 1, &ignore);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = ptx::idesc_bf16(128, n_pad, false, false);
      const uint32_t aQ = ptx::smem_u32(sQ), aA = ptx::smem_u32(sA);
      bool ok = ptx::mbar_wait(q_full, 0, abort_flag);
      // the tensor pipe runs only while this thread issues: stage, phase and descriptor words are
      // stepped, not recomputed, and the accumulate flag of all but a tile's first MMA is a constant
      const uint32_t a_lo0 = ptx::smem_desc_lo(aA, 16), q_lo0 = ptx::smem_desc_lo(aQ, 16);
      const uint32_t stage_step = kScanStageBytes >> 4, q_step = (uint32_t)q_box_bytes >> 4;
      uint32_t i = 0, s = 0, ph = 0, a_lo = a_lo0;
      for (int tile = blockIdx.x; ok && tile < tiles_per_seq; tile += gridDim.x, ++i) {
        const uint32_t buf = i & 1;
        const uint32_t d = tmem_base + buf * 64;
        if (!ptx::mbar_wait(acc_empty + buf, ((i >> 1) & 1) ^ 1, abort_flag)) break;
        uint32_t q_lo = q_lo0;
        for (int kb = 0; kb < KB; ++kb) {
          if (!ptx::mbar_wait(a_full + s, ph, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after();
          if (kb == 0) ptx::mma_ss_c<0>(d, a_lo, q_lo, ptx::kDescHiSw128, idesc);
          else ptx::mma_ss_c<1>(d, a_lo, q_lo, ptx::kDescHiSw128, idesc);
#pragma unroll
          for (int k = 1; k < 4; ++k) ptx::mma_ss_c<1>(d, a_lo + 2 * k, q_lo + 2 * k, ptx::kDescHiSw128, idesc);
          ptx::mma_commit(a_empty + s);
          q_lo += q_step;
          a_lo += stage_step;
          if (++s == (uint32_t)n_stages) { s = 0; ph ^= 1; a_lo = a_lo0; }
        }
        if (ok) ptx::mma_commit(acc_full + buf);
      }
    }
  } else {
    const int sub = warp & 3;
    const uint32_t lane_addr = (uint32_t)(32 * sub) << 16;
    uint32_t i = 0;
    for (int tile = blockIdx.x; tile < tiles_per_seq; tile += gridDim.x, ++i) {
      const uint32_t buf = i & 1;
      if (!ptx::mbar_wait(acc_full + buf, (i >> 1) & 1, abort_flag)) break;
      ptx::tc_fence_after();
      float best = -INFINITY;
      for (int c = 0; c < n_pad; c += 16) {
        uint32_t v[16];
        tmem_ld16_sync(tmem_base + buf * 64 + lane_addr + c, v);
#pragma unroll
        for (int q = 0; q < 16; ++q)
          if (c + q < nq) best = fmaxf(best, __uint_as_float(v[q]) * scale);
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(acc_empty + buf);
      const long long token = (long long)tile * kScanTileTokens + 32 * sub + lane;
      if (token < N) ts[(long long)b * N + token] = best;
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, kScanTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag) report_device_error(dev_status, REFORM_DEV_TIMEOUT);
}

// Returns REFORM_ERR_UNSUPPORTED when the shape does not fit this kernel (the caller then uses
// the generic scan).
inline int launch_scan_sm100(const void* bank, const void* queries, float* ts, int B, long long N,
                             long long N_cap, int E, int nq, float scale, int32_t* dev_status,
                             cudaStream_t st) {
  if (E % 64 != 0 || nq > 64 || N > 0x7fffff00LL) return REFORM_ERR_UNSUPPORTED;
  const int n_pad = (nq + 15) / 16 * 16;
  const size_t q_bytes = (size_t)n_pad * E * 2;
  const size_t fixed = 1024 + 512;
  if (q_bytes + 3 * kScanStageBytes + fixed > kScanSmemLimit) return REFORM_ERR_UNSUPPORTED;
  int n_stages = (int)((kScanSmemLimit - fixed - q_bytes) / kScanStageBytes);
  if (n_stages > 10) n_stages = 10;
  const size_t smem = q_bytes + (size_t)n_stages * kScanStageBytes + fixed;
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return REFORM_ERR_UNSUPPORTED;
  CUtensorMap tmBank, tmQ;
  {
    cuuint64_t dims[3] = {(cuuint64_t)E, (cuuint64_t)N, (cuuint64_t)B};
    cuuint64_t strides[2] = {(cuuint64_t)E * 2, (cuuint64_t)N_cap * E * 2};
    cuuint32_t box[3] = {64, 128, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    if (fn(&tmBank, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(bank), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return REFORM_ERR_UNSUPPORTED;
    cuuint64_t qdims[3] = {(cuuint64_t)E, (cuuint64_t)nq, (cuuint64_t)B};
    cuuint64_t qstrides[2] = {(cuuint64_t)E * 2, (cuuint64_t)nq * E * 2};
    cuuint32_t qbox[3] = {64, (cuuint32_t)n_pad, 1};
    if (fn(&tmQ, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(queries), qdims, qstrides, qbox, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return REFORM_ERR_UNSUPPORTED;
  }
  const int tiles = (int)((N + kScanTileTokens - 1) / kScanTileTokens);
  int per_b = (num_sms() + B - 1) / B;
  if (per_b > tiles) per_b = tiles;
  if (per_b < 1) per_b = 1;
  cudaFuncSetAttribute(scan_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  dim3 grid(per_b, B);
  scan_sm100_kernel<<<grid, kScanThreads, smem, st>>>(tmBank, tmQ, ts, N, E, nq, n_pad, n_stages, scale, tiles,
                                                     dev_status);
  count_launch();
  return check_launch();
}

}  // namespace reform
