// Tensor-core chunk step for bf16, head dimension 128 (sm_100a: tcgen05 MMA
// with TMEM accumulators, operands staged by TMA with 128-byte swizzle).
//
//   attn2_sm100_kernel  Sec. 3.1 chunk forward.  One block per SM owns two
//     128-row query tiles and walks the visible keys [cache ; chunk prefix] in
//     128-key tiles that both query tiles share:  S = Q K^T (SS MMA, fp32 in
//     TMEM) -> online softmax by 128 threads per tile, one query row each,
//     straight out of TMEM -> P (bf16) written back into the TMEM columns S
//     occupied -> O += P V (A operand from TMEM, V from shared memory,
//     MN-major).  O stays in TMEM for the whole walk and is rescaled only when
//     a row maximum grows by more than 2^8.  While one tile's softmax runs, the
//     other tile's MMAs keep the tensor pipe busy.  Details at the kernel.
//
//   score_sm100_kernel  H2O eviction score (Sec. 3.1; Sec. 4 "Common setup").
//     Key-stationary second pass: a block owns 128 keys (TMEM lanes) of one KV
//     head and revisits the trailing score_window query rows of the group's G
//     query heads: S^T = K Q^T, p = exp2(s*c - lse), summed along the queries
//     by the thread that owns the key.  One owner per key: no atomics, and the
//     result does not depend on scheduling.  Roles per block (192 threads):
//     warp 0 = TMA producer (one lane), warp 1 = MMA issuer (one lane) and
//     TMEM owner, warps 2..5 = 128 epilogue threads (TMEM lane = 32 * (warp %
//     4) + lane).
//
// All waits are bounded.
#pragma once

#include "common.cuh"
#include "chunk_simt.cuh"
#include "rope.cuh"
#include "sm100_ptx.cuh"

namespace reform {

constexpr int kT = 128;                   // tile edge: query rows, keys, head dimension
constexpr int kSm100Threads = 192;
constexpr uint32_t kTileBytes = kT * kT * 2;  // one 128 x 128 bf16 tile
constexpr uint32_t kHalfBytes = kTileBytes / 2;  // one TMA box: 128 rows x 64 columns
constexpr uint32_t kTmemCols = 256;
constexpr float kRescaleThreshold = 8.0f;  // log2 units

constexpr size_t kScoreSmemBytes = 3 * kTileBytes + 1024 + 256 + 2 * kT * sizeof(float);

__device__ __forceinline__ uint8_t* align_1024(uint8_t* p) {
  return reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~uintptr_t(1023));
}

// S (or S^T) = A B^T for two K-major 128 x 128 bf16 tiles in shared memory: 8 MMAs of K = 16
__device__ __forceinline__ void issue_kmajor_128x128x128(uint32_t d_tmem, uint32_t a_smem, uint32_t b_smem) {
  constexpr uint32_t idesc = ptx::idesc_bf16(kT, kT, false, false);
  const uint32_t a_lo = ptx::smem_desc_lo(a_smem, 16), b_lo = ptx::smem_desc_lo(b_smem, 16);
  ptx::mma_ss_c<0>(d_tmem, a_lo, b_lo, ptx::kDescHiSw128, idesc);
#pragma unroll
  for (int k = 1; k < 8; ++k) {
    constexpr uint32_t box = kHalfBytes >> 4;              // 64-column box, then 32 B per K = 16 step
    const uint32_t off = (k >> 2) * box + (k & 3) * 2;
    ptx::mma_ss_c<1>(d_tmem, a_lo + off, b_lo + off, ptx::kDescHiSw128, idesc);
  }
}

// O (+)= P V for keys [16 * K0, 16 * K0 + 64) of a key tile: P (bf16) from TMEM, V MN-major in shared memory
template <int K0>
__device__ __forceinline__ void issue_pv_half(uint32_t o_tmem, uint32_t p_tmem, uint32_t v_lo, bool first) {
  constexpr uint32_t idesc = ptx::idesc_bf16(kT, kT, false, true);
  if (K0 == 0 && first) ptx::mma_ts_c<0>(o_tmem, p_tmem, v_lo, ptx::kDescHiSw128, idesc);
  else ptx::mma_ts_c<1>(o_tmem, p_tmem + 8 * K0, v_lo + K0 * 128, ptx::kDescHiSw128, idesc);
#pragma unroll
  for (int k = K0 + 1; k < K0 + 4; ++k)
    ptx::mma_ts_c<1>(o_tmem, p_tmem + 8 * k, v_lo + k * 128, ptx::kDescHiSw128, idesc);
}

// ---------------------------------------------------------------------------
// Two query tiles per block, one block per SM.  The two tiles (normally the
// same 128 query rows of two query heads of one KV group, so their walks are
// identical) share every K/V tile a single TMA load brings in: half the
// L2 -> shared-memory traffic per flop of a one-tile block.  Each tile has its
// own S/P and O accumulators in tensor memory (4 x 128 = all 512 columns) and
// its own warpgroup of 128 softmax threads holding a whole 128-wide row in
// registers; the MMA issuer alternates between the tiles, so one tile's
// softmax hides behind the other tile's two MMAs.
// ---------------------------------------------------------------------------
constexpr int kAttn2Threads = 384;  // warps 0-3 / 4-7: softmax of tile 0 / 1; warp 8: TMA; warp 9: MMA
// setmaxnreg only redistributes the registers the block was launched with (what one warpgroup gives
// up is all the others can take; an increase that cannot be met blocks forever), so the split is
// checked here against the launch allocation and again, at run time, against the compiled kernel.
constexpr int kAttn2LaunchRegs = 168, kAttn2SoftmaxRegs = 224, kAttn2OtherRegs = 56;
static_assert(256 * kAttn2SoftmaxRegs + 128 * kAttn2OtherRegs <= kAttn2Threads * kAttn2LaunchRegs,
              "setmaxnreg split exceeds the block's launch allocation");
constexpr size_t kAttn2SmemBytes = 6 * kTileBytes + 1024 + 512;

struct Attn2Tile {
  int head;    // b * Hq + query head, or -1 if this block has no second tile
  int row0;    // first chunk row of the tile
  int n_kt;    // key tiles to walk (0 if absent)
};

__device__ __forceinline__ Attn2Tile attn2_tile(int u, int U, int G, int n_qt, int bg_q0, int Lc,
                                                int n_cache) {
  Attn2Tile t;
  if (u >= U) {
    t.head = -1; t.row0 = 0; t.n_kt = 0;
    return t;
  }
  const int qt = n_qt - 1 - u / G;  // longest walks first
  t.head = bg_q0 + u % G;
  t.row0 = qt * kT;
  const int last_row = min(t.row0 + kT - 1, Lc - 1);
  t.n_kt = (n_cache + last_row + 1 + kT - 1) / kT;
  return t;
}

// Rotary embedding of one row of a query tile in shared memory (Sec. 3.1: chunk row i sits at
// position n_cache + i once the cache rows have been renumbered).  The tile is two boxes of 64
// columns, 128 bytes per row, 16-byte chunks XOR-swizzled by (row & 7); column c of box 0 and
// column c of box 1 share an offset, which is where the two halves of a rotate-half pair live.
// tab: the row's 64 (cos, sin) pairs as 32 float4, fetched by the caller before it waited for the
// tile (the table does not depend on the tile, so its latency hides under the tile's copy).
__device__ __forceinline__ void rope_rotate_q_row(uint8_t* tile, int r, const float4 (&tab)[32], bool interleaved) {
  uint8_t* row0 = tile + r * 128;
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const int p = (c ^ (r & 7)) * 16;
    uint4 x = *reinterpret_cast<uint4*>(row0 + p);               // columns 8c .. 8c+7
    uint4 y = *reinterpret_cast<uint4*>(row0 + kHalfBytes + p);  // columns 64+8c .. 64+8c+7
    __nv_bfloat162* xe = reinterpret_cast<__nv_bfloat162*>(&x);
    __nv_bfloat162* ye = reinterpret_cast<__nv_bfloat162*>(&y);
    if (!interleaved) {  // pair i = (column i, column i + 64), i = 8c + e
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float4 cs = tab[4 * c + e];  // (cos, sin) of pairs 8c+2e and 8c+2e+1
        const float2 a = __bfloat1622float2(xe[e]), b = __bfloat1622float2(ye[e]);
        float a0, b0, a1, b1;
        rope_rotate(a.x, b.x, cs.x, cs.y, a0, b0);
        rope_rotate(a.y, b.y, cs.z, cs.w, a1, b1);
        xe[e] = __floats2bfloat162_rn(a0, a1);
        ye[e] = __floats2bfloat162_rn(b0, b1);
      }
    } else {             // pair i = (column 2i, column 2i + 1): box 0 holds pairs 4c+e, box 1 pairs 32+4c+e
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const float4 cx = tab[2 * c + e], cy = tab[16 + 2 * c + e];
        float2 a = __bfloat1622float2(xe[2 * e]), b = __bfloat1622float2(xe[2 * e + 1]);
        float r0, r1, r2, r3;
        rope_rotate(a.x, a.y, cx.x, cx.y, r0, r1);
        rope_rotate(b.x, b.y, cx.z, cx.w, r2, r3);
        xe[2 * e] = __floats2bfloat162_rn(r0, r1);
        xe[2 * e + 1] = __floats2bfloat162_rn(r2, r3);
        a = __bfloat1622float2(ye[2 * e]);
        b = __bfloat1622float2(ye[2 * e + 1]);
        rope_rotate(a.x, a.y, cy.x, cy.y, r0, r1);
        rope_rotate(b.x, b.y, cy.z, cy.w, r2, r3);
        ye[2 * e] = __floats2bfloat162_rn(r0, r1);
        ye[2 * e + 1] = __floats2bfloat162_rn(r2, r3);
      }
    }
    *reinterpret_cast<uint4*>(row0 + p) = x;
    *reinterpret_cast<uint4*>(row0 + kHalfBytes + p) = y;
  }
}

// rope_tab != nullptr: q holds un-rotated queries; each softmax warpgroup rotates its query tile in
// shared memory once, right after it lands (rope_tab[i * 64 + pair] = (cos, sin) for chunk row i),
// and the MMA issuer waits for that instead of for the copy.
__global__ void __launch_bounds__(kAttn2Threads, 1)
attn2_sm100_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, __nv_bfloat16* __restrict__ out,
                   float* __restrict__ lse, int Hq, int Hkv, int Lc, int n_cache, float scale_log2,
                   const float2* __restrict__ rope_tab, int rope_interleaved, int32_t* dev_status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align_1024(smem_raw);
  uint8_t* sQ = smem;                    // [2] query tiles
  uint8_t* sK = smem + 2 * kTileBytes;   // [2] stages
  uint8_t* sV = smem + 4 * kTileBytes;   // [2] stages
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 6 * kTileBytes);
  uint64_t* q_full = bars + 0;
  uint64_t* k_full = bars + 1;    // [2]
  uint64_t* k_empty = bars + 3;   // [2]
  uint64_t* v_full = bars + 5;    // [2]
  uint64_t* v_empty = bars + 7;   // [2]
  uint64_t* s_full = bars + 9;    // [2] per tile
  uint64_t* p_ready = bars + 11;  // [2 tiles][2 halves of the key tile]
  uint64_t* o_full = bars + 15;   // [2] per tile
  uint64_t* q_rot = bars + 17;    // [2] per tile: query tile rotated in place (rope_tab only)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 19);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = Hq / Hkv;
  const int g = blockIdx.y % Hkv, b = blockIdx.y / Hkv;
  const int n_qt = (Lc + kT - 1) / kT;
  const int U = G * n_qt;
  const Attn2Tile t0 = attn2_tile(2 * blockIdx.x, U, G, n_qt, b * Hq + g * G, Lc, n_cache);
  const Attn2Tile t1 = attn2_tile(2 * blockIdx.x + 1, U, G, n_qt, b * Hq + g * G, Lc, n_cache);
  const int kv_head = b * Hkv + g;
  const int n_kt0 = t0.n_kt, n_kt1 = t1.n_kt;  // n_kt0 >= n_kt1

  if (threadIdx.x == 0) {
    ptx::mbar_init(q_full, 1);
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(k_full + s, 1);
      ptx::mbar_init(k_empty + s, 1);
      ptx::mbar_init(v_full + s, 1);
      ptx::mbar_init(v_empty + s, 1);
      ptx::mbar_init(s_full + s, 1);
      ptx::mbar_init(p_ready + 2 * s, 128);
      ptx::mbar_init(p_ready + 2 * s + 1, 128);
      ptx::mbar_init(o_full + s, 1);
      ptx::mbar_init(q_rot + s, 128);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
  }
  if (warp == 9) {
    ptx::tmem_alloc(tmem_slot, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp >= 8) {
    ptx::setmaxnreg_dec<kAttn2OtherRegs>();
    if (warp == 8 && lane == 0) {
      ptx::prefetch_tmap(&tmQ);
      ptx::prefetch_tmap(&tmK);
      ptx::prefetch_tmap(&tmV);
      ptx::mbar_expect_tx(q_full, n_kt1 ? 2 * kTileBytes : kTileBytes);
      ptx::tma_load_3d(sQ, &tmQ, q_full, 0, t0.row0, t0.head);
      ptx::tma_load_3d(sQ + kHalfBytes, &tmQ, q_full, 64, t0.row0, t0.head);
      if (n_kt1) {
        ptx::tma_load_3d(sQ + kTileBytes, &tmQ, q_full, 0, t1.row0, t1.head);
        ptx::tma_load_3d(sQ + kTileBytes + kHalfBytes, &tmQ, q_full, 64, t1.row0, t1.head);
      }
      int issued_k = 0, issued_v = 0;
      for (int j = 0; j < n_kt0; ++j) {
        const int s = j & 1, ph = (j >> 1) & 1;
        if (!ptx::mbar_wait(k_empty + s, ph ^ 1, abort_flag)) break;
        ptx::mbar_expect_tx(k_full + s, kTileBytes);
        ptx::tma_load_3d(sK + s * kTileBytes, &tmK, k_full + s, 0, j * kT, kv_head);
        ptx::tma_load_3d(sK + s * kTileBytes + kHalfBytes, &tmK, k_full + s, 64, j * kT, kv_head);
        issued_k = j + 1;
        if (!ptx::mbar_wait(v_empty + s, ph ^ 1, abort_flag)) break;
        ptx::mbar_expect_tx(v_full + s, kTileBytes);
        ptx::tma_load_3d(sV + s * kTileBytes, &tmV, v_full + s, 0, j * kT, kv_head);
        ptx::tma_load_3d(sV + s * kTileBytes + kHalfBytes, &tmV, v_full + s, 64, j * kT, kv_head);
        issued_v = j + 1;
      }
      if (*abort_flag) {  // let copies in flight land before the block's shared memory is released
        volatile int ignore = 0;
        ptx::mbar_wait(q_full, 0, &ignore);
        for (int u = 1; u <= 2; ++u) {
          if (issued_k >= u) ptx::mbar_wait(k_full + ((issued_k - u) & 1), ((issued_k - u) >> 1) & 1, &ignore);
          if (issued_v >= u) ptx::mbar_wait(v_full + ((issued_v - u) & 1), ((issued_v - u) >> 1) & 1, &ignore);
        }
      }
    } else if (warp == 9 && lane == 0) {
      const uint32_t aQ = ptx::smem_u32(sQ), aK = ptx::smem_u32(sK), aV = ptx::smem_u32(sV);
      const uint32_t tS0 = tmem_base, tO0 = tmem_base + 128, tS1 = tmem_base + 256, tO1 = tmem_base + 384;
      bool ok = rope_tab ? ptx::mbar_wait(q_rot, 0, abort_flag) && (!n_kt1 || ptx::mbar_wait(q_rot + 1, 0, abort_flag))
                         : ptx::mbar_wait(q_full, 0, abort_flag);
      ok = ok && ptx::mbar_wait(k_full, 0, abort_flag);
      if (ok) {
        ptx::tc_fence_after();
        issue_kmajor_128x128x128(tS0, aQ, aK);
        ptx::mma_commit(s_full + 0);
        if (n_kt1) {
          issue_kmajor_128x128x128(tS1, aQ + kTileBytes, aK);
          ptx::mma_commit(s_full + 1);
        }
        ptx::mma_commit(k_empty + 0);
      }
      for (int j = 0; ok && j < n_kt0; ++j) {
        const int s = j & 1, s1 = (j + 1) & 1;
        // tile 0: O0 += P0 V[j], then S0 = Q0 K[j+1]^T
        // (thread 0 of tile 0's warpgroup has seen V[j] before its first arrival on p_ready and
        // K[j+1] before its second: a wait costs this thread one to two MMAs even when satisfied)
        if (!ptx::mbar_wait(p_ready + 0, j & 1, abort_flag)) break;
        ptx::tc_fence_after();
        const uint32_t v_lo = ptx::smem_desc_lo(aV + s * kTileBytes, kHalfBytes);
        issue_pv_half<0>(tO0, tS0, v_lo, j == 0);
        if (!ptx::mbar_wait(p_ready + 1, j & 1, abort_flag)) break;
        ptx::tc_fence_after();
        issue_pv_half<4>(tO0, tS0, v_lo, false);
        if (j + 1 < n_kt0) {
          issue_kmajor_128x128x128(tS0, aQ, aK + s1 * kTileBytes);
          ptx::mma_commit(s_full + 0);
        } else {
          ptx::mma_commit(o_full + 0);
        }
        // tile 1
        if (j < n_kt1) {
          if (!ptx::mbar_wait(p_ready + 2, j & 1, abort_flag)) break;
          ptx::tc_fence_after();
          issue_pv_half<0>(tO1, tS1, v_lo, j == 0);
          if (!ptx::mbar_wait(p_ready + 3, j & 1, abort_flag)) break;
          ptx::tc_fence_after();
          issue_pv_half<4>(tO1, tS1, v_lo, false);
        }
        ptx::mma_commit(v_empty + s);
        if (j + 1 < n_kt1) {
          issue_kmajor_128x128x128(tS1, aQ + kTileBytes, aK + s1 * kTileBytes);
          ptx::mma_commit(s_full + 1);
        } else if (j + 1 == n_kt1) {
          ptx::mma_commit(o_full + 1);
        }
        if (j + 1 < n_kt0) ptx::mma_commit(k_empty + s1);
      }
    }
  } else {
    ptx::setmaxnreg_inc<kAttn2SoftmaxRegs>();
    const int t = warp >> 2;                      // which tile this warpgroup serves
    const Attn2Tile tile = t ? t1 : t0;
    const int sub = warp & 3;                     // TMEM sub-partition of this warp
    const int r = 32 * sub + lane;                // row of the tile = TMEM lane
    const uint32_t lane_addr = (uint32_t)(32 * sub) << 16;
    const uint32_t tS = tmem_base + 256 * t + lane_addr, tO = tS + 128;
    const int row = tile.row0 + r;
    const int lim = n_cache + row;                // last visible key of this row
    float m = -INFINITY, l0 = 0.f, l1 = 0.f;
    bool ok = tile.n_kt > 0;
    if (rope_tab && ok) {
      float4 tab[32];   // this row's 64 (cos, sin) pairs, on their way while the tile's copy is in flight
      const float4* tr = reinterpret_cast<const float4*>(rope_tab + (long long)min(row, Lc - 1) * 64);
#pragma unroll
      for (int i = 0; i < 32; ++i) tab[i] = __ldg(tr + i);
      ok = ptx::mbar_wait(q_full, 0, abort_flag);
      if (ok && row < Lc) rope_rotate_q_row(sQ + t * kTileBytes, r, tab, rope_interleaved != 0);
      ptx::fence_proxy_async_smem();   // the rotated tile is read by the tensor cores (async proxy)
      ptx::mbar_arrive(q_rot + t);
    }
    for (int j = 0; ok && j < tile.n_kt; ++j) {
      if (!ptx::mbar_wait(s_full + t, j & 1, abort_flag)) { ok = false; break; }
      ptx::tc_fence_after();
      uint32_t v[128];
      ptx::tmem_ld128(tS, v);
      const int key0 = j * kT;
      if (key0 + kT - 1 > n_cache + tile.row0) {  // the walk reaches this tile's diagonal
        const int thr = lim - key0;               // columns past thr are invisible to this row
#pragma unroll
        for (int i = 0; i < 128; ++i)
          if (i > thr) v[i] = 0xff800000u;        // -inf
      }
      float mx[8];  // eight independent chains of 3-input maxima
#pragma unroll
      for (int c = 0; c < 8; ++c) mx[c] = ptx::max3(__uint_as_float(v[c]), __uint_as_float(v[c + 8]), __uint_as_float(v[c + 16]));
#pragma unroll
      for (int i = 24; i < 120; i += 16) {
#pragma unroll
        for (int c = 0; c < 8; ++c) mx[c] = ptx::max3(mx[c], __uint_as_float(v[i + c]), __uint_as_float(v[i + c + 8]));
      }
#pragma unroll
      for (int c = 0; c < 8; ++c) mx[c] = fmaxf(mx[c], __uint_as_float(v[120 + c]));
      const float mxa = ptx::max3(mx[0], mx[1], mx[2]), mxb = ptx::max3(mx[3], mx[4], mx[5]);
      const float m_new = fmaxf(m, ptx::max3(mxa, mxb, fmaxf(mx[6], mx[7])) * scale_log2);
      if (j == 0) {
        m = m_new;  // key 0 is visible to every row, so m is finite from here on
      } else {
        const bool grow = m_new > m + kRescaleThreshold;
        if (__any_sync(0xffffffffu, grow)) {
          const float alpha = grow ? ptx::ex2(m - m_new) : 1.0f;
          if (grow) m = m_new;
          l0 *= alpha;
          l1 *= alpha;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t o[32];
            ptx::tmem_ld32(tO + 32 * c, o);
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
            ptx::tmem_st32(tO + 32 * c, o);
          }
          ptx::tmem_st_wait();
        }
      }
      const float neg_m = -m;
      // P goes back to TMEM in two halves (keys 0-63, 64-127), each signalled on its own barrier,
      // so the first four PV MMAs start while the second half is still being exponentiated
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t pk[32];
        float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f;  // two independent pairs of partial row sums
#pragma unroll
        for (int i = 0; i < 64; i += 2) {
          const int e = 64 * half + i;
          float x0, x1;
          ptx::fma2(x0, x1, __uint_as_float(v[e]), __uint_as_float(v[e + 1]), scale_log2, neg_m);
          const float p0 = ptx::ex2(x0), p1 = ptx::ex2(x1);  // ex2(-inf) = 0 for masked columns
          if (i & 2) ptx::add2(b0, b1, p0, p1); else ptx::add2(a0, a1, p0, p1);
          pk[i >> 1] = ptx::pack_bf16(p0, p1);
        }
        ptx::add2(a0, a1, b0, b1);
        ptx::add2(l0, l1, a0, a1);
        ptx::tmem_st32(tS + 32 * half, pk);
        ptx::tmem_st_wait();
        ptx::tc_fence_before();
        if (threadIdx.x == 0) {  // on behalf of the MMA issuer: the operands its next MMAs read are in shared memory
          const int jn = j + 1;
          const bool there = half == 0 ? ptx::mbar_wait(v_full + (j & 1), (j >> 1) & 1, abort_flag)
                                       : (jn >= tile.n_kt || ptx::mbar_wait(k_full + (jn & 1), (jn >> 1) & 1, abort_flag));
          if (!there) { ok = false; break; }
        }
        ptx::mbar_arrive(p_ready + 2 * t + half);
      }
      if (!ok) break;
    }
    if (ok && ptx::mbar_wait(o_full + t, 0, abort_flag)) {
      ptx::tc_fence_after();
      const float l = l0 + l1;
      const float inv = 1.0f / l;
      __nv_bfloat16* op = out + ((long long)tile.head * Lc + row) * kT;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t o[32];
        ptx::tmem_ld32(tO + 32 * c, o);
        if (row < Lc) {
#pragma unroll
          for (int i = 0; i < 32; i += 8) {
            uint4 w;
            w.x = ptx::pack_bf16(__uint_as_float(o[i]) * inv, __uint_as_float(o[i + 1]) * inv);
            w.y = ptx::pack_bf16(__uint_as_float(o[i + 2]) * inv, __uint_as_float(o[i + 3]) * inv);
            w.z = ptx::pack_bf16(__uint_as_float(o[i + 4]) * inv, __uint_as_float(o[i + 5]) * inv);
            w.w = ptx::pack_bf16(__uint_as_float(o[i + 6]) * inv, __uint_as_float(o[i + 7]) * inv);
            *reinterpret_cast<uint4*>(op + 32 * c + i) = w;
          }
        }
      }
      if (row < Lc) lse[(long long)tile.head * Lc + row] = (m + log2f(l)) * kLn2;
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
  if (threadIdx.x == 0 && *abort_flag) report_device_error(dev_status, REFORM_DEV_TIMEOUT);
}


// Enumerates the (query head of the group, 128-row query tile of the window)
// pairs a key tile has to visit, skipping tiles none of whose rows sees it.
struct ScoreTiles {
  int G, Lc, n_cache, i_begin, j0;
  int hh, i0;
  __device__ ScoreTiles(int G_, int Lc_, int n_cache_, int window, int j0_)
      : G(G_), Lc(Lc_), n_cache(n_cache_), i_begin(Lc_ - window), j0(j0_), hh(0), i0(Lc_ - window) {
    skip();
  }
  __device__ bool valid() const { return hh < G; }
  __device__ void next() {
    i0 += kT;
    if (i0 >= Lc) { i0 = i_begin; ++hh; }
    skip();
  }
  __device__ void skip() {
    while (hh < G && j0 > n_cache + min(i0 + kT - 1, Lc - 1)) {
      i0 += kT;
      if (i0 >= Lc) { i0 = i_begin; ++hh; }
    }
  }
};

__global__ void __launch_bounds__(kSm100Threads, 2)
score_sm100_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const float* __restrict__ lse, float* __restrict__ score, int Hq, int Hkv, int Lc,
                   int n_cache, int cap, int window, float scale_log2, int accumulate, int q_first,
                   int32_t* dev_status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align_1024(smem_raw);
  uint8_t* sK = smem;
  uint8_t* sQ = smem + kTileBytes;  // two stages
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 3 * kTileBytes);
  uint64_t* k_full = bars + 0;
  uint64_t* q_full = bars + 1;   // [2]
  uint64_t* q_empty = bars + 3;  // [2]
  uint64_t* d_full = bars + 5;   // [2]
  uint64_t* d_empty = bars + 7;  // [2]
  uint64_t* lse_ready = bars + 9;  // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 11);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* lse2 = reinterpret_cast<float*>(smem + 3 * kTileBytes + 256);  // [2][128]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = blockIdx.y % Hkv, b = blockIdx.y / Hkv;
  const int G = Hq / Hkv;
  const int n = n_cache + Lc;
  const int j0 = blockIdx.x * kT;

  if (threadIdx.x == 0) {
    ptx::mbar_init(k_full, 1);
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(q_full + s, 1);
      ptx::mbar_init(q_empty + s, 1);
      ptx::mbar_init(d_full + s, 1);
      ptx::mbar_init(d_empty + s, 128);
      ptx::mbar_init(lse_ready + s, 128);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      ptx::prefetch_tmap(&tmQ);
      ptx::prefetch_tmap(&tmK);
      ptx::mbar_expect_tx(k_full, kTileBytes);
      ptx::tma_load_3d(sK, &tmK, k_full, 0, j0, b * Hkv + g);
      ptx::tma_load_3d(sK + kHalfBytes, &tmK, k_full, 64, j0, b * Hkv + g);
      int it = 0;
      for (ScoreTiles t(G, Lc, n_cache, window, j0); t.valid(); t.next(), ++it) {
        const int s = it & 1;
        if (!ptx::mbar_wait(q_empty + s, ((it >> 1) & 1) ^ 1, abort_flag)) break;
        ptx::mbar_expect_tx(q_full + s, kTileBytes);
        uint8_t* dst = sQ + s * kTileBytes;
        // tmQ starts at chunk row q_first (the whole chunk, or a rotated copy of the score window)
        ptx::tma_load_3d(dst, &tmQ, q_full + s, 0, t.i0 - q_first, b * Hq + g * G + t.hh);
        ptx::tma_load_3d(dst + kHalfBytes, &tmQ, q_full + s, 64, t.i0 - q_first, b * Hq + g * G + t.hh);
      }
      if (*abort_flag) {
        volatile int ignore = 0;
        ptx::mbar_wait(k_full, 0, &ignore);
        for (int u = 1; u <= 2 && u <= it; ++u) {
          int last = it - u;
          ptx::mbar_wait(q_full + (last & 1), (last >> 1) & 1, &ignore);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t aK = ptx::smem_u32(sK), aQ = ptx::smem_u32(sQ);
      bool ok = ptx::mbar_wait(k_full, 0, abort_flag);
      int it = 0;
      for (ScoreTiles t(G, Lc, n_cache, window, j0); ok && t.valid(); t.next(), ++it) {
        const int s = it & 1, ph = (it >> 1) & 1;
        if (!ptx::mbar_wait(q_full + s, ph, abort_flag)) break;
        if (!ptx::mbar_wait(d_empty + s, ph ^ 1, abort_flag)) break;
        ptx::tc_fence_after();
        issue_kmajor_128x128x128(tmem_base + s * kT, aK, aQ + s * kTileBytes);
        ptx::mma_commit(d_full + s);
        ptx::mma_commit(q_empty + s);
      }
    }
  } else {
    const int sub = warp & 3;
    const int r = 32 * sub + lane;
    const uint32_t lane_addr = (uint32_t)(32 * sub) << 16;
    const int key = j0 + r;
    float acc = 0.f;
    int it = 0;
    for (ScoreTiles t(G, Lc, n_cache, window, j0); t.valid(); t.next(), ++it) {
      const int s = it & 1, ph = (it >> 1) & 1;
      const int qi = t.i0 + r;
      lse2[s * kT + r] = (qi < Lc) ? lse[((long long)b * Hq + g * G + t.hh) * Lc + qi] * kLog2e : INFINITY;
      ptx::mbar_arrive(lse_ready + s);
      if (!ptx::mbar_wait(lse_ready + s, ph, abort_flag)) break;
      if (!ptx::mbar_wait(d_full + s, ph, abort_flag)) break;
      ptx::tc_fence_after();
      const int vis0 = key - n_cache - t.i0;  // column c sees this key iff c >= vis0
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t v[32];
        ptx::tmem_ld32(tmem_base + s * kT + lane_addr + 32 * c, v);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          float p = ptx::ex2(fmaf(__uint_as_float(v[i]), scale_log2, -lse2[s * kT + 32 * c + i]));
          if (32 * c + i >= vis0) acc += p;
        }
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(d_empty + s);
    }
    if (key < n && !*abort_flag) {
      long long o = ((long long)b * Hkv + g) * cap + key;
      float carry = (accumulate && key < n_cache) ? score[o] : 0.f;
      score[o] = carry + acc;
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag) report_device_error(dev_status, REFORM_DEV_TIMEOUT);
}

// The setmaxnreg split above draws on the registers the block is launched with: 384 threads times
// the kernel's register count.  If a compiler ever gave the kernel fewer than the split needs, the
// increase could not be met and would block forever, so such a build refuses to launch (with 384
// threads per block the count cannot exceed 168, and any count from 168 up holds the split).
inline bool attn_launch_regs_ok() {
  static int ok = -1;
  if (ok < 0) {
    cudaFuncAttributes a2;
    ok = cudaFuncGetAttributes(&a2, attn2_sm100_kernel) == cudaSuccess && a2.numRegs >= kAttn2LaunchRegs;
  }
  return ok == 1;
}

// Operands of a step whose rotary embedding is applied inside the call (REFORM_ROPE): the keys
// rotated at positions 0 .. n-1 into scratch, the queries the score pass reads rotated into
// scratch, and, for the attention kernel, either rotated queries or the table it rotates with.
struct RopeOperands {
  const void* k_rot = nullptr;       // [B*Hkv, cap, 128], the layout of k
  const void* q_score = nullptr;     // rotated query rows the score pass reads, [B*Hq, q_score_rows, 128]
  int q_score_rows = 0;              // Lc (all rows) or the score window
  int q_score_first = 0;             // chunk row of its row 0
  const void* q_attn = nullptr;      // rotated queries for the attention kernel, or nullptr ...
  const float2* table = nullptr;     // ... in which case it rotates at load with this table [Lc][64]
  int interleaved = 0;
};

// run_attention == false: only the score pass (lse already holds the row normalisers).
inline int launch_chunk_sm100(const reform_chunk_params* p, float* lse, float scale, cudaStream_t st,
                              bool run_attention = true, const RopeOperands* rope = nullptr) {
  if (!attn_launch_regs_ok()) return REFORM_ERR_UNSUPPORTED;
  const int n = p->n_cache + p->Lc;
  const float scale_log2 = scale * kLog2e;
  CUtensorMap tmQ, tmK, tmV, tmQs;
  const void* q_attn = rope && rope->q_attn ? rope->q_attn : p->q;
  const void* k_ptr = rope ? rope->k_rot : p->k;
  if (!make_tmap_bf16_d128(&tmQ, q_attn, (long long)p->B * p->Hq, p->Lc, p->Lc, kT) ||
      !make_tmap_bf16_d128(&tmK, k_ptr, (long long)p->B * p->Hkv, n, p->cap, kT) ||
      !make_tmap_bf16_d128(&tmV, p->v, (long long)p->B * p->Hkv, n, p->cap, kT)) {
    g_last_cuda_error = (int)cudaErrorInvalidValue;
    return REFORM_ERR_CUDA;
  }
  int q_first = 0;
  tmQs = tmQ;
  if (rope && !(p->flags & REFORM_NO_SCORE)) {
    q_first = rope->q_score_first;
    if (!make_tmap_bf16_d128(&tmQs, rope->q_score, (long long)p->B * p->Hq, rope->q_score_rows, rope->q_score_rows, kT)) {
      g_last_cuda_error = (int)cudaErrorInvalidValue;
      return REFORM_ERR_CUDA;
    }
  }
  if (run_attention) {
    cudaFuncSetAttribute(attn2_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttn2SmemBytes);
    const int units = (p->Hq / p->Hkv) * ((p->Lc + kT - 1) / kT);
    dim3 grid((units + 1) / 2, p->B * p->Hkv);
    attn2_sm100_kernel<<<grid, kAttn2Threads, kAttn2SmemBytes, st>>>(
        tmQ, tmK, tmV, (__nv_bfloat16*)p->out, lse, p->Hq, p->Hkv, p->Lc, p->n_cache, scale_log2,
        rope && !rope->q_attn ? rope->table : nullptr, rope ? rope->interleaved : 0, p->dev_status);
    count_launch();
    int rc = check_launch();
    if (rc != REFORM_OK) return rc;
  }
  if (p->flags & REFORM_NO_SCORE) return REFORM_OK;
  cudaFuncSetAttribute(score_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kScoreSmemBytes);
  dim3 grid2((n + kT - 1) / kT, p->B * p->Hkv);
  score_sm100_kernel<<<grid2, kSm100Threads, kScoreSmemBytes, st>>>(
      tmQs, tmK, lse, p->score, p->Hq, p->Hkv, p->Lc, p->n_cache, p->cap, p->score_window, scale_log2,
      (p->flags & REFORM_SCORE_ACCUMULATE) ? 1 : 0, q_first, p->dev_status);
  count_launch();
  return check_launch();
}

}  // namespace reform
