// Expert feed-forward with block-scaled FP8 operands (MXFP8): E4M3 elements, one E8M0 scale per 32 elements along K,
// applied by the tensor pipe inside the MMA (tcgen05.mma.kind::mxf8f6f4.block_scale, scales in tensor memory).
//
// One kernel, launched once for Linear-1 (gate | up, SwiGLU, h quantised in the epilogue) and once for Linear-2.
// Persistent CTAs, one per SM, tiles assigned round-robin (tile t goes to CTA t mod grid).  A tile is 128 rows of one
// expert x 256 accumulator columns: Linear-1 pairs 128 gate columns with the same 128 up columns, so a tile yields
// 128 columns of h = four whole 32-element scale blocks, which the epilogue quantises straight from the fp32
// accumulator (h never exists in bf16); Linear-2 writes 256 bf16 columns of y_perm.
//
// Tensor memory (512 columns) holds ONE 256-column accumulator plus 4 columns of A scales and 8 of B scales; two
// accumulators and the scales do not fit, and a 192-column tile with two accumulators was measured 13-15 % slower:
// an MMA costs about the same clocks in the running kernel at N = 192 as at N = 256.  So the epilogue does not
// overlap the next tile's mainloop; eight epilogue warps (two per lane quarter, half of the columns each) keep it
// short, and each hands the accumulator back right after its last load from tensor memory (the MMA thread waits
// for the accumulator 10 % of the time in Linear-1 on the Mixtral-like layer).
//
// Roles (448 threads): warp 0 = TMA producer (codes of A and of two 128-row weight boxes per 128-element K stage),
// warps 6-9 = scale loaders (one word per operand row per stage, loaded four stages ahead into registers and
// stored in the 512-byte layout tcgen05.cp expects, then a proxy fence and an arrival on the stage's full barrier),
// warp 1 = MMA issuer (per stage: three tcgen05.cp of scales into tensor memory, then four MMAs picking scale byte
// 0..3), warps 2-5 and 10-13 = epilogue.  Four stages of 49.5 KB.
// An expert of at most 64 rows is computed with swapped operands (weight box = M side, its rows padded to 16 = N
// side, the scale groups change roles with them): fewer multiply-adds on padding rows, which under the power cap is
// worth more than the clocks the extra instructions cost.  TMA loads carry L2 eviction priorities: weights only this
// tile reads go first, rows of A and weights other row blocks read again stay.
// Every wait is bounded; a wait that gives up is reported through the status word and the CTA unwinds.
#include <cuda_bf16.h>

#include <type_traits>

#include "ffn_math.cuh"
#include "moe_internal.h"
#include "mx_quant.cuh"
#include "ptx_sm100.cuh"

namespace {

constexpr int kThreads = 448;
constexpr int BM = 128;                 // rows per tile
constexpr int BNH = 128;                // rows of one weight box
constexpr int BN = 2 * BNH;             // accumulator columns
constexpr int BK = 128;                 // K elements (= bytes) per stage: one 128-byte swizzle row
constexpr int UMMA_K = 32;
constexpr int kABytes = BM * BK;
constexpr int kBBoxBytes = BNH * BK;
constexpr int kOperandBytes = kABytes + 2 * kBBoxBytes;
constexpr int kSfABytes = 512;          // 128 rows x 4 scale bytes
constexpr int kSfBytes = kSfABytes + 1024;
constexpr int kStages = 4;
constexpr int kAccBufs = 1;               // accumulators in tensor memory (two would leave no room for the scales)
constexpr int kTmemCols = 512;
constexpr uint32_t kTmemSfA = kAccBufs * BN;   // column of the A scales
constexpr uint32_t kTmemSfB = kAccBufs * BN + 4;
constexpr int kSfThreads = 128;
constexpr int kKernelIdMx = 9;          // in the detail word of a time-out: 9 * 65536 + role
constexpr int kMxSwapRows = 64;         // row blocks with at most this many rows run with swapped operands

struct MxParams {
  const int32_t* offsets;   // [E+1]
  int E;
  int N;                    // output columns of this GEMM: F (Linear-1) or H (Linear-2)
  int n_blocks;             // tiles along N: ceil(N / 128) gated, ceil(N / 256) otherwise
  int k_blocks;             // K / 128
  long long a_rows;         // R
  long long b_rows;         // E * N: rows of each weight matrix
  const uint32_t* sf_a;     // [K/128][R]
  const uint32_t* sf_b0;    // [K/128][E*N] gate resp. down
  const uint32_t* sf_b1;    // [K/128][E*N] up resp. down
  uint4* hq;                // Linear-1 out: E4M3 [R, N]
  unsigned char* sf_h;      // Linear-1 out: scale bytes, words [N/128][R]
  float* h_dbg;             // optional fp32 [R, N]
  __nv_bfloat16* y;         // Linear-2 out: bf16 [R, N]
  int32_t* status;
  unsigned long long* trace;   // null, or [CTAs][kMoeTraceFields] wait counters (the fields of the bf16 kernel)
  int cache_hints;          // L2 eviction priorities of the TMA loads: the bits of the bf16 kernel's knob (0, 1, 5)
  int swap_rows;            // row blocks with at most this many rows run with swapped operands (at most 64)
};

struct MxTile {
  int row0, row_end, n0, w_row0;
  int single;     // the expert has a single row block: no other tile reads these weight boxes
  int n_pad;      // 0, or the row count padded to 16 of a block of few rows, computed with swapped operands
};

struct MxTail {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
  int32_t blk_prefix[1025];   // exclusive prefix of ceil(count / 128) over experts
  int32_t offs[1025];         // the expert row offsets, copied once: tile decoding reads no global memory
};

__device__ __forceinline__ void mx_timeout(const MxParams& p, int role) {
  atomicCAS(&p.status[0], 0, MOE_ERR_TIMEOUT);
  atomicCAS(&p.status[1], 0, kKernelIdMx * 65536 + role);
}

// Tile t of the list ordered by (expert, column tile, row block): row blocks of one expert and column tile are
// neighbours, so CTAs that run side by side share the weight boxes in L2.
template <bool kGated>
__device__ __forceinline__ MxTile decode_tile(int t, const MxTail* st, const MxParams& p) {
  int lo = 0, hi = p.E;   // invariant: prefix(lo) * n_blocks <= t < prefix(hi) * n_blocks
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (st->blk_prefix[mid] * p.n_blocks <= t) lo = mid; else hi = mid;
  }
  const int e = lo;
  const int blocks_e = st->blk_prefix[e + 1] - st->blk_prefix[e];
  const int local = t - st->blk_prefix[e] * p.n_blocks;
  const int nb = local / blocks_e, mb = local - nb * blocks_e;
  MxTile tile;
  tile.row0 = st->offs[e] + mb * BM;
  tile.row_end = st->offs[e + 1];
  tile.n0 = nb * (kGated ? BNH : BN);
  tile.w_row0 = e * p.N + tile.n0;
  tile.single = blocks_e == 1 ? 1 : 0;
  const int rows = min(tile.row_end - tile.row0, BM);
  // swapped operands for small experts only: in clocks such a tile is slower than a 128-row tile (eight short
  // block-scaled MMAs per K block are bound by the issuing thread: 1060 against 810 clocks), what it saves is power,
  // which pays where such tiles are most of the launch (decode-like batches) and not for the odd short last block of
  // a many-row expert
  tile.n_pad = (blocks_e == 1 && rows <= p.swap_rows) ? ((rows + 15) & ~15) : 0;
  return tile;
}

template <bool kGated>
__global__ void __launch_bounds__(kThreads, 1)
expert_ffn_mx_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b0,
                     const __grid_constant__ CUtensorMap tm_b1, const MxParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
  unsigned char* base = smem_raw + pad;                      // 1024-byte aligned: required by the swizzle
  const uint32_t ring_u32 = raw + pad;                       // kStages operand stages
  const uint32_t sf_u32 = ring_u32 + kStages * kOperandBytes;   // kStages scale stages
  MxTail* st = reinterpret_cast<MxTail*>(base + kStages * (kOperandBytes + kSfBytes));

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(ptx::smem_u32(&st->full[s]), 1 + kSfThreads);   // the TMA arrival + every scale loader
      ptx::mbar_init(ptx::smem_u32(&st->empty[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(ptx::smem_u32(&st->tmem_full[a]), 1);
      ptx::mbar_init(ptx::smem_u32(&st->tmem_empty[a]), 8);          // one arrival per epilogue warp
    }
    st->abort_flag = 0;
    st->blk_prefix[0] = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async_smem();
  }
  if (warp == 0) {
    int32_t run = 0;
    for (int b0 = 0; b0 < p.E; b0 += 32) {
      const int e = b0 + lane;
      int32_t v = 0;
      if (e < p.E) {
        const int32_t lo = p.offsets[e], hi = p.offsets[e + 1];
        st->offs[e + 1] = hi;
        if (e == 0) st->offs[0] = lo;
        v = (hi - lo + BM - 1) / BM;
      }
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int32_t o = __shfl_up_sync(0xFFFFFFFFu, v, off);
        if (lane >= off) v += o;
      }
      if (e < p.E) st->blk_prefix[e + 1] = run + v;
      run += __shfl_sync(0xFFFFFFFFu, v, 31);
    }
    if (lane == 0) {
      ptx::prefetch_tensormap(&tm_a);
      ptx::prefetch_tensormap(&tm_b0);
      ptx::prefetch_tensormap(&tm_b1);
    }
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(&st->tmem_base), kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();

  const uint32_t tmem_base = st->tmem_base;
  const int total_tiles = st->blk_prefix[p.E] * p.n_blocks;
  const int b1_shift = kGated ? 0 : BNH;       // second weight box: same rows of the up matrix, or the next 128 rows
  volatile int* abort_flag = &st->abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      long long w_empty = 0;
      const long long t_begin = clock64();
      // L2 priorities as in the bf16 kernel: weights read by this tile alone go first, weights other row blocks read
      // again and the rows of A (read again by every column block) stay
      const uint64_t pol_first = ptx::l2_policy_evict_first(), pol_last = ptx::l2_policy_evict_last(),
                     pol_normal = ptx::l2_policy_evict_normal();
      const uint64_t pol_a = (p.cache_hints & 2) ? pol_last : pol_normal;
      for (int t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
        const MxTile tile = decode_tile<kGated>(t, st, p);
        const uint64_t pol_w = ((p.cache_hints & 1) && tile.single) ? pol_first
                               : ((p.cache_hints & 32) && !tile.single) ? pol_last : pol_normal;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!ptx::mbar_wait_timed(ptx::smem_u32(&st->empty[stage]), phase ^ 1u, abort_flag, &w_empty)) {
            mx_timeout(p, 1);
            ok = false;
            break;
          }
          const uint32_t full = ptx::smem_u32(&st->full[stage]);
          const uint32_t sa = ring_u32 + stage * kOperandBytes;
          ptx::mbar_expect_tx(full, kOperandBytes);
          ptx::tma_load_2d_hint(sa, &tm_a, full, kb * BK, tile.row0, pol_a);
          ptx::tma_load_2d_hint(sa + kABytes, &tm_b0, full, kb * BK, tile.w_row0, pol_w);
          ptx::tma_load_2d_hint(sa + kABytes + kBBoxBytes, &tm_b1, full, kb * BK, tile.w_row0 + b1_shift, pol_w);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (p.trace) {
        p.trace[blockIdx.x * kMoeTraceFields + 0] = static_cast<unsigned long long>(clock64() - t_begin);
        p.trace[blockIdx.x * kMoeTraceFields + 1] = static_cast<unsigned long long>(w_empty);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      long long w_full = 0, w_tmem = 0, t_swapped = 0, t_plain = 0;
      unsigned long long n_tiles = 0, n_swapped = 0;
      for (int t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
        const long long t_tile = clock64();
        const int n_pad = decode_tile<kGated>(t, st, p).n_pad;    // (decoded while the epilogue still drains)
        if (!ptx::mbar_wait_timed(ptx::smem_u32(&st->tmem_empty[acc]), acc_phase ^ 1u, abort_flag, &w_tmem)) {
          mx_timeout(p, 2);
          break;
        }
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
        // One K loop per tile kind (a run-time branch between the MMAs of a K block would cost the issuing thread
        // 100-200 clocks per block): wait for the stage, copy its scales to tensor memory, issue, free the stage.
        auto k_loop = [&](auto&& issue) -> bool {
          for (int kb = 0; kb < p.k_blocks; ++kb) {
            if (!ptx::mbar_wait_timed(ptx::smem_u32(&st->full[stage]), phase, abort_flag, &w_full)) {
              mx_timeout(p, 3);
              return false;
            }
            ptx::tc_fence_after_sync();
            const uint32_t sf = sf_u32 + stage * kSfBytes;
            ptx::tc_cp_32x128b_warpx4(tmem_base + kTmemSfA, sf);
            ptx::tc_cp_32x128b_warpx4(tmem_base + kTmemSfB, sf + kSfABytes);
            ptx::tc_cp_32x128b_warpx4(tmem_base + kTmemSfB + 4, sf + kSfABytes + 512);
            issue(ring_u32 + stage * kOperandBytes, kb != 0 ? 1u : 0u);
            ptx::tc_commit(ptx::smem_u32(&st->empty[stage]));   // codes and scales are free once these are done
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          return true;
        };
        // Swapped operands for a block of few rows: each 128-row weight box is the M side (its scales, the second and
        // third 512-byte group of the stage, are the A scales), the block's rows padded to 16 the N side (their
        // scales, the first group, the B scales); box 0 accumulates into columns 0.., box 1 into columns 128...
        auto swapped = [&](auto rows_tag) -> bool {
          constexpr int kRows = decltype(rows_tag)::value;
          return k_loop([&](uint32_t sa, uint32_t later) {
            const uint64_t r_desc = ptx::smem_desc_sw128(sa), w0_desc = ptx::smem_desc_sw128(sa + kABytes),
                           w1_desc = ptx::smem_desc_sw128(sa + kABytes + kBBoxBytes);
#pragma unroll
            for (int k4 = 0; k4 < BK / UMMA_K; ++k4) {
              const uint64_t adv = static_cast<uint64_t>(2 * k4);
              const uint32_t accum = k4 != 0 ? 1u : later;
              ptx::tc_mma_mx(d_tmem, w0_desc + adv, r_desc + adv, ptx::idesc_mx_e4m3(BNH, kRows, k4, k4),
                             tmem_base + kTmemSfB, tmem_base + kTmemSfA, accum);
              ptx::tc_mma_mx(d_tmem + BNH, w1_desc + adv, r_desc + adv, ptx::idesc_mx_e4m3(BNH, kRows, k4, k4),
                             tmem_base + kTmemSfB + 4, tmem_base + kTmemSfA, accum);
            }
          });
        };
        switch (n_pad >> 4) {
          case 0:
            ok = k_loop([&](uint32_t sa, uint32_t later) {
              const uint64_t a_desc = ptx::smem_desc_sw128(sa), b_desc = ptx::smem_desc_sw128(sa + kABytes);
#pragma unroll
              for (int k4 = 0; k4 < BK / UMMA_K; ++k4) {
                const uint64_t adv = static_cast<uint64_t>(2 * k4);   // +32 bytes along K inside the swizzle row
                ptx::tc_mma_mx(d_tmem, a_desc + adv, b_desc + adv, ptx::idesc_mx_e4m3(BM, BN, k4, k4),
                               tmem_base + kTmemSfA, tmem_base + kTmemSfB, k4 != 0 ? 1u : later);
              }
            });
            break;
          case 1: ok = swapped(std::integral_constant<int, 16>{}); break;
          case 2: ok = swapped(std::integral_constant<int, 32>{}); break;
          case 3: ok = swapped(std::integral_constant<int, 48>{}); break;
          default: ok = swapped(std::integral_constant<int, 64>{}); break;
        }
        if (!ok) break;
        ptx::tc_commit(ptx::smem_u32(&st->tmem_full[acc]));
        if (++acc == kAccBufs) { acc = 0; acc_phase ^= 1u; }
        ++n_tiles;
        if (n_pad != 0) {
          ++n_swapped;
          t_swapped += clock64() - t_tile;
        } else {
          t_plain += clock64() - t_tile;
        }
      }
      if (p.trace) {
        p.trace[blockIdx.x * kMoeTraceFields + 2] = static_cast<unsigned long long>(w_full);
        p.trace[blockIdx.x * kMoeTraceFields + 3] = static_cast<unsigned long long>(w_tmem);
        p.trace[blockIdx.x * kMoeTraceFields + 6] = n_tiles;
        p.trace[blockIdx.x * kMoeTraceFields + 8] = n_swapped;
        p.trace[blockIdx.x * kMoeTraceFields + 9] = static_cast<unsigned long long>(t_swapped);
        p.trace[blockIdx.x * kMoeTraceFields + 11] = static_cast<unsigned long long>(t_plain);
      }
    }
    __syncwarp();
  } else if (warp < 6 || warp >= 10) {
    // ------------------------------------------------------------------ epilogue (2 x 4 warps: 128 rows x two column halves)
    const int quarter = warp & 3;                 // TMEM lane quarter this warp may read
    const int half = warp >= 10 ? 1 : 0;          // which half of the tile's columns this warp drains
    int acc = 0;
    uint32_t acc_phase = 0;
    long long w_acc = 0, busy = 0;
    for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) {
      const MxTile tile = decode_tile<kGated>(t, st, p);
      if (!ptx::mbar_wait_timed(ptx::smem_u32(&st->tmem_full[acc]), acc_phase, abort_flag, &w_acc)) {
        if (lane == 0) mx_timeout(p, 4);
        break;
      }
      ptx::tc_fence_after_sync();
      const long long t_drain = clock64();
      const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(acc * BN);
      const int row = tile.row0 + quarter * 32 + lane;
      const bool row_ok = row < tile.row_end;
      const uint32_t empty_bar = ptx::smem_u32(&st->tmem_empty[acc]);
      auto release = [&]() {            // one arrival per warp and tile: its loads from the accumulator are complete
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(empty_bar);
      };
      if (tile.n_pad != 0) {
        // Swapped operands: this thread's lane is output column n0 + f (and n0 + 128 + f for Linear-2's second weight
        // box), accumulator column j is row row0 + j.  Few rows: the first four warps drain them all, the other four
        // only hand the accumulator back.  In Linear-1 the 32 lanes of a warp hold one 32-element block of h of a row,
        // so the block's maximum is a warp reduction and every lane converts and stores its own code byte: the same
        // bits as the per-thread quantisation of the 128-row tiles (maximum and conversion do not depend on order).
        if (half == 1) {
          release();
        } else {
          const int f = quarter * 32 + lane;
          const int col_a = tile.n0 + f, col_b = col_a + BNH;
#pragma unroll 1
          for (int j0 = 0; j0 < tile.n_pad; j0 += 16) {
            uint32_t va[16], vb[16];
            ptx::tmem_ld_32x16(t_addr + j0, va);
            ptx::tmem_ld_32x16(t_addr + BNH + j0, vb);
            ptx::tmem_ld_wait();
            if (j0 + 16 >= tile.n_pad) release();
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const int r = tile.row0 + j0 + i;
              if (r >= tile.row_end) continue;          // (the same for every lane of the warp)
              const float a = __uint_as_float(va[i]), b = __uint_as_float(vb[i]);
              if constexpr (kGated) {
                const float hv = silu_mul(a, b);
                const uint32_t amax_bits = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(fabsf(hv)));
                const uint32_t byte = mx::scale_byte(__uint_as_float(amax_bits));
                const unsigned char code = static_cast<unsigned char>(
                    __nv_cvt_float_to_fp8(hv * mx::inverse_scale(byte), __NV_SATFINITE, __NV_E4M3));
                if (col_a < p.N) {                      // N is a multiple of 32: a warp's block is inside or outside
                  reinterpret_cast<unsigned char*>(p.hq)[static_cast<size_t>(r) * p.N + col_a] = code;
                  if (lane == 0) p.sf_h[mx::scale_byte_index(p.a_rows, r, col_a >> 5)] = static_cast<unsigned char>(byte);
                  if (p.h_dbg != nullptr) p.h_dbg[static_cast<size_t>(r) * p.N + col_a] = hv;
                }
              } else {
                if (col_a < p.N) p.y[static_cast<size_t>(r) * p.N + col_a] = __float2bfloat16_rn(a);
                if (col_b < p.N) p.y[static_cast<size_t>(r) * p.N + col_b] = __float2bfloat16_rn(b);
              }
            }
          }
        }
      } else if constexpr (kGated) {
        // this warp's blocks of 32 h columns (N is a multiple of 32: blocks are whole); the accumulator is handed
        // back right after the warp's last load from tensor memory, before that block is processed and stored
        const int jb = half * (BNH / 64);
        const int je = min((half + 1) * (BNH / 64), (p.N - tile.n0) / 32);
        if (je <= jb) release();
#pragma unroll 1
        for (int j = jb; j < je; ++j) {
          const int col = tile.n0 + 32 * j;
          uint32_t g[32], u[32];
          ptx::tmem_ld_32x32(t_addr + 32 * j, g);
          ptx::tmem_ld_32x32(t_addr + BNH + 32 * j, u);
          ptx::tmem_ld_wait();
          if (j == je - 1) release();
          float h[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) h[i] = silu_mul(__uint_as_float(g[i]), __uint_as_float(u[i]));
          uint32_t c[8];
          const uint32_t byte = mx::quantize_block(h, c);
          if (row_ok) {
            uint4* dst = p.hq + (static_cast<size_t>(row) * p.N + col) / 16;
            dst[0] = make_uint4(c[0], c[1], c[2], c[3]);
            dst[1] = make_uint4(c[4], c[5], c[6], c[7]);
            p.sf_h[mx::scale_byte_index(p.a_rows, row, col >> 5)] = static_cast<unsigned char>(byte);
            if (p.h_dbg != nullptr) {
              float4* dbg = reinterpret_cast<float4*>(p.h_dbg + static_cast<size_t>(row) * p.N + col);
#pragma unroll
              for (int i = 0; i < 8; ++i) dbg[i] = make_float4(h[4 * i], h[4 * i + 1], h[4 * i + 2], h[4 * i + 3]);
            }
          }
        }
      } else {
        const int cb = half * (BN / 2);
        const int ce = min((half + 1) * (BN / 2), p.N - tile.n0);
        if (ce <= cb) release();
#pragma unroll 1
        for (int c0 = cb; c0 < ce; c0 += 32) {
          const int col = tile.n0 + c0;
          uint32_t v[32];
          ptx::tmem_ld_32x32(t_addr + c0, v);
          ptx::tmem_ld_wait();
          if (c0 + 32 >= ce) release();
          if (row_ok) {
            uint4* dst = reinterpret_cast<uint4*>(p.y + static_cast<size_t>(row) * p.N + col);
#pragma unroll
            for (int i = 0; i < 4; ++i)
              dst[i] = make_uint4(pack_bf16(__uint_as_float(v[8 * i]), __uint_as_float(v[8 * i + 1])),
                                  pack_bf16(__uint_as_float(v[8 * i + 2]), __uint_as_float(v[8 * i + 3])),
                                  pack_bf16(__uint_as_float(v[8 * i + 4]), __uint_as_float(v[8 * i + 5])),
                                  pack_bf16(__uint_as_float(v[8 * i + 6]), __uint_as_float(v[8 * i + 7])));
          }
        }
      }
      busy += clock64() - t_drain;
      if (++acc == kAccBufs) { acc = 0; acc_phase ^= 1u; }
    }
    if (p.trace && warp == 2 && lane == 0) {
      p.trace[blockIdx.x * kMoeTraceFields + 4] = static_cast<unsigned long long>(w_acc);
      p.trace[blockIdx.x * kMoeTraceFields + 5] = static_cast<unsigned long long>(busy);
    }
  } else {
    // ------------------------------------------------------------------ scale loaders (4 warps, one operand row each)
    const int w4 = warp - 6;                      // 0..3
    // Row of a 128-row group this thread serves.  Row r sits at (r % 32) * 16 + (r / 32) * 4 inside the group's
    // 512 bytes; with r = 32 * (lane % 4) + 8 * w4 + lane / 4 the 32 lanes of a warp store 32 consecutive words (one
    // shared-memory wavefront) and read four runs of eight consecutive rows from global memory.  Plain loads into
    // registers, kPrefetch stages ahead, then plain stores: a 4-byte cp.async costs 16 shared-memory wavefronts
    // per warp whatever the addresses, a quarter of the shared-memory pipe at this kernel's rate.
    const int idx = 32 * (lane & 3) + 8 * w4 + (lane >> 2);
    const uint32_t dst_a = (idx & 31) * 16 + (idx >> 5) * 4;
    const int n1 = idx + kSfThreads;              // second weight row of this thread
    const uint32_t dst_b1 = 512 + (n1 & 31) * 16 + ((n1 & 127) >> 5) * 4;
    constexpr int kPrefetch = 4;

    // prefetch cursor: the (tile, K block) whose scale words are loaded next
    int pf_t = blockIdx.x, pf_kb = 0;
    const uint32_t *pf_a = nullptr, *pf_b0 = nullptr, *pf_b1 = nullptr;   // null = outside the operand: scale byte 0
    auto pf_setup = [&]() {
      if (pf_t >= total_tiles) return;
      const MxTile tile = decode_tile<kGated>(pf_t, st, p);
      const long long a_row = static_cast<long long>(tile.row0) + idx;
      // weight row n of the tile: rows 0..127 come from the first box, 128..255 from the second
      const long long b_row_0 = idx < BNH ? static_cast<long long>(tile.w_row0) + idx
                                          : static_cast<long long>(tile.w_row0) + b1_shift + (idx - BNH);
      const long long b_row_1 = static_cast<long long>(tile.w_row0) + b1_shift + (n1 - BNH);
      pf_a = a_row < p.a_rows ? p.sf_a + a_row : nullptr;
      pf_b0 = b_row_0 < p.b_rows ? (idx < BNH ? p.sf_b0 : p.sf_b1) + b_row_0 : nullptr;
      pf_b1 = (n1 < BN && b_row_1 < p.b_rows) ? p.sf_b1 + b_row_1 : nullptr;
    };
    auto pf_load = [&](uint32_t (&w)[3]) {
      w[0] = pf_a ? __ldg(pf_a + pf_kb * p.a_rows) : 0u;
      w[1] = pf_b0 ? __ldg(pf_b0 + pf_kb * p.b_rows) : 0u;
      w[2] = pf_b1 ? __ldg(pf_b1 + pf_kb * p.b_rows) : 0u;
      if (++pf_kb == p.k_blocks) {
        pf_kb = 0;
        pf_t += gridDim.x;
        pf_setup();
      }
    };
    pf_setup();
    uint32_t buf[kPrefetch][3];
#pragma unroll
    for (int u = 0; u < kPrefetch; ++u) {
      buf[u][0] = buf[u][1] = buf[u][2] = 0u;
      if (pf_t < total_tiles) pf_load(buf[u]);
    }
    long long remaining = 0;                      // stages this CTA runs in all
    for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) remaining += p.k_blocks;
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    while (ok && remaining > 0) {
#pragma unroll
      for (int u = 0; u < kPrefetch; ++u) {
        if (remaining <= 0) break;
        if (!ptx::mbar_wait(ptx::smem_u32(&st->empty[stage]), phase ^ 1u, abort_flag)) {
          if (lane == 0) mx_timeout(p, 5);
          ok = false;
          break;
        }
        unsigned char* sf = base + kStages * kOperandBytes + stage * kSfBytes;
        *reinterpret_cast<uint32_t*>(sf + dst_a) = buf[u][0];
        *reinterpret_cast<uint32_t*>(sf + kSfABytes + dst_a) = buf[u][1];
        if (n1 < BN) *reinterpret_cast<uint32_t*>(sf + kSfABytes + dst_b1) = buf[u][2];
        ptx::fence_proxy_async_smem();      // the words were stored through the generic proxy, tcgen05.cp reads them
        ptx::mbar_arrive(ptx::smem_u32(&st->full[stage]));
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
        --remaining;
        if (pf_t < total_tiles) pf_load(buf[u]);
      }
    }
  }

  __syncthreads();
  if (st->abort_flag) {
    // a wait gave up: give copies still in flight time to land before the shared memory is released
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

// Tensor map over a row-major [rows, cols] matrix of E4M3 bytes: boxes of box_rows x 128 bytes, 128-byte swizzle.
CUresult encode_bytes(moe_ctx* ctx, CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(BK), box_rows};
  const cuuint32_t elem[2] = {1u, 1u};
  return ctx->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, elem,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

constexpr size_t kSmemBytes = 1024 + static_cast<size_t>(kStages) * (kOperandBytes + kSfBytes) + sizeof(MxTail);

}  // namespace

namespace moe {

cudaError_t prepare_expert_ffn_mx(moe_ctx* ctx) {
  (void)ctx;
  cudaError_t e = cudaFuncSetAttribute(expert_ffn_mx_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(kSmemBytes));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(expert_ffn_mx_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              static_cast<int>(kSmemBytes));
}

moe_status launch_expert_ffn_mx(moe_ctx* ctx, const moe_mx_ffn_args* a, cudaStream_t stream) {
  const moe_shape& s = ctx->shape;
  const uint64_t R = static_cast<uint64_t>(s.T) * s.k;
  CUtensorMap tm_x, tm_wg, tm_wu, tm_h, tm_wd;
  if (encode_bytes(ctx, &tm_x, a->xq_perm, R, s.H, BM) != CUDA_SUCCESS) return MOE_ERR_CUDA;
  if (encode_bytes(ctx, &tm_wg, a->wq_gate, static_cast<uint64_t>(s.E) * s.F, s.H, BNH) != CUDA_SUCCESS) return MOE_ERR_CUDA;
  if (encode_bytes(ctx, &tm_wu, a->wq_up, static_cast<uint64_t>(s.E) * s.F, s.H, BNH) != CUDA_SUCCESS) return MOE_ERR_CUDA;
  if (encode_bytes(ctx, &tm_h, a->hq_ws, R, s.F, BM) != CUDA_SUCCESS) return MOE_ERR_CUDA;
  if (encode_bytes(ctx, &tm_wd, a->wq_down, static_cast<uint64_t>(s.E) * s.H, s.F, BNH) != CUDA_SUCCESS) return MOE_ERR_CUDA;

  MxParams p1{};
  p1.offsets = a->offsets;
  p1.E = s.E;
  p1.N = s.F;
  p1.n_blocks = (s.F + BNH - 1) / BNH;
  p1.k_blocks = s.H / BK;
  p1.a_rows = static_cast<long long>(R);
  p1.b_rows = static_cast<long long>(s.E) * s.F;
  p1.sf_a = a->sfx_perm;
  p1.sf_b0 = a->sf_gate;
  p1.sf_b1 = a->sf_up;
  p1.hq = static_cast<uint4*>(a->hq_ws);
  p1.sf_h = reinterpret_cast<unsigned char*>(a->sfh_ws);
  p1.h_dbg = a->h_fp32_debug;
  p1.status = ctx->d_status;
  p1.trace = ctx->timing ? ctx->d_trace : nullptr;   // per-kernel timing also turns the wait counters on
  p1.cache_hints = moe_knob_value(ctx, "cache_hints", 35 | 8 | 64);   // (this kernel reads bits 0, 1 and 5)
  p1.swap_rows = moe_knob_value(ctx, "mx_swap_rows", kMxSwapRows);
  if (p1.swap_rows < 0 || p1.swap_rows > kMxSwapRows) p1.swap_rows = kMxSwapRows;

  MxParams p2{};
  p2.offsets = p1.offsets;
  p2.E = s.E;
  p2.N = s.H;
  p2.n_blocks = (s.H + BN - 1) / BN;
  p2.k_blocks = s.F / BK;
  p2.a_rows = static_cast<long long>(R);
  p2.b_rows = static_cast<long long>(s.E) * s.H;
  p2.sf_a = a->sfh_ws;
  p2.sf_b0 = a->sf_down;
  p2.sf_b1 = p2.sf_b0;
  p2.y = static_cast<__nv_bfloat16*>(a->y_perm);
  p2.status = ctx->d_status;
  p2.cache_hints = p1.cache_hints;
  p2.swap_rows = p1.swap_rows;
  p2.trace = ctx->timing ? ctx->d_trace + static_cast<size_t>(ctx->num_sms) * kMoeTraceFields : nullptr;

  const int grid = ctx->num_sms;
  if (ctx->timing &&
      cudaMemsetAsync(ctx->d_trace, 0, static_cast<size_t>(2) * ctx->num_sms * kMoeTraceFields * 8, stream) != cudaSuccess)
    return MOE_ERR_CUDA;
  expert_ffn_mx_kernel<true><<<grid, kThreads, kSmemBytes, stream>>>(tm_x, tm_wg, tm_wu, p1);
  moe_mark(ctx, 5, stream);
  expert_ffn_mx_kernel<false><<<grid, kThreads, kSmemBytes, stream>>>(tm_h, tm_wd, tm_wd, p2);
  moe_mark(ctx, 6, stream);
  ctx->last_launches += 2;
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

}  // namespace moe
