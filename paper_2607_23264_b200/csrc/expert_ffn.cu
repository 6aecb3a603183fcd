// Grouped expert GEMMs for sm_100a: Linear-1 (gate/up projections with the SiLU*mul epilogue) and
// Linear-2 (down projection), both as one persistent, warp-specialised tcgen05 kernel template.
//
// Tile: 128 rows of the expert-contiguous buffer x 256 fp32 accumulator columns in tensor memory.
//   Linear-1: columns 0..127 are gate outputs f0..f0+127, columns 128..255 the matching up outputs, so
//             the epilogue holds both halves of silu(g)*u for 128 h columns.
//   Linear-2: 256 output columns of y_perm.
// K is consumed in blocks of 64 bf16 (one 128-byte swizzle row); each block is 4 tcgen05.mma of K=16.
// Roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner, warps 2..5 = epilogue
// (warp w reads TMEM lanes 32*(w%4)..+31, i.e. tile rows).  A 4-stage shared-memory ring feeds the MMA;
// two 256-column accumulators let the epilogue of tile i overlap the mainloop of tile i+1.
// Expert row ranges are ragged: a tile may cover rows of the next expert (or past R, zero-filled by
// TMA); those rows are computed and discarded, stores are masked to the expert's own rows.
// Tile order inside an expert is N block, then M block (fastest), so the CTAs running at the same time
// share one weight tile through L2 and an expert's weights stream from HBM once.  Experts are split into
// "hot" ones (several 128-row blocks: their tiles are tensor-bound) and "cold" ones (few rows: their
// tiles only stream weights and are HBM-bound); the global order merges the hot and the cold tile lists
// at a fixed ratio so that both finish together, and CTAs draw tiles from it dynamically (one atomic
// counter).  At any time some SMs then keep the tensor pipes busy while others keep HBM busy, instead of
// the two kinds of work running one after the other.
#include <cuda_bf16.h>

#include "moe_internal.h"
#include "ptx_sm100.cuh"

namespace {

constexpr int BM = 128;            // rows per tile
constexpr int BN_ACC = 256;        // accumulator columns per tile
constexpr int BK = 64;             // K elements per pipeline stage (128 bytes of bf16)
constexpr int UMMA_K = 16;
constexpr int kStages = 4;
constexpr int kABytes = BM * BK * 2;          // 16 KiB
constexpr int kBHalfBytes = 128 * BK * 2;     // 16 KiB: one 128-row weight box
constexpr int kStageBytes = kABytes + 2 * kBHalfBytes;   // 48 KiB
constexpr int kThreads = 192;
constexpr int kMaxExperts = 1024;
constexpr int kTmemCols = 512;
constexpr int kChunkCols = 32;     // accumulator columns per tcgen05.ld = columns of one store tile
constexpr int kRing = 4;           // tile ids the producer may publish ahead of the consumers
constexpr int kHotBlocks = 2;      // experts with at least this many 128-row blocks count as tensor-bound

struct SharedTail {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint64_t ring_full[kRing];
  uint64_t ring_empty[kRing];
  int32_t ring_tile[kRing];         // tile ids drawn by the producer; -1 = no more tiles
  uint32_t tmem_base;
  volatile int abort_flag;
  volatile uint32_t mma_progress;   // K-blocks issued so far by the MMA warp (pacing clock)
  volatile int mma_idle;            // 1 while the MMA warp waits for an accumulator or has finished
  int32_t hot_prefix[kMaxExperts + 1];    // exclusive prefix of 128-row blocks over hot experts (cold count 0)
  int32_t cold_prefix[kMaxExperts + 1];   // the same over cold experts
};

constexpr size_t kSmemBytes = 1024 /* alignment slack */ + static_cast<size_t>(kStages) * kStageBytes + sizeof(SharedTail);

struct FfnParams {
  const int32_t* offsets;   // [E+1]
  int E;
  int N;                    // output columns of this GEMM per row (F for Linear-1, H for Linear-2)
  int K;                    // reduction length (H for Linear-1, F for Linear-2)
  int n_blocks;             // tiles along N
  int out_cols_per_tile;    // 128 (Linear-1) or 256 (Linear-2)
  int w_rows_per_expert;    // rows of the weight matrix per expert (= N)
  int b1_row_shift;         // row offset of the second weight box: 0 (up matrix) or 128 (same matrix)
  __nv_bfloat16* out;       // [R, N]
  float* h_dbg;             // Linear-1 only: fp32 copy of h before rounding, or nullptr
  int burst, mode, ik;      // store pacing
  int32_t* status;          // [2]
  int32_t* sched;           // [2] next tile to draw, CTAs finished; both zero between launches
  unsigned long long* trace;   // nullptr, or [gridDim.x][kMoeTraceFields] wait counters in SM clocks
  int kernel_id;
};

struct Tile {
  int row0;      // first row in the expert-contiguous buffer
  int row_end;   // end of the expert's rows (exclusive)
  int n0;        // first output column
  int w_row0;    // first row of the weight box in the [E*N, K] weight matrix
};

// Position `pos` of the merged order -> tile.  Among the first `pos` positions floor(pos*cold/total) are
// cold tiles; position pos is itself cold when that count steps up at pos+1.
__device__ __forceinline__ Tile decode_tile(int pos, const SharedTail* st, const FfnParams& p) {
  const long long hot_tiles = static_cast<long long>(st->hot_prefix[p.E]) * p.n_blocks;
  const long long cold_tiles = static_cast<long long>(st->cold_prefix[p.E]) * p.n_blocks;
  const long long total = hot_tiles + cold_tiles;
  const long long cold_before = (static_cast<long long>(pos) * cold_tiles) / total;
  const bool is_cold = ((static_cast<long long>(pos) + 1) * cold_tiles) / total > cold_before;
  const int tile = static_cast<int>(is_cold ? cold_before : pos - cold_before);
  const int32_t* prefix = is_cold ? st->cold_prefix : st->hot_prefix;
  const int q = tile / p.n_blocks;   // lies in [prefix[e], prefix[e+1]) of the owning expert
  int lo = 0, hi = p.E;              // invariant: prefix[lo] <= q < prefix[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (prefix[mid] <= q) lo = mid; else hi = mid;
  }
  const int e = lo;
  const int mb = prefix[e + 1] - prefix[e];
  const int local = tile - p.n_blocks * prefix[e];
  const int n_blk = local / mb;
  const int m_blk = local - n_blk * mb;
  Tile t;
  t.row0 = p.offsets[e] + m_blk * BM;
  t.row_end = p.offsets[e + 1];
  t.n0 = n_blk * p.out_cols_per_tile;
  t.w_row0 = e * p.w_rows_per_expert + t.n0;
  return t;
}

__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.f + __expf(-g)) * u; }

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// Hold the epilogue until the MMA warp has issued `ik` more K-blocks than at `start`, or cannot advance.
__device__ __forceinline__ void pace_gap(SharedTail* st, uint32_t start, int ik) {
  for (int spin = 0; spin < (1 << 16); ++spin) {
    if (st->mma_progress - start >= static_cast<uint32_t>(ik) || st->mma_idle || st->abort_flag) return;
    __nanosleep(64);
  }
}

template <bool kGated>
__global__ void __launch_bounds__(kThreads, 1)
expert_gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b0,
                   const __grid_constant__ CUtensorMap tm_b1, const FfnParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
  unsigned char* stage_base = smem_raw + pad;                 // 1024-byte aligned: required by the swizzle
  const uint32_t stage_u32 = raw + pad;
  SharedTail* st = reinterpret_cast<SharedTail*>(stage_base + static_cast<size_t>(kStages) * kStageBytes);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(ptx::smem_u32(&st->full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&st->empty[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(ptx::smem_u32(&st->tmem_full[a]), 1);
      ptx::mbar_init(ptx::smem_u32(&st->tmem_empty[a]), 4);   // one arrival per epilogue warp
    }
    for (int r = 0; r < kRing; ++r) {
      ptx::mbar_init(ptx::smem_u32(&st->ring_full[r]), 1);
      ptx::mbar_init(ptx::smem_u32(&st->ring_empty[r]), 5);   // MMA thread + four epilogue warps
    }
    st->abort_flag = 0;
    st->mma_progress = 0;
    st->mma_idle = 0;
    st->hot_prefix[0] = 0;
    st->cold_prefix[0] = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async_smem();
  }
  if (warp == 0) {
    // exclusive prefixes of ceil(count/128) over experts (hot and cold apart), 32 experts per step
    int32_t run_hot = 0, run_cold = 0;
    for (int base = 0; base < p.E; base += 32) {
      const int e = base + lane;
      int32_t v = 0;
      if (e < p.E) v = (p.offsets[e + 1] - p.offsets[e] + BM - 1) / BM;
      int32_t hot = v >= kHotBlocks ? v : 0;
      int32_t cold = v - hot;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int32_t oh = __shfl_up_sync(0xFFFFFFFFu, hot, off);
        const int32_t oc = __shfl_up_sync(0xFFFFFFFFu, cold, off);
        if (lane >= off) { hot += oh; cold += oc; }
      }
      if (e < p.E) {
        st->hot_prefix[e + 1] = run_hot + hot;
        st->cold_prefix[e + 1] = run_cold + cold;
      }
      run_hot += __shfl_sync(0xFFFFFFFFu, hot, 31);
      run_cold += __shfl_sync(0xFFFFFFFFu, cold, 31);
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
  const int total_tiles = (st->hot_prefix[p.E] + st->cold_prefix[p.E]) * p.n_blocks;
  const int k_blocks = (p.K + BK - 1) / BK;
  volatile int* abort_flag = &st->abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int slot = 0;
      uint32_t ring_phase = 0;
      bool ok = true;
      long long w_empty = 0;
      const long long t_begin = clock64();
      while (ok) {
        // draw the next tile and publish it to the MMA and epilogue roles
        if (!ptx::mbar_wait(ptx::smem_u32(&st->ring_empty[slot]), ring_phase ^ 1u, abort_flag)) {
          atomicCAS(&p.status[0], 0, MOE_ERR_TIMEOUT);
          atomicCAS(&p.status[1], 0, p.kernel_id * 65536 + 5);
          break;
        }
        int pos = atomicAdd(&p.sched[0], 1);
        if (pos >= total_tiles) pos = -1;
        st->ring_tile[slot] = pos;
        ptx::mbar_arrive(ptx::smem_u32(&st->ring_full[slot]));
        if (++slot == kRing) { slot = 0; ring_phase ^= 1u; }
        if (pos < 0) break;
        const Tile t = decode_tile(pos, st, p);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!ptx::mbar_wait_timed(ptx::smem_u32(&st->empty[stage]), phase ^ 1u, abort_flag, &w_empty)) {
            atomicCAS(&p.status[0], 0, MOE_ERR_TIMEOUT);
            atomicCAS(&p.status[1], 0, p.kernel_id * 65536 + 1);
            ok = false;
            break;
          }
          const uint32_t full = ptx::smem_u32(&st->full[stage]);
          const uint32_t sa = stage_u32 + stage * kStageBytes;
          ptx::mbar_expect_tx(full, kStageBytes);
          ptx::tma_load_2d(sa, &tm_a, full, kb * BK, t.row0);
          ptx::tma_load_2d(sa + kABytes, &tm_b0, full, kb * BK, t.w_row0);
          ptx::tma_load_2d(sa + kABytes + kBHalfBytes, &tm_b1, full, kb * BK, t.w_row0 + p.b1_row_shift);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (p.trace) {
        p.trace[blockIdx.x * kMoeTraceFields + 0] = static_cast<unsigned long long>(clock64() - t_begin);
        p.trace[blockIdx.x * kMoeTraceFields + 1] = static_cast<unsigned long long>(w_empty);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::idesc_bf16_f32(BM, BN_ACC);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      uint32_t progress = 0;
      int slot = 0;
      uint32_t ring_phase = 0;
      bool ok = true;
      long long w_full = 0, w_tmem = 0;
      unsigned long long n_tiles = 0;
      while (ok) {
        st->mma_idle = 1;
        if (!ptx::mbar_wait(ptx::smem_u32(&st->ring_full[slot]), ring_phase, abort_flag)) {
          atomicCAS(&p.status[0], 0, MOE_ERR_TIMEOUT);
          atomicCAS(&p.status[1], 0, p.kernel_id * 65536 + 6);
          break;
        }
        const int pos = st->ring_tile[slot];
        ptx::mbar_arrive(ptx::smem_u32(&st->ring_empty[slot]));
        if (++slot == kRing) { slot = 0; ring_phase ^= 1u; }
        if (pos < 0) break;
        if (!ptx::mbar_wait_timed(ptx::smem_u32(&st->tmem_empty[acc]), acc_phase ^ 1u, abort_flag, &w_tmem)) {
          atomicCAS(&p.status[0], 0, MOE_ERR_TIMEOUT);
          atomicCAS(&p.status[1], 0, p.kernel_id * 65536 + 2);
          break;
        }
        st->mma_idle = 0;
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN_ACC);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!ptx::mbar_wait_timed(ptx::smem_u32(&st->full[stage]), phase, abort_flag, &w_full)) {
            atomicCAS(&p.status[0], 0, MOE_ERR_TIMEOUT);
            atomicCAS(&p.status[1], 0, p.kernel_id * 65536 + 3);
            ok = false;
            break;
          }
          ptx::tc_fence_after_sync();
          const uint32_t sa = stage_u32 + stage * kStageBytes;
          const uint64_t a_desc = ptx::smem_desc_sw128(sa);
          const uint64_t b_desc = ptx::smem_desc_sw128(sa + kABytes);
#pragma unroll
          for (int k4 = 0; k4 < BK / UMMA_K; ++k4) {
            // +32 bytes along K inside the swizzle row = +2 in the descriptor's 16-byte address units
            ptx::tc_mma_bf16(d_tmem, a_desc + static_cast<uint64_t>(2 * k4), b_desc + static_cast<uint64_t>(2 * k4),
                             idesc, (kb | k4) != 0 ? 1u : 0u);
          }
          ptx::tc_commit(ptx::smem_u32(&st->empty[stage]));   // stage is free once these MMAs have read it
          st->mma_progress = ++progress;
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ptx::tc_commit(ptx::smem_u32(&st->tmem_full[acc]));    // accumulator complete
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
        ++n_tiles;
      }
      st->mma_idle = 1;
      if (p.trace) {
        p.trace[blockIdx.x * kMoeTraceFields + 2] = static_cast<unsigned long long>(w_full);
        p.trace[blockIdx.x * kMoeTraceFields + 3] = static_cast<unsigned long long>(w_tmem);
        p.trace[blockIdx.x * kMoeTraceFields + 6] = n_tiles;
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue (4 warps = 128 rows)
    const int quarter = warp & 3;                 // TMEM lane quarter this warp may read
    const int r_in_tile = quarter * 32 + lane;
    int acc = 0;
    uint32_t acc_phase = 0;
    const int burst = p.burst;
    int slot = 0;
    uint32_t ring_phase = 0;
    long long w_acc = 0, busy = 0, w_gap = 0;
    while (true) {
      if (!ptx::mbar_wait(ptx::smem_u32(&st->ring_full[slot]), ring_phase, abort_flag)) {
        if (lane == 0) {
          atomicCAS(&p.status[0], 0, MOE_ERR_TIMEOUT);
          atomicCAS(&p.status[1], 0, p.kernel_id * 65536 + 7);
        }
        break;
      }
      const int pos = st->ring_tile[slot];
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&st->ring_empty[slot]));
      if (++slot == kRing) { slot = 0; ring_phase ^= 1u; }
      if (pos < 0) break;
      const Tile t = decode_tile(pos, st, p);
      if (!ptx::mbar_wait_timed(ptx::smem_u32(&st->tmem_full[acc]), acc_phase, abort_flag, &w_acc)) {
        if (lane == 0) {
          atomicCAS(&p.status[0], 0, MOE_ERR_TIMEOUT);
          atomicCAS(&p.status[1], 0, p.kernel_id * 65536 + 4);
        }
        break;
      }
      ptx::tc_fence_after_sync();
      const long long t_store = clock64();
      const int row = t.row0 + r_in_tile;
      const bool row_ok = row < t.row_end;
      const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                              static_cast<uint32_t>(acc * BN_ACC);
      __nv_bfloat16* out_row = p.out + static_cast<size_t>(row) * p.N + t.n0;
      constexpr int kChunks = kGated ? (128 / kChunkCols) : (BN_ACC / kChunkCols);
      int in_burst = 0;
      uint32_t gap_start = st->mma_progress;
#pragma unroll 1
      for (int c = 0; c < kChunks; ++c) {
        uint32_t v[32];
        float o[32];
        if constexpr (kGated) {
          uint32_t u[32];
          ptx::tmem_ld_32x32(t_addr + c * kChunkCols, v);
          ptx::tmem_ld_32x32(t_addr + 128 + c * kChunkCols, u);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] = silu_mul(__uint_as_float(v[i]), __uint_as_float(u[i]));
        } else {
          ptx::tmem_ld_32x32(t_addr + c * kChunkCols, v);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] = __uint_as_float(v[i]);
        }
        const int col0 = t.n0 + c * kChunkCols;
        if (row_ok) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            if (col0 + q * 8 < p.N) {     // N is a multiple of 8: a 16-byte vector is inside or outside
              uint4 w;
              w.x = pack_bf16(o[q * 8 + 0], o[q * 8 + 1]);
              w.y = pack_bf16(o[q * 8 + 2], o[q * 8 + 3]);
              w.z = pack_bf16(o[q * 8 + 4], o[q * 8 + 5]);
              w.w = pack_bf16(o[q * 8 + 6], o[q * 8 + 7]);
              *reinterpret_cast<uint4*>(out_row + c * kChunkCols + q * 8) = w;
            }
          }
          if constexpr (kGated) {
            if (p.h_dbg != nullptr) {
              float* dbg = p.h_dbg + static_cast<size_t>(row) * p.N + col0;
#pragma unroll
              for (int q = 0; q < 8; ++q) {
                if (col0 + q * 4 < p.N) {
                  *reinterpret_cast<float4*>(dbg + q * 4) = make_float4(o[q * 4], o[q * 4 + 1], o[q * 4 + 2], o[q * 4 + 3]);
                }
              }
            }
          }
        }
        if (p.mode == 1 && ++in_burst >= burst && c + 1 < kChunks) {
          const long long t_gap = clock64();
          pace_gap(st, gap_start, p.ik);
          w_gap += clock64() - t_gap;
          gap_start = st->mma_progress;
          in_burst = 0;
        }
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&st->tmem_empty[acc]));
      busy += clock64() - t_store;
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
    if (p.trace && warp == 2 && lane == 0) {
      p.trace[blockIdx.x * kMoeTraceFields + 4] = static_cast<unsigned long long>(w_acc);
      p.trace[blockIdx.x * kMoeTraceFields + 5] = static_cast<unsigned long long>(busy);
      p.trace[blockIdx.x * kMoeTraceFields + 7] = static_cast<unsigned long long>(w_gap);
    }
  }

  __syncthreads();
  if (st->abort_flag) {
    // Give copies and MMAs still in flight a bounded time to land before the CTA's memory is released.
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
  // Every CTA has drawn its last tile by now.  The last CTA to leave re-arms the scheduler for the next launch.
  if (tid == 0) {
    const int done = atomicAdd(&p.sched[1], 1);
    if (done == static_cast<int>(gridDim.x) - 1) {
      p.sched[0] = 0;
      p.sched[1] = 0;
      __threadfence();
    }
  }
}

// Calibration probe: one CTA issues `iters` tcgen05.mma of shape M x N x 16 back to back on resident
// shared-memory operands and reports the SM clocks from the first issue to the completion of the last.
__global__ void __launch_bounds__(128, 1) mma_cycle_probe(int M, int N, int iters, long long* out) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ uint64_t bar;
  __shared__ uint32_t tmem_base_s;
  __shared__ volatile int abort_flag;
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
  const uint32_t base = raw + pad;
  for (int i = threadIdx.x; i < kStageBytes / 4; i += blockDim.x)
    reinterpret_cast<uint32_t*>(smem_raw + pad)[i] = 0x3c003c00u;   // bf16 values near 0.0078
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    abort_flag = 0;
    ptx::fence_barrier_init();
  }
  ptx::fence_proxy_async_smem();
  if (threadIdx.x < 32) {
    ptx::tmem_alloc(ptx::smem_u32(&tmem_base_s), kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tb = tmem_base_s;
  if (threadIdx.x == 0) {
    const uint32_t idesc = ptx::idesc_bf16_f32(M, N);
    const uint64_t a = ptx::smem_desc_sw128(base), b = ptx::smem_desc_sw128(base + kABytes);
    const long long t0 = clock64();
    for (int i = 0; i < iters; ++i) {
      const uint64_t adv = static_cast<uint64_t>(2 * (i & 3));
      ptx::tc_mma_bf16(tb, a + adv, b + adv, idesc, i > 0 ? 1u : 0u);
    }
    ptx::tc_commit(ptx::smem_u32(&bar));
    ptx::mbar_wait(ptx::smem_u32(&bar), 0, &abort_flag);
    out[0] = abort_flag ? -1 : clock64() - t0;
  }
  __syncthreads();
  if (threadIdx.x < 32) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tb, kTmemCols);
  }
}

CUresult encode_2d(moe_ctx* ctx, CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(BK), 128u};
  const cuuint32_t elem[2] = {1u, 1u};
  return ctx->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                           elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

}  // namespace

extern "C" moe_status moe_probe_mma_cycles(moe_ctx* ctx, int32_t M, int32_t N, int32_t iters, double* cycles_per_mma,
                                           void* stream) {
  if (!ctx || !cycles_per_mma) return MOE_ERR_INVALID_ARG;
  if (!(M == 64 || M == 128) || N < 16 || N > 256 || N % 16 != 0 || iters < 1 || iters > (1 << 20))
    return MOE_ERR_INVALID_ARG;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  long long* d_out = reinterpret_cast<long long*>(ctx->d_trace);   // reuse the first trace word as the result slot
  const size_t smem = 1024 + kStageBytes;
  if (cudaFuncSetAttribute(mma_cycle_probe, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) !=
      cudaSuccess)
    return MOE_ERR_CUDA;
  mma_cycle_probe<<<1, 128, smem, cs>>>(M, N, iters, d_out);
  long long clocks = 0;
  if (cudaMemcpyAsync(&clocks, d_out, sizeof(clocks), cudaMemcpyDeviceToHost, cs) != cudaSuccess) return MOE_ERR_CUDA;
  if (cudaStreamSynchronize(cs) != cudaSuccess) return MOE_ERR_CUDA;
  if (clocks < 0) return MOE_ERR_TIMEOUT;
  *cycles_per_mma = static_cast<double>(clocks) / iters;
  return MOE_OK;
}

namespace moe {

cudaError_t prepare_expert_ffn(moe_ctx*) {
  cudaError_t e = cudaFuncSetAttribute(expert_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(kSmemBytes));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(expert_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              static_cast<int>(kSmemBytes));
}

moe_status launch_expert_ffn(moe_ctx* ctx, const void* x_perm, const int32_t* offsets, const void* w_gate,
                             const void* w_up, const void* w_down, void* h_ws, void* y_perm,
                             float* h_fp32_debug, const moe_tuning* tuning, cudaStream_t stream) {
  const moe_shape& s = ctx->shape;
  const uint64_t R = static_cast<uint64_t>(s.T) * s.k;
  if (R == 0) return MOE_OK;
  moe_tuning tn = {1, 0, 1, 0, 0, 0};
  if (tuning) tn = *tuning;

  CUtensorMap tm_x, tm_wg, tm_wu, tm_h, tm_wd;
  if (encode_2d(ctx, &tm_x, x_perm, R, s.H) != CUDA_SUCCESS) return MOE_ERR_CUDA;
  if (encode_2d(ctx, &tm_wg, w_gate, static_cast<uint64_t>(s.E) * s.F, s.H) != CUDA_SUCCESS) return MOE_ERR_CUDA;
  if (encode_2d(ctx, &tm_wu, w_up, static_cast<uint64_t>(s.E) * s.F, s.H) != CUDA_SUCCESS) return MOE_ERR_CUDA;
  if (encode_2d(ctx, &tm_h, h_ws, R, s.F) != CUDA_SUCCESS) return MOE_ERR_CUDA;
  if (encode_2d(ctx, &tm_wd, w_down, static_cast<uint64_t>(s.E) * s.H, s.F) != CUDA_SUCCESS) return MOE_ERR_CUDA;

  FfnParams p1{};
  p1.offsets = offsets;
  p1.E = s.E;
  p1.N = s.F;
  p1.K = s.H;
  p1.n_blocks = (s.F + 127) / 128;
  p1.out_cols_per_tile = 128;
  p1.w_rows_per_expert = s.F;
  p1.b1_row_shift = 0;
  p1.out = static_cast<__nv_bfloat16*>(h_ws);
  p1.h_dbg = h_fp32_debug;
  p1.burst = tn.store_burst_tiles;
  p1.mode = tn.interleave_mode;
  p1.ik = tn.interleave_k;
  p1.status = ctx->d_status;
  p1.sched = ctx->d_sched;
  p1.trace = (tn.debug_flags & 1) ? ctx->d_trace : nullptr;
  p1.kernel_id = 1;

  FfnParams p2 = p1;
  p2.N = s.H;
  p2.K = s.F;
  p2.n_blocks = (s.H + 255) / 256;
  p2.out_cols_per_tile = 256;
  p2.w_rows_per_expert = s.H;
  p2.b1_row_shift = 128;
  p2.out = static_cast<__nv_bfloat16*>(y_perm);
  p2.h_dbg = nullptr;
  p2.sched = ctx->d_sched + 2;
  p2.trace = p1.trace ? p1.trace + static_cast<size_t>(ctx->num_sms) * kMoeTraceFields : nullptr;
  p2.kernel_id = 2;

  const int grid = ctx->num_sms;   // persistent: one CTA per SM (shared memory allows no second)
  expert_gemm_kernel<true><<<grid, kThreads, kSmemBytes, stream>>>(tm_x, tm_wg, tm_wu, p1);
  moe_mark(ctx, 5, stream);
  expert_gemm_kernel<false><<<grid, kThreads, kSmemBytes, stream>>>(tm_h, tm_wd, tm_wd, p2);
  moe_mark(ctx, 6, stream);
  ctx->last_launches += 2;
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

}  // namespace moe
