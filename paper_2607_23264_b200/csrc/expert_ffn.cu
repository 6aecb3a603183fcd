// Grouped expert GEMMs for sm_100a: Linear-1 (gate/up projections with the SiLU*mul epilogue) and
// Linear-2 (down projection) in one persistent, warp-specialised tcgen05 kernel.
//
// Tile: 128 rows of the expert-contiguous buffer x 256 fp32 accumulator columns in tensor memory.
//   Linear-1: columns 0..127 are gate outputs f0..f0+127, columns 128..255 the matching up outputs, so
//             the epilogue holds both halves of silu(g)*u for 128 h columns.
//   Linear-2: 256 output columns of y_perm.
// K is consumed in blocks of 64 bf16 (one 128-byte swizzle row); each block is 4 tcgen05.mma of K=16.
// Roles (192 threads): warp 0 = TMA producer and tile scheduler, warp 1 = MMA issuer and TMEM owner,
// warps 2..5 = epilogue (warp w reads TMEM lanes 32*(w%4)..+31, i.e. tile rows).  A 4-stage
// shared-memory ring feeds the MMA; two 256-column accumulators let the epilogue of tile i overlap the
// mainloop of tile i+1.  The producer publishes the tiles it draws to the other roles through a small
// ring of tile codes.
// Expert row ranges are ragged: a tile may cover rows of the next expert (or past R, zero-filled by
// TMA); those rows are computed and discarded, stores are masked to the expert's own rows.
// Stores: an epilogue warp whose 32 rows all belong to the expert packs 64 output columns at a time into a
// swizzled 4 KiB box of shared memory and one lane hands the box to the TMA unit (whole 128-byte lines, no
// load/store-unit work per row); a warp with rows of the next expert, a paced run and a launch whose Linear-2 tiles
// wait for h store 16 bytes per lane and row from registers instead.  Both ways write the same values.  The CTA-pair
// kernel further down stores the same way.
//
// Tile orders (moe_tuning.schedule):
//   0  Expert-Wave: all Linear-1 tiles, then all Linear-2 tiles.  Inside a GEMM the order within an expert is
//      N block, then M block (fastest), so the CTAs running at the same time share one weight tile through L2
//      and an expert's weights stream from HBM once.  Experts are split into "hot" ones (several 128-row
//      blocks: tensor-bound tiles) and "cold" ones (one block: their tiles only stream weights, HBM-bound);
//      the order merges the hot and the cold tile lists at a fixed ratio so that both finish together, and
//      CTAs draw tiles dynamically from one atomic counter.  Run as two launches (the kernel boundary is the
//      Linear-1 -> Linear-2 dependency) or as one launch with per-block ready counters.
//   1  Interleaved (Algorithm 1 of the paper): both GEMMs' tiles are listed row-major (row = one 128-row block),
//      CTA g of G owns tiles g, g+G, ... of each list and splices its Linear-2 tiles between its Linear-1 tiles as
//      early as a row lead of D allows (InterleaveCursor below).  One launch; a Linear-2 tile waits (bounded)
//      until all Linear-1 tiles of its row have published their h rows.
// An expert with at most 64 rows is computed with the operands swapped: each 128-row weight box is the MMA's M
// side and the expert's rows, padded to a multiple of 16, its N side.  A tcgen05.mma costs 128 clocks at N = 256 but
// 46 at N <= 32, so the two instructions per K step (one per weight box) take 92 clocks instead of 128; the
// shared-memory stage is the same three boxes, only the MMA issue and the epilogue (lane = output column) differ.
// A launch whose experts all hold at most 16 rows runs on six 34 KiB stages (16-row A box + two weight boxes).
// A CTA-pair variant (256-row tiles over a cluster of two CTAs, cta_group::2) follows further down; it runs on request
// and for Linear-1 of the E4M3 path on layers of many-row experts.
#include <cuda_bf16.h>

#include <type_traits>

#include "ffn_math.cuh"
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
// Wide mode (launches with many-row experts, see below): a stage holds a second 128-row A box, and three such stages
// take the room of the four.
constexpr int kWideStages = 3;
constexpr int kWideStageBytes = 2 * kABytes + 2 * kBHalfBytes;   // 64 KiB
static_assert(kWideStages * kWideStageBytes <= kStages * kStageBytes, "the wide ring must fit in the ring's shared memory");
// A launch whose experts all hold at most 16 rows (decode-like layers): a stage is one 16-row box of A and the two
// weight boxes, and six of them fit in the ring plus the store boxes such a launch does not use.  These tiles live on
// the bytes in flight.
constexpr int kSmallStages = 6;
constexpr int kSmallABytes = 16 * BK * 2;                          // 2 KiB
constexpr int kSmallStageBytes = kSmallABytes + 2 * kBHalfBytes;   // 34 KiB
constexpr int kMaxStages = kSmallStages;
constexpr int kWideFlag = 1 << 16;   // in the per-tile word next to the tile code: a 256-row tile on both accumulators
constexpr int kThreads = 192;
constexpr int kMaxExperts = 1024;
constexpr int kTmemCols = 512;
constexpr int kChunkCols = 32;     // accumulator columns per tcgen05.ld = columns of one store tile
constexpr int kRing = 4;           // tile codes the producer may publish ahead of the consumers
constexpr int kHotBlocks = 2;      // experts with at least this many 128-row blocks count as tensor-bound
constexpr int kSwapRows = 64;      // row blocks with at most this many rows (small experts, short last blocks) run with swapped operands
constexpr int kPhaseShift = 30;    // tile code = phase << 30 | index in the phase's tile list; -1 = no more tiles

struct SharedTail {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint64_t ring_full[kRing];
  uint64_t ring_empty[kRing];
  int32_t ring_tile[kRing];
  int32_t ring_kind[kRing];         // 0, the padded row count of a tile computed with swapped operands, or kWideFlag
  uint32_t tmem_base;
  volatile int abort_flag;
  volatile uint32_t mma_progress;   // K-blocks issued so far by the MMA warp (pacing clock)
  volatile int mma_idle;            // 1 while the MMA warp waits for an accumulator or has finished
  int wide;                         // this launch cuts many-row experts into 256-row blocks (wide mode)
  int small;                        // every expert of this launch holds at most 16 rows: six 34 KiB stages
  int32_t hot_prefix[kMaxExperts + 1];    // exclusive prefix of row blocks over hot experts (cold count 0): 128-row
                                          // blocks, or 256-row blocks in wide mode
  int32_t cold_prefix[kMaxExperts + 1];   // the same over cold experts
  int32_t offs[kMaxExperts + 1];          // the expert row offsets, copied once: tile decoding reads no global memory
};

// Staging for the epilogue's bulk tensor stores: per epilogue warp one box of 32 rows x 64 bf16 columns (4 KiB, rows
// of 128 bytes in the 128-byte swizzle), between the ring and the tail.
constexpr int kStoreBoxCols = 64;
constexpr int kStoreBoxBytes = 32 * kStoreBoxCols * 2;
constexpr int kStoreStagingBytes = 4 * kStoreBoxBytes;
constexpr size_t kSmemBytes = 1024 /* alignment slack */ + static_cast<size_t>(kStages) * kStageBytes + kStoreStagingBytes +
                              sizeof(SharedTail);
static_assert(kSmemBytes + 64 <= 227 * 1024, "ring + store staging + tail must fit in one CTA's shared memory");
static_assert(kSmallStages * kSmallStageBytes <= kStages * kStageBytes + kStoreStagingBytes, "the small ring must fit too");

// How one epilogue warp stores: smem == 0 = 16-byte stores from registers (each lane its own row); else the warp
// stages 32 rows x 64 columns there and one lane hands them to the TMA unit as whole 128-byte lines.
struct StoreStage {
  uint32_t smem;               // this warp's box (1024-byte aligned), or 0
  const CUtensorMap* map;      // the [R, N] output in boxes of 32 rows x 64 columns, 128-byte swizzle
};

struct PhaseDesc {          // one of the two GEMMs
  int N;                    // output columns per row (F for Linear-1, H for Linear-2) = weight rows per expert
  int K;                    // reduction length (H for Linear-1, F for Linear-2)
  int n_blocks;             // tiles along N
  int k_blocks;             // 64-deep K blocks
  int out_cols_per_tile;    // 128 (Linear-1) or 256 (Linear-2)
  int b1_row_shift;         // row offset of the second weight box: 0 (up matrix) or 128 (same matrix)
  __nv_bfloat16* out;       // [R, N]
  // FP8 (E4M3) operands: fp32 scales applied in the epilogue, out = acc * row_scale[row] * col_scale[weight row];
  // all nullptr for bf16 operands.  col_scale0 belongs to the first weight box, col_scale1 to the second.
  const float* row_scale;   // [R]
  const float* col_scale0;  // [E * N]
  const float* col_scale1;  // [E * N]
};

struct FfnParams {
  const int32_t* offsets;   // [E+1]
  int E;
  PhaseDesc ph[2];
  float* h_dbg;             // fp32 copy of h before rounding, or nullptr
  int burst, mode, ik;      // store pacing
  int32_t* status;          // [2]
  int32_t* sched;           // [2] next tile to draw, CTAs finished; both zero between launches
  int32_t* ready;           // [128-row blocks] Linear-1 warps that published their part of the block's h rows
  unsigned long long* trace;   // nullptr, or [gridDim.x][kMoeTraceFields] wait counters in SM clocks
  int32_t* order_log;       // nullptr, or [gridDim.x][kMoeOrderLogCap] tile codes in the order this CTA drew them
  int phase_lo, phase_hi;   // GEMMs in this launch: [0,1) Linear-1, [1,2) Linear-2, [0,2) both
  int schedule;             // 0 merged order drawn dynamically, 1 Algorithm 1
  int lead_D;               // Algorithm 1: minimum row lead of Linear-1 over Linear-2 (>= 1)
  int fp8;                  // operands are E4M3 bytes (128 per swizzle row) instead of bf16 (64 per row)
  int k_elems;              // K elements per pipeline stage: 64 (bf16) or 128 (E4M3)
  int swap_rows;            // row blocks with at most this many rows run with swapped operands
  int wide_allowed;         // the launch may use wide mode (two-launch Expert-Wave runs)
  int cache_hints;          // L2 eviction priorities of the TMA loads, bit mask (see run_ffn)
  int small_a;              // swapped-operand tiles of at most this many padded rows load A in 16-row boxes (0: never)
  int bulk_stores;          // single-CTA kernel: whole 32-row groups of a tile leave through shared memory and TMA stores
  int small_ring;           // launches whose experts all hold at most 16 rows use six 34 KiB stages
  int expert_class;         // 0: all experts.  A GEMM split into two launches: 1 = the experts of at most 16 rows (all
                            // experts, if the layer does not hold both kinds), 2 = the others (none, if it does not)
  int withhold_ready;       // host-requested failure drill: Linear-1 never publishes its rows (one-launch runs)
  long long wait_budget;    // clocks a cross-CTA wait may last before it gives up
  int kernel_id;
};

struct Tile {
  int phase;     // 0 Linear-1, 1 Linear-2
  int row0;      // first row in the expert-contiguous buffer
  int row_end;   // end of the expert's rows (exclusive)
  int n0;        // first output column
  int w_row0;    // first row of the weight box in the [E*N, K] weight matrix
  int block;     // global index of the 128-row block (ready counter)
  int n_pad;     // 0 for a 128-row tile; else operands are swapped and this is the row count padded to 16
  int wide;      // 1: the tile covers rows row0 .. row0 + 255 on both accumulators (rows row0 + 128.. on the second)
  int single;    // 1: the expert has a single row block, so no other tile reads these weight boxes
};

// Largest e with prefix(e) <= q, prefix non-decreasing with prefix(0) = 0 and q < prefix(E).
template <class F>
__device__ __forceinline__ int find_expert(F prefix, int q, int E) {
  int lo = 0, hi = E;   // invariant: prefix(lo) <= q < prefix(hi)
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (prefix(mid) <= q) lo = mid; else hi = mid;
  }
  return lo;
}

// m_blk counts the expert's row blocks in the unit of its class: 256 rows for a hot expert in wide mode, else 128.
__device__ __forceinline__ Tile make_tile(int phase, int e, int m_blk, int n_blk, bool hot, const SharedTail* st,
                                          const FfnParams& p) {
  const PhaseDesc& d = p.ph[phase];
  const int unit = (hot && st->wide) ? 2 * BM : BM;
  Tile t;
  t.phase = phase;
  t.row0 = st->offs[e] + m_blk * unit;
  t.row_end = st->offs[e + 1];
  t.n0 = n_blk * d.out_cols_per_tile;
  t.w_row0 = e * d.N + t.n0;
  t.block = st->hot_prefix[e] + st->cold_prefix[e] + m_blk;
  const int rows = min(t.row_end - t.row0, unit);                 // rows of this block: a whole small expert, or the
  t.wide = rows > BM ? 1 : 0;                                     // (short) last block of a larger one
  t.n_pad = rows <= p.swap_rows ? ((rows + 15) & ~15) : 0;        // few rows: swapped operands
  t.single = st->offs[e + 1] - st->offs[e] <= BM ? 1 : 0;
  return t;
}

// Tile code -> tile.
//  schedule 0: index = position in the merged hot/cold order of the phase.  Among the first `pos` positions
//              floor(pos*cold/total) are cold tiles; position pos is itself cold when that count steps up at
//              pos+1.  Inside a class the order is expert, N block, M block (fastest).
//  schedule 1: index = row-major tile number k: row k / n_blocks (a global 128-row block), column k % n_blocks.
__device__ __forceinline__ Tile decode_tile(int code, const SharedTail* st, const FfnParams& p) {
  const int phase = code >> kPhaseShift;
  const int idx = code & ((1 << kPhaseShift) - 1);
  const int nb = p.ph[phase].n_blocks;
  if (p.schedule == 1) {
    const int row = idx / nb;
    const int n_blk = idx - row * nb;
    const int e = find_expert([&](int i) { return st->hot_prefix[i] + st->cold_prefix[i]; }, row, p.E);
    return make_tile(phase, e, row - (st->hot_prefix[e] + st->cold_prefix[e]), n_blk, false, st, p);   // never wide
  }
  const long long hot_tiles = static_cast<long long>(st->hot_prefix[p.E]) * nb;
  const long long cold_tiles = static_cast<long long>(st->cold_prefix[p.E]) * nb;
  const long long total = hot_tiles + cold_tiles;
  const long long cold_before = (static_cast<long long>(idx) * cold_tiles) / total;
  const bool is_cold = ((static_cast<long long>(idx) + 1) * cold_tiles) / total > cold_before;
  const int tile = static_cast<int>(is_cold ? cold_before : idx - cold_before);
  const int32_t* prefix = is_cold ? st->cold_prefix : st->hot_prefix;
  const int e = find_expert([&](int i) { return prefix[i]; }, tile / nb, p.E);
  const int mb = prefix[e + 1] - prefix[e];
  const int local = tile - nb * prefix[e];
  const int n_blk = local / mb;
  return make_tile(phase, e, local - n_blk * mb, n_blk, !is_cold, st, p);
}

// Schedule 1 (the paper's Algorithm 1): a CTA owns every stride-th tile of each GEMM's row-major tile list and keeps
// the tiles of one GEMM in list order; what is decided per draw is only which GEMM goes next.  Linear-2 goes when
// it has a tile left whose row lies at least `lead` rows behind the row of the CTA's pending Linear-1 tile (or
// Linear-1 has none left); otherwise Linear-1 goes.  Returns the tile code, -1 when both lists are exhausted.
struct InterleaveCursor {
  int next1, next2;   // this CTA's pending tile of Linear-1 / Linear-2
  int stride;         // scheduler instances = CTAs of the launch
  __device__ __forceinline__ int draw(int tiles1, int tiles2, int per_row1, int per_row2, int lead) {
    const bool left1 = next1 < tiles1, left2 = next2 < tiles2;
    if (!left1 && !left2) return -1;
    const bool linear2_may_go = left2 && (!left1 || next2 / per_row2 + lead <= next1 / per_row1);
    int code;
    if (linear2_may_go) {
      code = (1 << kPhaseShift) | next2;
      next2 += stride;
    } else {
      code = next1;
      next1 += stride;
    }
    return code;
  }
};

__device__ __forceinline__ void report_timeout(const FfnParams& p, int role) {
  atomicCAS(&p.status[0], 0, MOE_ERR_TIMEOUT);
  atomicCAS(&p.status[1], 0, p.kernel_id * 65536 + role);
}

// Store pacing of one epilogue warp.  The state lives across the CTA's tiles, so a burst of `burst` store tiles may
// span accumulators.  After a burst the next store is held until the MMA warp (this CTA's, or the pair leader's: the
// words are read through their shared::cluster addresses) has issued `ik` more K blocks than when the burst ended,
// or cannot advance (it waits for an accumulator or has finished), or the CTA is aborting, or a spin cap expires.
struct Pacer {
  uint32_t progress_addr, idle_addr;   // shared::cluster addresses of mma_progress / mma_idle
  int in_burst;                        // store tiles written since the last gap
  uint32_t burst_end;                  // mma_progress when the current burst was completed
  long long held;                      // clocks spent holding stores
  __device__ __forceinline__ void before_store(const int burst, const int ik, volatile int* aborting) {
    if (in_burst < burst) return;
    const long long t0 = clock64();
    for (int spin = 0; spin < (1 << 16); ++spin) {
      if (ptx::ld_cluster_u32(progress_addr) - burst_end >= static_cast<uint32_t>(ik) ||
          ptx::ld_cluster_u32(idle_addr) != 0u || *aborting)
        break;
      __nanosleep(64);
    }
    held += clock64() - t0;
    in_burst = 0;
  }
  __device__ __forceinline__ void after_store(const int burst) {
    if (++in_burst >= burst) burst_end = ptx::ld_cluster_u32(progress_addr);
  }
};

// Bounded wait until `*counter` (written by other CTAs with release ordering) reaches `target`.
__device__ __forceinline__ bool wait_counter(const int32_t* counter, int target, volatile int* abort_flag,
                                             long long budget) {
  const long long t0 = clock64();
  for (uint32_t it = 0;; ++it) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
    if (v >= target) return true;
    if ((it & 0xFu) == 0xFu) {
      if (*abort_flag) return false;
      if (clock64() - t0 > budget) {
        *abort_flag = 1;
        return false;
      }
    }
    __nanosleep(100);
  }
}

// Drain one finished accumulator: rows of this thread's TMEM lane, kGated ? silu(g)*u of 128 columns
// : 256 plain columns, written as bf16 with 16-byte stores masked to the expert's rows and to N.
template <bool kGated, bool kFp8>
__device__ __forceinline__ void drain_accumulator(const Tile& t, const FfnParams& p, uint32_t t_addr, int row,
                                                  Pacer& pacer, volatile int* aborting, const StoreStage& ss) {
  const PhaseDesc& d = p.ph[kGated ? 0 : 1];
  const bool row_ok = row < t.row_end;
  const int lane = threadIdx.x & 31;
  // Bulk stores when all 32 rows of the warp belong to the expert (a box cannot be masked by rows) and the stores
  // are not paced (a paced store tile is one 32-column chunk)
  const bool bulk = ss.smem != 0 && p.mode == 0 && p.h_dbg == nullptr && row - lane + 32 <= t.row_end;
  __nv_bfloat16* out_row = d.out + static_cast<size_t>(row) * d.N + t.n0;
  constexpr int kChunks = kGated ? (128 / kChunkCols) : (BN_ACC / kChunkCols);
#pragma unroll 1
  for (int c = 0; c < kChunks; ++c) {
    uint32_t v[32];
    float o[32];
    if (p.mode == 1) pacer.before_store(p.burst, p.ik, aborting);
    if constexpr (kGated) {
      uint32_t u[32];
      ptx::tmem_ld_32x32(t_addr + c * kChunkCols, v);
      ptx::tmem_ld_32x32(t_addr + 128 + c * kChunkCols, u);
      ptx::tmem_ld_wait();
      if constexpr (kFp8) {
        const float rs = row_ok ? d.row_scale[row] : 0.f;
        // the chunk's 32 column scales of each matrix as eight 16-byte loads (the same addresses in every lane);
        // N is a multiple of 32, so a chunk is inside the matrix or outside as a whole
        const bool in = t.n0 + c * kChunkCols < d.N;
        const float4* g4 = reinterpret_cast<const float4*>(d.col_scale0 + t.w_row0 + c * kChunkCols);
        const float4* u4 = reinterpret_cast<const float4*>(d.col_scale1 + t.w_row0 + c * kChunkCols);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const float4 sg = in ? __ldg(g4 + q) : make_float4(0.f, 0.f, 0.f, 0.f);
          const float4 su = in ? __ldg(u4 + q) : make_float4(0.f, 0.f, 0.f, 0.f);
          o[4 * q + 0] = silu_mul(__uint_as_float(v[4 * q + 0]) * (rs * sg.x), __uint_as_float(u[4 * q + 0]) * (rs * su.x));
          o[4 * q + 1] = silu_mul(__uint_as_float(v[4 * q + 1]) * (rs * sg.y), __uint_as_float(u[4 * q + 1]) * (rs * su.y));
          o[4 * q + 2] = silu_mul(__uint_as_float(v[4 * q + 2]) * (rs * sg.z), __uint_as_float(u[4 * q + 2]) * (rs * su.z));
          o[4 * q + 3] = silu_mul(__uint_as_float(v[4 * q + 3]) * (rs * sg.w), __uint_as_float(u[4 * q + 3]) * (rs * su.w));
        }
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = silu_mul(__uint_as_float(v[i]), __uint_as_float(u[i]));
      }
    } else {
      ptx::tmem_ld_32x32(t_addr + c * kChunkCols, v);
      ptx::tmem_ld_wait();
      if constexpr (kFp8) {
        const float rs = row_ok ? d.row_scale[row] : 0.f;
        // columns 0..127 of the tile come from the first weight box, 128..255 from the second (same matrix)
        const bool in = t.n0 + c * kChunkCols < d.N;
        const float4* s4 = reinterpret_cast<const float4*>(d.col_scale0 + t.w_row0 + c * kChunkCols);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const float4 sc = in ? __ldg(s4 + q) : make_float4(0.f, 0.f, 0.f, 0.f);
          o[4 * q + 0] = __uint_as_float(v[4 * q + 0]) * (rs * sc.x);
          o[4 * q + 1] = __uint_as_float(v[4 * q + 1]) * (rs * sc.y);
          o[4 * q + 2] = __uint_as_float(v[4 * q + 2]) * (rs * sc.z);
          o[4 * q + 3] = __uint_as_float(v[4 * q + 3]) * (rs * sc.w);
        }
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = __uint_as_float(v[i]);
      }
    }
    const int col0 = t.n0 + c * kChunkCols;
    if (bulk) {
      if ((c & 1) == 0) {             // the box is free again once the TMA unit has read the previous one
        if (lane == 0) ptx::bulk_wait_group_read_all();
        __syncwarp();
      }
      const uint32_t row_smem = ss.smem + static_cast<uint32_t>(lane) * 128u;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint32_t j = static_cast<uint32_t>((c & 1) * 4 + q);          // 16-byte piece of the 128-byte row
        const uint32_t dst = row_smem + ((j ^ (static_cast<uint32_t>(lane) & 7u)) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(pack_bf16(o[q * 8 + 0], o[q * 8 + 1])),
                     "r"(pack_bf16(o[q * 8 + 2], o[q * 8 + 3])), "r"(pack_bf16(o[q * 8 + 4], o[q * 8 + 5])),
                     "r"(pack_bf16(o[q * 8 + 6], o[q * 8 + 7]))
                     : "memory");
      }
      if (c & 1) {
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0 && col0 - kChunkCols < d.N) {   // (a box that starts beyond N has nothing to write)
          ptx::tma_store_2d(ss.map, ss.smem, col0 - kChunkCols, row);
          ptx::bulk_commit_group();
        }
      }
    } else if (row_ok) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (col0 + q * 8 < d.N) {     // N is a multiple of 8: a 16-byte vector is inside or outside
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
          float* dbg = p.h_dbg + static_cast<size_t>(row) * d.N + col0;
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            if (col0 + q * 4 < d.N) {
              *reinterpret_cast<float4*>(dbg + q * 4) = make_float4(o[q * 4], o[q * 4 + 1], o[q * 4 + 2], o[q * 4 + 3]);
            }
          }
        }
      }
    }
    if (p.mode == 1) pacer.after_store(p.burst);
  }
}

// Drain an accumulator computed with swapped operands: this thread's TMEM lane is output column n0 + f (and
// n0 + 128 + f for Linear-2's second weight box); accumulator column j is row row0 + j.  Few rows, so plain 2-byte
// stores (a warp writes 64 contiguous bytes per row).  Not paced: these tiles are a few rows long.
template <bool kGated, bool kFp8>
__device__ __forceinline__ void drain_swapped(const Tile& t, const FfnParams& p, uint32_t t_addr, int f) {
  const PhaseDesc& d = p.ph[kGated ? 0 : 1];
  const int col_a = t.n0 + f;
  const int col_b = col_a + 128;
  float sa = 1.f, sb = 1.f;                       // column scales of this lane's weight rows (E4M3 operands)
  if constexpr (kFp8) {
    if (kGated) {
      if (col_a < d.N) { sa = d.col_scale0[t.w_row0 + f]; sb = d.col_scale1[t.w_row0 + f]; }
    } else {
      if (col_a < d.N) sa = d.col_scale0[t.w_row0 + f];
      if (col_b < d.N) sb = d.col_scale0[t.w_row0 + 128 + f];
    }
  }
#pragma unroll 1
  for (int j0 = 0; j0 < t.n_pad; j0 += 16) {
    uint32_t va[16], vb[16];
    ptx::tmem_ld_32x16(t_addr + j0, va);
    ptx::tmem_ld_32x16(t_addr + 128 + j0, vb);
    ptx::tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int r = t.row0 + j0 + i;
      if (r < t.row_end) {
        float a = __uint_as_float(va[i]), b = __uint_as_float(vb[i]);
        if constexpr (kFp8) {
          const float rs = d.row_scale[r];
          a *= rs * sa;
          b *= rs * sb;
        }
        const size_t base = static_cast<size_t>(r) * d.N;
        if constexpr (kGated) {
          if (col_a < d.N) {
            const float hv = silu_mul(a, b);
            d.out[base + col_a] = __float2bfloat16_rn(hv);
            if (p.h_dbg != nullptr) p.h_dbg[base + col_a] = hv;
          }
        } else {
          if (col_a < d.N) d.out[base + col_a] = __float2bfloat16_rn(a);
          if (col_b < d.N) d.out[base + col_b] = __float2bfloat16_rn(b);
        }
      }
    }
  }
}

// The eight MMAs of one K block of a swapped-operand tile: weight box 0 into columns 0.., weight box 1 into columns
// 128.., N = kRows (the tile's rows padded to 16).  kRows is a template parameter because the instruction descriptor
// must be a compile-time constant: with the descriptor in an ordinary register each of these short instructions took
// about 100 clocks to issue, twice what the tensor pipe needs for them (measured with a stand-alone loop: 58 against
// 95 to 190 clocks per instruction).
template <bool kFp8, int kRows>
__device__ __forceinline__ void issue_swapped(uint32_t d_tmem, uint64_t w0_desc, uint64_t w1_desc, uint64_t rows_desc,
                                              uint32_t accumulate_first) {
  constexpr uint32_t idesc = kFp8 ? ptx::idesc_e4m3_f32(BM, kRows) : ptx::idesc_bf16_f32(BM, kRows);
#pragma unroll
  for (int k4 = 0; k4 < BK / UMMA_K; ++k4) {
    const uint64_t adv = static_cast<uint64_t>(2 * k4);
    const uint32_t accum = k4 != 0 ? 1u : accumulate_first;
    if constexpr (kFp8) {
      ptx::tc_mma_e4m3(d_tmem, w0_desc + adv, rows_desc + adv, idesc, accum);
      ptx::tc_mma_e4m3(d_tmem + 128u, w1_desc + adv, rows_desc + adv, idesc, accum);
    } else {
      ptx::tc_mma_bf16(d_tmem, w0_desc + adv, rows_desc + adv, idesc, accum);
      ptx::tc_mma_bf16(d_tmem + 128u, w1_desc + adv, rows_desc + adv, idesc, accum);
    }
  }
}

template <bool kFp8>
__global__ void __launch_bounds__(kThreads, 1)
expert_ffn_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_wg,
                  const __grid_constant__ CUtensorMap tm_wu, const __grid_constant__ CUtensorMap tm_h,
                  const __grid_constant__ CUtensorMap tm_wd, const __grid_constant__ CUtensorMap tm_x16,
                  const __grid_constant__ CUtensorMap tm_h16, const __grid_constant__ CUtensorMap tm_h_out,
                  const __grid_constant__ CUtensorMap tm_y_out, const FfnParams p) {
  // tm_x16, tm_h16: 16-row boxes of A; tm_h_out, tm_y_out: the two outputs in boxes of 32 rows x 64 columns (stores)
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
  unsigned char* stage_base = smem_raw + pad;                 // 1024-byte aligned: required by the swizzle
  const uint32_t stage_u32 = raw + pad;
  const uint32_t store_u32 = stage_u32 + kStages * kStageBytes;
  SharedTail* st = reinterpret_cast<SharedTail*>(stage_base + static_cast<size_t>(kStages) * kStageBytes + kStoreStagingBytes);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid == 0) {
    for (int s = 0; s < kMaxStages; ++s) {
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
    // Wide mode is chosen per launch, by every CTA alike, from the expert row counts.  An expert with several 128-row
    // blocks is then cut into 256-row blocks, each one tile on both accumulators: its two halves
    // share the weight boxes of a stage, a third less to bring into shared memory per flop, which is what holds
    // these tiles back when the weights of many experts stream through L2 at once.
    // The price is one stage of the ring (three stages of 64 KiB), which the one-block tiles of small experts feel
    // (they stream weights and live on the bytes in flight), so wide mode needs enough many-row work to pay for
    // it: at least three 256-row blocks for every four single-block experts.  (Measured in steady state on the
    // DeepSeek-V3-like layer at 1024 to 16384 tokens, where that ratio runs from 0.31 to 3.4: +3 %, -0.7 %, -3.1 %,
    // -5.2 %, -6.3 % with wide mode; the crossover lies near 0.5.)
    // A GEMM split by expert size (every CTA of both launches decides alike from the same counts): the split applies
    // when the layer holds experts of at most 16 rows and larger ones; otherwise the first launch computes everything
    // and the second nothing.  take(rows) says whether this launch computes an expert of that many rows.
    int tiny = 0, larger = 0;
    if (p.expert_class != 0) {
      for (int base = 0; base < p.E; base += 32) {
        const int e = base + lane;
        const int rows = e < p.E ? p.offsets[e + 1] - p.offsets[e] : 0;
        tiny += (rows > 0 && rows <= 16) ? 1 : 0;
        larger += rows > 16 ? 1 : 0;
      }
      tiny = __reduce_add_sync(0xFFFFFFFFu, tiny);
      larger = __reduce_add_sync(0xFFFFFFFFu, larger);
    }
    const bool both_kinds = tiny > 0 && larger > 0;
    const int cls = p.expert_class;
    auto take = [&](int rows) -> bool {
      if (cls == 0) return true;
      if (!both_kinds) return cls == 1;
      return cls == 1 ? rows <= 16 : rows > 16;
    };
    int hot_wide_blocks = 0, cold_blocks = 0, max_rows = 0;
    for (int base = 0; base < p.E; base += 32) {
      const int e = base + lane;
      int rows = e < p.E ? p.offsets[e + 1] - p.offsets[e] : 0;
      if (!take(rows)) rows = 0;
      if (rows > BM * (kHotBlocks - 1)) hot_wide_blocks += (rows + 2 * BM - 1) / (2 * BM);
      else if (rows > 0) cold_blocks += 1;
      max_rows = max(max_rows, rows);
    }
    hot_wide_blocks = __reduce_add_sync(0xFFFFFFFFu, hot_wide_blocks);
    cold_blocks = __reduce_add_sync(0xFFFFFFFFu, cold_blocks);
    max_rows = __reduce_max_sync(0xFFFFFFFFu, max_rows);
    // every tile of the launch is then a swapped-operand tile that loads one 16-row box of A
    if (lane == 0)
      st->small = (p.small_ring != 0 && max_rows <= 16 && p.small_a >= 16 && p.swap_rows >= 16 && p.schedule == 0) ? 1 : 0;
    // (E4M3 operands: the weight-streaming tiles are a larger share of the time there, and on the same layer wide mode
    // costs 2 % at 4096 tokens; they keep the stricter rule of four 256-row blocks per single-block expert.)
    const bool enough_hot = p.fp8 ? 4 * cold_blocks <= hot_wide_blocks : 3 * cold_blocks <= 4 * hot_wide_blocks;
    const bool wide_mode = p.wide_allowed != 0 && hot_wide_blocks > 0 && (enough_hot || p.wide_allowed == 2);
    if (lane == 0) st->wide = wide_mode ? 1 : 0;
    // exclusive prefixes of the row-block counts over experts (hot and cold apart), 32 experts per step
    int32_t run_hot = 0, run_cold = 0;
    if (lane == 0) st->offs[0] = p.offsets[0];
    for (int base = 0; base < p.E; base += 32) {
      const int e = base + lane;
      int32_t v = 0, rows = 0;
      if (e < p.E) {
        const int32_t lo = p.offsets[e], hi = p.offsets[e + 1];
        st->offs[e + 1] = hi;
        rows = hi - lo;
        if (!take(rows)) rows = 0;          // (an expert of another launch: no blocks here)
        v = (rows + BM - 1) / BM;
      }
      int32_t hot = v >= kHotBlocks ? (wide_mode ? (rows + 2 * BM - 1) / (2 * BM) : v) : 0;
      int32_t cold = v >= kHotBlocks ? 0 : v;
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
      ptx::prefetch_tensormap(&tm_x);
      ptx::prefetch_tensormap(&tm_wg);
      ptx::prefetch_tensormap(&tm_wu);
      ptx::prefetch_tensormap(&tm_h);
      ptx::prefetch_tensormap(&tm_wd);
      ptx::prefetch_tensormap(&tm_x16);
      ptx::prefetch_tensormap(&tm_h16);
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
  // ring geometry of this launch: [A][B0][B1] x 4 stages, or in wide mode [A][A'][B0][B1] x 3 stages
  const bool wide_mode = st->wide != 0;
  const bool small_mode = st->small != 0;                          // (never together: wide mode needs many-row experts)
  const int n_stages = wide_mode ? kWideStages : small_mode ? kSmallStages : kStages;
  const uint32_t stage_bytes = wide_mode ? kWideStageBytes : small_mode ? kSmallStageBytes : kStageBytes;
  // offset of the first weight box inside a stage
  const uint32_t b_off = wide_mode ? 2 * kABytes : small_mode ? kSmallABytes : kABytes;
  const int total_blocks = st->hot_prefix[p.E] + st->cold_prefix[p.E];
  const int tiles1 = p.phase_lo == 0 ? total_blocks * p.ph[0].n_blocks : 0;   // Linear-1 tiles of this launch
  const int tiles2 = p.phase_hi == 2 ? total_blocks * p.ph[1].n_blocks : 0;   // Linear-2 tiles of this launch
  const bool chained = tiles1 > 0 && tiles2 > 0;   // Linear-2 tiles depend on Linear-1 tiles of the same launch
  volatile int* abort_flag = &st->abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------------ tile scheduler + TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int slot = 0;
      uint32_t ring_phase = 0;
      bool ok = true;
      long long w_empty = 0;
      InterleaveCursor cursor{static_cast<int>(blockIdx.x), static_cast<int>(blockIdx.x), static_cast<int>(gridDim.x)};
      int n_drawn = 0;
      const long long t_begin = clock64();
      // Schedule 0 draws positions from a global counter.  The round trip of that atomic would sit between two tiles
      // with nothing new in flight, so the position of the following tile is requested a few K blocks before the
      // current tile's loads end (kDrawAhead) and is only looked at when that tile begins.
      constexpr int kDrawAhead = 8;
      const uint64_t pol_first = ptx::l2_policy_evict_first(), pol_last = ptx::l2_policy_evict_last(),
                     pol_normal = ptx::l2_policy_evict_normal();
      int pos_next = p.schedule == 0 ? atomicAdd(&p.sched[0], 1) : 0;
      while (ok) {
        if (!ptx::mbar_wait(ptx::smem_u32(&st->ring_empty[slot]), ring_phase ^ 1u, abort_flag)) {
          report_timeout(p, 5);
          break;
        }
        // ---- next tile of this CTA
        int code = -1;
        bool drawn_next = false;
        if (p.schedule == 1) {
          code = cursor.draw(tiles1, tiles2, p.ph[0].n_blocks, p.ph[1].n_blocks, p.lead_D);
        } else {
          const int pos = pos_next;
          if (pos < tiles1) code = pos;
          else if (pos < tiles1 + tiles2) code = (1 << kPhaseShift) | (pos - tiles1);
        }
        if (p.order_log && n_drawn < kMoeOrderLogCap) p.order_log[blockIdx.x * kMoeOrderLogCap + n_drawn++] = code;
        Tile t{};
        if (code >= 0) t = decode_tile(code, st, p);
        st->ring_tile[slot] = code;
        st->ring_kind[slot] = t.wide ? kWideFlag : t.n_pad;
        ptx::mbar_arrive(ptx::smem_u32(&st->ring_full[slot]));
        if (++slot == kRing) { slot = 0; ring_phase ^= 1u; }
        if (code < 0) break;
        const PhaseDesc& d = p.ph[t.phase];
        // L2 priorities: the weights of an expert with a single row block are read by this tile alone (bit 0: they go
        // first); the rows of A are read once per column block (bit 1: they stay, Linear-2 only: bit 2)
        const uint64_t pol_w = ((p.cache_hints & 1) && t.single) ? pol_first
                               : ((p.cache_hints & 32) && !t.single) ? pol_last : pol_normal;
        const uint64_t pol_a = ((p.cache_hints & 2) && (t.phase == 1 || !(p.cache_hints & 4))) ? pol_last : pol_normal;
        const CUtensorMap* ma = t.phase == 0 ? &tm_x : &tm_h;
        const CUtensorMap* ma16 = t.phase == 0 ? &tm_x16 : &tm_h16;
        const bool small_a = p.small_a != 0 && t.n_pad != 0 && t.n_pad <= p.small_a;
        const CUtensorMap* mb0 = t.phase == 0 ? &tm_wg : &tm_wd;
        const CUtensorMap* mb1 = t.phase == 0 ? &tm_wu : &tm_wd;
        if (chained && t.phase == 1) {
          // every Linear-1 tile of this row (n_blocks tiles x 4 epilogue warps) must have published its h rows
          if (!wait_counter(&p.ready[t.block], 4 * p.ph[0].n_blocks, abort_flag, p.wait_budget)) {
            report_timeout(p, 8);
            break;
          }
          ptx::fence_proxy_async_all();   // h was written through the generic proxy, TMA reads through the async one
        }
        for (int kb = 0; kb < d.k_blocks; ++kb) {
          if (p.schedule == 0 && !drawn_next && kb + kDrawAhead >= d.k_blocks) {
            pos_next = atomicAdd(&p.sched[0], 1);
            drawn_next = true;
          }
          if (!ptx::mbar_wait_timed(ptx::smem_u32(&st->empty[stage]), phase ^ 1u, abort_flag, &w_empty)) {
            report_timeout(p, 1);
            ok = false;
            break;
          }
          const uint32_t full = ptx::smem_u32(&st->full[stage]);
          const uint32_t sa = stage_u32 + stage * stage_bytes;
          if (small_a) {
            // a swapped-operand tile reads only its own rows (padded to 16): bring those, in 16-row boxes, instead of
            // a 128-row box of mostly other experts' rows
            ptx::mbar_expect_tx(full, t.n_pad * 128 + 2 * kBHalfBytes);
            for (int r16 = 0; r16 < t.n_pad; r16 += 16)
              ptx::tma_load_2d_hint(sa + r16 * 128, ma16, full, kb * p.k_elems, t.row0 + r16, pol_a);
          } else {
            ptx::mbar_expect_tx(full, t.wide ? kWideStageBytes : kStageBytes);
            ptx::tma_load_2d_hint(sa, ma, full, kb * p.k_elems, t.row0, pol_a);
          }
          if (t.wide) ptx::tma_load_2d_hint(sa + kABytes, ma, full, kb * p.k_elems, t.row0 + BM, pol_a);
          ptx::tma_load_2d_hint(sa + b_off, mb0, full, kb * p.k_elems, t.w_row0, pol_w);
          ptx::tma_load_2d_hint(sa + b_off + kBHalfBytes, mb1, full, kb * p.k_elems, t.w_row0 + d.b1_row_shift, pol_w);
          if (++stage == n_stages) { stage = 0; phase ^= 1u; }
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
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;                    // accumulator of the next one-accumulator tile
      uint32_t acc_uses[2] = {0, 0};  // tiles that have used each accumulator so far (the barriers' phases)
      uint32_t progress = 0;
      int slot = 0;
      uint32_t ring_phase = 0;
      bool ok = true;
      long long w_full = 0, w_tmem = 0, t_swapped = 0, w_swapped = 0, t_full_tiles = 0;
      unsigned long long n_tiles = 0, n_swapped = 0;

      // One K block: wait for the stage, issue its MMAs, release the stage.  `issue` gets the stage's address.
      auto k_block = [&](auto&& issue) -> bool {
        if (!ptx::mbar_wait_timed(ptx::smem_u32(&st->full[stage]), phase, abort_flag, &w_full)) {
          report_timeout(p, 3);
          return false;
        }
        ptx::tc_fence_after_sync();
        issue(stage_u32 + stage * stage_bytes);
        ptx::tc_commit(ptx::smem_u32(&st->empty[stage]));   // stage is free once these MMAs have read it
        st->mma_progress = ++progress;
        if (++stage == n_stages) { stage = 0; phase ^= 1u; }
        return true;
      };
      // The K loop of one tile, one instantiation per tile kind: a run-time branch between the MMAs of a K block costs
      // 100 to 200 clocks per block (measured with a stand-alone issue loop: a never-taken branch around four dependent
      // N = 16 instructions takes them from 65 to 115 clocks each), which is nothing next to four 128-clock instructions
      // but doubles the time of a swapped-operand tile.  kKind: 0 = 128 rows on accumulator `acc`; -1 = 256 rows on
      // both accumulators; otherwise the padded row count of a swapped-operand tile.
      auto run_tile = [&](auto kind_tag, int k_blocks, uint32_t d_tmem) -> bool {
        constexpr int kKind = decltype(kind_tag)::value;
        constexpr uint32_t idesc = kFp8 ? ptx::idesc_e4m3_f32(BM, BN_ACC) : ptx::idesc_bf16_f32(BM, BN_ACC);
        auto mma = [](uint32_t d, uint64_t a, uint64_t b, uint32_t accumulate) {
          if constexpr (kFp8) ptx::tc_mma_e4m3(d, a, b, idesc, accumulate);
          else ptx::tc_mma_bf16(d, a, b, idesc, accumulate);
        };
        if constexpr (kKind == 0) {
          for (int kb = 0; kb < k_blocks; ++kb) {
            const uint32_t later = kb != 0 ? 1u : 0u;
            if (!k_block([&](uint32_t sa) {
                  const uint64_t a_desc = ptx::smem_desc_sw128(sa), b_desc = ptx::smem_desc_sw128(sa + b_off);
                  // +32 bytes along K inside the swizzle row = +2 in the descriptor's 16-byte address units
                  // (16 bf16 or 32 E4M3 elements per instruction: 32 bytes either way)
#pragma unroll
                  for (int k4 = 0; k4 < BK / UMMA_K; ++k4) mma(d_tmem, a_desc + 2 * k4, b_desc + 2 * k4, k4 != 0 ? 1u : later);
                }))
              return false;
          }
        } else if constexpr (kKind == -1) {
          // rows 0..127 into accumulator 0, rows 128..255 (the second A box) into accumulator 1, same weight boxes.
          // The first K block is peeled: accumulator 1 may still be draining (the previous tile's epilogue) while
          // the first MMAs into accumulator 0 run.
          auto half = [&](uint32_t sa, uint32_t a_off, uint32_t d, uint32_t later) {
            const uint64_t a_desc = ptx::smem_desc_sw128(sa + a_off), b_desc = ptx::smem_desc_sw128(sa + b_off);
#pragma unroll
            for (int k4 = 0; k4 < BK / UMMA_K; ++k4) mma(d, a_desc + 2 * k4, b_desc + 2 * k4, k4 != 0 ? 1u : later);
          };
          bool acc1_ok = true;
          if (!k_block([&](uint32_t sa) {
                half(sa, 0, tmem_base, 0u);
                st->mma_idle = 1;   // (a paced epilogue must not hold its stores for an MMA warp that waits for it)
                acc1_ok = ptx::mbar_wait_timed(ptx::smem_u32(&st->tmem_empty[1]), (acc_uses[1] & 1u) ^ 1u, abort_flag, &w_tmem);
                st->mma_idle = 0;
                ptx::tc_fence_after_sync();
                if (acc1_ok) half(sa, kABytes, tmem_base + BN_ACC, 0u);
              }))
            return false;
          if (!acc1_ok) {
            report_timeout(p, 2);
            return false;
          }
          for (int kb = 1; kb < k_blocks; ++kb) {
            if (!k_block([&](uint32_t sa) {
                  half(sa, 0, tmem_base, 1u);
                  half(sa, kABytes, tmem_base + BN_ACC, 1u);
                }))
              return false;
          }
        } else {
          // swapped operands: each 128-row weight box is the M side, the expert's rows (the A box) the N side; the
          // first weight box accumulates into columns 0.., the second into columns 128..
          auto issue = [&](uint32_t sa, uint32_t later) {
            issue_swapped<kFp8, kKind>(d_tmem, ptx::smem_desc_sw128(sa + b_off),
                                       ptx::smem_desc_sw128(sa + b_off + kBHalfBytes), ptx::smem_desc_sw128(sa), later);
          };
          // Two K blocks per wait: the sixteen short MMAs of two stages are issued without a branch between them (the
          // bubble a branch opens in the issue stream costs as much as three of these instructions; with one wait per
          // two blocks the stand-alone loop goes from 723 to 588 clocks per block).
          int kb = 0;
          for (; n_stages >= kStages && kb + 2 <= k_blocks; kb += 2) {   // (the three-stage ring cannot spare two stages)
            const int s0 = stage, s1 = stage + 1 == n_stages ? 0 : stage + 1;
            const uint32_t ph1 = s1 == 0 ? phase ^ 1u : phase;
            const uint32_t bar0 = ptx::smem_u32(&st->full[s0]), bar1 = ptx::smem_u32(&st->full[s1]);
            if (!(ptx::mbar_try_wait(bar0, phase) & ptx::mbar_try_wait(bar1, ph1))) {
              if (!ptx::mbar_wait_timed(bar0, phase, abort_flag, &w_full) || !ptx::mbar_wait_timed(bar1, ph1, abort_flag, &w_full)) {
                report_timeout(p, 3);
                return false;
              }
            }
            ptx::tc_fence_after_sync();
            issue(stage_u32 + s0 * stage_bytes, kb != 0 ? 1u : 0u);
            ptx::tc_commit(ptx::smem_u32(&st->empty[s0]));
            issue(stage_u32 + s1 * stage_bytes, 1u);
            ptx::tc_commit(ptx::smem_u32(&st->empty[s1]));
            progress += 2;
            st->mma_progress = progress;
            stage = s1 + 1 == n_stages ? 0 : s1 + 1;
            phase = stage == 0 ? ph1 ^ 1u : ph1;
          }
          for (; kb < k_blocks; ++kb) {
            if (!k_block([&](uint32_t sa) { issue(sa, kb != 0 ? 1u : 0u); })) return false;
          }
        }
        return true;
      };

      while (ok) {
        st->mma_idle = 1;
        if (!ptx::mbar_wait(ptx::smem_u32(&st->ring_full[slot]), ring_phase, abort_flag)) {
          report_timeout(p, 6);
          break;
        }
        const int code = st->ring_tile[slot];
        const int kind = st->ring_kind[slot];
        ptx::mbar_arrive(ptx::smem_u32(&st->ring_empty[slot]));
        if (++slot == kRing) { slot = 0; ring_phase ^= 1u; }
        if (code < 0) break;
        const bool wide = kind == kWideFlag;
        const int n_pad = wide ? 0 : kind;
        const int k_blocks = p.ph[code >> kPhaseShift].k_blocks;
        // a wide tile takes both accumulators, first rows on accumulator 0; the tile after it starts on 0 again,
        // the one the epilogue hands back first
        if (wide) acc = 0;
        if (!ptx::mbar_wait_timed(ptx::smem_u32(&st->tmem_empty[acc]), (acc_uses[acc] & 1u) ^ 1u, abort_flag, &w_tmem)) {
          report_timeout(p, 2);
          break;
        }
        st->mma_idle = 0;
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN_ACC);
        const long long t_tile = clock64(), w_full_before = w_full;
        if (wide) {
          ok = run_tile(std::integral_constant<int, -1>{}, k_blocks, d_tmem);
        } else {
          switch (n_pad >> 4) {
            case 0: ok = run_tile(std::integral_constant<int, 0>{}, k_blocks, d_tmem); break;
            case 1: ok = run_tile(std::integral_constant<int, 16>{}, k_blocks, d_tmem); break;
            case 2: ok = run_tile(std::integral_constant<int, 32>{}, k_blocks, d_tmem); break;
            case 3: ok = run_tile(std::integral_constant<int, 48>{}, k_blocks, d_tmem); break;
            case 4: ok = run_tile(std::integral_constant<int, 64>{}, k_blocks, d_tmem); break;
            case 5: ok = run_tile(std::integral_constant<int, 80>{}, k_blocks, d_tmem); break;
            case 6: ok = run_tile(std::integral_constant<int, 96>{}, k_blocks, d_tmem); break;
            case 7: ok = run_tile(std::integral_constant<int, 112>{}, k_blocks, d_tmem); break;
            default: ok = run_tile(std::integral_constant<int, 128>{}, k_blocks, d_tmem); break;
          }
        }
        if (!ok) break;
        if (wide) {
          ptx::tc_commit(ptx::smem_u32(&st->tmem_full[0]));    // both accumulators complete
          ptx::tc_commit(ptx::smem_u32(&st->tmem_full[1]));
          ++acc_uses[0];
          ++acc_uses[1];
          acc = 0;
        } else {
          ptx::tc_commit(ptx::smem_u32(&st->tmem_full[acc]));  // accumulator complete
          ++acc_uses[acc];
          acc ^= 1;
        }
        ++n_tiles;
        if (n_pad != 0) {
          ++n_swapped;
          t_swapped += clock64() - t_tile;
          w_swapped += w_full - w_full_before;
        } else {
          t_full_tiles += clock64() - t_tile;
        }
      }
      st->mma_idle = 1;
      if (p.trace) {
        p.trace[blockIdx.x * kMoeTraceFields + 2] = static_cast<unsigned long long>(w_full);
        p.trace[blockIdx.x * kMoeTraceFields + 3] = static_cast<unsigned long long>(w_tmem);
        p.trace[blockIdx.x * kMoeTraceFields + 6] = n_tiles;
        p.trace[blockIdx.x * kMoeTraceFields + 8] = n_swapped;
        p.trace[blockIdx.x * kMoeTraceFields + 9] = static_cast<unsigned long long>(t_swapped);
        p.trace[blockIdx.x * kMoeTraceFields + 10] = static_cast<unsigned long long>(w_swapped);
        p.trace[blockIdx.x * kMoeTraceFields + 11] = static_cast<unsigned long long>(t_full_tiles);
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue (4 warps = 128 rows)
    const int quarter = warp & 3;                 // TMEM lane quarter this warp may read
    const int r_in_tile = quarter * 32 + lane;
    int acc = 0;                    // accumulator of the next one-accumulator tile (the MMA warp counts the same way)
    uint32_t acc_uses[2] = {0, 0};
    int slot = 0;
    uint32_t ring_phase = 0;
    long long w_acc = 0, busy = 0;
    Pacer pacer{ptx::smem_u32(const_cast<uint32_t*>(&st->mma_progress)), ptx::smem_u32(const_cast<int*>(&st->mma_idle)), 0, 0u, 0};
    // Bulk stores of whole row blocks unless Linear-2 tiles of this launch wait for h (their release is a plain
    // fence after plain stores) or the knob switches them off
    // (a launch on the small ring has no 128-row tiles, and its ring reaches into the boxes)
    const uint32_t my_box = (chained || !p.bulk_stores || small_mode) ? 0u
                                                                      : store_u32 + static_cast<uint32_t>(quarter) * kStoreBoxBytes;
    const StoreStage ss_h{my_box, &tm_h_out}, ss_y{my_box, &tm_y_out};
    bool ok = true;
    while (ok) {
      if (!ptx::mbar_wait(ptx::smem_u32(&st->ring_full[slot]), ring_phase, abort_flag)) {
        if (lane == 0) report_timeout(p, 7);
        break;
      }
      const int code = st->ring_tile[slot];
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&st->ring_empty[slot]));
      if (++slot == kRing) { slot = 0; ring_phase ^= 1u; }
      if (code < 0) break;
      Tile t = decode_tile(code, st, p);
      // a wide tile is drained as two 128-row parts, accumulator 0 then accumulator 1
      const int parts = t.wide ? 2 : 1;
      if (t.wide) acc = 0;
      for (int part = 0; part < parts; ++part) {
        if (!ptx::mbar_wait_timed(ptx::smem_u32(&st->tmem_full[acc]), acc_uses[acc] & 1u, abort_flag, &w_acc)) {
          if (lane == 0) report_timeout(p, 4);
          ok = false;
          break;
        }
        ptx::tc_fence_after_sync();
        const long long t_store = clock64();
        const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                                static_cast<uint32_t>(acc * BN_ACC);
        if (t.n_pad != 0) {
          if (t.phase == 0) drain_swapped<true, kFp8>(t, p, t_addr, r_in_tile);
          else drain_swapped<false, kFp8>(t, p, t_addr, r_in_tile);
        } else if (t.phase == 0) {
          drain_accumulator<true, kFp8>(t, p, t_addr, t.row0 + r_in_tile, pacer, abort_flag, ss_h);
        } else {
          drain_accumulator<false, kFp8>(t, p, t_addr, t.row0 + r_in_tile, pacer, abort_flag, ss_y);
        }
        ptx::tc_fence_before_sync();
        if (chained && t.phase == 0) {
          // publish this warp's 32 rows x 128 columns of h to the Linear-2 tiles of the block
          __threadfence();
          ptx::fence_proxy_async_all();
        }
        __syncwarp();
        if (lane == 0) {
          ptx::mbar_arrive(ptx::smem_u32(&st->tmem_empty[acc]));
          if (chained && t.phase == 0 && !p.withhold_ready) atomicAdd(&p.ready[t.block], 1);
        }
        busy += clock64() - t_store;
        ++acc_uses[acc];
        acc ^= 1;
        t.row0 += BM;               // the second part of a wide tile
      }
      if (t.wide) acc = 0;
    }
    if (lane == 0) ptx::bulk_wait_group_all();      // this warp's bulk stores have landed
    if (p.trace && warp == 2 && lane == 0) {
      p.trace[blockIdx.x * kMoeTraceFields + 4] = static_cast<unsigned long long>(w_acc);
      p.trace[blockIdx.x * kMoeTraceFields + 5] = static_cast<unsigned long long>(busy);
      p.trace[blockIdx.x * kMoeTraceFields + 7] = static_cast<unsigned long long>(pacer.held);
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
  // Every CTA has drawn its last tile by now.  The last CTA to leave re-arms the scheduler and, after a
  // chained launch, the ready counters for the next launch.
  __shared__ int s_last;
  if (tid == 0) s_last = atomicAdd(&p.sched[1], 1) == static_cast<int>(gridDim.x) - 1;
  __syncthreads();
  if (s_last) {
    if (chained)
      for (int i = tid; i < total_blocks; i += kThreads) p.ready[i] = 0;
    if (tid == 0) {
      p.sched[0] = 0;
      p.sched[1] = 0;
    }
    __threadfence();
  }
}


// ------------------------------------------------------------------------------------------------------------
// CTA-pair variant (on request: debug_flags bit 3) for layers whose experts hold many rows: a cluster of two CTAs computes a 256-row x 256-column
// tile with tcgen05.mma.cta_group::2.  Each CTA loads its own 128 rows of A and one 128-row weight box (for
// Linear-1 the leader holds the gate box, its peer the up box), so a stage is 32 KiB per CTA instead of 48 and
// six stages fit; the leader's MMA thread issues for both, reading the peer's operands from the peer's shared
// memory, and each CTA's epilogue drains its own 128 accumulator rows.  Static schedule: pair c takes tiles
// c, c + pairs, ... in the order expert -> N block -> 256-row block (fastest); one GEMM per launch.
// ------------------------------------------------------------------------------------------------------------
constexpr int kPairStages = 6;
constexpr int kPairStageBytes = kABytes + kBHalfBytes;   // 32 KiB per CTA

struct PairTail {
  uint64_t full[kPairStages];       // used in the leader: its own expect_tx arrival + the bytes of both CTAs
  uint64_t empty[kPairStages];      // one per CTA, both arrived on by the leader's multicast commit
  uint64_t tmem_full[2];            // one per CTA, multicast commit
  uint64_t tmem_empty[2];           // used in the leader: 4 epilogue warps of each CTA
  uint32_t tmem_base;
  volatile int abort_flag;
  volatile uint32_t mma_progress;
  volatile int mma_idle;
  int32_t pair_prefix[kMaxExperts + 1];   // exclusive prefix of 256-row blocks per expert
  int32_t offs[kMaxExperts + 1];          // the expert row offsets, copied once
};
constexpr size_t kPairSmemBytes = 1024 + static_cast<size_t>(kPairStages) * kPairStageBytes + kStoreStagingBytes +
                                  sizeof(PairTail);   // ring, the epilogue warps' store boxes, tail

__device__ __forceinline__ Tile decode_pair_tile(int tile, int phase, uint32_t rank, const PairTail* st,
                                                 const FfnParams& p) {
  const PhaseDesc& d = p.ph[phase];
  const int e = find_expert([&](int i) { return st->pair_prefix[i]; }, tile / d.n_blocks, p.E);
  const int pb = st->pair_prefix[e + 1] - st->pair_prefix[e];
  const int local = tile - d.n_blocks * st->pair_prefix[e];
  const int n_blk = local / pb;
  const int pair_row = local - n_blk * pb;
  Tile t;
  t.phase = phase;
  t.row0 = st->offs[e] + pair_row * 2 * BM + static_cast<int>(rank) * BM;   // this CTA's 128 rows
  t.row_end = st->offs[e + 1];
  t.n0 = n_blk * d.out_cols_per_tile;
  t.w_row0 = e * d.N + t.n0;
  t.block = 0;
  t.n_pad = 0;
  t.wide = 0;
  t.single = 0;
  return t;
}

template <bool kFp8>
__global__ void __launch_bounds__(kThreads, 1)
expert_ffn_pair_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b0,
                       const __grid_constant__ CUtensorMap tm_b1, const __grid_constant__ CUtensorMap tm_out,
                       const FfnParams p) {   // tm_out: this GEMM's output in boxes of 32 rows x 64 columns (stores)
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
  unsigned char* stage_base = smem_raw + pad;
  const uint32_t stage_u32 = raw + pad;
  const uint32_t store_u32 = stage_u32 + kPairStages * kPairStageBytes;
  PairTail* st = reinterpret_cast<PairTail*>(stage_base + static_cast<size_t>(kPairStages) * kPairStageBytes + kStoreStagingBytes);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t rank = ptx::cluster_ctarank();            // 0 = leader (issues the MMAs), 1 = peer
  const int pair = blockIdx.x >> 1, pairs = gridDim.x >> 1;
  const int phase = p.phase_lo;
  const PhaseDesc& d = p.ph[phase];

  if (tid == 0) {
    for (int s = 0; s < kPairStages; ++s) {
      ptx::mbar_init(ptx::smem_u32(&st->full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&st->empty[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(ptx::smem_u32(&st->tmem_full[a]), 1);
      ptx::mbar_init(ptx::smem_u32(&st->tmem_empty[a]), 8);   // four epilogue warps in each CTA of the pair
    }
    st->abort_flag = 0;
    st->mma_progress = 0;
    st->mma_idle = 0;
    st->pair_prefix[0] = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async_smem();
  }
  if (warp == 0) {
    int32_t run = 0;
    for (int base = 0; base < p.E; base += 32) {
      const int e = base + lane;
      int32_t v = 0;
      if (e < p.E) {
        const int32_t lo = p.offsets[e], hi = p.offsets[e + 1];
        st->offs[e + 1] = hi;
        if (e == 0) st->offs[0] = lo;
        v = (hi - lo + 2 * BM - 1) / (2 * BM);
      }
      int32_t incl = v;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl += o;
      }
      if (e < p.E) st->pair_prefix[e + 1] = run + incl;
      run += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
    if (lane == 0) {
      ptx::prefetch_tensormap(&tm_a);
      ptx::prefetch_tensormap(&tm_b0);
      ptx::prefetch_tensormap(&tm_b1);
    }
  }
  if (warp == 1) {
    ptx::tmem_alloc_pair(ptx::smem_u32(&st->tmem_base), kTmemCols);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::cluster_sync();            // both CTAs' barriers exist before anything signals across the pair
  ptx::tc_fence_after_sync();

  const uint32_t tmem_base = st->tmem_base;
  const int total_tiles = st->pair_prefix[p.E] * d.n_blocks;
  volatile int* abort_flag = &st->abort_flag;
  const CUtensorMap* mb = (rank == 0) ? &tm_b0 : &tm_b1;      // this CTA's half of the 256 weight rows
  const int b_shift = (rank == 0) ? 0 : d.b1_row_shift;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t ph = 0;
      bool ok = true;
      long long w_empty = 0;
      const long long t_begin = clock64();
      // L2 priorities (bits of cache_hints): 8 = the rows of A stay (they are read once per column block), 64 = the
      // weight boxes stay (every row block of the expert reads them), 16 = the weight boxes go first
      const uint64_t pol_a = ((p.cache_hints & 8) && (phase == 1 || !(p.cache_hints & 4))) ? ptx::l2_policy_evict_last()
                                                                                          : ptx::l2_policy_evict_normal();
      const uint64_t pol_w = (p.cache_hints & 16) ? ptx::l2_policy_evict_first()
                             : (p.cache_hints & 64) ? ptx::l2_policy_evict_last() : ptx::l2_policy_evict_normal();
      for (int tile = pair; ok && tile < total_tiles; tile += pairs) {
        const Tile t = decode_pair_tile(tile, phase, rank, st, p);
        for (int kb = 0; kb < d.k_blocks; ++kb) {
          if (!ptx::mbar_wait_timed(ptx::smem_u32(&st->empty[stage]), ph ^ 1u, abort_flag, &w_empty)) {
            report_timeout(p, 1);
            ok = false;
            break;
          }
          const uint32_t full_local = ptx::smem_u32(&st->full[stage]);
          const uint32_t full_leader = ptx::map_to_cta(full_local, 0);
          const uint32_t sa = stage_u32 + stage * kPairStageBytes;
          if (rank == 0) ptx::mbar_expect_tx(full_local, 2 * kPairStageBytes);   // the bytes of both CTAs
          ptx::tma_load_2d_pair_hint(sa, &tm_a, full_leader, kb * p.k_elems, t.row0, pol_a);
          ptx::tma_load_2d_pair_hint(sa + kABytes, mb, full_leader, kb * p.k_elems, t.w_row0 + b_shift, pol_w);
          if (++stage == kPairStages) { stage = 0; ph ^= 1u; }
        }
      }
      if (p.trace) {
        p.trace[blockIdx.x * kMoeTraceFields + 0] = static_cast<unsigned long long>(clock64() - t_begin);
        p.trace[blockIdx.x * kMoeTraceFields + 1] = static_cast<unsigned long long>(w_empty);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = kFp8 ? ptx::idesc_e4m3_f32(2 * BM, BN_ACC) : ptx::idesc_bf16_f32(2 * BM, BN_ACC);
      int stage = 0;
      uint32_t ph = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      uint32_t progress = 0;
      bool ok = true;
      long long w_full = 0, w_tmem = 0;
      unsigned long long n_tiles = 0;
      for (int tile = pair; ok && tile < total_tiles; tile += pairs) {
        st->mma_idle = 1;
        if (!ptx::mbar_wait_timed(ptx::smem_u32(&st->tmem_empty[acc]), acc_phase ^ 1u, abort_flag, &w_tmem)) {
          report_timeout(p, 2);
          break;
        }
        st->mma_idle = 0;
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN_ACC);
        for (int kb = 0; kb < d.k_blocks; ++kb) {
          if (!ptx::mbar_wait_timed(ptx::smem_u32(&st->full[stage]), ph, abort_flag, &w_full)) {
            report_timeout(p, 3);
            ok = false;
            break;
          }
          ptx::tc_fence_after_sync();
          const uint32_t sa = stage_u32 + stage * kPairStageBytes;
          const uint64_t a_desc = ptx::smem_desc_sw128(sa);
          const uint64_t b_desc = ptx::smem_desc_sw128(sa + kABytes);
#pragma unroll
          for (int k4 = 0; k4 < BK / UMMA_K; ++k4) {
            const uint64_t adv = static_cast<uint64_t>(2 * k4);
            if constexpr (kFp8) ptx::tc_mma_e4m3_pair(d_tmem, a_desc + adv, b_desc + adv, idesc, (kb | k4) != 0 ? 1u : 0u);
            else ptx::tc_mma_bf16_pair(d_tmem, a_desc + adv, b_desc + adv, idesc, (kb | k4) != 0 ? 1u : 0u);
          }
          ptx::tc_commit_pair(ptx::smem_u32(&st->empty[stage]), 3);    // frees the stage in both CTAs
          st->mma_progress = ++progress;
          if (++stage == kPairStages) { stage = 0; ph ^= 1u; }
        }
        if (!ok) break;
        ptx::tc_commit_pair(ptx::smem_u32(&st->tmem_full[acc]), 3);    // accumulator complete, both CTAs
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
    // ------------------------------------------------------------------ epilogue (both CTAs, own 128 rows)
    const int quarter = warp & 3;
    const int r_in_tile = quarter * 32 + lane;
    int acc = 0;
    uint32_t acc_phase = 0;
    long long w_acc = 0, busy = 0;
    // the MMA warp whose progress paces the stores is the leader's: both CTAs read its words
    Pacer pacer{ptx::map_to_cta(ptx::smem_u32(const_cast<uint32_t*>(&st->mma_progress)), 0),
                ptx::map_to_cta(ptx::smem_u32(const_cast<int*>(&st->mma_idle)), 0), 0, 0u, 0};
    const uint32_t empty_leader0 = ptx::map_to_cta(ptx::smem_u32(&st->tmem_empty[0]), 0);
    const uint32_t empty_leader1 = ptx::map_to_cta(ptx::smem_u32(&st->tmem_empty[1]), 0);
    const StoreStage ss{p.bulk_stores ? store_u32 + static_cast<uint32_t>(quarter) * kStoreBoxBytes : 0u, &tm_out};
    for (int tile = pair; tile < total_tiles; tile += pairs) {
      const Tile t = decode_pair_tile(tile, phase, rank, st, p);
      if (!ptx::mbar_wait_timed(ptx::smem_u32(&st->tmem_full[acc]), acc_phase, abort_flag, &w_acc)) {
        if (lane == 0) report_timeout(p, 4);
        break;
      }
      ptx::tc_fence_after_sync();
      const long long t_store = clock64();
      const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                              static_cast<uint32_t>(acc * BN_ACC);
      if (phase == 0)
        drain_accumulator<true, kFp8>(t, p, t_addr, t.row0 + r_in_tile, pacer, abort_flag, ss);
      else
        drain_accumulator<false, kFp8>(t, p, t_addr, t.row0 + r_in_tile, pacer, abort_flag, ss);
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive_cluster(acc ? empty_leader1 : empty_leader0);
      busy += clock64() - t_store;
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
    if (lane == 0) ptx::bulk_wait_group_all();      // this warp's bulk stores have landed
    if (p.trace && warp == 2 && lane == 0) {
      p.trace[blockIdx.x * kMoeTraceFields + 4] = static_cast<unsigned long long>(w_acc);
      p.trace[blockIdx.x * kMoeTraceFields + 5] = static_cast<unsigned long long>(busy);
      p.trace[blockIdx.x * kMoeTraceFields + 7] = static_cast<unsigned long long>(pacer.held);
    }
  }

  __syncthreads();
  if (st->abort_flag) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    __syncthreads();
  }
  ptx::cluster_sync();            // the peer's shared memory and barriers stay alive until both CTAs are done
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

// Calibration probe: one CTA issues `iters` tcgen05.mma of shape M x N x 16 back to back on resident
// shared-memory operands and reports the SM clocks from the first issue to the completion of the last.
template <int kKind>
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
    const uint64_t a = ptx::smem_desc_sw128(base), b = ptx::smem_desc_sw128(base + kABytes);
    // block-scaled kind: scale columns behind the accumulator, filled once from the (constant) operand bytes
    const uint32_t sfa = tb + 256, sfb = tb + 260;
    if constexpr (kKind >= 2) {
      ptx::tc_cp_32x128b_warpx4(sfa, base);
      ptx::tc_cp_32x128b_warpx4(sfb, base + 512);
      ptx::tc_cp_32x128b_warpx4(sfb + 4, base + 1024);
    }
    // descriptors out of the loop: the loop must cost less than the instruction it times
    uint32_t idesc[4];
#pragma unroll
    for (int k4 = 0; k4 < 4; ++k4)
      idesc[k4] = kKind == 0 ? ptx::idesc_bf16_f32(M, N) : kKind == 1 ? ptx::idesc_e4m3_f32(M, N)
                                                                      : ptx::idesc_mx_e4m3(M, N, k4, k4);
    const long long t0 = clock64();
    for (int i = 0; i < iters; i += 4) {
      if constexpr (kKind == 3) {        // as a K stage of the block-scaled GEMM: three scale copies, then four MMAs
        ptx::tc_cp_32x128b_warpx4(sfa, base);
        ptx::tc_cp_32x128b_warpx4(sfb, base + 512);
        ptx::tc_cp_32x128b_warpx4(sfb + 4, base + 1024);
      }
#pragma unroll
      for (int k4 = 0; k4 < 4; ++k4) {
        const uint64_t adv = static_cast<uint64_t>(2 * k4);
        const uint32_t acc = (i | k4) != 0 ? 1u : 0u;
        if constexpr (kKind == 0) ptx::tc_mma_bf16(tb, a + adv, b + adv, idesc[k4], acc);
        else if constexpr (kKind == 1) ptx::tc_mma_e4m3(tb, a + adv, b + adv, idesc[k4], acc);
        else ptx::tc_mma_mx(tb, a + adv, b + adv, idesc[k4], sfa, sfb, acc);
      }
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

// Tensor map over a row-major [rows, cols] matrix of bf16 (elem_bytes 2) or E4M3 bytes (elem_bytes 1): boxes of
// box_rows rows x 128 bytes, 128-byte swizzle.  Encoding a map costs a few microseconds of host time, and a serving
// loop calls with the same buffers every step, so the context keeps the last maps it built, keyed by everything
// that goes into one.
bool tensor_map_2d(moe_ctx* ctx, const void* base, uint64_t rows, uint64_t cols, int elem_bytes, int box_rows,
                   CUtensorMap* out) {
  for (int i = 0; i < ctx->num_maps; ++i) {
    const moe_map_entry& m = ctx->maps[i];
    if (m.base == base && m.rows == rows && m.cols == cols && m.elem_bytes == elem_bytes && m.box_rows == box_rows) {
      *out = m.map;
      return true;
    }
  }
  moe_map_entry& m = ctx->maps[ctx->num_maps < kMoeMapCache ? ctx->num_maps++ : ctx->next_map_victim++ % kMoeMapCache];
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * static_cast<uint64_t>(elem_bytes)};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(128 / elem_bytes), static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t elem[2] = {1u, 1u};
  const CUresult r = ctx->encode_tiled(&m.map, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                                               : CU_TENSOR_MAP_DATA_TYPE_UINT8, 2,
                                       const_cast<void*>(base), dims, strides, box, elem,
                                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                       static_cast<CUtensorMapL2promotion>(moe_knob_value(ctx, "l2_promo", 3)),
                                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    m.base = nullptr;
    m.rows = 0;
    return false;
  }
  m.base = base;
  m.rows = rows;
  m.cols = cols;
  m.elem_bytes = elem_bytes;
  m.box_rows = box_rows;
  *out = m.map;
  return true;
}

}  // namespace

extern "C" moe_status moe_probe_mma_cycles(moe_ctx* ctx, int32_t M, int32_t N, int32_t iters, double* cycles_per_mma,
                                           void* stream) {
  return moe_probe_mma_cycles_kind(ctx, 0, M, N, iters, cycles_per_mma, stream);
}

extern "C" moe_status moe_probe_mma_cycles_kind(moe_ctx* ctx, int32_t kind, int32_t M, int32_t N, int32_t iters,
                                                double* cycles_per_mma, void* stream) {
  if (!ctx || !cycles_per_mma) return MOE_ERR_INVALID_ARG;
  if (kind < 0 || kind > 3 || (kind >= 2 && M != 128)) return MOE_ERR_INVALID_ARG;
  if (!(M == 64 || M == 128) || N < 16 || N > 256 || N % 16 != 0 || iters < 1 || iters > (1 << 20))
    return MOE_ERR_INVALID_ARG;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  long long* d_out = reinterpret_cast<long long*>(ctx->d_trace);   // reuse the first trace word as the result slot
  const size_t smem = 1024 + kStageBytes;
  auto kernel = kind == 0 ? mma_cycle_probe<0> : kind == 1 ? mma_cycle_probe<1> : kind == 2 ? mma_cycle_probe<2> : mma_cycle_probe<3>;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
    return MOE_ERR_CUDA;
  iters = (iters + 3) / 4 * 4;
  kernel<<<1, 128, smem, cs>>>(M, N, iters, d_out);
  long long clocks = 0;
  if (cudaMemcpyAsync(&clocks, d_out, sizeof(clocks), cudaMemcpyDeviceToHost, cs) != cudaSuccess) return MOE_ERR_CUDA;
  if (cudaStreamSynchronize(cs) != cudaSuccess) return MOE_ERR_CUDA;
  if (clocks < 0) return MOE_ERR_TIMEOUT;
  *cycles_per_mma = static_cast<double>(clocks) / iters;
  return MOE_OK;
}

namespace moe {

cudaError_t prepare_expert_ffn(moe_ctx* ctx) {
  cudaError_t e = cudaSuccess;
  const int smem1 = static_cast<int>(kSmemBytes), smem2 = static_cast<int>(kPairSmemBytes);
  if ((e = cudaFuncSetAttribute(expert_ffn_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem1)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(expert_ffn_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem1)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(expert_ffn_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem2)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(expert_ffn_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem2)) != cudaSuccess) return e;
  // how many CTA pairs can be resident at once (an SM left over in a GPC cannot join a pair)
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * (ctx->num_sms / 2));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kPairSmemBytes;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  int clusters = 0;
  e = cudaOccupancyMaxActiveClusters(&clusters, expert_ffn_pair_kernel<false>, &cfg);
  if (e != cudaSuccess) return e;
  ctx->max_pairs = clusters < ctx->num_sms / 2 ? clusters : ctx->num_sms / 2;
  return cudaSuccess;
}

namespace {
cudaError_t launch_pair(moe_ctx* ctx, const CUtensorMap& a, const CUtensorMap& b0, const CUtensorMap& b1,
                        const CUtensorMap& out, const FfnParams& p, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * ctx->max_pairs);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kPairSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return p.fp8 ? cudaLaunchKernelEx(&cfg, expert_ffn_pair_kernel<true>, a, b0, b1, out, p)
               : cudaLaunchKernelEx(&cfg, expert_ffn_pair_kernel<false>, a, b0, b1, out, p);
}
}  // namespace

struct FfnMaps {
  CUtensorMap x, wg, wu, h, wd;   // copies: the kernels take them by value
  CUtensorMap x16, h16;           // the two A matrices in boxes of 16 rows (swapped-operand tiles)
  CUtensorMap h_out, y_out;       // the two outputs (bf16) in boxes of 32 rows (the epilogue's bulk stores)
};

static void launch_single(int grid, const FfnMaps& m, const FfnParams& p, cudaStream_t stream) {
  if (p.fp8)
    expert_ffn_kernel<true><<<grid, kThreads, kSmemBytes, stream>>>(m.x, m.wg, m.wu, m.h, m.wd, m.x16, m.h16, m.h_out, m.y_out, p);
  else
    expert_ffn_kernel<false><<<grid, kThreads, kSmemBytes, stream>>>(m.x, m.wg, m.wu, m.h, m.wd, m.x16, m.h16, m.h_out, m.y_out, p);
}

// Everything one expert-FFN call needs on the host side; fp8 selects E4M3 operands with epilogue scales.
struct FfnCall {
  const void* a1;          // Linear-1 input rows [R,H]
  const void* w_gate;
  const void* w_up;
  const void* w_down;
  void* h_bf16;            // Linear-1 output [R,F] bf16
  const void* a2;          // Linear-2 input rows [R,F]: h_bf16 itself, or its E4M3 copy
  void* y_perm;            // [R,H] bf16
  float* h_dbg;
  int fp8;
  const float *s_a1, *s_gate, *s_up, *s_a2, *s_down;   // fp8 scales
};

static moe_status run_ffn(moe_ctx* ctx, const FfnCall& c, const int32_t* offsets, const moe_tuning* tuning,
                          cudaStream_t stream, bool second_phase_only, bool first_phase_only) {
  const moe_shape& s = ctx->shape;
  const uint64_t R = static_cast<uint64_t>(s.T) * s.k;
  if (R == 0) return MOE_OK;
  const moe_tuning tn = moe_effective_tuning(ctx, tuning);
  if (c.fp8 && (tn.schedule != 0 || (tn.debug_flags & 6) != 0)) return MOE_ERR_UNSUPPORTED;   // bf16-only modes
  const int eb = c.fp8 ? 1 : 2;
  const int k_elems = 128 / eb;

  FfnMaps m;
  {
    const uint64_t EF = static_cast<uint64_t>(s.E) * s.F, EH = static_cast<uint64_t>(s.E) * s.H;
    const bool ok = tensor_map_2d(ctx, c.a1, R, s.H, eb, 128, &m.x) && tensor_map_2d(ctx, c.w_gate, EF, s.H, eb, 128, &m.wg) &&
                    tensor_map_2d(ctx, c.w_up, EF, s.H, eb, 128, &m.wu) && tensor_map_2d(ctx, c.a2, R, s.F, eb, 128, &m.h) &&
                    tensor_map_2d(ctx, c.w_down, EH, s.F, eb, 128, &m.wd) &&
                    tensor_map_2d(ctx, c.a1, R, s.H, eb, 16, &m.x16) && tensor_map_2d(ctx, c.a2, R, s.F, eb, 16, &m.h16) &&
                    tensor_map_2d(ctx, c.h_bf16, R, s.F, 2, 32, &m.h_out) && tensor_map_2d(ctx, c.y_perm, R, s.H, 2, 32, &m.y_out);
    if (!ok) return MOE_ERR_CUDA;
  }

  FfnParams p{};
  p.offsets = offsets;
  p.E = s.E;
  p.ph[0] = PhaseDesc{s.F, s.H, (s.F + 127) / 128, (s.H + k_elems - 1) / k_elems, 128, 0,
                      static_cast<__nv_bfloat16*>(c.h_bf16), c.s_a1, c.s_gate, c.s_up};
  p.ph[1] = PhaseDesc{s.H, s.F, (s.H + 255) / 256, (s.F + k_elems - 1) / k_elems, 256, 128,
                      static_cast<__nv_bfloat16*>(c.y_perm), c.s_a2, c.s_down, c.s_down};
  p.h_dbg = c.h_dbg;
  p.burst = tn.store_burst_tiles;
  p.mode = tn.interleave_mode;
  p.ik = tn.interleave_k;
  p.status = ctx->d_status;
  p.ready = ctx->d_ready;
  p.schedule = tn.schedule;
  p.fp8 = c.fp8;
  p.k_elems = k_elems;
  p.swap_rows = moe_knob_value(ctx, "swap_rows", kSwapRows);
  // L2 eviction priorities of the TMA loads (development knob cache_hints, a bit mask).  Default 35 = in the
  // single-CTA kernel the weights of an expert with a single row block go first (bit 0: no other tile reads them, and
  // on layers of many small experts they are nearly all of the traffic), the rows of A stay (bit 1: every column block
  // of the expert reads them again) and so do the weights of experts with several row blocks (bit 5: each of those
  // blocks reads them).  Measured in the power-capped steady state: bits 0 and 1 -6 % on the decode-like layer and
  // -3.7 % on the DeepSeek-V3-like one; bit 5 another -1.2 % there and -1 to -2 % on the Mixtral-like layer at 1024 to
  // 3072 tokens.  Bit 2 restricts bit 1 to Linear-2.  In the CTA-pair kernel bit 3 = rows of A stay, bit 6 = weights
  // stay (together -3 % on the Mixtral-like layer, both on by default), bit 4 = weights go first (17 % slower: the row
  // blocks that share a weight box do not run closely enough together).
  p.cache_hints = moe_knob_value(ctx, "cache_hints", 35 | 8 | 64);
  // Swapped-operand tiles of at most 16 rows (most tiles of a decode-like batch) load those rows as one 16-row box
  // instead of a 128-row box of mostly other experts' rows: a third less to move per K block; -1 % on the decode-like
  // layer, -0.4 % on the DeepSeek-V3-like one in steady state (larger row counts, several boxes per K block: no gain).
  p.small_a = moe_knob_value(ctx, "small_a", 16);
  p.bulk_stores = moe_knob_value(ctx, "bulk_stores", 1);
  p.small_ring = moe_knob_value(ctx, "small_ring", 1);
  const int grid = ctx->num_sms;   // persistent: one CTA per SM (shared memory allows no second)
  // Algorithm 1's lead; 0 asks for the anti-starvation knee ceil(b_n K_SM / (2 h_inter)) with b_n = 128
  p.lead_D = tn.dep_lead_D > 0 ? tn.dep_lead_D : (128 * grid + 2 * s.F - 1) / (2 * s.F);
  p.withhold_ready = (tn.debug_flags & 4) != 0;
  p.wait_budget = p.withhold_ready ? 200000000LL : ptx::kWaitClockBudget;   // the drill gives up after ~0.1 s
  const bool trace = (tn.debug_flags & 1) != 0;
  if (trace && !second_phase_only &&
      cudaMemsetAsync(ctx->d_trace, 0, static_cast<size_t>(2) * ctx->num_sms * kMoeTraceFields * 8, stream) !=
          cudaSuccess)
    return MOE_ERR_CUDA;   // roles that do not run in a variant (the peer's MMA warp) leave zeros, not stale counts
  const bool split = second_phase_only || first_phase_only;   // the caller runs something between the two GEMMs
  // Launch-latency-bound layers (every tile fits in about one wave of CTAs) run both GEMMs in one launch.
  const long long max_blocks = static_cast<long long>(R / 128) + s.E;
  const bool tiny = max_blocks * (p.ph[0].n_blocks + p.ph[1].n_blocks) <= 2LL * grid;
  const bool one_launch = !split && (tn.schedule == 1 || (tn.debug_flags & 6) != 0 || tiny);
  // The CTA-pair kernel runs on request only.  It used to be the default for layers averaging 1024 rows per expert or
  // more; since the TMA loads carry L2 eviction priorities the single-CTA kernel with 256-row tiles is the faster one
  // there as well (Mixtral-like layer, steady state: -1.6 to -4 % at 8192 tokens, -6 % at 4096, -9 % at 16384; burst
  // equal): it computes an expert's remainder rows as a 128-row or swapped-operand tile instead of a whole 256-row
  // tile, draws tiles dynamically instead of in rounds, and holds a higher SM clock under the power cap.
  // One exception, per GEMM (bit 0 Linear-1, bit 1 Linear-2): with E4M3 operands on a layer averaging 1024 rows per
  // expert or more, Linear-1 runs as CTA pairs.  Its 128-row tiles (256-row tiles do not pay there, see below) need 96
  // operand bytes per clock and SM where an SM takes 64, which holds an E4M3 mainloop at two thirds of its rate; a pair
  // needs 64 (Mixtral-like layer, steady state, alternating runs: Linear-1 1.94 -> 1.77 ms, the step 3.13 -> 2.92 ms;
  // Linear-2 stays on 256-row tiles: 1.07 against 1.09 ms).  debug_flags bit 4 keeps the single-CTA kernel everywhere.
  const bool dense = R / static_cast<uint64_t>(s.E) >= 1024;
  const int pair_phases = !(!one_launch && ctx->max_pairs > 0) ? 0
                          : (tn.debug_flags & 8)               ? 3
                          : (c.fp8 && dense && !(tn.debug_flags & 16)) ? moe_knob_value(ctx, "fp8_pair_phases", 1)
                                                                       : 0;
  unsigned long long* trace2 = trace ? ctx->d_trace + static_cast<size_t>(ctx->num_sms) * kMoeTraceFields : nullptr;

  if (one_launch) {
    p.phase_lo = 0;
    p.phase_hi = 2;
    p.sched = ctx->d_sched;
    p.trace = trace ? ctx->d_trace : nullptr;
    p.order_log = trace ? ctx->d_order : nullptr;
    p.kernel_id = 3;
    launch_single(grid, m, p, stream);
    moe_mark(ctx, 5, stream);
    moe_mark(ctx, 6, stream);
    ctx->last_launches += 1;
    return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
  }
  // two separate launches: many-row experts may run as 256-row tiles (decided in the kernel from the row counts)
  const int wide_knob = moe_knob_value(ctx, "wide_tiles", 1);   // 0 never, 1 by the kernel's rule, 2 whenever an expert has several blocks
  // Which GEMMs may use them (bit 0 Linear-1, bit 1 Linear-2).  A 256-row tile holds both accumulators, so the next
  // tile waits for the drain of the first; with E4M3 operands the mainloop is half as long and that wait weighs twice
  // as much in Linear-1 (gated epilogue): there 256-row tiles pay in Linear-2 only (Mixtral-like layer, per-row FP8,
  // steady state: 3.07 against 3.18-3.24 ms with both, 3.22-3.23 with Linear-1 only); bf16 gains from both (4.85-4.89
  // against 5.05-5.13 ms with either one alone).
  const int wide_phases = moe_knob_value(ctx, "wide_phases", c.fp8 ? 2 : 3);
  // Fine-grained bf16 layers (16 to 256 rows per expert on average): each GEMM as two launches, first the experts of
  // at most 16 rows, which then run on the six-stage ring, then the others (DeepSeek-V3-like layer, steady state,
  // alternating runs: 4.60 -> 4.53 ms through the bench, 4.52 -> 4.47 through the library alone; with E4M3 operands the
  // same split costs 2 %, so that path keeps one launch per GEMM).  A layer without both kinds of experts runs its
  // first launch on everything and its second on nothing.  Not while tracing (one set of counters per GEMM).
  // (Below 16 rows per expert on average, decode-like layers, larger experts are unlikely and the empty second launch
  // of each GEMM would cost 1 %.)
  const uint64_t mean_rows = R / static_cast<uint64_t>(s.E);
  const bool split_sizes = !trace && !c.fp8 && moe_knob_value(ctx, "split_sizes", 1) != 0 && mean_rows >= 16 &&
                           mean_rows <= 256;
  if (!second_phase_only) {
    p.wide_allowed = (wide_phases & 1) ? wide_knob : 0;
    p.phase_lo = 0;
    p.phase_hi = 1;
    p.sched = ctx->d_sched;
    p.trace = trace ? ctx->d_trace : nullptr;
    p.kernel_id = (pair_phases & 1) ? 4 : 1;
    if (pair_phases & 1) {
      if (launch_pair(ctx, m.x, m.wg, m.wu, m.h_out, p, stream) != cudaSuccess) return MOE_ERR_CUDA;
    } else if (split_sizes) {
      p.expert_class = 1;
      launch_single(grid, m, p, stream);
      p.expert_class = 2;
      launch_single(grid, m, p, stream);
      p.expert_class = 0;
      ctx->last_launches += 1;
    } else {
      launch_single(grid, m, p, stream);
    }
    moe_mark(ctx, 5, stream);
    ctx->last_launches += 1;
  }
  if (!first_phase_only) {
    p.wide_allowed = (wide_phases & 2) ? wide_knob : 0;
    p.phase_lo = 1;
    p.phase_hi = 2;
    p.sched = ctx->d_sched + 2;
    p.trace = trace2;
    p.kernel_id = (pair_phases & 2) ? 5 : 2;
    if (pair_phases & 2) {
      if (launch_pair(ctx, m.h, m.wd, m.wd, m.y_out, p, stream) != cudaSuccess) return MOE_ERR_CUDA;
    } else if (split_sizes) {
      p.expert_class = 1;
      launch_single(grid, m, p, stream);
      p.expert_class = 2;
      launch_single(grid, m, p, stream);
      p.expert_class = 0;
      ctx->last_launches += 1;
    } else {
      launch_single(grid, m, p, stream);
    }
    moe_mark(ctx, 6, stream);
    ctx->last_launches += 1;
  }
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

moe_status launch_expert_ffn(moe_ctx* ctx, const void* x_perm, const int32_t* offsets, const void* w_gate,
                             const void* w_up, const void* w_down, void* h_ws, void* y_perm,
                             float* h_fp32_debug, const moe_tuning* tuning, cudaStream_t stream) {
  FfnCall c{};
  c.a1 = x_perm;
  c.w_gate = w_gate;
  c.w_up = w_up;
  c.w_down = w_down;
  c.h_bf16 = h_ws;
  c.a2 = h_ws;
  c.y_perm = y_perm;
  c.h_dbg = h_fp32_debug;
  return run_ffn(ctx, c, offsets, tuning, stream, false, false);
}

moe_status launch_expert_ffn_fp8(moe_ctx* ctx, const moe_fp8_ffn_args* a, const moe_tuning* tuning,
                                 cudaStream_t stream) {
  const moe_shape& s = ctx->shape;
  FfnCall c{};
  c.a1 = a->xq_perm;
  c.w_gate = a->wq_gate;
  c.w_up = a->wq_up;
  c.w_down = a->wq_down;
  c.h_bf16 = a->h_ws;
  c.a2 = a->hq_ws;
  c.y_perm = a->y_perm;
  c.fp8 = 1;
  c.s_a1 = a->sx_perm;
  c.s_gate = a->s_gate;
  c.s_up = a->s_up;
  c.s_a2 = a->sh_ws;
  c.s_down = a->s_down;
  moe_status st = run_ffn(ctx, c, a->offsets, tuning, stream, false, true);          // Linear-1 -> h (bf16)
  if (st != MOE_OK) return st;
  if (launch_quantize_rows(ctx, a->h_ws, static_cast<long long>(s.T) * s.k, s.F, a->hq_ws, a->sh_ws, stream) !=
      cudaSuccess)
    return MOE_ERR_CUDA;                                                              // h -> E4M3 + row scales
  return run_ffn(ctx, c, a->offsets, tuning, stream, true, false);                    // Linear-2
}

}  // namespace moe
