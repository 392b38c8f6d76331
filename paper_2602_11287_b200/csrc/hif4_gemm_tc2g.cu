// Grouped (MoE) tensor-core HiF4 GEMM on CTA pairs with the operands swapped: per expert g,
// C[off[g]:off[g+1], :] = A[off[g]:off[g+1], :] * B[g]^T (Eq. 3 summed over unit pairs).
//
// Experts get very different numbers of rows (a few hot ones thousands, the median a few dozen), so
// the tokens go on the flexible side of the MMA: a work unit is 256 weight rows of one expert (the
// MMA's M side, 128 rows per CTA of the pair) times a token tile of T rows of that expert, T a multiple
// of 32 up to 256 (the MMA's N side, T/2 rows per CTA).  A unit decodes 128 weight rows + T/2 token rows
// per CTA and 64-wide K block, so a 40-row expert costs little more than the decode of its weights,
// which every row of the expert needs anyway.  The accumulator holds C transposed (lane = weight row,
// column = token); the epilogue stores it back with 32 lanes writing 32 consecutive columns of one
// token's row, which is coalesced without staging and lets the last tile of a group stop at its end.
//
// Pipeline, barriers and bounded waits are those of the dense CTA-pair kernel: TMA producer warp (raw
// units, K = 256 per stage, each CTA fetches its own rows), 16 decode warps, the MMA-issuing thread
// on rank 0 with multicast commits, 4 epilogue warps, two accumulator stages.
//
// Small token tiles (T <= 64, three quarters of the tiles of a Zipf-routed layer): the time of a K chunk is the
// serial decode of two units per decode thread whatever T is, and with T / 2 <= 32 token rows per CTA almost all
// of the 256 "token row" threads would idle.  Such a tile is therefore multiplied with TWO weight tiles at once:
// the token-row threads decode the 128 rows of the second weight tile instead, four extra warps decode the few
// token rows (one unit per thread and chunk, read straight from global memory into a small operand buffer of
// their own), the MMA thread issues both products against the same token block into two accumulators, and the
// epilogue stores both.  The unit count of those tiles halves.
#include "hif4_common.cuh"
#include "hif4_gemm_internal.cuh"
#include "hif4_tc2_common.cuh"

namespace hif4 {
namespace {

constexpr int kWRows = 128;                           // weight rows per CTA (256 per pair)
constexpr int kMaxTok = 256;                          // token rows per unit (128 per CTA)
constexpr int kRawHalfBytes = 128 * kRawRowBytes;     // 18432
constexpr int kRawStageBytes = 2 * kRawHalfBytes;     // weight rows then token rows
constexpr int kDecHalfBytes = 128 * 128;              // 128 rows x 64 BF16
constexpr int kDecStageBytes = 2 * kDecHalfBytes;
constexpr int kRawStages = 2;
constexpr int kDecStages = 4;
constexpr int kTmemCols = 512;

constexpr int kDecodeWarp0 = 6;
constexpr int kDecodeThreads = 512;
constexpr int kTokWarp0 = kDecodeWarp0 + kDecodeThreads / 32;  // 22: the four token warps of the small-tile mode
constexpr int kTokThreads = 128;                               // (unit of the chunk, token row): 4 x 32
constexpr int kSmallT = 64;                                    // token tiles up to this many rows take two weight tiles
constexpr int kTokBufBytes = 32 * 128;                         // decoded token rows of one K = 64 block (small mode)
constexpr int kThreads = kDecodeWarp0 * 32 + kDecodeThreads + kTokThreads;   // 832
constexpr int kEpiBufBytes = 16 * 32 * 4;                      // epilogue staging of one warp: 16 token rows x 32 columns of C
constexpr int kSmemBytes = 1024 + kDecStages * kDecStageBytes + kRawStages * kRawStageBytes + kDecStages * kTokBufBytes + 256 + 1024;
constexpr int kSmemBytesStaged = kSmemBytes + 4 * kEpiBufBytes;

// tcgen05.mma kind::f16 descriptor without the N field: D = F32, A = B = BF16, K-major, M = 256.
constexpr uint32_t kInstrDescM256 = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(256 >> 4) << 24);

// One work record: token rows [tok0, tok0 + T) of a group (valid below tok_end) times weight rows [w_row0, +256) of
// that group's matrix (columns [n0, +256) of C); tiles = 2: also the next 256 weight rows (small-tile mode).
struct WorkRec { int tok0; int tok_end; int w_row0; int n0; int T; int tiles; };
constexpr int kTableHeaderBytes = 32;                 // record count, then the records

struct GroupedParams {
  float* C;
  int64_t ldc;
  int64_t N;            // weight rows per expert = columns of C
  int num_kc;           // K / 256
  int n_wtiles;         // ceil(N / 256)
  int max_entries;          // dense problems: 1
  const WorkRec* table;     // nullptr: one dense problem of dense_rows token rows (a single tile)
  const int* table_count;   // number of records (written by the table kernel)
  const uint32_t* tok_units;    // the token operand again, for the token warps of the small-tile mode
  int64_t tok_rows;
  int64_t upr;              // units per row
  int dense_rows;
  // Dense problems with fewer weight tiles than CTA pairs: every tile is cut into `slices` K ranges on pairs of
  // their own.  Slice 0 stores its part of C, slice s > 0 adds to it after the same epilogue warp of slice s - 1
  // is done with the same columns, so every element is summed in slice order.
  int slices;               // 1: not split (always 1 with a table)
  unsigned int* flags;      // [n_wtiles][slices][8]: "this epilogue warp of this slice is done" (zero at launch)
  unsigned int* error_word;
  // Keep the multipliers here, behind the 8-byte fields and 8 bytes off a 16-byte boundary of the parameter block: the
  // decode loop reads them as instruction operands, and with the same six words 4 or 8 bytes further the kernel
  // measured 7-8 % slower (ncu durations, config-5 gate/up 3.18-3.21 vs 2.96 ms), at the head of the block 1 %.
  DecodeMul mul;
};

// Work table from the device-side offsets: every group is cut into token tiles of 256 rows, the last one padded
// to a multiple of 32; a tile of more than kSmallT rows gives one record per 256 weight rows, a smaller one a
// record per PAIR of weight tiles.  Thread g counts the records of group g and a block-wide scan places them; then
// the records of the 256 groups are written as one flat list, record i by thread i % 256 of block (i / 256) % blocks
// (it finds the group of a record by bisection in the scanned counts), so a hot expert's hundreds of records cost no
// more than anyone else's.  Every block repeats the counting and the scan (a few microseconds) and writes its share
// of the list; block 0 writes the record count.  Groups are taken 256 at a time.
constexpr int kTableBlocks = 16;
__global__ void __launch_bounds__(256)
build_work_table_kernel(const int64_t* __restrict__ offsets, int num_groups, int64_t N, int n_wtiles, uint8_t* table_mem,
                        int max_records) {
  __shared__ int warp_sums[8];
  __shared__ int s_first[257];                 // first record of each group of the batch (relative), and their total
  __shared__ int64_t s_lo[256], s_hi[256];
  __shared__ int s_base;
  WorkRec* table = reinterpret_cast<WorkRec*>(table_mem + kTableHeaderBytes);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) s_base = 0;
  __syncthreads();
  for (int g0 = 0; g0 < num_groups; g0 += 256) {
    const int g = g0 + threadIdx.x;
    int64_t lo = 0, hi = 0;
    if (g < num_groups) { lo = offsets[g]; hi = offsets[g + 1]; }
    if (hi < lo) hi = lo;
    const int64_t rows = hi - lo;
    const int64_t full = rows / kMaxTok;
    const int rest = static_cast<int>(rows - full * kMaxTok);
    const int rest_units = rest == 0 ? 0 : rest <= kSmallT ? (n_wtiles + 1) / 2 : n_wtiles;
    const int mine = static_cast<int>(full) * n_wtiles + rest_units;
    // exclusive scan of `mine` over the block
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    int before = 0;
    for (int w = 0; w < warp; ++w) before += warp_sums[w];
    s_first[threadIdx.x] = before + incl - mine;
    if (threadIdx.x == 255) s_first[256] = before + incl;
    s_lo[threadIdx.x] = lo; s_hi[threadIdx.x] = hi;
    __syncthreads();
    const int batch_total = s_first[256], base = s_base;
    for (int i = blockIdx.x * 256 + threadIdx.x; i < batch_total && base + i < max_records; i += 256 * gridDim.x) {
      int a = 0, b = 256;                               // the last group whose first record is <= i (empty groups skipped)
      while (b - a > 1) {
        const int m = (a + b) >> 1;
        if (s_first[m] <= i) a = m; else b = m;
      }
      const int64_t g_lo = s_lo[a], g_hi = s_hi[a];
      const int j = i - s_first[a];
      const int g_full = static_cast<int>((g_hi - g_lo) / kMaxTok), g_rest = static_cast<int>((g_hi - g_lo) - static_cast<int64_t>(g_full) * kMaxTok);
      WorkRec rec;
      int t_rows, wt, step;
      if (j < g_full * n_wtiles) {                        // a whole token tile
        const int tile = j / n_wtiles;
        wt = j - tile * n_wtiles; step = 1; t_rows = kMaxTok;
        rec.tok0 = static_cast<int>(g_lo + static_cast<int64_t>(tile) * kMaxTok);
      } else {                                          // the last tile of the group
        step = g_rest <= kSmallT ? 2 : 1;
        wt = (j - g_full * n_wtiles) * step; t_rows = g_rest;
        rec.tok0 = static_cast<int>(g_lo + static_cast<int64_t>(g_full) * kMaxTok);
      }
      rec.tok_end = static_cast<int>(g_hi);
      rec.n0 = wt * 256;
      rec.w_row0 = static_cast<int>(static_cast<int64_t>(g0 + a) * N) + rec.n0;
      rec.T = (t_rows + 31) & ~31;
      rec.tiles = step == 2 ? (wt + 1 < n_wtiles ? 2 : 3) : 1;       // 3: small-tile mode whose second weight tile does not exist
      table[base + i] = rec;
    }
    __syncthreads();
    if (threadIdx.x == 0) s_base = base + batch_total;
    __syncthreads();
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) *reinterpret_cast<int*>(table_mem) = s_base < max_records ? s_base : max_records;
}

struct Unit { int tok0; int tok_end; int T; int w_row0; int n0; int kc0; int kc1; int wt; int slice; int tiles; };
__device__ __forceinline__ Unit unit_of(const GroupedParams& p, int u) {
  Unit r;
  if (p.table == nullptr) {                 // dense: unit = (K slice, weight tile)
    r.slice = u / p.n_wtiles; r.wt = u - r.slice * p.n_wtiles;
    r.tok0 = 0; r.tok_end = p.dense_rows; r.T = (p.dense_rows + 31) & ~31;
    r.tiles = 1;
    r.n0 = r.wt * 256;
    r.w_row0 = r.n0;
    r.kc0 = static_cast<int>(static_cast<int64_t>(r.slice) * p.num_kc / p.slices);
    r.kc1 = static_cast<int>(static_cast<int64_t>(r.slice + 1) * p.num_kc / p.slices);
    return r;
  }
  const WorkRec t = p.table[u];
  r.wt = 0; r.slice = 0;
  r.tok0 = t.tok0; r.tok_end = t.tok_end; r.T = t.T; r.tiles = t.tiles;
  r.n0 = t.n0;
  r.w_row0 = t.w_row0;
  r.kc0 = 0; r.kc1 = p.num_kc;
  return r;
}
__device__ __forceinline__ int total_units_of(const GroupedParams& p) {
  return p.table == nullptr ? p.n_wtiles * p.slices : *p.table_count;
}

// Decodes the two units held in raw words W[0..8], W[9..17] into decoded stages 2h and 2h+1 (skipped for
// rows that the tile does not use; the barrier protocol runs either way).
__device__ __forceinline__ bool decode_two_units_g(const uint32_t (&W)[18], bool active, const uint32_t (&chunk_addr)[8],
                                                   uint32_t lut, const DecodeMul& mul, uint32_t dec_empty0,
                                                   uint32_t dec_full0_leader, uint32_t parity_free,
                                                   volatile uint32_t* abort_flag) {
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    if (!__all_sync(0xFFFFFFFFu, mbar_wait(dec_empty0 + 8 * u, parity_free, abort_flag))) return false;
    if (active) decode_unit_balanced(W[9 * u], &W[9 * u + 1], chunk_addr, u * kDecStageBytes, lut, mul);
    fence_proxy_async_smem();
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive_cluster(dec_full0_leader + 8 * u);
  }
  return true;
}

// Bounded wait until a word in global memory, written by another CTA after a __threadfence(), has reached `want`.
__device__ __noinline__ bool wait_word(const unsigned int* word, unsigned int want, volatile uint32_t* abort_flag) {
  const uint64_t t0 = global_ns();
  for (uint32_t it = 1;; ++it) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(word) : "memory");
    if (v >= want) return true;
    __nanosleep(32);
    if ((it & 63u) == 0u) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > kWaitBudgetNs) {
        *abort_flag = 1u;
        return false;
      }
    }
  }
}

// kStagedEpi: the epilogue passes C through a staging block in shared memory (see there); the other instantiation
// stores straight from the accumulator registers.  Two kernels rather than one with both paths: records with a long K
// gain nothing from the staged form and keep the smaller kernel.  What only the staged epilogue needs rides behind
// the common parameters, so that the other instantiation's parameter block keeps its layout.
template <bool kStagedEpi> struct EpilogueArgs {};
template <> struct EpilogueArgs<true> {
  CUtensorMap tmC;          // FP32 view of C, box = 32 columns x 16 rows
  int tma_store;            // 1: whole 16-row chunks of C go out through tmC
};
template <bool kStagedEpi>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_tc2g_kernel(const __grid_constant__ CUtensorMap tmTok, const __grid_constant__ CUtensorMap tmW,
                 const GroupedParams p, const __grid_constant__ EpilogueArgs<kStagedEpi> epi) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t dec_base = smem_base;                                        // 1024-byte aligned stages
  const uint32_t raw_base = dec_base + kDecStages * kDecStageBytes;
  const uint32_t tok_base = raw_base + kRawStages * kRawStageBytes;        // 1024-byte aligned: small-mode token blocks
  const uint32_t epi_base = tok_base + kDecStages * kTokBufBytes;          // 1024-byte aligned: epilogue staging, one block per warp
  const uint32_t bar_base = epi_base + (kStagedEpi ? 4 * kEpiBufBytes : 0);
  const uint32_t raw_full = bar_base, raw_empty = bar_base + 16, dec_full = bar_base + 32, dec_empty = bar_base + 64,
                 tmem_full = bar_base + 96, tmem_empty = bar_base + 112;
  uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
  volatile uint32_t* tmem_ptr_smem = reinterpret_cast<volatile uint32_t*>(gen_base + (bar_base - smem_base) + 128);
  volatile uint32_t* abort_flag = tmem_ptr_smem + 1;
  const uint32_t lut = bar_base + 256;
  if (threadIdx.x < 256)
    reinterpret_cast<uint32_t*>(gen_base + (lut - smem_base))[threadIdx.x] = spread_e8_entry(threadIdx.x);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const int total_units = total_units_of(p);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kRawStages; ++s) {
      mbar_init(raw_full + 8 * s, 1);
      mbar_init(raw_empty + 8 * s, kDecodeThreads);
    }
    for (int s = 0; s < kDecStages; ++s) {
      mbar_init(dec_full + 8 * s, kDecodeThreads / 32 + 2);   // 8 decode warps + 1 token warp of each CTA per stage (used on rank 0)
      mbar_init(dec_empty + 8 * s, 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(tmem_full + 8 * s, 1);
      mbar_init(tmem_empty + 8 * s, 8);                   // 4 epilogue warps of each CTA (used on rank 0)
    }
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(bar_base + 128),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();            // the peer's barriers are initialised before anyone arrives on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_smem;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      uint32_t n = 0;
      bool ok = true;
      for (int u = pair; u < total_units && ok; u += num_pairs) {
        const Unit un = unit_of(p, u);
        for (int kc = un.kc0; kc < un.kc1; ++kc, ++n) {
          const uint32_t s = n & 1u, ph = (n >> 1) & 1u;
          if (!(ok = mbar_wait(raw_empty + 8 * s, ph ^ 1u, abort_flag, 128))) break;
          mbar_expect_tx(raw_full + 8 * s, kRawStageBytes);
          const uint32_t dst = raw_base + s * kRawStageBytes;
          tma_load_2d(dst, &tmW, kc * kRawRowBytes, un.w_row0 + static_cast<int>(rank) * kWRows, raw_full + 8 * s);
          if (un.tiles == 1)
            tma_load_2d(dst + kRawHalfBytes, &tmTok, kc * kRawRowBytes, un.tok0 + static_cast<int>(rank) * (un.T >> 1),
                        raw_full + 8 * s);
          else            // small-tile mode: the second weight tile takes the place of the token rows
            tma_load_2d(dst + kRawHalfBytes, &tmW, kc * kRawRowBytes, un.w_row0 + 256 + static_cast<int>(rank) * kWRows,
                        raw_full + 8 * s);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer (rank 0 only)
    if (rank == 0 && lane == 0) {
      uint32_t n = 0, ucount = 0;
      bool ok = true;
      for (int u = pair; u < total_units && ok; u += num_pairs) {
        const Unit un = unit_of(p, u);
        const uint32_t acc = ucount & 1u, aph = (ucount >> 1) & 1u;
        if (!(ok = mbar_wait_cluster(tmem_empty + 8 * acc, aph ^ 1u, abort_flag))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * kMaxTok;
        const uint32_t idesc = kInstrDescM256 | (static_cast<uint32_t>(un.T >> 3) << 17);
        for (int kc = un.kc0; kc < un.kc1 && ok; ++kc, ++n) {
          // stages 0 and 2 are filled first (see the dense pair kernel): consume 0, 2, 1, 3
#pragma unroll
          for (int i = 0; i < kDecStages; ++i) {
            const int st = ((i & 1) << 1) | (i >> 1);
            if (!(ok = mbar_wait_cluster(dec_full + 8 * st, n & 1u, abort_flag))) break;
            tc_fence_after();
            const uint64_t adesc = make_desc(dec_base + st * kDecStageBytes);                  // weights: M side
            if (un.tiles == 1) {
              const uint64_t bdesc = make_desc(dec_base + st * kDecStageBytes + kDecHalfBytes);  // tokens: N side
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                tc2_mma(d_tmem, adesc + 2 * kk, bdesc + 2 * kk, idesc, ((kc - un.kc0) | i | kk) != 0 ? 1u : 0u);
            } else {
              // small-tile mode: both halves of the stage are weight tiles, the tokens sit in their own block
              const uint64_t a2desc = make_desc(dec_base + st * kDecStageBytes + kDecHalfBytes);
              const uint64_t bdesc = make_desc(tok_base + st * kTokBufBytes);
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                tc2_mma(d_tmem, adesc + 2 * kk, bdesc + 2 * kk, idesc, ((kc - un.kc0) | i | kk) != 0 ? 1u : 0u);
              if (un.tiles == 2) {
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                  tc2_mma(d_tmem + 128, a2desc + 2 * kk, bdesc + 2 * kk, idesc, ((kc - un.kc0) | i | kk) != 0 ? 1u : 0u);
              }
            }
            tc2_commit_both(dec_empty + 8 * st);
          }
        }
        if (!ok) break;
        tc2_commit_both(tmem_full + 8 * acc);
        ++ucount;
      }
    }
  } else if (warp < kDecodeWarp0) {
    // ---------------------------------------------------------------- epilogue: C^T tile -> rows of C
    const int q = warp & 3;                      // TMEM lane quadrant this warp may read
    const uint32_t tmem_empty_leader = mapa(tmem_empty, 0);
    [[maybe_unused]] const uint32_t my_buf = epi_base + static_cast<uint32_t>(q) * kEpiBufBytes;
    uint32_t ucount = 0;
    for (int u = pair; u < total_units; u += num_pairs) {
      const Unit un = unit_of(p, u);
      const uint32_t acc = ucount & 1u, aph = (ucount >> 1) & 1u;
      if (!__all_sync(0xFFFFFFFFu, mbar_wait(tmem_full + 8 * acc, aph, abort_flag, 256))) break;
      tc_fence_after();
      const int chunks = un.T >> 4;
      // K-sliced dense tile: slices after the first add to what the previous slice has left in C
      const bool adds = un.slice > 0;
      unsigned int* my_flag = p.slices > 1 ? p.flags + (static_cast<size_t>(un.wt) * p.slices + un.slice) * 8 + rank * 4 + q : nullptr;
      if (adds && !__all_sync(0xFFFFFFFFu, wait_word(my_flag - 8, 1u, abort_flag))) break;
      const int n_acc = un.tiles == 2 ? 2 : 1;   // small-tile mode: a second accumulator 128 columns further, 256 columns of C further
#pragma unroll 1
      for (int a = 0; a < n_acc; ++a) {
        const int64_t col = static_cast<int64_t>(un.n0) + a * 256 + rank * kWRows + q * 32 + lane;   // column of C = weight row
        const bool col_ok = col < p.N;
#pragma unroll 1
        for (int c = 0; c < chunks; ++c) {
          uint32_t r[16];
          tc_ld16(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * kMaxTok + a * 128 + c * 16, r);
          tc_wait_ld();
          if (a == n_acc - 1 && c == chunks - 1) {   // accumulator fully read: hand it back before the stores
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(tmem_empty_leader + 8 * acc);
          }
          if constexpr (kStagedEpi) {
            const int tok = un.tok0 + c * 16;
            // The lanes put their column of the 16 x 32 chunk into the warp's staging block (row v = 32 consecutive
            // floats: no bank conflicts).  A chunk whose sixteen token rows all exist then goes out as one TMA store,
            // which also clips columns past N; the last rows of a group, a C that the tensor map cannot describe and the
            // adding slices of a K-sliced tile are written row by row from the block (each lane its own column) -- a
            // short rolled loop instead of sixteen tested, 64-bit-addressed stores per lane in the instruction stream.
            const int64_t col0 = static_cast<int64_t>(un.n0) + a * 256 + rank * kWRows + q * 32;
            const int n_rows = un.tok_end - tok < 16 ? un.tok_end - tok : 16;        // warp-uniform, may be <= 0
            if (col0 >= p.N || n_rows <= 0) continue;
            if (lane == 0) bulk_wait_read<0>();        // the previous TMA store has read the block
            __syncwarp();
#pragma unroll
            for (int v = 0; v < 16; ++v)
              asm volatile("st.shared.u32 [%0], %1;" ::"r"(my_buf + static_cast<uint32_t>(v * 128 + lane * 4)), "r"(r[v]) : "memory");
            if (epi.tma_store && !adds && n_rows == 16) {
              fence_proxy_async_smem();
              __syncwarp();
              if (lane == 0) {
                tma_store_2d(&epi.tmC, static_cast<int>(col0), tok, my_buf);
                bulk_commit();
              }
            } else if (col_ok) {
              float* cp = p.C + static_cast<int64_t>(tok) * p.ldc + col;
#pragma unroll 1
              for (int v = 0; v < n_rows; ++v, cp += p.ldc) {
                const float x = __uint_as_float(lds32(my_buf + static_cast<uint32_t>(v * 128 + lane * 4)));
                if (adds) asm volatile("red.global.add.f32 [%0], %1;" ::"l"(cp), "f"(x) : "memory");
                else __stcs(cp, x);                  // C is written once and not read again by this kernel
              }
            }
          } else {
            const int tok = un.tok0 + c * 16;
            float* cp = p.C + static_cast<int64_t>(tok) * p.ldc + col;
#pragma unroll
            for (int v = 0; v < 16; ++v)
              if (col_ok && tok + v < un.tok_end) {
                float* dst = cp + static_cast<int64_t>(v) * p.ldc;
                if (adds) asm volatile("red.global.add.f32 [%0], %1;" ::"l"(dst), "f"(__uint_as_float(r[v])) : "memory");
                else __stcs(dst, __uint_as_float(r[v]));       // C is written once and not read again by this kernel
              }
          }
        }
      }
      if (p.slices > 1 && un.slice + 1 < p.slices) {      // the next slice may add to these columns now
        if (kStagedEpi && lane == 0) bulk_wait_all();     // (its own stores, if any went through the tensor map, have landed)
        __threadfence();
        __syncwarp();
        if (lane == 0) asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(my_flag), "r"(1u) : "memory");
      }
      ++ucount;
    }
    if (kStagedEpi && lane == 0) bulk_wait_all();  // shared memory stays valid until the last store has read it
  } else if (warp >= kTokWarp0) {
    // ---------------------------------------------------------------- token warps (small-tile mode): warp w = unit w of the chunk
    const int w = warp - kTokWarp0;
    const uint32_t r7 = static_cast<uint32_t>(lane) & 7u;
    const uint32_t dec_row = tok_base + static_cast<uint32_t>(w) * kTokBufBytes + static_cast<uint32_t>(lane) * 128u;
    uint32_t chunk_addr[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) chunk_addr[j] = dec_row + ((static_cast<uint32_t>(j) ^ r7) << 4);
    const uint32_t my_empty = dec_empty + 8 * w;
    const uint32_t my_full_leader = mapa(dec_full, 0) + 8 * w;
    uint32_t n = 0;
    bool ok = true;
    for (int u = pair; u < total_units && ok; u += num_pairs) {
      const Unit un = unit_of(p, u);
      const int64_t tok = static_cast<int64_t>(un.tok0) + rank * (un.T >> 1) + lane;      // this lane's token row
      const bool active = un.tiles != 1 && lane < (un.T >> 1) && tok < p.tok_rows;
      const uint32_t* src = p.tok_units + (tok * p.upr + static_cast<int64_t>(un.kc0) * kRawUnits + w) * kUnitWords;
      uint32_t W[9];
      if (active) {
#pragma unroll
        for (int i = 0; i < 9; ++i) W[i] = __ldg(src + i);
      }
      for (int kc = un.kc0; kc < un.kc1 && ok; ++kc, ++n) {
        uint32_t Wn[9];
        const bool more = active && kc + 1 < un.kc1;          // the next chunk's unit is requested before this one is decoded
        if (more) {
#pragma unroll
          for (int i = 0; i < 9; ++i) Wn[i] = __ldg(src + (kc + 1 - un.kc0) * (kRawUnits * kUnitWords) + i);
        }
        if (!(ok = __all_sync(0xFFFFFFFFu, mbar_wait(my_empty, (n & 1u) ^ 1u, abort_flag, 32)))) break;
        if (active) decode_unit_balanced(W[0], &W[1], chunk_addr, 0u, lut, p.mul);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(my_full_leader);
        if (more) {
#pragma unroll
          for (int i = 0; i < 9; ++i) W[i] = Wn[i];
        }
      }
    }
  } else {
    // ---------------------------------------------------------------- decode
    const int d = threadIdx.x - kDecodeWarp0 * 32;            // 0..511
    const int h = d >> 8;                                     // which unit pair of the raw chunk
    const int row = d & 255;                                  // 0..127 weight rows, 128..255 token rows
    const uint32_t r7 = static_cast<uint32_t>(row) & 7u;
    const uint32_t raw_row = static_cast<uint32_t>(row) * kRawRowBytes + static_cast<uint32_t>(h) * 64u;
    const uint32_t dec_row = dec_base + static_cast<uint32_t>(2 * h) * kDecStageBytes + static_cast<uint32_t>(row) * 128u;
    uint32_t chunk_addr[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) chunk_addr[j] = dec_row + ((static_cast<uint32_t>(j) ^ r7) << 4);
    const uint32_t dec_empty0 = dec_empty + 16 * h;
    const uint32_t dec_full0_leader = mapa(dec_full, 0) + 16 * h;
    uint32_t n = 0;
    bool ok = true;
    for (int u = pair; u < total_units && ok; u += num_pairs) {
      const Unit un = unit_of(p, u);
      const bool active = row < 128 || un.tiles != 1 || (row - 128) < (un.T >> 1);    // small-tile mode: rows 128.. are weight rows too
      for (int kc = un.kc0; kc < un.kc1 && ok; ++kc, ++n) {
        const uint32_t s = n & 1u, ph = (n >> 1) & 1u;
        if (!(ok = __all_sync(0xFFFFFFFFu, mbar_wait(raw_full + 8 * s, ph, abort_flag)))) break;
        uint32_t L[20];
        const uint32_t src = raw_base + s * kRawStageBytes + raw_row;
#pragma unroll
        for (int i = 0; i < 5; ++i) {
          const uint4 v = lds128(src + 16 * i);
          L[4 * i] = v.x; L[4 * i + 1] = v.y; L[4 * i + 2] = v.z; L[4 * i + 3] = v.w;
        }
        fence_proxy_async_smem();                // reads ordered before the async proxy refills the stage
        mbar_arrive(raw_empty + 8 * s);
        // one copy of the decoder for both halves: units 2h, 2h+1 start at word 0 or 2 of the window
        uint32_t W[18];
#pragma unroll
        for (int i = 0; i < 18; ++i) W[i] = h ? L[i + 2] : L[i];
        ok = decode_two_units_g(W, active, chunk_addr, lut, p.mul, dec_empty0, dec_full0_leader, (n & 1u) ^ 1u, abort_flag);
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  if (*abort_flag) {
    const uint64_t t0 = global_ns();
    while (global_ns() - t0 < 2000000ull) {}     // let copies and MMAs that are still in flight land
    if (threadIdx.x == 0) atomicExch(p.error_word, 1u);
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();            // neither CTA leaves while the other may still read its shared memory or arrive on its barriers
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// FP32 view of C [rows, N] for the epilogue's TMA stores: box = 32 columns x 16 rows.
bool make_c_map_g(CUtensorMap* map, float* C, int64_t rows, int64_t N, int64_t ldc) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ldc) * 4};
  const cuuint32_t box[2] = {32, 16};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, C, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

hif4_status launch_swapped(const void* A, const void* B, int64_t a_rows, int64_t b_rows, GroupedParams p, int64_t K,
                           cudaStream_t st) {
  static uint64_t smem_opt_in = 0, smem_opt_in_staged = 0;
  if (!ensure_dynamic_smem(gemm_tc2g_kernel<false>, kSmemBytes, smem_opt_in) ||
      !ensure_dynamic_smem(gemm_tc2g_kernel<true>, kSmemBytesStaged, smem_opt_in_staged))
    return HIF4_ERR_CUDA;
  CUtensorMap tmTok, tmW;
  const int64_t upr = K / kUnitElems;
  if (!make_unit_map(&tmTok, A, a_rows, upr, 128) || !make_unit_map(&tmW, B, b_rows, upr, kWRows)) return HIF4_ERR_CUDA;
  p.num_kc = static_cast<int>(K / (kRawUnits * kUnitElems));
  p.upr = upr;
  p.n_wtiles = static_cast<int>(ceil_div64(p.N, 256));
  p.error_word = device_error_word();
  if (!p.error_word) return HIF4_ERR_CUDA;
  p.mul = make_decode_mul();
  if (p.slices < 1) p.slices = 1;
  const int64_t units = static_cast<int64_t>(p.max_entries) * p.n_wtiles * p.slices;
  if (units > 0x7FFFFFFFll) return HIF4_ERR_SHAPE;
  const int pairs = static_cast<int>(units < sm_count() / 2 ? units : sm_count() / 2);
  // The staged epilogue where it pays (ncu durations, staged against plain stores).  A dense problem has about one
  // record per pair, so its epilogue is not hidden behind a next main loop: M = 128, N = K = 4096 30.9 vs 33.3 us,
  // N = 14336 38.0 vs 41.1 us, M = 64 36.3 vs 37.4 us.  A grouped problem hides the epilogue and gains only while its
  // instructions weigh against a short main loop: K = 2048 -12 %, K = 2560 -4.6 %, K = 3072 equal, K = 4096 +1 %,
  // K = 5120 +2 %, K = 7168 +3 to +6 % (the staging adds to the shared-memory pipe, which the main loop owns there).
  // The TMA stores need a C that a tensor map can describe; a TMA store clips the innermost dimension in 16-byte pieces,
  // so N must be a multiple of four columns.
  if (p.table == nullptr || ceil_div64(p.num_kc, p.slices) <= 10) {
    EpilogueArgs<true> epi;
    epi.tmC = tmW;                                    // placeholder when the store path is not used
    epi.tma_store = ((reinterpret_cast<uintptr_t>(p.C) & 15u) == 0 && p.ldc % 4 == 0 && p.N % 4 == 0 && a_rows < (1ll << 31) &&
                     make_c_map_g(&epi.tmC, p.C, a_rows, p.N, p.ldc)) ? 1 : 0;
    gemm_tc2g_kernel<true><<<2 * pairs, kThreads, kSmemBytesStaged, st>>>(tmTok, tmW, p, epi);
  } else {
    gemm_tc2g_kernel<false><<<2 * pairs, kThreads, kSmemBytes, st>>>(tmTok, tmW, p, EpilogueArgs<false>{});
  }
  note_launch();
  return launch_status();
}

}  // namespace

// K slices of a dense problem with few rows.  All slices of all weight tiles must be resident at once (they wait
// for one another), and a slice starts its epilogue when the one before it has finished its own, which costs
// about the time of 3.5 K = 256 chunks per extra slice: take the count with the shortest critical path, at most 4.
static int swapped_slices(int64_t N, int64_t K) {
  const int64_t tiles = ceil_div64(N, 256), pairs = sm_count() / 2, chunks = K / 256;
  int64_t s_max = tiles > 0 ? pairs / tiles : 1;
  if (s_max > 4) s_max = 4;
  int64_t best = 1, best_cost = 2 * chunks;
  for (int64_t s = 2; s <= s_max; ++s) {
    const int64_t cost = 2 * ceil_div64(chunks, s) + 7 * (s - 1);       // in half chunks
    if (cost < best_cost) { best = s; best_cost = cost; }
  }
  return static_cast<int>(best);
}

size_t gemm_tc2_swapped_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  if (M <= 0 || N <= 0 || K <= 0 || K % 256 != 0) return 0;
  const int s = swapped_slices(N, K);
  return s > 1 ? static_cast<size_t>((ceil_div64(N, 256) * s * 8 * sizeof(unsigned int) + 255) / 256 * 256) : 0;
}

// Dense problem with few rows (M <= 128): the same kernel with a single token tile.
hif4_status launch_gemm_tc2_swapped(const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K,
                                    int64_t ldc, void* workspace, size_t workspace_bytes, cudaStream_t st) {
  GroupedParams p{};
  p.C = C; p.ldc = ldc; p.N = N;
  p.max_entries = 1;
  p.table = nullptr;
  p.dense_rows = static_cast<int>(M);
  p.slices = swapped_slices(N, K);
  if (p.slices > 1) {
    const size_t need = gemm_tc2_swapped_workspace_bytes(M, N, K);
    if (!workspace || workspace_bytes < need) return HIF4_ERR_WORKSPACE;
    p.flags = static_cast<unsigned int*>(workspace);
    if (cudaMemsetAsync(p.flags, 0, need, st) != cudaSuccess) return HIF4_ERR_CUDA;
  }
  return launch_swapped(A, B, M, N, p, K, st);
}

size_t grouped_tc2_workspace_bytes(int num_groups, int64_t total_rows, int64_t N) {
  const int64_t max_records = (ceil_div64(total_rows, kMaxTok) + num_groups) * ceil_div64(N, 256);
  return static_cast<size_t>((kTableHeaderBytes + max_records * static_cast<int64_t>(sizeof(WorkRec)) + 255) / 256 * 256);
}

hif4_status launch_grouped_gemm_tc2(const void* A, const void* B, float* C, const int64_t* offsets, int num_groups,
                                    int64_t total_rows, int64_t N, int64_t K, int64_t ldc, void* workspace,
                                    cudaStream_t st) {
  const int n_wtiles = static_cast<int>(ceil_div64(N, 256));
  const int64_t max_records = (ceil_div64(total_rows, kMaxTok) + num_groups) * n_wtiles;
  if (max_records > 0x7FFFFFFFll) return HIF4_ERR_SHAPE;
  uint8_t* table_mem = static_cast<uint8_t*>(workspace);
  build_work_table_kernel<<<kTableBlocks, 256, 0, st>>>(offsets, num_groups, N, n_wtiles, table_mem, static_cast<int>(max_records));
  note_launch();
  if (cudaGetLastError() != cudaSuccess) return HIF4_ERR_CUDA;
  GroupedParams p{};
  p.C = C; p.ldc = ldc; p.N = N;
  p.max_entries = static_cast<int>(max_records / n_wtiles);
  p.table = reinterpret_cast<const WorkRec*>(table_mem + kTableHeaderBytes);
  p.table_count = reinterpret_cast<const int*>(table_mem);
  p.tok_units = static_cast<const uint32_t*>(A);
  p.tok_rows = total_rows;
  return launch_swapped(A, B, total_rows, static_cast<int64_t>(num_groups) * N, p, K, st);
}

}  // namespace hif4
