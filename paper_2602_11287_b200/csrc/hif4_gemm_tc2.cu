// Tensor-core HiF4 x HiF4 -> FP32 GEMM for sm_100a on CTA pairs: C = A * B^T (Eq. 3 summed over unit
// pairs), 256 x 256 output tile per pair of SMs (tcgen05.mma cta_group::2).
//
// Same arithmetic as the single-CTA kernel (every HiF4 value, level-1 scale included, is exactly a
// BF16; products are exact in the FP32 accumulator), different work split.  The cost that bounds
// this GEMM is the decode of packed units into BF16 operand tiles on the CUDA cores; a 128 x 256 tile
// on one SM decodes 128 + 256 rows per 64-wide K block, a 256 x 256 tile on two SMs only 128 + 128 rows
// per SM for the same tensor work per SM.  Cluster of two CTAs, rank r:
//   warp 0       TMA producer: raw units of A rows [m0 + 128 r, +128) and B rows [n0 + 128 r, +128),
//                4 units (K = 256, 144 bytes) per row per stage, two stages; each CTA fetches its own rows
//   warps 6-21   decode: 512 threads = 256 tile rows x 2; thread (row, h) loads 80 bytes of the row's
//                raw chunk and decodes units 2h and 2h+1 (Eq. 2) into K-major SWIZZLE_128B operand
//                rows of decoded stages 2h and 2h+1 (a K = 64 block each, four stages)
//   warp 1       rank 0 only: issues tcgen05.mma.cta_group::2 (256 x 256 x 16, four per K block), which
//                reads A and B halves from both CTAs' shared memory and accumulates into both CTAs'
//                tensor memory; commits are multicast to the barriers of both CTAs
//   warps 2-5    epilogue: tcgen05.ld of this CTA's 128 accumulator rows, 32 x 16 FP32 slabs staged in
//                shared memory (SWIZZLE_64B) and written to C with TMA stores, which also clip the
//                ragged edges; plain per-thread stores when C is not 16-byte aligned
// Cross-CTA signalling: "decoded stage full" and "accumulator drained" are mbarriers of rank 0 on which
// the warps of both CTAs arrive (one remote arrive per warp after fence.proxy.async); "stage free" and
// "accumulator complete" arrive in both CTAs through the multicast commit.
//
// Every wait on an mbarrier is bounded: when the budget runs out the CTA raises an error word, every
// role leaves its loop, both CTAs meet at the final cluster barrier, tensor memory is released and
// the kernel returns.
#include "hif4_common.cuh"
#include "hif4_gemm_internal.cuh"
#include "hif4_quantize_device.cuh"
#include "hif4_tc_common.cuh"
#include "hif4_tc2_common.cuh"

namespace hif4 {
namespace {

constexpr int kPairM = 256, kPairN = 256;             // output tile of a CTA pair
constexpr int kRows = 128;                            // A rows and B rows per CTA
constexpr int kRawHalfBytes = kRows * kRawRowBytes;   // 18432
constexpr int kRawStageBytes = 2 * kRawHalfBytes;     // A rows then B rows
constexpr int kDecHalfBytes = kRows * 128;            // 128 rows x 64 BF16
constexpr int kDecStageBytes = 2 * kDecHalfBytes;
constexpr int kRawStages = 2;
constexpr int kDecStages = 4;                         // one per unit of a raw chunk
constexpr int kTmemCols = 512;                        // two 256-column accumulators

constexpr int kDecodeWarp0 = 6;
constexpr int kDecodeThreads = 4 * kRows;             // 512: (A rows + B rows) x 2 unit pairs
constexpr int kThreads = kDecodeWarp0 * 32 + kDecodeThreads;   // 704

constexpr int kEpiCols = 16;                          // FP32 columns per staged slab (64-byte rows)
constexpr int kEpiSlabBytes = 32 * kEpiCols * 4;      // 32 rows of one epilogue warp: 2048
constexpr int kEpiBytes = 4 * 2 * kEpiSlabBytes;      // 4 warps x 2 buffers
constexpr int kSmemBytes = 1024 /*alignment slack*/ + kDecStages * kDecStageBytes + kRawStages * kRawStageBytes + kEpiBytes +
                           256 /*barriers*/ + 1024 /*spread table*/;

// tcgen05.mma kind::f16 instruction descriptor: D = F32, A = B = BF16, both K-major, N/8, M/16.
constexpr uint32_t kInstrDesc2 = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kPairN >> 3) << 17) |
                                 (static_cast<uint32_t>(kPairM >> 4) << 24);

struct Gemm2Params {
  float* C;
  int64_t ldc;
  int64_t M;
  int64_t N;
  int num_kc;           // K / 256
  int n_tiles;          // ceil(N / 256)
  int total_tiles;
  unsigned int* error_word;
  int tma_store;        // 1: C goes out through the tensor map tmC, 0: per-thread stores
  // Tile schedule: every pair computes `full_rounds` whole tiles.  Fewer tiles than pairs (full_rounds == 0): the
  // `tail_tiles` tiles are cut into `slices` K ranges each, on pairs of their own, so that the single round
  // keeps tail_tiles * slices pairs busy instead of tail_tiles.  Slice 0 of a tile stores its part to C,
  // slice s > 0 adds its part with TMA reduce-add stores once slice s - 1 has finished the same rows
  // (warp to warp: an epilogue warp owns 32 rows of the tile), so every element is summed in slice order.
  int full_rounds;
  int tail_tiles;
  int slices;               // 1: tail tiles are not split
  // Balanced last rounds (sk_tiles > 0; then tail_tiles is 0 and slices is 2): after `full_rounds` whole tiles per
  // pair, the K = 256 chunks of the remaining `sk_tiles` tiles (between one and two per pair, starting at tile
  // `sk_tile0`), laid end to end, are dealt out in equal contiguous runs.  A run begins with the last chunks of a
  // tile whose first chunks end the previous pair's run: the pair that has the end of a tile computes it first and
  // stores it (slice 0, flag row = the index of its run), the pair that has the beginning computes it last and adds
  // (slice 1), so the addition hardly ever waits.
  int sk_tiles;
  int sk_tile0;
  unsigned int* flags;      // [tail_tiles or pairs + 1][slices][8]: "this epilogue warp's rows of this slice are in C" (zero at launch)
  DecodeMul mul;
  // Fused activation conversion (kFusedA): the A operand is not packed units but BF16 activations [M, K], row stride
  // ld_x elements; the A-side decode threads run Algorithm 1 on the two units they are about to decode.
  const uint16_t* x;
  int64_t ld_x;
};

constexpr int kMaxSlices = 4;

struct WorkItem {
  int m0, n0;           // tile origin
  int kc0, kc1;         // K = 256 chunks [kc0, kc1)
  int tail;             // index among the tail tiles, -1 for a whole tile
  int slice;            // K slice of a tail tile
};
// First and last chunk (exclusive) of a pair's run in the balanced rounds, in chunks of the sk_tiles tiles laid end to
// end.  The runs go to the pairs in descending order (`run` = num_pairs - 1 - pair), so that the pair that waits
// for its neighbour's part of a shared tile has the higher index: CTAs are handed out in index order, and a
// grid that is only partly resident still cannot wait for a CTA that has not started.
__device__ __forceinline__ int balanced_run(const Gemm2Params& p, int pair, int num_pairs, int64_t& c0, int64_t& c1) {
  const int64_t total = static_cast<int64_t>(p.sk_tiles) * p.num_kc;
  const int run = num_pairs - 1 - pair;
  c0 = total * run / num_pairs;
  c1 = total * (run + 1) / num_pairs;
  return run;
}
__device__ __forceinline__ int num_work_items(const Gemm2Params& p, int pair, int num_pairs) {
  if (p.sk_tiles > 0) {
    int64_t c0, c1;
    balanced_run(p, pair, num_pairs, c0, c1);
    return p.full_rounds + static_cast<int>((c1 - 1) / p.num_kc - c0 / p.num_kc) + 1;
  }
  return p.full_rounds + (pair < p.tail_tiles * p.slices ? 1 : 0);
}
__device__ __forceinline__ WorkItem work_item(const Gemm2Params& p, int pair, int num_pairs, int i) {
  WorkItem w;
  int t;
  if (i < p.full_rounds) {
    t = i * num_pairs + pair;
    w.kc0 = 0; w.kc1 = p.num_kc; w.tail = -1; w.slice = 0;
  } else if (p.sk_tiles > 0) {
    int64_t c0, c1;
    const int run = balanced_run(p, pair, num_pairs, c0, c1);
    const int64_t tr = c0 / p.num_kc + (i - p.full_rounds);
    const int64_t first = tr * p.num_kc;
    w.kc0 = c0 > first ? static_cast<int>(c0 - first) : 0;
    w.kc1 = c1 < first + p.num_kc ? static_cast<int>(c1 - first) : p.num_kc;
    t = p.sk_tile0 + static_cast<int>(tr);
    if (w.kc0 > 0) { w.tail = run; w.slice = 0; }                        // end of a tile: computed first, stored
    else if (w.kc1 < p.num_kc) { w.tail = run + 1; w.slice = 1; }        // beginning of a tile: computed last, added
    else { w.tail = -1; w.slice = 0; }
  } else {
    w.tail = pair % p.tail_tiles;
    w.slice = pair / p.tail_tiles;
    t = p.full_rounds * num_pairs + w.tail;
    w.kc0 = static_cast<int>(static_cast<int64_t>(w.slice) * p.num_kc / p.slices);
    w.kc1 = static_cast<int>(static_cast<int64_t>(w.slice + 1) * p.num_kc / p.slices);
  }
  const int mt = t / p.n_tiles;
  w.m0 = mt * kPairM;
  w.n0 = (t - mt * p.n_tiles) * kPairN;
  return w;
}

// Bounded wait until a word in global memory, written by another CTA after a __threadfence(), has reached
// `want`.  Returns false when the budget ran out or another thread has already given up.
__device__ __noinline__ bool wait_count(const unsigned int* counter, unsigned int want, volatile uint32_t* abort_flag) {
  const uint64_t t0 = global_ns();
  for (uint32_t it = 1;; ++it) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
    if (v >= want) return true;
    __nanosleep(128);
    if ((it & 63u) == 0u) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > kWaitBudgetNs) {
        *abort_flag = 1u;
        return false;
      }
    }
  }
}

// Decodes the two units held in raw words W[0..8] and W[9..17] into decoded stages 2h and 2h+1.  Returns
// false when a wait gave up.
__device__ __forceinline__ bool decode_two_units(const uint32_t (&W)[18], const uint32_t (&chunk_addr)[8], uint32_t lut,
                                                 const DecodeMul& mul, uint32_t dec_empty0, uint32_t dec_full0_leader,
                                                 uint32_t parity_free, volatile uint32_t* abort_flag) {
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    // warp-uniform outcome, so that the warp barrier below is never reached by a part of the warp
    if (!__all_sync(0xFFFFFFFFu, mbar_wait(dec_empty0 + 8 * u, parity_free, abort_flag))) return false;
    decode_unit_balanced(W[9 * u], &W[9 * u + 1], chunk_addr, u * kDecStageBytes, lut, mul);
    fence_proxy_async_smem();                  // generic-proxy writes -> visible to the tensor core
    // One remote arrive per warp; the warp barrier orders the other lanes' writes and proxy fences
    // before it.
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive_cluster(dec_full0_leader + 8 * u);
  }
  return true;
}

template <bool kFusedA>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ CUtensorMap tmC, const Gemm2Params p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t dec_base = smem_base;                                        // 1024-byte aligned stages
  const uint32_t raw_base = dec_base + kDecStages * kDecStageBytes;
  const uint32_t epi_base = raw_base + kRawStages * kRawStageBytes;          // 1024-byte aligned as well
  const uint32_t bar_base = epi_base + kEpiBytes;
  // barriers (8 bytes each)
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
  const int n_items = num_work_items(p, pair, num_pairs);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kRawStages; ++s) {
      mbar_init(raw_full + 8 * s, 1);
      mbar_init(raw_empty + 8 * s, kDecodeThreads);
    }
    for (int s = 0; s < kDecStages; ++s) {
      mbar_init(dec_full + 8 * s, kDecodeThreads / 32);   // 8 warps of each CTA per stage (used on rank 0)
      mbar_init(dec_empty + 8 * s, 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(tmem_full + 8 * s, 1);
      mbar_init(tmem_empty + 8 * s, 8);               // 4 epilogue warps of each CTA (used on rank 0)
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
      for (int i = 0; i < n_items && ok; ++i) {
        const WorkItem w = work_item(p, pair, num_pairs, i);
        for (int kc = w.kc0; kc < w.kc1; ++kc, ++n) {
          const uint32_t s = n & 1u, ph = (n >> 1) & 1u;
          if (!(ok = mbar_wait(raw_empty + 8 * s, ph ^ 1u, abort_flag, 128))) break;
          mbar_expect_tx(raw_full + 8 * s, kFusedA ? kRawHalfBytes : kRawStageBytes);
          const uint32_t dst = raw_base + s * kRawStageBytes;
          if (!kFusedA) tma_load_2d(dst, &tmA, kc * kRawRowBytes, w.m0 + static_cast<int>(rank) * kRows, raw_full + 8 * s);
          tma_load_2d(dst + kRawHalfBytes, &tmB, kc * kRawRowBytes, w.n0 + static_cast<int>(rank) * kRows,
                      raw_full + 8 * s);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer (rank 0 only)
    if (rank == 0 && lane == 0) {
      uint32_t n = 0, tcount = 0;
      bool ok = true;
      for (int it = 0; it < n_items && ok; ++it, ++tcount) {
        const WorkItem w = work_item(p, pair, num_pairs, it);
        const uint32_t acc = tcount & 1u, aph = (tcount >> 1) & 1u;
        if (!(ok = mbar_wait_cluster(tmem_empty + 8 * acc, aph ^ 1u, abort_flag))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * kPairN;
        for (int kc = w.kc0; kc < w.kc1 && ok; ++kc, ++n) {
          // The two halves of the decode threads fill stages (0, 1) and (2, 3) side by side, so stages
          // 0 and 2 are ready first: the K blocks of a chunk are consumed in the order 0, 2, 1, 3.
#pragma unroll
          for (int i = 0; i < kDecStages; ++i) {
            const int u = ((i & 1) << 1) | (i >> 1);
            if (!(ok = mbar_wait_cluster(dec_full + 8 * u, n & 1u, abort_flag))) break;
            tc_fence_after();
            const uint64_t adesc = make_desc(dec_base + u * kDecStageBytes);
            const uint64_t bdesc = make_desc(dec_base + u * kDecStageBytes + kDecHalfBytes);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              tc2_mma(d_tmem, adesc + 2 * kk, bdesc + 2 * kk, kInstrDesc2, ((kc - w.kc0) | i | kk) != 0 ? 1u : 0u);
            tc2_commit_both(dec_empty + 8 * u);       // both CTAs may overwrite the stage once these MMAs have read it
          }
        }
        if (!ok) break;
        tc2_commit_both(tmem_full + 8 * acc);         // accumulator complete, in both CTAs
      }
    }
  } else if (warp < kDecodeWarp0) {
    // ---------------------------------------------------------------- epilogue
    const int q = warp & 3;                      // TMEM lane quadrant this warp may read
    const uint32_t tmem_empty_leader = mapa(tmem_empty, 0);
    uint32_t tcount = 0;
    if (p.tma_store) {
      // Slab = this warp's 32 rows x 16 columns, 64-byte rows, 16-byte chunk c of row r stored at chunk
      // c ^ ((r >> 1) & 3) (SWIZZLE_64B): conflict-free 128-bit stores, and the TMA store undoes it.
      const uint32_t slab0 = epi_base + static_cast<uint32_t>(q) * (2 * kEpiSlabBytes);
      const uint32_t my_row = slab0 + static_cast<uint32_t>(lane) * 64u;
      const uint32_t sw = (static_cast<uint32_t>(lane) >> 1) & 3u;
      uint32_t slabs = 0;
      for (int it = 0; it < n_items; ++it, ++tcount) {
        const WorkItem w = work_item(p, pair, num_pairs, it);
        const uint32_t acc = tcount & 1u, aph = (tcount >> 1) & 1u;
        if (!__all_sync(0xFFFFFFFFu, mbar_wait(tmem_full + 8 * acc, aph, abort_flag, 256))) break;
        tc_fence_after();
        // K-sliced tail tile: slice 0 stores, slice s > 0 adds once the same warp of slice s - 1 is done
        const bool sliced = w.tail >= 0 && p.slices > 1;
        const bool adds = sliced && w.slice > 0;
        unsigned int* my_flag = sliced ? p.flags + (static_cast<size_t>(w.tail) * p.slices + w.slice) * 8 + rank * 4 + q : nullptr;
        if (adds && !__all_sync(0xFFFFFFFFu, wait_count(my_flag - 8, 1u, abort_flag))) break;
        const int row0 = w.m0 + static_cast<int>(rank) * kRows + q * 32;
#pragma unroll 1
        for (int c = 0; c < kPairN / kEpiCols; ++c) {
          // slabs that lie entirely outside C are neither read nor staged: the two staging buffers
          // alternate over the slabs that are stored, which is what the wait below counts on
          const bool stored = row0 < p.M && w.n0 + c * kEpiCols < p.N;             // same for the whole warp
          uint32_t r[16];
          if (stored) {
            tc_ld16(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * kPairN + c * kEpiCols, r);
            tc_wait_ld();
          }
          if (c == kPairN / kEpiCols - 1) {          // accumulator fully read: hand it back before the stores
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(tmem_empty_leader + 8 * acc);
          }
          if (!stored) continue;
          const uint32_t buf = (slabs & 1u) * kEpiSlabBytes;
          if (lane == 0) bulk_wait_read<1>();        // the store that used this buffer two slabs ago has read it
          __syncwarp();
#pragma unroll
          for (int v = 0; v < 4; ++v)
            sts128(my_row + buf + ((static_cast<uint32_t>(v) ^ sw) << 4), r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
          fence_proxy_async_smem();                  // generic-proxy writes -> visible to the TMA store
          __syncwarp();
          if (lane == 0) {
            if (adds) tma_reduce_add_2d(&tmC, w.n0 + c * kEpiCols, row0, slab0 + buf);
            else tma_store_2d(&tmC, w.n0 + c * kEpiCols, row0, slab0 + buf);
            bulk_commit();
          }
          ++slabs;
        }
        if (sliced && w.slice + 1 < p.slices && lane == 0) {      // the next slice may add to these rows now
          bulk_wait_all();
          __threadfence();
          asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(my_flag), "r"(1u) : "memory");
        }
      }
      if (lane == 0) bulk_wait_all();                // shared memory stays valid until the last store has read it
    } else {
      const bool vec_ok = ((reinterpret_cast<uintptr_t>(p.C) & 15u) == 0) && (p.ldc % 4 == 0);
      for (int it = 0; it < n_items; ++it, ++tcount) {         // (tail tiles are never K-sliced on this path)
        const WorkItem w = work_item(p, pair, num_pairs, it);
        const uint32_t acc = tcount & 1u, aph = (tcount >> 1) & 1u;
        if (!__all_sync(0xFFFFFFFFu, mbar_wait(tmem_full + 8 * acc, aph, abort_flag, 256))) break;
        tc_fence_after();
        const int64_t row = static_cast<int64_t>(w.m0) + rank * kRows + q * 32 + lane;
        const bool row_ok = row < p.M;
        float* crow = p.C + row * p.ldc + w.n0;
#pragma unroll 1
        for (int c = 0; c < kPairN / 32; ++c) {
          uint32_t r[32];
          tc_ld32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * kPairN + c * 32, r);
          tc_wait_ld();
          const int64_t col0 = static_cast<int64_t>(w.n0) + c * 32;
          if (row_ok && col0 < p.N) {
            if (vec_ok && col0 + 32 <= p.N) {
#pragma unroll
              for (int v = 0; v < 8; ++v)
                *reinterpret_cast<uint4*>(crow + c * 32 + 4 * v) = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
            } else {
#pragma unroll
              for (int v = 0; v < 32; ++v)
                if (col0 + v < p.N) crow[c * 32 + v] = __uint_as_float(r[v]);
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(tmem_empty_leader + 8 * acc);
      }
    }
  } else {
    // ---------------------------------------------------------------- decode
    const int d = threadIdx.x - kDecodeWarp0 * 32;            // 0..511
    const int h = d >> 8;                                     // which unit pair of the raw chunk
    const int row = d & 255;                                  // 0..127 A rows, 128..255 B rows
    const uint32_t r7 = static_cast<uint32_t>(row) & 7u;
    // bytes [0, 80) of the row chunk hold units 0 and 1, bytes [64, 144) units 2 and 3
    const uint32_t raw_row = static_cast<uint32_t>(row) * kRawRowBytes + static_cast<uint32_t>(h) * 64u;
    const uint32_t dec_row = dec_base + static_cast<uint32_t>(2 * h) * kDecStageBytes + static_cast<uint32_t>(row) * 128u;
    uint32_t chunk_addr[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) chunk_addr[j] = dec_row + ((static_cast<uint32_t>(j) ^ r7) << 4);
    const uint32_t dec_empty0 = dec_empty + 16 * h;
    const uint32_t dec_full0_leader = mapa(dec_full, 0) + 16 * h;
    uint32_t n = 0;
    bool ok = true;
    for (int i = 0; i < n_items && ok; ++i) {
      const WorkItem w = work_item(p, pair, num_pairs, i);
      for (int kc = w.kc0; kc < w.kc1 && ok; ++kc, ++n) {
        const uint32_t s = n & 1u, ph = (n >> 1) & 1u;
        if (kFusedA && row < kRows) {
          // A rows: 128 BF16 activations of this row (units 2h, 2h+1 of the chunk) from global memory, converted with
          // Algorithm 1 (round-half-to-even) by this thread, then decoded like packed units.  Rows past M read as zeros.
          const int64_t gr = static_cast<int64_t>(w.m0) + rank * kRows + row;
          uint32_t W[18];
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            uint4 v[8];
            if (gr < p.M) {
              const uint4* src = reinterpret_cast<const uint4*>(p.x + gr * p.ld_x + static_cast<int64_t>(kc) * 256 + (2 * h + u) * 64);
#pragma unroll
              for (int g = 0; g < 8; ++g) v[g] = __ldg(src + g);
            } else {
#pragma unroll
              for (int g = 0; g < 8; ++g) v[g] = make_uint4(0u, 0u, 0u, 0u);
            }
            uint32_t codes[8], meta;
            encode_unit_bf16_single<false>(v, codes, meta);
            W[9 * u] = meta;
#pragma unroll
            for (int g = 0; g < 8; ++g) W[9 * u + 1 + g] = codes[g];
          }
          // the raw stage holds only B rows here, but its barriers are shared by all decode threads
          if (!(ok = __all_sync(0xFFFFFFFFu, mbar_wait(raw_full + 8 * s, ph, abort_flag)))) break;
          mbar_arrive(raw_empty + 8 * s);
          ok = decode_two_units(W, chunk_addr, lut, p.mul, dec_empty0, dec_full0_leader, (n & 1u) ^ 1u, abort_flag);
          continue;
        }
        if (!(ok = __all_sync(0xFFFFFFFFu, mbar_wait(raw_full + 8 * s, ph, abort_flag)))) break;
        uint32_t L[20];
        const uint32_t src = raw_base + s * kRawStageBytes + raw_row;
#pragma unroll
        for (int i = 0; i < 5; ++i) {
          const uint4 v = lds128(src + 16 * i);
          L[4 * i] = v.x; L[4 * i + 1] = v.y; L[4 * i + 2] = v.z; L[4 * i + 3] = v.w;
        }
        // The stage is refilled through the async proxy (TMA) while it was read through the generic
        // proxy: the proxy fence orders these reads before the release.
        fence_proxy_async_smem();
        mbar_arrive(raw_empty + 8 * s);
        // units 2h, 2h+1 start at word 0 (h = 0) or 2 (h = 1) of the loaded window; one copy of the decoder
        // serves both halves (two copies run side by side cost instruction-cache misses)
        uint32_t W[18];
#pragma unroll
        for (int i = 0; i < 18; ++i) W[i] = h ? L[i + 2] : L[i];
        ok = decode_two_units(W, chunk_addr, lut, p.mul, dec_empty0, dec_full0_leader, (n & 1u) ^ 1u, abort_flag);
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  if (*abort_flag) {
    // Some wait gave up: give copies and MMAs that are still in flight time to land before the
    // shared and tensor memory they target is released.
    const uint64_t t0 = global_ns();
    while (global_ns() - t0 < 2000000ull) {}
    if (threadIdx.x == 0) atomicExch(p.error_word, 1u);
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();            // neither CTA leaves while the other may still read its shared memory or arrive on its barriers
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// FP32 view of C for the TMA stores of the epilogue: box = 16 columns x 32 rows, SWIZZLE_64B.
bool make_c_map(CUtensorMap* map, float* C, int64_t M, int64_t N, int64_t ldc) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(M)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ldc) * 4};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(kEpiCols), 32};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, C, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Tile schedule of the dense pair kernel for this shape on this device (see Gemm2Params).
struct Tc2Plan {
  int pairs, full_rounds, tail_tiles, slices, sk_tiles, sk_tile0;
  size_t flag_bytes, bytes;          // workspace: the slices' completion words
};
static Tc2Plan tc2_plan(int64_t M, int64_t N, int64_t K) {
  Tc2Plan pl{};
  const int64_t tiles = ceil_div64(M, kPairM) * ceil_div64(N, kPairN);
  const int64_t max_pairs = sm_count() / 2;
  pl.pairs = static_cast<int>(tiles < max_pairs ? tiles : max_pairs);
  pl.slices = 1;
  if (pl.pairs <= 0 || tiles > 0x7FFFFFFFll) return pl;
  pl.full_rounds = static_cast<int>(tiles / pl.pairs);
  pl.tail_tiles = static_cast<int>(tiles % pl.pairs);
  if (tiles < max_pairs) {            // a single, partial round: all its tiles are "tail" tiles
    pl.full_rounds = 0;
    pl.tail_tiles = static_cast<int>(tiles);
  }
  if (pl.tail_tiles > 0) {
    // Slice s starts its epilogue when slice s - 1 has finished its own, which adds about the time of
    // 3.5 K = 256 chunks per extra slice (measured): take the slice count with the shortest critical path.
    int64_t s_max = max_pairs / pl.tail_tiles;
    if (s_max > kMaxSlices) s_max = kMaxSlices;
    const int64_t chunks = K / 256;
    int64_t best = 1, best_cost = 2 * chunks;
    for (int64_t s = 2; s <= s_max; ++s) {
      const int64_t cost = 2 * ceil_div64(chunks, s) + 7 * (s - 1);       // in half chunks
      if (cost < best_cost) { best = s; best_cost = cost; }
    }
    pl.slices = static_cast<int>(best);
  }
  if (pl.full_rounds >= 1 && pl.tail_tiles > 0) {
    // Several rounds and a partial one: the last whole round and the partial one are balanced chunk by chunk
    // instead (every pair then works tail_tiles / pairs of a tile longer than the whole rounds take, which is never
    // more than the K slices of the partial round alone would cost).
    pl.full_rounds -= 1;
    pl.sk_tile0 = pl.full_rounds * pl.pairs;
    pl.sk_tiles = pl.pairs + pl.tail_tiles;
    pl.tail_tiles = 0;
    pl.slices = 2;
    pl.flag_bytes = (static_cast<size_t>(pl.pairs + 1) * 2 * 8 * sizeof(unsigned int) + 255) / 256 * 256;
    pl.bytes = pl.flag_bytes;
  } else if (pl.slices > 1) {
    pl.flag_bytes = (static_cast<size_t>(pl.tail_tiles) * pl.slices * 8 * sizeof(unsigned int) + 255) / 256 * 256;
    pl.bytes = pl.flag_bytes;
  }
  return pl;
}

size_t gemm_tc2_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  if (M <= 0 || N <= 0 || K <= 0 || K % 256 != 0) return 0;
  return tc2_plan(M, N, K).bytes;
}

bool gemm_tc2_supported(const void* A, const void* B, int64_t M, int64_t N, int64_t K) {
  if (!gemm_tc_supported(A, B, M, N, N, K)) return false;
  return M < (1ll << 31) - kPairM && N < (1ll << 31) - kPairN && sm_count() >= 2;
}

// x != nullptr: the A operand is BF16 activations converted inside the kernel (A is then unused).
static hif4_status launch_gemm_tc2_any(const void* A, const uint16_t* x, int64_t ld_x, const void* B, float* C, int64_t M,
                                       int64_t N, int64_t K, int64_t ldc, void* workspace, size_t workspace_bytes,
                                       cudaStream_t st) {
  static uint64_t smem_opt_in = 0, smem_opt_in_fused = 0;
  if (!(x ? ensure_dynamic_smem(gemm_tc2_kernel<true>, kSmemBytes, smem_opt_in_fused)
          : ensure_dynamic_smem(gemm_tc2_kernel<false>, kSmemBytes, smem_opt_in)))
    return HIF4_ERR_CUDA;
  CUtensorMap tmA, tmB;
  const int64_t upr = K / kUnitElems;
  if (!make_unit_map(&tmB, B, N, upr, kRows)) return HIF4_ERR_CUDA;
  if (x) tmA = tmB;                                   // placeholder: the fused kernel never loads A through TMA
  else if (!make_unit_map(&tmA, A, M, upr, kRows)) return HIF4_ERR_CUDA;
  Gemm2Params p{};
  p.x = x; p.ld_x = ld_x;
  p.C = C; p.ldc = ldc; p.M = M; p.N = N;
  p.num_kc = static_cast<int>(K / (kRawUnits * kUnitElems));
  p.n_tiles = static_cast<int>(ceil_div64(N, kPairN));
  const int64_t tiles = ceil_div64(M, kPairM) * p.n_tiles;
  if (tiles > 0x7FFFFFFFll) return HIF4_ERR_SHAPE;
  p.total_tiles = static_cast<int>(tiles);
  p.error_word = device_error_word();
  if (!p.error_word) return HIF4_ERR_CUDA;
  p.mul = make_decode_mul();
  CUtensorMap tmC = tmA;                              // placeholder when the store path is not used
  // (a TMA store clips the innermost dimension in 16-byte pieces: with N % 4 != 0 it would write up to three columns
  // past N, so such shapes take the per-thread stores)
  p.tma_store = ((reinterpret_cast<uintptr_t>(C) & 15u) == 0 && ldc % 4 == 0 && N % 4 == 0 && make_c_map(&tmC, C, M, N, ldc)) ? 1 : 0;
  const Tc2Plan pl = tc2_plan(M, N, K);
  p.full_rounds = pl.full_rounds;
  p.tail_tiles = pl.tail_tiles;
  p.slices = p.tma_store ? pl.slices : 1;             // the plain-store epilogue cannot add to C
  p.sk_tiles = pl.sk_tiles;
  p.sk_tile0 = pl.sk_tile0;
  if (p.sk_tiles > 0 && !p.tma_store) {               // back to whole tiles: full rounds and an unsliced partial one
    p.full_rounds += 1;
    p.tail_tiles = p.sk_tiles - pl.pairs;
    p.sk_tiles = 0;
  }
  if (p.slices > 1) {
    if (!workspace || workspace_bytes < pl.bytes) return HIF4_ERR_WORKSPACE;
    p.flags = static_cast<unsigned int*>(workspace);
    if (cudaMemsetAsync(p.flags, 0, pl.flag_bytes, st) != cudaSuccess) return HIF4_ERR_CUDA;
  }
  const int pairs = p.full_rounds == 0 && p.sk_tiles == 0 ? p.tail_tiles * p.slices : pl.pairs;      // a single round: one pair per slice
  if (x) gemm_tc2_kernel<true><<<2 * pairs, kThreads, kSmemBytes, st>>>(tmA, tmB, tmC, p);
  else gemm_tc2_kernel<false><<<2 * pairs, kThreads, kSmemBytes, st>>>(tmA, tmB, tmC, p);
  note_launch();
  return launch_status();
}

hif4_status launch_gemm_tc2(const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K, int64_t ldc,
                            void* workspace, size_t workspace_bytes, cudaStream_t st) {
  return launch_gemm_tc2_any(A, nullptr, 0, B, C, M, N, K, ldc, workspace, workspace_bytes, st);
}

hif4_status launch_gemm_tc2_fused_bf16(const void* X, int64_t ld_x, const void* B, float* C, int64_t M, int64_t N, int64_t K,
                                       int64_t ldc, void* workspace, size_t workspace_bytes, cudaStream_t st) {
  return launch_gemm_tc2_any(nullptr, static_cast<const uint16_t*>(X), ld_x, B, C, M, N, K, ldc, workspace, workspace_bytes, st);
}

}  // namespace hif4
