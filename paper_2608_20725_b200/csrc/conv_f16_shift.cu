// fp16-input / fp32-accumulate im2win convolution on the sm_100a tensor cores:
// the "shifted-view" kernel (paper Algorithm 1's GEMM, "TC" variant, with the
// operand staging redesigned around the im2win layout).
//
// In the im2win tensor a strip (n, c, ho) is a row of Wp "columns", column k'
// being the Kh contiguous elements {u}.  The window of output wo is columns
// wo*s .. wo*s + Kw - 1, so for a fixed kernel column v the operand of output
// wo is column wo*s + v: the SAME data as for v = 0, shifted by v columns.
// The kernel therefore stages each column ONCE per channel block,
//     S[row = virtual column][k2 = c*Kh + u]     (64 halves = 128 bytes per row),
// in the k-major 128-byte-swizzled layout, and issues the MMAs of the Kw kernel
// columns against row-shifted views of the same tile: the shared-memory
// descriptor of kernel column v starts (v div s) rows further, inside sub-tile
// (v mod s).  (With stride s the columns are de-interleaved into s sub-tiles,
// sub-tile j holding columns k' = j mod s, which turns the column stride s of
// consecutive outputs into a row stride of 1.)  Every element of the window
// tensor is read from L2/HBM once per output-channel tile and written to shared
// memory once, instead of Kw times as in an im2col-style expansion.
//
// The MMA rows are "virtual positions" q = (n*Ho + ho)*Wq + kq with Wq = ceil(Wp/s):
// q runs over ALL columns of a strip, also the (Wq - Wo) trailing ones that are
// no output; their accumulator rows are computed and dropped.  (When s does not
// divide Wp the last virtual position of a strip lacks some columns; they are
// staged as zeros and only dropped rows read them.)  Tiles are 128
// consecutive q and may span strips and images.  Useful work is Wo/Wq of the
// MMA work (0.97 for 56-wide rows, 0.78 for 7-wide rows).
//
//   GEMM:  acc[q][co] += sum_{k2} S_v[q][k2] * Fp2[v][co][k2]   for v = 0..Kw-1
//
// Roles: 8 producer warps gather S (one 16-byte chunk = 8 k2 per work item, lanes
// on consecutive rows so that global reads are contiguous Kh-element records),
// one warp streams the filter tiles Fp2[v][n0:n0+BN][kb*64:+64] by TMA, one
// thread issues tcgen05.mma and commits to the "empty" mbarriers; afterwards the
// producer warps read the accumulator from tensor memory and store the real
// outputs.  Two rings of stages: S tiles (each used by Kw MMA groups) and
// filter tiles (each used by one).  All mbarrier waits are bounded.
#include <cuda.h>
#include <stdlib.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace im2win {
namespace {

using namespace ptx;

constexpr int TILE_M = 128;
constexpr int KB = kF16KBlock;
constexpr int PRODUCER_WARPS = 8;
constexpr int PRODUCER_THREADS = PRODUCER_WARPS * 32;
constexpr int NUM_THREADS = PRODUCER_THREADS + 64;   // + TMA warp + MMA warp
constexpr int MAX_STAGES = 8;
constexpr int ITEM_GROUP = 5;                        // work items whose loads are issued together

struct ShiftParams {
  const uint16_t* __restrict__ win;
  const int32_t* __restrict__ koff2;   // k2 -> c*chan_stride + u, -1 for padded k2
  float* __restrict__ y;
  uint32_t* status;
  int64_t VQ, img_stride, strip, chan_stride, window_elems;
  int32_t C, N;
  int32_t Wq, Wp, Ho, Wo, HoWo, Co, Kh, Kw, s, num_kb;
  int32_t chunks;         // 16-byte chunks of a row that are staged (8, fewer when one short k-block is all)
  int32_t chunks_last;    // ... of them in the last k-block, = 2 * nks_last
  int32_t nks_last;       // 16-wide MMA steps of the last k-block
  int32_t halo8;          // halo rows of a sub-tile, rounded up to 8
  int32_t nbig;           // the first nbig tiles are 256 positions tall (two MMA halves), the rest 128
  int32_t a_stage_bytes, sa, sb;
};


template <int BN, int ITEMS>
__global__ void __launch_bounds__(NUM_THREADS, (BN <= 128 ? 2 : 1))
conv_f16_shift_kernel(const __grid_constant__ CUtensorMap fmap, ShiftParams q) {
  constexpr int B_STAGE_BYTES = BN * KB * 2;

  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) uint64_t bars[4 * MAX_STAGES + 1];
  __shared__ uint32_t tmem_base_slot;
  __shared__ volatile uint32_t abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t a_ring = smem_u32(smem);
  const uint32_t b_ring = a_ring + q.sa * q.a_stage_bytes;
  const uint32_t a_full0 = smem_u32(&bars[0]);
  const uint32_t a_empty0 = smem_u32(&bars[MAX_STAGES]);
  const uint32_t b_full0 = smem_u32(&bars[2 * MAX_STAGES]);
  const uint32_t b_empty0 = smem_u32(&bars[3 * MAX_STAGES]);
  const uint32_t acc_bar = smem_u32(&bars[4 * MAX_STAGES]);

  // Tall tiles (two 128-row MMA halves sharing every filter stage) come first in the grid.
  const bool big = (int)blockIdx.x < q.nbig;
  const int mt = big ? 2 : 1;
  const int64_t q0 = big ? (int64_t)blockIdx.x * (2 * TILE_M)
                         : (int64_t)q.nbig * (2 * TILE_M) + (int64_t)((int)blockIdx.x - q.nbig) * TILE_M;
  const int n0 = blockIdx.y * BN;
  const int rows = TILE_M * mt + q.halo8;          // rows of one sub-tile
  const int total_rows = q.s * rows;
  const int sub_bytes = rows * 128;

  if (threadIdx.x == 0) {
    abort_flag = 0u;
    for (int i = 0; i < MAX_STAGES; ++i) {
      mbar_init(a_full0 + 8 * i, PRODUCER_WARPS);
      mbar_init(a_empty0 + 8 * i, 1);
      mbar_init(b_full0 + 8 * i, 1);
      mbar_init(b_empty0 + 8 * i, 1);
    }
    mbar_init(acc_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == PRODUCER_WARPS + 1) tmem_alloc(smem_u32(&tmem_base_slot), 2 * BN);
  // k2 -> element offset table of the whole reduction, kept in shared memory
  int32_t* koff_s = reinterpret_cast<int32_t*>(smem + q.sa * q.a_stage_bytes + q.sb * B_STAGE_BYTES);
  for (int i = threadIdx.x; i < q.num_kb * KB; i += NUM_THREADS) koff_s[i] = __ldg(q.koff2 + i);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_acc = tmem_base_slot;

  if (warp < PRODUCER_WARPS) {
    // ---------------- producers of the S tile ---------------------------------
    // Work item = (row, 16-byte chunk); item = chunk * total_rows + row so that the
    // lanes of a warp walk consecutive rows (contiguous records in the window tensor).
    // Per item: rel = element offset of (row, channel 0, u 0) from the tile's first image,
    // meta = swizzled byte offset of the chunk in a stage | chunk index (bits 0-2) |
    // row-inside-tensor flag (bit 3); 0xffffffff marks "no such item".
    // Loads are unconditional (a dead row or a padded k2 reads element 0 of the tile's
    // image and is masked afterwards) so that the compiler can issue all of a group's
    // loads back to back.
    uint32_t rel[ITEMS], meta[ITEMS];
    // Rows are numbered in blocks of 8 per sub-tile (row i of sub-tile j <-> strip column i*s + j), so
    // that the lanes of a warp read 32 neighbouring columns whatever the stride and the eight lanes of
    // a store phase hit eight different rows of the swizzle pattern.
    const int n_items = total_rows * q.chunks;
    const uint32_t img_rows = (uint32_t)(q.Ho * q.Wq);       // virtual positions per image
    const uint32_t n_first = (uint32_t)q0 / img_rows;
    const uint16_t* __restrict__ tile_win = q.win + (int64_t)n_first * q.img_stride;
    const int blk_rows = 8 * q.s;
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
      const int item = threadIdx.x + it * PRODUCER_THREADS;
      rel[it] = 0;
      meta[it] = 0xffffffffu;
      if (item < n_items) {
        const int ch = item / total_rows;
        const int ri = item - ch * total_rows;
        const int blk = ri / blk_rows;
        const int w = ri - blk * blk_rows;
        const int sub = w >> 3;
        const int i = blk * 8 + (w & 7);
        meta[it] = (uint32_t)(sub * sub_bytes + i * 128 + ((ch ^ (i & 7)) << 4)) | (uint32_t)ch;
        const uint32_t vq = (uint32_t)q0 + (uint32_t)i;
        if (vq < (uint32_t)q.VQ) {
          const uint32_t sg = vq / (uint32_t)q.Wq;
          const int col = (int)(vq - sg * (uint32_t)q.Wq) * q.s + sub;
          const uint32_t n = sg / (uint32_t)q.Ho;
          const int ho = (int)(sg - n * (uint32_t)q.Ho);
          if (col < q.Wp) {                    // the last virtual column of a strip may be cut short
            rel[it] = (uint32_t)((int64_t)(n - n_first) * q.img_stride + ho * q.strip + (int64_t)col * q.Kh);
            meta[it] |= 8u;
          }
        }
      }
    }

    bool ok = true;
    TIMER_DECL;
    if (threadIdx.x == 0) TIMER_LAP(0);   // setup
    // The stage is produced in units of ITEM_GROUP items whose loads are issued back to back.
    // Dead rows and padded k2 read a word of the status block that is always zero, so nothing
    // needs masking afterwards.  (Holding the next unit's loads in a second register buffer,
    // and L2 prefetches of the next k-blocks' runs, were measured and did not pay.)
    constexpr int G = ITEM_GROUP;
    constexpr int NG = ITEMS / G;
    const uint16_t* __restrict__ zero16 = reinterpret_cast<const uint16_t*>(q.status + 2);
    auto issue = [&](int kb, int climit, int gidx, uint32_t (&h)[G][8]) {
      const int4* kt = reinterpret_cast<const int4*>(koff_s + kb * KB);   // this k-block's offsets (shared memory)
#pragma unroll
      for (int gi = 0; gi < G; ++gi) {
        const int it = gidx * G + gi;
        const int ch = (int)(meta[it] & 7u);
        const int4 o0 = kt[ch * 2], o1 = kt[ch * 2 + 1];
        const int32_t off[8] = {o0.x, o0.y, o0.z, o0.w, o1.x, o1.y, o1.z, o1.w};
        const uint16_t* src = tile_win + rel[it];
        const bool row_ok = (meta[it] & 8u) != 0 && ch < climit;
#pragma unroll
        for (int e = 0; e < 8; ++e) h[gi][e] = (uint32_t)__ldg((row_ok && off[e] >= 0) ? src + off[e] : zero16);
      }
    };
    auto store = [&](uint32_t a_stage, int climit, int gidx, const uint32_t (&h)[G][8]) {
#pragma unroll
      for (int gi = 0; gi < G; ++gi) {
        const int it = gidx * G + gi;
        if (meta[it] != 0xffffffffu && (int)(meta[it] & 7u) < climit) {
          const uint32_t w0 = h[gi][0] | (h[gi][1] << 16), w1 = h[gi][2] | (h[gi][3] << 16);
          const uint32_t w2 = h[gi][4] | (h[gi][5] << 16), w3 = h[gi][6] | (h[gi][7] << 16);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_stage + (meta[it] & ~15u)), "r"(w0),
                       "r"(w1), "r"(w2), "r"(w3)
                       : "memory");
        }
      }
    };

    int st = 0;                 // ring slot and its phase bit, advanced without divisions
    uint32_t ph = 0;
    uint32_t buf[G][8];
    for (int kb = 0; kb < q.num_kb && ok; ++kb) {
      const uint32_t a_stage = a_ring + st * q.a_stage_bytes;
      const int climit = kb == q.num_kb - 1 ? q.chunks_last : 8;   // the MMAs skip the padded tail of k
#pragma unroll
      for (int gidx = 0; gidx < NG; ++gidx) {
        issue(kb, climit, gidx, buf);
        if (gidx == 0) {
          if (threadIdx.x == 0) TIMER_LAP(2);   // issuing loads
          if (lane == 0) ok = mbar_wait(a_empty0 + 8 * st, ph ^ 1u, &abort_flag, q.status);
          ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
          __syncwarp();   // lane 0 observed the barrier: orders the other lanes' accesses after it
          if (threadIdx.x == 0) TIMER_LAP(1);   // wait for a free stage
        }
        if (ok) store(a_stage, climit, gidx, buf);
      }
      if (!ok) break;
      if (threadIdx.x == 0) TIMER_LAP(3);   // waiting for the loads, pack + store
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(a_full0 + 8 * st);
      if (threadIdx.x == 0) TIMER_LAP(4);   // fence + arrive
      if (++st == q.sa) {
        st = 0;
        ph ^= 1u;
      }
    }

    // ---------------- epilogue --------------------------------------------------
    if (ok && lane == 0) ok = mbar_wait(acc_bar, 0u, &abort_flag, q.status);
    ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
    __syncwarp();   // lane 0 observed the barrier: orders the other lanes' accesses after it
    if (threadIdx.x == 0) TIMER_LAP(5);     // wait for the accumulator
    if (ok) {
      tc_fence_after();
      const int lq = warp & 3;                 // tensor-memory lane quadrant this warp may read
      const int chalf = warp >> 2;             // which half of the channel tile
      for (int half = 0; half < mt; ++half) {
        const uint32_t vq = (uint32_t)q0 + (uint32_t)(half * TILE_M + lq * 32 + lane);   // accumulator row = virtual position
        bool valid = false;
        float* yrow = q.y;
        if (vq < (uint32_t)q.VQ) {
          const uint32_t sg = vq / (uint32_t)q.Wq;
          const int kq = (int)(vq - sg * (uint32_t)q.Wq);
          const uint32_t n = sg / (uint32_t)q.Ho;
          const int ho = (int)(sg - n * (uint32_t)q.Ho);
          valid = kq < q.Wo;                   // trailing columns of a strip are no output
          yrow += ((int64_t)n * q.Co) * q.HoWo + ho * q.Wo + kq;
        }
        const uint32_t lane_base = tmem_acc + ((uint32_t)(lq * 32) << 16) + (uint32_t)(half * BN);
#pragma unroll 1
        for (int c0 = chalf * (BN / 2); c0 < (chalf + 1) * (BN / 2); c0 += 32) {
          if (n0 + c0 >= q.Co) break;
          uint32_t v[32];
          tmem_ld32(lane_base + (uint32_t)c0, v);
          if (valid) store_strided32(yrow + (int64_t)(n0 + c0) * q.HoWo, q.HoWo, v, q.Co - n0 - c0);
        }
      }
    }
    if (threadIdx.x == 0) { TIMER_LAP(6); TIMER_FLUSH(); }     // epilogue
  } else if (warp == PRODUCER_WARPS) {
    // ---------------- TMA producer of the filter tiles -------------------------
    // The whole warp walks the loop (warp-uniform values can stay in uniform registers, which
    // the TMA and MMA instructions take their operands from); one elected lane issues.
    const bool leader = elect_one();
    bool ok = true;
    int st = 0;
    uint32_t ph = 0;
    for (int kb = 0; kb < q.num_kb && ok; ++kb) {
      for (int v = 0; v < q.Kw; ++v) {
        ok = mbar_wait(b_empty0 + 8 * st, ph ^ 1u, &abort_flag, q.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const uint32_t bar = b_full0 + 8 * st;
        if (leader) {
          mbar_arrive_expect_tx(bar, B_STAGE_BYTES);
          tma_load_3d(b_ring + st * B_STAGE_BYTES, &fmap, kb * KB, n0, v, bar);
        }
        __syncwarp();
        if (++st == q.sb) {
          st = 0;
          ph ^= 1u;
        }
      }
    }
  } else {
    // ---------------- MMA issuer ------------------------------------------------
    constexpr uint32_t idesc = instr_desc_f16(TILE_M, BN);
    const bool leader = elect_one();
    bool ok = true;
    int sta = 0, stb = 0;                 // ring slots and phase bits, advanced without divisions
    uint32_t pha = 0, phb = 0, first = 0;
    // Descriptor low words (16-byte units) of the ring bases; kernel column v reads sub-tile
    // v mod s shifted down v div s rows (128 bytes each).
    const uint32_t a_lo0 = smem_desc_lo(a_ring), b_lo0 = smem_desc_lo(b_ring);
    const uint32_t sub_lo = (uint32_t)sub_bytes >> 4;
    TIMER_DECL;
    for (int kb = 0; kb < q.num_kb && ok; ++kb) {
      TIMER_LAP(8);
      ok = mbar_wait(a_full0 + 8 * sta, pha, &abort_flag, q.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      TIMER_LAP(9);                         // MMA warp: wait for an S stage
      const uint32_t a_lo_stage = a_lo0 + (uint32_t)(sta * (q.a_stage_bytes >> 4));
      const int nks = kb == q.num_kb - 1 ? q.nks_last : KB / 16;
      uint32_t a_view = 0;                  // offset of kernel column v's view inside the stage
      int sub = 0;
      for (int v = 0; v < q.Kw; ++v) {
        TIMER_LAP(8);
        ok = mbar_wait(b_full0 + 8 * stb, phb, &abort_flag, q.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        TIMER_LAP(10);                      // MMA warp: wait for a filter stage
        tc_fence_after();
        const uint32_t b_lo = b_lo0 + (uint32_t)(stb * (B_STAGE_BYTES >> 4));
        uint32_t a_lo = a_lo_stage + a_view;
        // next kernel column: next sub-tile, or back to sub-tile 0 one row (128 bytes) further down
        if (++sub == q.s) {
          sub = 0;
          a_view += 8u - (uint32_t)(q.s - 1) * sub_lo;
        } else {
          a_view += sub_lo;
        }
        if (leader) {
          uint32_t acc_col = tmem_acc;
          for (int half = 0; half < mt; ++half) {
#pragma unroll
            for (int j = 0; j < KB / 16; ++j)
              if (j < nks) umma_f16_lohi(acc_col, a_lo + 2 * j, b_lo + 2 * j, idesc, first | (uint32_t)j);
            a_lo += (uint32_t)(TILE_M * 128) >> 4;
            acc_col += (uint32_t)BN;
          }
          umma_commit(b_empty0 + 8 * stb);
        }
        __syncwarp();
        TIMER_LAP(11);                      // MMA warp: issue + commit
        first = 1u;                         // every later MMA accumulates
        if (++stb == q.sb) {
          stb = 0;
          phb ^= 1u;
        }
      }
      if (ok && leader) umma_commit(a_empty0 + 8 * sta);
      __syncwarp();
      if (++sta == q.sa) {
        sta = 0;
        pha ^= 1u;
      }
    }
    if (ok && leader) umma_commit(acc_bar);
    __syncwarp();
    if (leader) {
      TIMER_LAP(8);
      TIMER_FLUSH();
    }
  }

  // ---------------- teardown ---------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == PRODUCER_WARPS + 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_acc, 2 * BN);
  }
}

// ------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(p);
  return fn;
}

constexpr int kSmemBudget = 220 * 1024;

template <int BN>
void choose_stages(const ShiftPlan& plan, int a_bytes, int* sa, int* sb) {
  const int b_bytes = BN * KB * 2;
  // Narrow channel tiles leave room for two CTAs per SM: give each half of the budget.
  const int budget = (BN <= 128 ? kSmemBudget / 2 : kSmemBudget) - 2048 - (int)plan.K2p * 4;
  int a = 2, b = 2;
  // Filter stages turn over Kw (x2 for tall tiles) times faster than S stages and hide the
  // L2 latency of the TMA loads: grow them to 4 first, then S to 3, then both further.
  auto fits = [&](int aa, int bb) { return aa * a_bytes + bb * b_bytes <= budget; };
  while (b < 4 && fits(a, b + 1)) ++b;
  if (fits(a + 1, b)) ++a;
  while (b < 6 && fits(a, b + 1)) ++b;
  if (a < 4 && fits(a + 1, b)) ++a;
  *sa = a;
  *sb = b;
}

template <int BN, int ITEMS>
cudaError_t launch_variant(const CUtensorMap& fmap, const ShiftParams& q0, const ShiftPlan& plan, int co,
                           cudaStream_t stream) {
  ShiftParams q = q0;
  int sa, sb;
  choose_stages<BN>(plan, q.a_stage_bytes, &sa, &sb);
  q.sa = sa;
  q.sb = sb;
  const int smem_bytes = sa * q.a_stage_bytes + sb * BN * KB * 2 + (int)plan.K2p * 4 + 1024;
  cudaError_t e = cudaFuncSetAttribute(conv_f16_shift_kernel<BN, ITEMS>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  if (e != cudaSuccess) return e;
  const int64_t units = (plan.VQ + TILE_M - 1) / TILE_M;
  dim3 grid((unsigned)(units - q.nbig), (unsigned)((co + BN - 1) / BN));   // a tall tile covers two units
  conv_f16_shift_kernel<BN, ITEMS><<<grid, NUM_THREADS, smem_bytes, stream>>>(fmap, q);
  return cudaGetLastError();
}

// Number of 256-position tiles: whole waves of tall tiles while two units per slot remain, and
// in the last round as many tall tiles as it takes for the rest to fit in one wave.
int choose_nbig(int64_t units, int cotiles, int ctas_per_sm, int kw) {
  const char* force = debug_getenv("IM2WIN_F16_TALL");     // testing aid: 1 = all tall, 0 = none
  if (force) return atoi(force) ? (int)(units / 2) : 0;
  // Tall tiles halve the filter traffic per flop, which is what bounds wide kernels (measured:
  // +40 % at 11x11, +25 % at 5x5); with three kernel columns the S producers are the bound and
  // a tall tile only doubles their per-stage latency (measured: -30 % on 3x3 stride 2).
  if (kw < 5) return 0;
  int64_t slots = (int64_t)148 * ctas_per_sm / cotiles;
  if (slots < 1) slots = 1;
  const int64_t full = units / (2 * slots) * slots;
  const int64_t rest = units - 2 * full;
  const int64_t extra = rest > slots ? rest - slots : 0;
  return (int)(full + extra);
}

template <int BN>
cudaError_t launch_bn(const CUtensorMap& fmap, const ShiftParams& q0, const ShiftPlan& plan, int co,
                      int s, cudaStream_t stream) {
  ShiftParams q = q0;
  const int64_t units = (plan.VQ + TILE_M - 1) / TILE_M;
  q.nbig = choose_nbig(units, (co + BN - 1) / BN, BN <= 128 ? 2 : 1, q.Kw);
  const int mt = q.nbig > 0 ? 2 : 1;
  const int total_rows = s * (TILE_M * mt + q.halo8);
  q.a_stage_bytes = total_rows * 128;
  if (2 * q.a_stage_bytes + 2 * BN * KB * 2 + (int)plan.K2p * 4 > (BN <= 128 ? kSmemBudget / 2 : kSmemBudget) - 2048) {
    q.nbig = 0;                                   // tall tiles do not fit: fall back to 128-row tiles
    q.a_stage_bytes = s * (TILE_M + q.halo8) * 128;
  }
  const int rows_all = q.a_stage_bytes / 128;
  const int items = (rows_all * q.chunks + PRODUCER_THREADS - 1) / PRODUCER_THREADS;
  if (items <= 5) return launch_variant<BN, 5>(fmap, q, plan, co, stream);
  if (items <= 10) return launch_variant<BN, 10>(fmap, q, plan, co, stream);
  if (items <= 15) return launch_variant<BN, 15>(fmap, q, plan, co, stream);
  if (items <= 20) return launch_variant<BN, 20>(fmap, q, plan, co, stream);
  q.nbig = 0;
  q.a_stage_bytes = s * (TILE_M + q.halo8) * 128;
  return launch_variant<BN, 15>(fmap, q, plan, co, stream);
}

}  // namespace

ShiftPlan plan_f16_shift(const Geometry& g) {
  ShiftPlan p{};
  p.eligible = false;
  p.Wq = (g.Wp + g.s - 1) / g.s;
  const int halo = (g.Kw - 1 + g.s - 1) / g.s;
  p.rows = TILE_M + (halo + 7) / 8 * 8;
  p.total_rows = g.s * p.rows;
  p.K2 = (int64_t)g.C * g.Kh;
  p.K2p = (p.K2 + KB - 1) / KB * KB;
  p.VQ = (int64_t)g.N * g.Ho * p.Wq;
  // the MMAs stop at the last 16-wide step that holds real k2; a single short k-block is staged that narrow
  p.nks_last = (int32_t)((p.K2 - (p.K2p - KB) + 15) / 16);
  p.chunks = p.K2p == KB ? 2 * p.nks_last : 8;
  p.items = (p.total_rows * p.chunks + PRODUCER_THREADS - 1) / PRODUCER_THREADS;
  if (p.items > 15) return p;
  if (p.K2p * 4 > 24 * 1024) return p;                    // offset table lives in shared memory
  if (g.img_stride >= ((int64_t)1 << 30)) return p;       // 32-bit offsets relative to the tile's first image
  // two stages of each ring must fit even for the widest channel tile
  if (2 * p.total_rows * 128 + 2 * 256 * KB * 2 + p.K2p * 4 > kSmemBudget - 2048) return p;
  if (p.VQ + 2 * TILE_M >= ((int64_t)1 << 31)) return p;   // 32-bit position arithmetic
  p.eligible = true;
  return p;
}

cudaError_t launch_conv_f16_shift(const uint16_t* window, float* y, void* scratch, const Geometry& g,
                                  const ScratchLayout& l, cudaStream_t stream) {
  const ShiftPlan plan = plan_f16_shift(g);
  if (!plan.eligible) return cudaErrorInvalidValue;
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return cudaErrorNotSupported;
  unsigned char* base = static_cast<unsigned char*>(scratch);
  const int bn = g.Co <= 64 ? 64 : (g.Co <= 128 ? 128 : 256);

  // Filter as Fp2[v][co][k2p] halves: a 3-D tensor (k2 fastest), one box = 64 k2 x BN channels of one v.
  CUtensorMap fmap;
  const cuuint64_t dims[3] = {(cuuint64_t)plan.K2p, (cuuint64_t)g.Co, (cuuint64_t)g.Kw};
  const cuuint64_t strides[2] = {(cuuint64_t)plan.K2p * 2, (cuuint64_t)plan.K2p * 2 * (cuuint64_t)g.Co};
  const cuuint32_t box[3] = {(cuuint32_t)KB, (cuuint32_t)bn, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  CUresult cr = encode(&fmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, base + l.filter_off, dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (cr != CUDA_SUCCESS) return cudaErrorInvalidValue;

  ShiftParams q;
  q.win = window;
  q.koff2 = reinterpret_cast<const int32_t*>(base + l.koff_off);
  q.y = y;
  q.status = reinterpret_cast<uint32_t*>(base);
  q.VQ = plan.VQ; q.img_stride = g.img_stride; q.strip = g.strip;
  q.chan_stride = g.chan_stride; q.window_elems = g.window_elems; q.C = g.C; q.N = g.N;
  q.Wq = plan.Wq; q.Wp = g.Wp; q.chunks = plan.chunks; q.nks_last = plan.nks_last;
  q.chunks_last = 2 * plan.nks_last; q.Ho = g.Ho; q.Wo = g.Wo; q.HoWo = g.Ho * g.Wo; q.Co = g.Co;
  q.Kh = g.Kh; q.Kw = g.Kw; q.s = g.s; q.num_kb = (int32_t)(plan.K2p / KB);
  q.halo8 = plan.rows - TILE_M;
  q.nbig = 0;
  q.a_stage_bytes = plan.total_rows * 128;
  q.sa = q.sb = 2;
  if (bn == 64) return launch_bn<64>(fmap, q, plan, g.Co, g.s, stream);
  if (bn == 128) return launch_bn<128>(fmap, q, plan, g.Co, g.s, stream);
  return launch_bn<256>(fmap, q, plan, g.Co, g.s, stream);
}

}  // namespace im2win
