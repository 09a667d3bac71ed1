// fp16-input / fp32-accumulate im2win convolution on the sm_100a tensor cores:
// shifted-view kernel for layers whose whole reduction over (channel, kernel row) fits ONE
// k-block, K2 = C*Kh <= 64 (network stems: few input channels, any kernel size and stride).
//
// GEMM formulation as in conv_f16_shift.cu (paper Algorithm 1 with the S tile of im2win columns,
// S[row = virtual column][k2 = c*Kh + u], and Kw row-shifted views of it, one per kernel column).
// Such layers are bound by the output they write and by how cheaply S is built, not by the MMAs,
// and their window tensors are the awkward ones: strides that do not divide the strip width,
// channel planes that start on odd addresses.  This kernel makes no alignment assumption at all:
//
//   * raw stage: for one channel the columns a tile needs are ONE contiguous run of the window
//     tensor per strip segment (per image when s divides Wp, per strip otherwise).  Each run is
//     brought in by one untiled bulk copy that starts at the 16-byte boundary below the run and
//     ends at the one above it; where the run really starts inside the copy (its "phase", 0..7
//     elements) differs per channel and segment and is added when the data is read back.
//   * S stage without swizzle, S[sub-tile][16-byte unit of k2][row]: only the units that hold
//     real k2 exist (K2 = 33 -> 6 units, not 8), the MMAs stop at the last 16-wide step with
//     real k2, and a view shifted by r rows starts 16*r bytes further.
//   * re-layout: one work item = one row of one sub-tile: K2 2-byte shared loads (lanes on
//     consecutive rows, i.e. records s*Kh elements apart: at most 2-way bank conflicts) and one
//     conflict-free 16-byte store per unit.  The kernel is bound by instruction issue, so the
//     common stems (3 channels, Kh = 3, 5, 7, 11) get instantiations in which the (channel, u)
//     loops are unrolled: one address per channel, immediate offsets for u, the packing of
//     halves into words resolved at compile time.  Any other (C, Kh) takes a table-driven loop.
//   * filter: Fp2[v][co][64] as for the other shifted-view kernels, resident in shared memory for
//     the whole kernel when the layer has one channel tile and the Kw tiles fit, streamed
//     otherwise.  The channel tile is Co rounded up to 16 (MMA N), not to a power of two.
//
// Virtual positions q = (n*Ho + ho)*Wq + kq with Wq = ceil(Wp/s); when s does not divide Wp the
// last virtual column of a strip lacks some columns, which are staged as zeros and only feed
// accumulator rows that are dropped.  Persistent CTAs; S stage i and accumulator i (two to four of
// each, in tensor memory) belong together, so that one commit per tile tells the epilogue that the
// accumulator is complete and the re-layout warps that the S stage is free; bounded mbarrier waits.
// Warp roles: 0-7 and 11 re-layout, 8 filter copies, 9 MMA issue (and tensor-memory allocation),
// 10 raw copies, 12-15 epilogue (a second epilogue warp per lane quadrant was measured: 5 % faster on
// a 3-channel 3x3 layer, 5-8 % slower on the 7x7 and 11x11 stems).
#include <cuda.h>
#include <stdlib.h>

#include "common.cuh"
#define IM2WIN_INLINE_SLOW_WAIT   // the slow path of the bounded waits expanded in place: faster in this kernel
#include "ptx_sm100.cuh"

namespace im2win {
namespace {

using namespace ptx;

constexpr int TILE_M = 128;
constexpr int KB = kF16KBlock;
constexpr int REPACK_WARPS = 9;                      // warps 0-7 and warp 11
constexpr int REPACK_THREADS = REPACK_WARPS * 32;
constexpr int WARP_TMA = 8, WARP_MMA = 9, WARP_RAW = 10, WARP_REPACK9 = 11, WARP_EPI0 = 12;
constexpr int NUM_WARPS = 16;
constexpr int NUM_THREADS = NUM_WARPS * 32;
constexpr int MAX_STAGES = 4;                        // S stages / accumulators
constexpr int MAX_RAW = 8;                           // most raw stages a testing switch may ask for (3 or 4 are used)
constexpr int MAX_B = 16;                            // filter stages (a resident filter needs Kw of them)
constexpr int SEG_MAX = 6;                           // strip segments (or images) one tile may touch
constexpr int SEG_GAP = 48;                          // bytes between the copies of consecutive segments
constexpr int EPI_PITCH = 136;                       // floats per output plane in an epilogue staging buffer
constexpr int EPI_BUF_BYTES = 32 * EPI_PITCH * 4;    // 32 planes x (128 positions + alignment slack)

struct StemParams {
  const uint16_t* __restrict__ win;
  float* __restrict__ y;
  uint32_t* status;
  int64_t chan_stride, img_stride, strip, window_elems;
  int32_t VQ, C, N, Wq, Wp, Ho, Wo, HoWo, Co, Kh, Kw, s;
  int32_t sKh;              // s * Kh: elements per virtual column
  int32_t K2;               // C * Kh
  int32_t rows;             // virtual positions staged per tile: 128 + (Kw-1)/s
  int32_t R;                // rows per unit plane of an S sub-tile: rows rounded up to 8
  int32_t nks;              // 16-wide MMA steps: ceil(K2 / 16)
  int32_t chunks;           // 16-byte units of k2 per row: 2 * nks
  int32_t ragged;           // 1: s does not divide Wp, segments are strips; 0: segments are images
  int32_t chan_region;      // bytes of one channel's part of a raw stage
  int32_t raw_stage_bytes, a_stage_bytes, b_stage_bytes;
  int32_t bn, bnr;          // channel tile (multiple of 16) and its round-up to 32 (accumulator pitch)
  int32_t tmem_cols;
  uint32_t idesc;
  int32_t rs, sa, sb, resident;
  int32_t ntm, nwork;
  int32_t cbits;            // bits of a channel index: ceil(log2 C)
  int32_t epi_bufs;         // staging buffers of the aligned-store epilogue (0: stores straight from registers)
};

struct Segment {            // the part of a tile that is one contiguous run per channel
  int64_t e0;               // element index (channel 0) of the run's first element in the window tensor
  int32_t row0, cnt;        // tile rows [row0, row0 + cnt)
  int32_t elems;            // valid elements of the run (a multiple of Kh)
  int32_t dst;              // byte offset of the run's copy inside a channel region
};

// Where a tile starts: strip (s does not divide Wp) or image u0, row a0 inside it, and for strips
// the image n0 and output row ho0 of strip u0.  Worked out with divisions once and then advanced
// from tile to tile of the persistent loop with additions (a lone warp runs this code on the
// critical path of the raw copies: every division there costs a hundred cycles).
struct TilePos { int u0, a0, n0, ho0; };

__device__ __forceinline__ void pos_init(const StemParams& q, int q0, TilePos& p) {
  const int per = q.ragged ? q.Wq : q.Ho * q.Wq;       // rows of a whole strip / image
  p.u0 = q0 / per;
  p.a0 = q0 - p.u0 * per;
  p.n0 = q.ragged ? p.u0 / q.Ho : p.u0;
  p.ho0 = q.ragged ? p.u0 - p.n0 * q.Ho : 0;
}
// adv = rows between consecutive tiles of this CTA, split as adv = du*per + da and du = dn*Ho + dho
__device__ __forceinline__ void pos_advance(const StemParams& q, TilePos& p, int du, int da, int dn, int dho) {
  const int per = q.ragged ? q.Wq : q.Ho * q.Wq;
  p.a0 += da;
  p.u0 += du;
  const int carry = p.a0 >= per ? 1 : 0;
  p.a0 -= carry ? per : 0;
  p.u0 += carry;
  if (q.ragged) {
    p.n0 += dn;
    p.ho0 += dho + carry;
    if (p.ho0 >= q.Ho) { p.ho0 -= q.Ho; ++p.n0; }
  } else {
    p.n0 = p.u0;
  }
}

// Splits the rows of the tile at `p` into contiguous runs: lane g of the calling warp works out
// run g (no loop: the runs after the first start on strip / image boundaries); returns whether
// the lane's run exists.
__device__ __forceinline__ bool split_tile(const StemParams& q, const TilePos& p, int lane, Segment& sg) {
  const int per = q.ragged ? q.Wq : q.Ho * q.Wq;
  const int first_cnt = q.rows < per - p.a0 ? q.rows : per - p.a0;
  const int unit = p.u0 + lane;
  const int row0 = lane == 0 ? 0 : first_cnt + (lane - 1) * per;
  const int a = lane == 0 ? p.a0 : 0;
  int cnt = q.rows - row0;
  if (cnt > per - a) cnt = per - a;
  const bool valid = lane < SEG_MAX && row0 < q.rows && unit < (q.ragged ? q.N * q.Ho : q.N);
  if (valid) {
    if (q.ragged) {
      int n = p.n0, ho = p.ho0 + lane;
      while (ho >= q.Ho) { ho -= q.Ho; ++n; }
      int cend = (a + cnt) * q.s;
      if (cend > q.Wp) cend = q.Wp;
      sg.e0 = (int64_t)n * q.img_stride + (int64_t)ho * q.strip + (int64_t)a * q.sKh;
      sg.elems = cend * q.Kh - a * q.sKh;
    } else {
      sg.e0 = (int64_t)unit * q.img_stride + (int64_t)a * q.sKh;
      sg.elems = cnt * q.sKh;
    }
    sg.row0 = row0;
    sg.cnt = cnt;
    sg.dst = ((row0 * q.sKh * 2) & ~15) + SEG_GAP * lane;
  }
  return valid;
}

// One row of S for compile-time (C, Kh): returns the row's K2 halves packed into words.
template <int C_, int KH_>
__device__ __forceinline__ void load_row(uint32_t src, uint32_t phase0, uint32_t cs7, uint32_t chan_region,
                                         uint32_t (&w)[8 * ((C_ * KH_ + 15) / 16)]) {
#pragma unroll
  for (int c = 0; c < C_; ++c) {
    // where channel c's run starts inside its copy: the 16-byte phase of its first element
    const uint32_t base = src + (uint32_t)c * chan_region + ((((uint32_t)c * cs7 + phase0) & 7u) << 1);
#pragma unroll
    for (int u = 0; u < KH_; ++u) {
      uint16_t v;
      asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(base + 2u * (uint32_t)u));   // folds into the load's offset
      const int k2 = c * KH_ + u;
      if (k2 & 1) w[k2 >> 1] |= (uint32_t)v << 16;
      else w[k2 >> 1] = (uint32_t)v;
    }
  }
}

// C_ = KH_ = KW_ = 0: any (C, Kh, Kw) with C*Kh <= 64: table-driven re-layout, looped MMA issue.
// STAGED: the epilogue that writes aligned runs through a staging buffer (opt-in, see plan_f16_stem).
template <int C_, int KH_, int KW_, bool STAGED>
__global__ void __launch_bounds__(NUM_THREADS, 1)
conv_f16_stem_kernel(const __grid_constant__ CUtensorMap fmap, StemParams q) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) uint64_t bars[3 * MAX_STAGES + 2 * MAX_RAW + 2 * MAX_B];
  __shared__ uint32_t tmem_base_slot;
  __shared__ volatile uint32_t abort_flag;
  __shared__ Segment seg_ring[MAX_RAW][SEG_MAX];      // the segments of the tile in each raw stage (written by the loader)
  __shared__ int32_t nseg_ring[MAX_RAW];
  __shared__ __align__(16) uint32_t tab_s[KB];           // k2 -> channel region + 2*u | (c*chan_stride mod 8) << 24
  __shared__ __align__(16) uint32_t zero_s[4];           // what padded k2 read

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // shared-memory map: filter ring (1024-byte aligned stages) | S ring | raw ring
  const uint32_t b_ring = smem_u32(smem);
  const uint32_t a_ring = b_ring + q.sb * q.b_stage_bytes;
  const uint32_t raw_ring = a_ring + q.sa * q.a_stage_bytes;
  const uint32_t epi_ring = raw_ring + q.rs * q.raw_stage_bytes;
  const uint32_t a_full0 = smem_u32(&bars[0]);
  const uint32_t acc_empty0 = smem_u32(&bars[MAX_STAGES]);
  const uint32_t acc_full0 = smem_u32(&bars[2 * MAX_STAGES]);
  const uint32_t r_full0 = smem_u32(&bars[3 * MAX_STAGES]);
  const uint32_t r_empty0 = smem_u32(&bars[3 * MAX_STAGES + MAX_RAW]);
  const uint32_t b_full0 = smem_u32(&bars[3 * MAX_STAGES + 2 * MAX_RAW]);
  const uint32_t b_empty0 = smem_u32(&bars[3 * MAX_STAGES + 2 * MAX_RAW + MAX_B]);

  if (threadIdx.x == 0) {
    abort_flag = 0u;
    for (int i = 0; i < MAX_STAGES; ++i) {
      mbar_init(a_full0 + 8 * i, REPACK_WARPS);
      mbar_init(acc_empty0 + 8 * i, NUM_WARPS - WARP_EPI0);      // the epilogue warps
      mbar_init(acc_full0 + 8 * i, 1);
    }
    for (int i = 0; i < MAX_RAW; ++i) {
      mbar_init(r_full0 + 8 * i, 1);
      mbar_init(r_empty0 + 8 * i, REPACK_WARPS);
    }
    for (int i = 0; i < MAX_B; ++i) {
      mbar_init(b_full0 + 8 * i, 1);
      mbar_init(b_empty0 + 8 * i, 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == WARP_MMA) tmem_alloc(smem_u32(&tmem_base_slot), (uint32_t)q.tmem_cols);
  if (threadIdx.x < KB) {
    const int k2 = threadIdx.x;
    uint32_t t = 0x80000000u;                // padded k2
    if (k2 < q.K2) {
      const int c = k2 / q.Kh, u = k2 - c * q.Kh;
      t = (uint32_t)(c * q.chan_region + 2 * u) | ((uint32_t)((c * (int)(q.chan_stride & 7)) & 7) << 24);
    }
    tab_s[k2] = t;
  }
  if (threadIdx.x < 4) zero_s[threadIdx.x] = 0u;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_acc = tmem_base_slot;

  if (warp < 8 || warp == WARP_REPACK9) {
    // ---------------- re-layout: raw stage -> S stage ---------------------------
    const uint32_t zero_addr = smem_u32(zero_s);
    const uint32_t r16 = (uint32_t)q.R * 16u;
    const uint32_t cs7 = (uint32_t)q.chan_stride & 7u;
    bool ok = true;
    int st = 0, rst = 0;
    uint32_t ph = 0, rph = 0;
    const int n_ri = q.s * q.rows;
    // nine warps: 288 threads take the 262 rows of a 7x7 stride-2 tile in one pass and the 520 rows of
    // an 11x11 stride-4 tile in two (eight warps need two and three)
    const int rt = warp < 8 ? (int)threadIdx.x : 256 + lane;
    TIMER_DECL;
    for (int w = blockIdx.x; w < q.nwork && ok; w += gridDim.x) {
      if (lane == 0) {
        ok = mbar_wait(r_full0 + 8 * rst, rph, &abort_flag, q.status);
        if (threadIdx.x == 0) TIMER_LAP(1);     // wait for the raw stage
        // S stage st is free once the MMAs of the tile that used it last are complete
        if (ok) ok = mbar_wait(acc_full0 + 8 * st, ph ^ 1u, &abort_flag, q.status);
        if (threadIdx.x == 0) TIMER_LAP(2);     // wait for a free S stage
      }
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
      if (!ok) break;
      __syncwarp();                             // lane 0 observed the barrier; orders the other lanes' reads after it
      const Segment* segs = seg_ring[rst];      // published by the loader's arrival on the raw stage's barrier
      const int nseg = nseg_ring[rst];
      const uint32_t a_stage = a_ring + st * q.a_stage_bytes;
      const uint32_t raw_stage = raw_ring + rst * q.raw_stage_bytes;
      for (int ri = rt; ri < n_ri; ri += REPACK_THREADS) {
        int sub = 0, i = ri;
        while (i >= q.rows) { i -= q.rows; ++sub; }
        // the segment of row i, the row's record inside the segment's run, the run's phase
        bool live = false;
        uint32_t src = raw_stage, phase0 = 0;
        for (int g = 0; g < nseg; ++g) {
          const int d = i - segs[g].row0;
          if (d >= 0 && d < segs[g].cnt) {
            const int rel = (d * q.s + sub) * q.Kh;
            live = rel < segs[g].elems;
            src = raw_stage + (uint32_t)(segs[g].dst + 2 * rel);
            phase0 = (uint32_t)segs[g].e0 & 7u;
          }
        }
        uint32_t dst = a_stage + (uint32_t)((sub * q.chunks * q.R + i) << 4);
        if constexpr (C_ > 0) {
          constexpr int NW = 8 * ((C_ * KH_ + 15) / 16);
          uint32_t wd[NW];
#pragma unroll
          for (int k = 0; k < NW; ++k) wd[k] = 0u;
          if (live) load_row<C_, KH_>(src, phase0, cs7, (uint32_t)q.chan_region, wd);
#pragma unroll
          for (int ch = 0; ch < NW / 4; ++ch)
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (uint32_t)ch * r16), "r"(wd[4 * ch]),
                         "r"(wd[4 * ch + 1]), "r"(wd[4 * ch + 2]), "r"(wd[4 * ch + 3])
                         : "memory");
        } else {
          for (int ch = 0; ch < q.chunks; ++ch, dst += r16) {
            uint32_t w0 = 0, w1 = 0, w2 = 0, w3 = 0;
            if (live) {
              const uint4 t0 = *reinterpret_cast<const uint4*>(tab_s + ch * 8);
              const uint4 t1 = *reinterpret_cast<const uint4*>(tab_s + ch * 8 + 4);
              const uint32_t t[8] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
              uint32_t h[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const uint32_t a = (t[e] >> 31) ? zero_addr
                                                : src + (t[e] & 0xffffffu) + ((((t[e] >> 24) + phase0) & 7u) << 1);
                uint16_t v;
                asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a));
                h[e] = v;
              }
              w0 = h[0] | (h[1] << 16); w1 = h[2] | (h[3] << 16);
              w2 = h[4] | (h[5] << 16); w3 = h[6] | (h[7] << 16);
            }
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(w0), "r"(w1), "r"(w2), "r"(w3)
                         : "memory");
          }
        }
      }
      if (threadIdx.x == 0) TIMER_LAP(3);       // re-layout
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(a_full0 + 8 * st);
        mbar_arrive(r_empty0 + 8 * rst);
      }
      if (threadIdx.x == 0) TIMER_LAP(4);       // fence + arrive
      if (++st == q.sa) { st = 0; ph ^= 1u; }
      if (++rst == q.rs) { rst = 0; rph ^= 1u; }
    }
    if (threadIdx.x == 0) TIMER_FLUSH();
  } else if (warp == WARP_TMA) {
    // ---------------- TMA loader of the filter tiles ---------------------------
    const bool leader = elect_one();
    bool ok = true;
    if (q.resident) {
      // one channel tile whose Kw filter tiles fit: loaded once, never released
      if (leader)
        for (int v = 0; v < q.Kw; ++v) {
          mbar_arrive_expect_tx(b_full0 + 8 * v, (uint32_t)q.b_stage_bytes);
          tma_load_3d(b_ring + v * q.b_stage_bytes, &fmap, 0, 0, v, b_full0 + 8 * v);
        }
      __syncwarp();
    } else {
      int st = 0;
      uint32_t ph = 0;
      for (int w = blockIdx.x; w < q.nwork && ok; w += gridDim.x) {
        const int n0 = (w / q.ntm) * q.bn;
        for (int v = 0; v < q.Kw; ++v) {
          ok = mbar_wait(b_empty0 + 8 * st, ph ^ 1u, &abort_flag, q.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          if (leader) {
            mbar_arrive_expect_tx(b_full0 + 8 * st, (uint32_t)q.b_stage_bytes);
            tma_load_3d(b_ring + st * q.b_stage_bytes, &fmap, 0, n0, v, b_full0 + 8 * st);
          }
          __syncwarp();
          if (++st == q.sb) { st = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == WARP_MMA) {
    // ---------------- MMA issuer ------------------------------------------------
    const bool leader = elect_one();
    bool ok = true;
    int sta = 0, stb = 0;
    uint32_t pha = 0, phb = 0;
    uint32_t it = 0;                             // work items done by this CTA
    const uint32_t a_lo0 = smem_desc_lo_noswz(a_ring, (uint32_t)q.R * 16u), b_lo0 = smem_desc_lo(b_ring);
    const uint32_t sub_units = (uint32_t)(q.chunks * q.R);   // 16-byte units per sub-tile
    const uint32_t kstep_units = 2u * (uint32_t)q.R;         // 16-byte units per 16-element k step
    // compile-time kernel width: the issue loops unroll completely and every operand address is a
    // stage base plus a value worked out here, once (back-to-back MMAs of N = 64 need 48 cycles each,
    // a looped issue sequence spends twice that per MMA on its own address arithmetic)
    constexpr int KWU = KW_ > 0 ? KW_ : 1;
    constexpr int NKS = KW_ > 0 ? (C_ * KH_ + 15) / 16 : 1;
    uint32_t aoff[KWU];
    if constexpr (KW_ > 0) {
      uint32_t sub = 0, shift = 0;
#pragma unroll
      for (int v = 0; v < KW_; ++v) {
        aoff[v] = sub * sub_units + shift;
        if (++sub == (uint32_t)q.s) { sub = 0; ++shift; }
      }
    }
    const uint32_t b_step = (uint32_t)(q.b_stage_bytes >> 4);
    TIMER_DECL;
    for (int w = blockIdx.x; w < q.nwork && ok; w += gridDim.x, ++it) {
      const uint32_t buf = (uint32_t)sta;       // accumulator i goes with S stage i
      TIMER_LAP(11);
      ok = mbar_wait(acc_empty0 + 8 * buf, pha ^ 1u, &abort_flag, q.status);   // drained by the epilogue
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      TIMER_LAP(9);                              // MMA warp: wait for a free accumulator
      ok = mbar_wait(a_full0 + 8 * sta, pha, &abort_flag, q.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      TIMER_LAP(10);                             // MMA warp: wait for an S stage
      tc_fence_after();
      const uint32_t acc = tmem_acc + buf * (uint32_t)q.bnr;
      const uint32_t a_lo_stage = a_lo0 + (uint32_t)(sta * (q.a_stage_bytes >> 4));
      // kernel column v reads sub-tile v mod s from row v div s on.  A single thread issuing branchy
      // code takes hundreds of cycles per kernel column, so the loops below are kept straight-line.
      if (q.resident) {
        if (it == 0) {                          // the resident filter is complete after the first wait
          for (int v = 0; v < q.Kw && ok; ++v) {
            ok = mbar_wait(b_full0 + 8 * v, 0u, &abort_flag, q.status);
            ok = __all_sync(0xffffffffu, ok);
          }
          if (!ok) break;
          tc_fence_after();
        }
        if constexpr (KW_ > 0) {
          if (leader) {
#pragma unroll
            for (int v = 0; v < KW_; ++v)
#pragma unroll
              for (int j = 0; j < NKS; ++j)
                umma_f16_ab(acc, a_lo_stage + aoff[v] + (uint32_t)j * kstep_units, kSmemDescHiNoSwz128,
                            b_lo0 + (uint32_t)v * b_step + 2 * j, kSmemDescHiSw128, q.idesc, (v | j) ? 1u : 0u);
            umma_commit(acc_full0 + 8 * buf);   // accumulator complete = S stage free
          }
        } else if (leader) {
          uint32_t a_v = a_lo_stage, b_v = b_lo0, sub = 0, accf = 0;
          const uint32_t wrap_step = 1u - (uint32_t)(q.s - 1) * sub_units;   // back to sub-tile 0, one row further
          const uint32_t last_sub = (uint32_t)q.s - 1u;
#pragma unroll 1
          for (int v = 0; v < q.Kw; ++v) {
#pragma unroll
            for (int j = 0; j < KB / 16; ++j)
              if (j < q.nks)
                umma_f16_ab(acc, a_v + (uint32_t)j * kstep_units, kSmemDescHiNoSwz128, b_v + 2 * j, kSmemDescHiSw128,
                            q.idesc, accf | (uint32_t)j);
            accf = 1u;
            b_v += b_step;
            const bool wrap = sub == last_sub;
            a_v += wrap ? wrap_step : sub_units;
            sub = wrap ? 0u : sub + 1u;
          }
          umma_commit(acc_full0 + 8 * buf);     // accumulator complete = S stage free
        }
        __syncwarp();
      } else if constexpr (KW_ > 0) {
#pragma unroll
        for (int v = 0; v < KW_; ++v) {
          ok = mbar_wait(b_full0 + 8 * stb, phb, &abort_flag, q.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          if (leader) {
            const uint32_t b_lo = b_lo0 + (uint32_t)stb * b_step;
#pragma unroll
            for (int j = 0; j < NKS; ++j)
              umma_f16_ab(acc, a_lo_stage + aoff[v] + (uint32_t)j * kstep_units, kSmemDescHiNoSwz128, b_lo + 2 * j,
                          kSmemDescHiSw128, q.idesc, (v | j) ? 1u : 0u);
            umma_commit(b_empty0 + 8 * stb);
          }
          __syncwarp();
          if (++stb == q.sb) { stb = 0; phb ^= 1u; }
        }
        if (!ok) break;
        if (leader) umma_commit(acc_full0 + 8 * buf);       // accumulator complete = S stage free
        __syncwarp();
      } else {
        uint32_t sub = 0, shift = 0, first = 0;
        for (int v = 0; v < q.Kw; ++v) {
          ok = mbar_wait(b_full0 + 8 * stb, phb, &abort_flag, q.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          if (leader) {
            const uint32_t a_lo = a_lo_stage + sub * sub_units + shift;
            const uint32_t b_lo = b_lo0 + (uint32_t)(stb * (q.b_stage_bytes >> 4));
#pragma unroll
            for (int j = 0; j < KB / 16; ++j)
              if (j < q.nks)
                umma_f16_ab(acc, a_lo + (uint32_t)j * kstep_units, kSmemDescHiNoSwz128, b_lo + 2 * j, kSmemDescHiSw128,
                            q.idesc, first | (uint32_t)j);
            first = 1u;
            umma_commit(b_empty0 + 8 * stb);
          }
          __syncwarp();
          if (++sub == (uint32_t)q.s) { sub = 0; ++shift; }
          if (++stb == q.sb) { stb = 0; phb ^= 1u; }
        }
        if (!ok) break;
        if (leader) umma_commit(acc_full0 + 8 * buf);       // accumulator complete = S stage free
        __syncwarp();
      }
      if (++sta == q.sa) { sta = 0; pha ^= 1u; }
    }
    if (leader) { TIMER_LAP(11); TIMER_FLUSH(); }   // MMA warp: filter waits, issue, commits
  } else if (warp == WARP_RAW) {
    // ---------------- raw loader: one bulk copy per (segment, channel) ----------
    bool ok = true;
    int rst = 0;
    uint32_t rph = 0;
    const int64_t lim16 = (q.window_elems * 2) & ~(int64_t)15;   // bytes of the tensor that whole 16-byte copies may touch
    // one channel tile: this CTA's tiles are gridDim.x apart and the position is advanced by additions
    const bool stepping = q.nwork == q.ntm;
    TilePos pos;
    pos_init(q, (int)blockIdx.x * TILE_M, pos);
    const int per = q.ragged ? q.Wq : q.Ho * q.Wq;
    const int adv = (int)gridDim.x * TILE_M;
    const int du = adv / per, da = adv - du * per;
    const int dn = q.ragged ? du / q.Ho : 0, dho = q.ragged ? du - dn * q.Ho : 0;
    const int cmask = (1 << q.cbits) - 1;       // copies are numbered (run << cbits) | channel
    const bool drop_first_arrive = *reinterpret_cast<volatile uint32_t*>(q.status + 2) == ptx::kDebugDropArrive;
    TIMER_DECL;
    for (int w = blockIdx.x; w < q.nwork && ok; w += gridDim.x) {
      if (!stepping) pos_init(q, (w % q.ntm) * TILE_M, pos);
      // the split does not need the raw stage: done before the wait
      Segment sg = {};
      const bool have = split_tile(q, pos, lane, sg);
      const int nseg = __popc(__ballot_sync(0xffffffffu, have));
      if (stepping) pos_advance(q, pos, du, da, dn, dho);
      if (lane == 0) TIMER_LAP(6);               // raw loader: splitting the tile, issuing copies
      ok = mbar_wait(r_empty0 + 8 * rst, rph ^ 1u, &abort_flag, q.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (lane == 0) TIMER_LAP(5);               // raw loader: wait for a free raw stage
      // the tile's segments go with the raw stage: the re-layout warps read them once the stage is full
      if (have) seg_ring[rst][lane] = sg;
      if (lane == 0) nseg_ring[rst] = nseg;
      const uint32_t bar = r_full0 + 8 * rst;
      const uint32_t stage = raw_ring + rst * q.raw_stage_bytes;
      const int ncopy = nseg << q.cbits;
      for (int idx0 = 0; idx0 < ncopy; idx0 += 32) {
        const int idx = idx0 + lane;
        const int g = idx >> q.cbits, c = idx & cmask;
        // the run's description comes from the lane that worked it out
        const int64_t e0 = __shfl_sync(0xffffffffu, sg.e0, g & 31);
        const int elems = __shfl_sync(0xffffffffu, sg.elems, g & 31);
        const int sdst = __shfl_sync(0xffffffffu, sg.dst, g & 31);
        if (idx >= ncopy || c >= q.C) continue;
        const int64_t e = e0 + (int64_t)c * q.chan_stride;
        const int64_t src_off = (e & ~(int64_t)7) * 2;            // bytes, 16-byte aligned
        const int phase = (int)(e & 7);
        int64_t bytes = ((int64_t)(phase + elems) * 2 + 15) & ~(int64_t)15;
        const uint32_t dst = stage + (uint32_t)(c * q.chan_region + sdst);
        if (src_off + bytes > lim16) {
          // the run ends in the last, partial 16 bytes of the tensor: those elements are fetched
          // with plain loads so that no copy reads beyond the tensor
          const int64_t end_e = e + elems;
          int64_t e1 = lim16 / 2;
          if (e1 < e - phase) e1 = e - phase;
          for (; e1 < end_e; ++e1) {
            const uint16_t v = __ldg(q.win + e1);
            asm volatile("st.shared.u16 [%0], %1;" ::"r"(dst + (uint32_t)((e1 - (e - phase)) * 2)), "h"(v) : "memory");
          }
          bytes = lim16 - src_off;
        }
        if (bytes > 0) {
          mbar_expect_tx(bar, (uint32_t)bytes);
          bulk_load(dst, reinterpret_cast<const unsigned char*>(q.win) + src_off, (uint32_t)bytes, bar);
        }
      }
      __syncwarp();
      // after every lane has announced its bytes (testing aid: with the marker in word 2 of the status
      // block the first arrival of each CTA is left out, so that the waits on this stage run out)
      if (lane == 0 && !(drop_first_arrive && w == (int)blockIdx.x)) mbar_arrive(bar);
      if (++rst == q.rs) { rst = 0; rph ^= 1u; }
    }
    if (lane == 0) { TIMER_LAP(6); TIMER_FLUSH(); }
  } else if (warp >= WARP_EPI0) {
    // ---------------- epilogue: tensor memory -> NCHW output --------------------
    const int lq = warp & 3;                     // tensor-memory lane quadrant this warp may read
    bool ok = true;
    uint32_t it = 0;
    TIMER_DECL;
    uint32_t buf = 0, eph = 0, chunk_ctr = 0;
    // Meeting point of the four epilogue warps: hardware barrier 1.  It has no time-out, so the warps
    // first agree (through the same barrier, which every warp reaches because the wait before it is
    // bounded) whether all of them got their accumulator; from there on they take the same path.
    auto epi_sync = [&]() { asm volatile("bar.sync 1, 128;" ::: "memory"); };
    // ragged run ends: lane -> (plane lane/6, end element lane%6) in two passes of 32
    const int bi0 = lane / 6, bt0 = lane - 6 * bi0, bi1 = (lane + 32) / 6, bt1 = lane + 32 - 6 * bi1;
    for (int w = blockIdx.x; w < q.nwork && ok; w += gridDim.x, ++it) {
      const int q0 = (w % q.ntm) * TILE_M;
      const int n0 = (w / q.ntm) * q.bn;
      const int vq = q0 + lq * 32 + lane;        // accumulator row = virtual position
      bool valid = false;
      float* yrow = q.y;
      int o = 0;                                 // index of the row's output inside its plane
      if (vq < q.VQ) {
        const int sg = vq / q.Wq;
        const int kq = vq - sg * q.Wq;
        const int n = sg / q.Ho;
        const int ho = sg - n * q.Ho;
        valid = kq < q.Wo;                       // trailing columns of a strip are no output
        o = ho * q.Wo + kq;
        yrow += ((int64_t)n * q.Co + n0) * q.HoWo + o;
      }
      // The tile's outputs: first and last valid position (the same for every thread).  When both lie
      // in one image the outputs are ONE contiguous run of each output plane, [o0, o0 + nv).
      bool staged = false;
      int o0 = 0, nv = 0;
      int64_t plane0 = 0;
      if constexpr (STAGED) {
        const int sgF0 = q0 / q.Wq, kqF0 = q0 - sgF0 * q.Wq;
        const int sgF = kqF0 < q.Wo ? sgF0 : sgF0 + 1;         // a tile that starts on a dropped column
        const int kqF = kqF0 < q.Wo ? kqF0 : 0;
        const int nF = sgF / q.Ho, hoF = sgF - nF * q.Ho;
        const int vqL = q0 + TILE_M - 1 < q.VQ - 1 ? q0 + TILE_M - 1 : q.VQ - 1;
        const int sgL = vqL / q.Wq, kqL0 = vqL - sgL * q.Wq;
        const int kqL = kqL0 < q.Wo ? kqL0 : q.Wo - 1;
        const int nL = sgL / q.Ho, hoL = sgL - nL * q.Ho;
        o0 = hoF * q.Wo + kqF;
        nv = hoL * q.Wo + kqL - o0 + 1;
        staged = nF == nL && nF < q.N && nv > 0;
        plane0 = ((int64_t)nF * q.Co + n0) * q.HoWo;
      }
      if (lane == 0) ok = mbar_wait(acc_full0 + 8 * buf, eph, &abort_flag, q.status);
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
      __syncwarp();   // lane 0 observed the barrier: orders the other lanes' accesses after it
      if constexpr (STAGED) {
        uint32_t all_ok;
        asm volatile(
            "{\n\t.reg .pred p, pq;\n\t"
            "setp.ne.b32 pq, %1, 0;\n\t"
            "bar.red.and.pred p, 1, 128, pq;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(all_ok)
            : "r"((uint32_t)ok)
            : "memory");
        ok = all_ok != 0;
      }
      if (!ok) break;
      if (threadIdx.x == WARP_EPI0 * 32) TIMER_LAP(7);   // epilogue: address arithmetic, wait for the accumulator
      tc_fence_after();
      const uint32_t lane_base = tmem_acc + buf * (uint32_t)q.bnr + ((uint32_t)(lq * 32) << 16);
      const int nco = q.Co - n0 < q.bn ? q.Co - n0 : q.bn;   // real channels of this tile
      if ((!STAGED || !staged) && nco > 64) {
#pragma unroll 1
        for (int c0 = 0; c0 < nco; c0 += 32) {
          uint32_t v[32];
          tmem_ld32(lane_base + (uint32_t)c0, v);
          if (valid) store_strided32(yrow + (int64_t)c0 * q.HoWo, q.HoWo, v, nco - c0);
        }
      } else if (!STAGED || !staged) {
        // up to 64 channels: both tensor-memory loads are in flight together (one costs the warp some
        // 500 cycles when the tensor core is busy with the next tiles); measured 1-3 % on the 64-channel
        // stems, while wider tiles (96 channels: a dual round and a single one) lost 8 % with it
#pragma unroll 1
        for (int c0 = 0; c0 < nco; c0 += 64) {
          uint32_t v[32], v2[32];
          tmem_ld32_issue(lane_base + (uint32_t)c0, v);
          const bool second = c0 + 32 < nco;
          if (second) tmem_ld32_issue(lane_base + (uint32_t)(c0 + 32), v2);
          tmem_ld_wait();
          if (valid) {
            store_strided32(yrow + (int64_t)c0 * q.HoWo, q.HoWo, v, nco - c0);
            if (second) store_strided32(yrow + (int64_t)(c0 + 32) * q.HoWo, q.HoWo, v2, nco - c0 - 32);
          }
        }
      } else if constexpr (STAGED) {
        // Through the staging buffer: the rows are compacted (dropped columns leave no gap) and every
        // plane is shifted by the 16-byte phase of its run, so that the run can be written with aligned
        // 16-byte stores.  Plane c0 + j starts (g0 + j*hw) mod 4 floats after a 16-byte boundary (c0 is a
        // multiple of 32); warp lq writes planes lq, lq + 4, ..., which all have the same phase.
        const uint32_t g0 = (uint32_t)((plane0 + o0) & 3);
        const uint32_t hw = (uint32_t)q.HoWo & 3u;
        const int h = (int)((g0 + (uint32_t)lq * hw) & 3u);
        const int e0 = 4 * lane - h;                         // run element of the lane's first float
        const bool full = e0 >= 0 && e0 + 3 < nv;
        const int nhead = h ? 4 - h : 0;                     // floats before the first 16-byte boundary
        const int tail0 = (h + nv) & ~3, ntail = (h + nv) & 3;   // floats after the last one start at column tail0
#pragma unroll 1
        for (int c0 = 0; c0 < nco && ok; c0 += 32) {
          uint32_t v[32];
          tmem_ld32(lane_base + (uint32_t)c0, v);
          if (threadIdx.x == WARP_EPI0 * 32) TIMER_LAP(12);   // tmem load
          const uint32_t stage = epi_ring + (q.epi_bufs == 2 ? (chunk_ctr & 1u) : 0u) * EPI_BUF_BYTES;
          ++chunk_ctr;
          if (q.epi_bufs == 1) epi_sync();                    // the readers of the last chunk are done
          if (valid) {
            uint32_t colb[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) colb[k] = stage + (uint32_t)((o - o0) + (int)((g0 + (uint32_t)k * hw) & 3u)) * 4u;
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (c0 + j < nco)
                asm volatile("st.shared.b32 [%0], %1;" ::"r"(colb[j & 3] + (uint32_t)(j * EPI_PITCH * 4)), "r"(v[j])
                             : "memory");
          }
          if (threadIdx.x == WARP_EPI0 * 32) TIMER_LAP(13);   // staging stores
          epi_sync();                                        // the chunk is staged
          if (threadIdx.x == WARP_EPI0 * 32) TIMER_LAP(14);   // barrier
          // per lane, the same for every plane: 16-byte store, or which of its four floats exist
          {
            const uint32_t src0 = stage + (uint32_t)(lq * EPI_PITCH * 4) + 16u * lane;
            float* gp0 = q.y + plane0 + (int64_t)(c0 + lq) * q.HoWo + (o0 - h) + 4 * lane;   // 16-byte aligned
            const int nplanes = (nco - c0 - lq + 3) >> 2 < 8 ? (nco - c0 - lq + 3) >> 2 : 8;   // planes lq, lq+4, .. < nco
            const int64_t pstep = (int64_t)4 * q.HoWo;
            uint32_t f[8][4];
#pragma unroll
            for (int i = 0; i < 8; ++i)
              if (i < nplanes)
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(f[i][0]), "=r"(f[i][1]), "=r"(f[i][2]), "=r"(f[i][3])
                             : "r"(src0 + (uint32_t)(i * 4 * EPI_PITCH * 4)));
            if (full) {
#pragma unroll
              for (int i = 0; i < 8; ++i)
                if (i < nplanes)
                  *reinterpret_cast<float4*>(gp0 + i * pstep) = make_float4(
                      __uint_as_float(f[i][0]), __uint_as_float(f[i][1]), __uint_as_float(f[i][2]), __uint_as_float(f[i][3]));
            }
            if (threadIdx.x == WARP_EPI0 * 32) TIMER_LAP(15);   // reads + stores
            // The ragged ends of the runs (at most three floats before the first and after the last
            // 16-byte boundary) of all eight planes go out in two store instructions, lane = (plane,
            // end element): a store instruction costs the warp some 30 cycles however few lanes it
            // has, so one instruction per element and plane would double the epilogue's time.
#pragma unroll
            for (int pass = 0; pass < 2; ++pass) {
              const int i = pass ? bi1 : bi0, t = pass ? bt1 : bt0;
              const int col = t < 3 ? h + t : tail0 + t - 3;
              const bool exists = i < nplanes && (t < 3 ? (t < nhead && col < h + nv) : (t - 3 < ntail && col >= h));
              if (exists) {
                uint32_t x;
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(x) : "r"(stage + (uint32_t)(((lq + 4 * i) * EPI_PITCH + col) * 4)));
                (q.y + plane0 + (int64_t)(c0 + lq + 4 * i) * q.HoWo + (o0 - h))[col] = __uint_as_float(x);
              }
            }
          }
        }
        if (!ok) break;
      }
      // the buffer may be overwritten once all four warps have read it
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty0 + 8 * buf);
      if (++buf == (uint32_t)q.sa) { buf = 0; eph ^= 1u; }
      if (threadIdx.x == WARP_EPI0 * 32) TIMER_LAP(8);   // epilogue: tensor memory -> global
    }
    if (threadIdx.x == WARP_EPI0 * 32) TIMER_FLUSH();
  }

  // ---------------- teardown ---------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == WARP_MMA) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_acc, (uint32_t)q.tmem_cols);
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

constexpr int kSmemMax = 227 * 1024;
constexpr int kStaticSmem = 3 * 1024;        // barriers, segment copies, tables (rounded up)

}  // namespace

StemPlan plan_f16_stem(const Geometry& g) {
  StemPlan p{};
  p.eligible = false;
  const int64_t K2 = (int64_t)g.C * g.Kh;
  if (K2 > KB) return p;
  p.Wq = (g.Wp + g.s - 1) / g.s;
  p.ragged = g.Wp % g.s != 0;
  p.rows = TILE_M + (g.Kw - 1) / g.s;
  p.R = (p.rows + 7) / 8 * 8;
  p.nks = (int32_t)((K2 + 15) / 16);
  p.VQ = (int64_t)g.N * g.Ho * p.Wq;
  if (p.VQ >= ((int64_t)1 << 31) - 4 * TILE_M) return p;        // 32-bit position arithmetic
  const int64_t seg_rows = p.ragged ? p.Wq : (int64_t)g.Ho * p.Wq;
  if ((p.rows - 2) / seg_rows + 2 > SEG_MAX) return p;
  const int64_t skh = (int64_t)g.s * g.Kh;
  if ((int64_t)p.rows * skh * 2 > 64 * 1024) return p;
  p.chan_region = (int32_t)((((int64_t)p.rows * skh * 2 + 15) & ~(int64_t)15) + SEG_GAP * SEG_MAX + 32);
  p.raw_stage_bytes = g.C * p.chan_region;
  p.a_stage_bytes = (g.s * 2 * p.nks * p.R * 16 + 127) / 128 * 128;
  p.bn = g.Co >= 256 ? 256 : (g.Co + 15) / 16 * 16;
  p.b_stage_bytes = p.bn * KB * 2;
  const int nct = (g.Co + p.bn - 1) / p.bn;
  if ((p.VQ + TILE_M - 1) / TILE_M * nct >= ((int64_t)1 << 31)) return p;
  // rings: S stages (= accumulators) 2, raw 2, filter resident if one channel tile and its Kw tiles
  // fit, else 2..4 stages; then what is left goes to a third raw stage and to more S stages
  const int budget = kSmemMax - 1024 - kStaticSmem;
  const int base = 2 * p.a_stage_bytes + 2 * p.raw_stage_bytes;
  const int bnr = (p.bn + 31) / 32 * 32;
  p.sa = 2;
  p.rs = 2;
  p.resident = 0;
  if (nct == 1 && g.Kw <= MAX_B && base + g.Kw * p.b_stage_bytes <= budget) {
    p.resident = 1;
    p.sb = g.Kw;
  } else {
    p.sb = 4;
    while (p.sb > 2 && base + p.sb * p.b_stage_bytes > budget) --p.sb;
    if (base + p.sb * p.b_stage_bytes > budget) return p;
  }
  int used = base + p.sb * p.b_stage_bytes;
  if (used + p.raw_stage_bytes <= budget) { p.rs = 3; used += p.raw_stage_bytes; }
  while (p.sa < MAX_STAGES && (p.sa + 1) * bnr <= 512 && used + p.a_stage_bytes <= budget) {
    ++p.sa;
    used += p.a_stage_bytes;
  }
  // three raw stages by default (measured: eight in flight slow a 3-channel 3x3 layer down from 1.01 ms
  // to 1.27 ms, as a second CTA per SM does); IM2WIN_F16_STEM_RAW = 2..8 sets another depth (a testing aid)
  const char* force_rs = debug_getenv("IM2WIN_F16_STEM_RAW");
  // (per-strip runs are many small copies: a fourth stage pays there, 273 -> 250 us on the 7x7 stride-2
  // layer with 227-wide strips; with per-image runs it changes nothing or costs, see above)
  const int rs_max = force_rs && atoi(force_rs) >= 2 && atoi(force_rs) <= MAX_RAW ? atoi(force_rs) : (p.ragged ? 4 : 3);
  if (rs_max < p.rs) { used -= (p.rs - rs_max) * p.raw_stage_bytes; p.rs = rs_max; }
  while (p.rs < rs_max && (p.rs + 1) * p.raw_stage_bytes <= 48 * 1024 && used + p.raw_stage_bytes <= budget) {
    ++p.rs;
    used += p.raw_stage_bytes;
  }

  const char* force_sa = debug_getenv("IM2WIN_F16_STEM_STAGES");   // testing aid: S stages / accumulators (2..4)
  if (force_sa && atoi(force_sa) >= 2 && atoi(force_sa) < p.sa) p.sa = atoi(force_sa);
  // Staging buffers of the aligned-store epilogue.  Off by default: measured, the staged path is exact
  // but twice as slow as storing from the registers (cfg3 300 us against 155 us: the two passes through
  // shared memory and the second tensor-memory round trip cost the epilogue warps more than the aligned
  // stores save).  IM2WIN_F16_STEM_EPI=1|2 turns it on with one or two buffers where they fit (tests do).
  p.epi_bufs = 0;
  const char* want_epi = debug_getenv("IM2WIN_F16_STEM_EPI");
  const int epi_want = want_epi ? atoi(want_epi) : 0;
  if (epi_want >= 2 && used + 2 * EPI_BUF_BYTES <= budget) p.epi_bufs = 2;
  else if (epi_want >= 1 && used + EPI_BUF_BYTES <= budget) p.epi_bufs = 1;
  p.smem_bytes = p.sa * p.a_stage_bytes + p.rs * p.raw_stage_bytes + p.sb * p.b_stage_bytes +
                 p.epi_bufs * EPI_BUF_BYTES + 1024;
  p.eligible = true;
  return p;
}

cudaError_t launch_conv_f16_stem(const uint16_t* window, float* y, void* scratch, const Geometry& g,
                                 const ScratchLayout& l, cudaStream_t stream) {
  const StemPlan plan = plan_f16_stem(g);
  if (!plan.eligible) return cudaErrorInvalidValue;
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return cudaErrorNotSupported;
  unsigned char* base = static_cast<unsigned char*>(scratch);

  // Filter as Fp2[v][co][64] halves: a 3-D tensor (k2 fastest), one box = 64 k2 x bn channels of one v.
  CUtensorMap fmap;
  const cuuint64_t dims[3] = {(cuuint64_t)KB, (cuuint64_t)g.Co, (cuuint64_t)g.Kw};
  const cuuint64_t strides[2] = {(cuuint64_t)KB * 2, (cuuint64_t)KB * 2 * (cuuint64_t)g.Co};
  const cuuint32_t box[3] = {(cuuint32_t)KB, (cuuint32_t)plan.bn, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  CUresult cr = encode(&fmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, base + l.filter_off, dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (cr != CUDA_SUCCESS) return cudaErrorInvalidValue;

  StemParams q;
  q.win = window;
  q.y = y;
  q.status = reinterpret_cast<uint32_t*>(base);
  q.chan_stride = g.chan_stride; q.img_stride = g.img_stride; q.strip = g.strip; q.window_elems = g.window_elems;
  q.VQ = (int32_t)plan.VQ; q.C = g.C; q.N = g.N; q.Wq = plan.Wq; q.Wp = g.Wp; q.Ho = g.Ho; q.Wo = g.Wo;
  q.HoWo = g.Ho * g.Wo; q.Co = g.Co; q.Kh = g.Kh; q.Kw = g.Kw; q.s = g.s;
  q.sKh = g.s * g.Kh; q.K2 = g.C * g.Kh;
  q.rows = plan.rows; q.R = plan.R; q.nks = plan.nks; q.chunks = 2 * plan.nks; q.ragged = plan.ragged;
  q.chan_region = plan.chan_region; q.raw_stage_bytes = plan.raw_stage_bytes;
  q.a_stage_bytes = plan.a_stage_bytes; q.b_stage_bytes = plan.b_stage_bytes;
  q.bn = plan.bn; q.bnr = (plan.bn + 31) / 32 * 32;
  q.tmem_cols = 32;
  while (q.tmem_cols < plan.sa * q.bnr) q.tmem_cols *= 2;
  q.idesc = instr_desc_f16(TILE_M, plan.bn);
  q.rs = plan.rs; q.sa = plan.sa; q.sb = plan.sb; q.resident = plan.resident;
  const int64_t ntm = (plan.VQ + TILE_M - 1) / TILE_M;
  q.ntm = (int32_t)ntm;
  q.nwork = (int32_t)(ntm * ((g.Co + plan.bn - 1) / plan.bn));
  q.epi_bufs = plan.epi_bufs;
  q.cbits = 0;
  while ((1 << q.cbits) < g.C) ++q.cbits;

  const char* generic = debug_getenv("IM2WIN_F16_STEM_GENERIC");   // testing aid: the table-driven re-layout everywhere
  int kh = (g.C == 3 && g.Kh == g.Kw && !(generic && atoi(generic))) ? g.Kh : 0;   // the common stems: square kernels on 3 channels
  if (kh != 3 && kh != 5 && kh != 7 && kh != 11) kh = 0;
  void (*kernel)(const CUtensorMap, StemParams);
  if (plan.epi_bufs > 0)
    kernel = kh == 3 ? conv_f16_stem_kernel<3, 3, 3, true> : kh == 5 ? conv_f16_stem_kernel<3, 5, 5, true>
           : kh == 7 ? conv_f16_stem_kernel<3, 7, 7, true> : kh == 11 ? conv_f16_stem_kernel<3, 11, 11, true>
                                                                      : conv_f16_stem_kernel<0, 0, 0, true>;
  else
    kernel = kh == 3 ? conv_f16_stem_kernel<3, 3, 3, false> : kh == 5 ? conv_f16_stem_kernel<3, 5, 5, false>
           : kh == 7 ? conv_f16_stem_kernel<3, 7, 7, false> : kh == 11 ? conv_f16_stem_kernel<3, 11, 11, false>
                                                                      : conv_f16_stem_kernel<0, 0, 0, false>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, plan.smem_bytes);
  if (e != cudaSuccess) return e;
  // persistent CTAs: one per SM (measured: a second CTA per SM, where it fits, only slows the layer
  // down, 1.30 ms against 1.00 ms on a 3-channel 3x3 layer); IM2WIN_F16_STEM_CTAS=2 asks for two (a testing aid)
  int per_sm = 1;
  const char* force = debug_getenv("IM2WIN_F16_STEM_CTAS");
  if (force && atoi(force) == 2) {
    per_sm = (kSmemMax + 1024) / (plan.smem_bytes + kStaticSmem + 1024);
    if (per_sm > 512 / q.tmem_cols) per_sm = 512 / q.tmem_cols;
    if (per_sm > 2) per_sm = 2;
    if (per_sm < 1) per_sm = 1;
  }
  const int slots = 148 * per_sm;
  const unsigned grid = (unsigned)(q.nwork < slots ? q.nwork : slots);
  kernel<<<grid, NUM_THREADS, plan.smem_bytes, stream>>>(fmap, q);
  return cudaGetLastError();
}

}  // namespace im2win
