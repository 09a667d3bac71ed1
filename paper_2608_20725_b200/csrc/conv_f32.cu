// fp32 im2win convolution on CUDA cores (paper Eq. 3, "CC" variant) for sm_100a.
//
// GEMM view (Algorithm 1's dimensions with positions as rows):
//     y[p][co] = sum_k A[p][k] * Fk[k][co],  p = (n, ho, wo),  k = (c, v, u),
//     A[p][k]  = window[n][c][ho][(wo*s)*Kh + v*Kh + u].
// A CTA computes a BM x BN tile of y.  Per k-block of 16 it gathers the A tile
// from the window tensor (lanes walk consecutive positions, i.e. addresses
// s*Kh elements apart inside one strip; the k -> offset table is precomputed)
// and the Fk tile (contiguous) into a three-slot shared-memory ring with
// asynchronous copies (cp.async: no registers, two k-blocks in flight while the
// current one is multiplied).  Each thread accumulates an 8 x 8 register tile with 128-bit
// shared-memory loads (2 x 4 positions by 2 x 4 output channels).  The tile is
// held as 8 x 4 pairs of adjacent output channels and updated with the packed
// fma.rn.f32x2 instruction: one issue slot per two FMAs (the FMA pipe rate is
// unchanged -- measured 74 TFLOP/s for both forms -- but the kernel is bound by
// issue slots, which the packed form halves).  Positions run along the lanes,
// so stores to the NCHW output are contiguous per output channel.
// Large layers (128-position tiles) take a second form with a 16 x 8 register tile whose pairs are
// adjacent POSITIONS (conv_f32_tall_kernel below).
#include "common.cuh"

namespace im2win {
namespace {

struct ConvF32Params {
  const float* __restrict__ win;
  const float* __restrict__ fk;      // [Kp][Co_pad]
  const int32_t* __restrict__ koff;  // [Kp]
  float* __restrict__ y;
  int64_t P, img_stride, strip;
  int32_t HoWo, Wo, sKh, Co, Co_pad, Kp;
};


__device__ __forceinline__ void ffma2(unsigned long long& d, unsigned long long a, unsigned long long b) {
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b));
}
__device__ __forceinline__ unsigned long long dup2(float a) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %1};" : "=l"(r) : "f"(a));
  return r;
}
__device__ __forceinline__ float2 unpack2(unsigned long long v) {
  float2 r;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(r.x), "=f"(r.y) : "l"(v));
  return r;
}

// Position p -> (image n, offset r inside the image's Ho*Wo outputs).  A 64-bit division costs about a
// hundred instructions; with fewer than 2^31 positions (every layer but the very largest) a 32-bit one does.
__device__ __forceinline__ void split_position(int64_t p, const ConvF32Params& q, int64_t& n, int& r) {
  if (q.P < ((int64_t)1 << 31)) {
    const uint32_t nq = (uint32_t)p / (uint32_t)q.HoWo;
    n = nq;
    r = (int)((uint32_t)p - nq * (uint32_t)q.HoWo);
  } else {
    n = p / q.HoWo;
    r = (int)(p - n * q.HoWo);
  }
}

// Threads along the channel direction of a BM x BN tile: every thread holds 8 positions x 8 channels, or,
// for the 96-channel tile (layers of 96, 192, ... output channels, which 64- and 128-channel tiles would
// pad by a third), 8 x 6: four channels from the tile's first 64 and two from its last 32.
__host__ __device__ constexpr int f32_tn(int bn) { return bn == 96 ? 16 : bn / 8; }

// BK: the k-block, 16 or 32 (see plan_f32).  KLANES: which way the window operand is gathered.  false: the
// lanes of a warp are 32 consecutive positions at one k (their elements lie s*Kh apart).  true: the lanes
// are 8 consecutive k (contiguous in the im2win tensor within a channel) of 4 consecutive positions, so a
// copy instruction touches about four 32-byte sectors instead of one per lane; shared-memory rows are
// BM + 4 words apart so that the 32 lanes still write 32 different banks.  Measured: with windows 176
// bytes apart (11x11, stride 4) 10 % faster; 3 % SLOWER where windows lie 12-56 bytes apart (the sectors
// of neighbouring positions overlap anyway, and every thread then tracks several positions).
template <int BM, int BN, int BK, bool KLANES>
__global__ void __launch_bounds__((BM / 8) * f32_tn(BN), ((BM / 8) * f32_tn(BN) == 256 ? 2 : 3))
conv_f32_kernel(ConvF32Params q) {
  constexpr int THREADS = (BM / 8) * f32_tn(BN);
  constexpr int NPT = BN / f32_tn(BN);                     // channels per thread: 8 or 6
  constexpr int NP2 = NPT / 2;                             // ... as pairs
  constexpr int LO = BN == 96 ? 64 : BN / 2;               // channels of the first group (four per thread)
  constexpr int A_PER_THREAD = BK * BM / THREADS;         // scalar gathers per k-block
  constexpr int A_KK_STEP = THREADS / BM;                 // 2 (256 threads) or 1 (128 threads)
  constexpr int KG = BK / 8;                              // KLANES: groups of eight consecutive k per k-block,
  constexpr int NPOS = A_PER_THREAD / KG;                 // positions per loader thread,
  constexpr int APITCH = KLANES ? BM + 4 : BM;            // row pitch of the window operand in shared memory
  static_assert(!KLANES || (NPOS >= 1 && (THREADS / 32) * NPOS * 4 == BM), "loader mapping (k along lanes)");
  constexpr int B_VEC_PER_THREAD = (BK * BN / 4 + THREADS - 1) / THREADS; // float4 loads per k-block
  static_assert(THREADS % BM == 0 && A_PER_THREAD * A_KK_STEP == BK, "loader mapping");

  constexpr int STAGES = 3;          // shared-memory ring filled by asynchronous copies
  extern __shared__ __align__(16) unsigned char smem_f32[];
  float (*As)[BK][APITCH] = reinterpret_cast<float (*)[BK][APITCH]>(smem_f32);
  float (*Bs)[BK][BN] = reinterpret_cast<float (*)[BK][BN]>(smem_f32 + sizeof(float) * STAGES * BK * APITCH);

  const int tid = threadIdx.x;
  const int tm = tid % (BM / 8);     // position direction: fastest across lanes
  const int tn = tid / (BM / 8);
  const int64_t m0 = (int64_t)blockIdx.x * BM;
  const int n0 = blockIdx.y * BN;

  // Loader role: one fixed position (row of A) per thread, or (KLANES) NPOS positions lm + 4 j and
  // the k's kq + 8 g of every k-block.
  constexpr int NBASE = KLANES ? NPOS : 1;
  constexpr int NOFF = KLANES ? KG : A_PER_THREAD;
  const int kq = tid & 7;
  const int lm = KLANES ? (tid >> 5) * (NPOS * 4) + ((tid >> 3) & 3) : tid % BM;
  const int lkk0 = tid / BM;
  const float* abase[NBASE];
  uint32_t lvalid = 0;
#pragma unroll
  for (int j = 0; j < NBASE; ++j) {
    const int64_t lp = m0 + lm + 4 * j;
    abase[j] = q.win;
    if (lp < q.P) {
      int64_t n;
      int r;
      split_position(lp, q, n, r);
      const int ho = r / q.Wo;
      const int wo = r - ho * q.Wo;
      abase[j] += n * q.img_stride + ho * q.strip + (int64_t)wo * q.sKh;
      lvalid |= 1u << j;
    }
  }

  int offreg[NOFF];                  // offsets of the next k-block to be issued

  // The offset table is read one k-block ahead of the copies it addresses, so that issuing
  // the copies never waits for it.
  auto load_offsets = [&](int kb) {
    const int k0 = kb * BK;
#pragma unroll
    for (int i = 0; i < NOFF; ++i) offreg[i] = __ldg(q.koff + k0 + (KLANES ? i * 8 + kq : lkk0 + i * A_KK_STEP));
  };
  // Asynchronous copies (global -> shared, no registers) of k-block kb into ring slot `buf`:
  // 4-byte gathers of the window operand (zero-filled outside the tensor and in the padded
  // tail of k), 16-byte copies of the filter rows.
  auto issue_copies = [&](int kb, int buf, bool more) {
    const int k0 = kb * BK;
#pragma unroll
    for (int i = 0; i < NOFF; ++i) {
      const int off = offreg[i];
#pragma unroll
      for (int j = 0; j < NBASE; ++j) {
        const bool ok = ((lvalid >> j) & 1u) && off >= 0;
        const float* src = ok ? abase[j] + off : q.win;
        const uint32_t dst = (uint32_t)__cvta_generic_to_shared(
            KLANES ? &As[buf][i * 8 + kq][lm + 4 * j] : &As[buf][lkk0 + i * A_KK_STEP][lm]);
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(ok ? 4 : 0) : "memory");
      }
    }
#pragma unroll
    for (int i = 0; i < B_VEC_PER_THREAD; ++i) {
      const int e = tid + i * THREADS;       // float4 index inside the BK x BN tile
      if ((BK * BN / 4) % THREADS != 0 && e >= BK * BN / 4) break;
      const int kk = e / (BN / 4);
      const int nn = (e - kk * (BN / 4)) * 4;
      const float* src = q.fk + (int64_t)(k0 + kk) * q.Co_pad + n0 + nn;
      const uint32_t dst = (uint32_t)__cvta_generic_to_shared(&Bs[buf][kk][nn]);
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
    }
    if (more) load_offsets(kb + 1);
  };

  unsigned long long acc2[8][NP2];   // acc2[i][jp] = (acc[i][2jp], acc[i][2jp+1])
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int jp = 0; jp < NP2; ++jp) acc2[i][jp] = 0ull;

  const int nkb = q.Kp / BK;
  load_offsets(0);
#pragma unroll
  for (int s = 0; s < STAGES - 1; ++s) {
    if (s < nkb) issue_copies(s, s, s + 1 < nkb);
    asm volatile("cp.async.commit_group;" ::: "memory");
  }

  int buf = 0;                        // ring slot of k-block kb
  for (int kb = 0; kb < nkb; ++kb) {
    asm volatile("cp.async.wait_group %0;" ::"n"(STAGES - 2) : "memory");
    __syncthreads();                  // k-block kb has landed for everyone; slot (kb-1) is free
    {
      const int nk = kb + STAGES - 1;
      int nbuf = buf + STAGES - 1;
      if (nbuf >= STAGES) nbuf -= STAGES;
      if (nk < nkb) issue_copies(nk, nbuf, nk + 1 < nkb);
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      const float4 a0 = *reinterpret_cast<const float4*>(&As[buf][kk][tm * 4]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[buf][kk][BM / 2 + tm * 4]);
      const ulonglong2 b0 = *reinterpret_cast<const ulonglong2*>(&Bs[buf][kk][tn * 4]);
      unsigned long long b[4];
      b[0] = b0.x; b[1] = b0.y;
      if (NPT == 8) {
        const ulonglong2 b1 = *reinterpret_cast<const ulonglong2*>(&Bs[buf][kk][LO + tn * 4]);
        b[2] = b1.x; b[3] = b1.y;
      } else {
        b[2] = *reinterpret_cast<const unsigned long long*>(&Bs[buf][kk][LO + tn * 2]);
        b[3] = 0ull;
      }
      const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const unsigned long long ad = dup2(a[i]);
#pragma unroll
        for (int jp = 0; jp < NP2; ++jp) ffma2(acc2[i][jp], ad, b[jp]);
      }
    }
    if (++buf == STAGES) buf = 0;
  }

  float acc[8][NPT];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int jp = 0; jp < NP2; ++jp) {
      const float2 v = unpack2(acc2[i][jp]);
      acc[i][2 * jp] = v.x;
      acc[i][2 * jp + 1] = v.y;
    }

  // Epilogue: positions of one half-tile are 4 consecutive p; NCHW output is
  // contiguous in p within an image for a fixed output channel.
  const bool vec_ok = (q.HoWo % 4) == 0;
#pragma unroll
  for (int hm = 0; hm < 2; ++hm) {
    const int64_t p = m0 + hm * (BM / 2) + tm * 4;
    if (p >= q.P) continue;
    int64_t n;
    int r;
    split_position(p, q, n, r);
    // (image, offset) of the four positions: the offset advances by one and wraps into the next image
    int64_t nn[4];
    int rr[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      nn[i] = n; rr[i] = r + i;
      while (rr[i] >= q.HoWo) { rr[i] -= q.HoWo; ++nn[i]; }
    }
#pragma unroll
    for (int j = 0; j < NPT; ++j) {
      const int co = j < 4 ? n0 + tn * 4 + j : n0 + LO + tn * (NPT - 4) + (j - 4);
      if (co >= q.Co) continue;
      if (vec_ok) {
        float4 v = make_float4(acc[hm * 4 + 0][j], acc[hm * 4 + 1][j], acc[hm * 4 + 2][j], acc[hm * 4 + 3][j]);
        *reinterpret_cast<float4*>(q.y + (n * q.Co + co) * q.HoWo + r) = v;
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (p + i >= q.P) break;
          q.y[(nn[i] * q.Co + co) * q.HoWo + rr[i]] = acc[hm * 4 + i][j];
        }
      }
    }
  }
}


// Second form of the same kernel: 16 positions x 8 channels per thread, accumulators packed as pairs of
// adjacent POSITIONS.  The pairs come straight out of the 128-bit loads of the window operand; only the
// eight filter values of a k are duplicated with moves: per 128 FMAs 64 fma.rn.f32x2 + 8 moves + 6 shared
// loads against 64 + 16 + 8 in the 8 x 8 form, i.e. 6 % fewer FMA-pipe cycles and 11 % fewer issue slots.
// (BM/16)*(BN/8) threads: 64 for the 128 x 64 and 64 x 128 tiles, 128 for 128 x 128.  The register cap of 200
// keeps five 64-thread CTAs on an SM (206 registers uncapped: four CTAs, and 2 % slower than the 8 x 8 form
// instead of 5 % faster; a cap of 168: spills, 30 % slower).  Every loader thread tracks BM/threads positions;
// the offsets of the next k-block are prefetched as in the first form.
// 96-channel tiles: 16 x 6 per thread (channels as in the first form); KLANES as in the first form.
// STAGED: the epilogue for outputs whose rows do not start on 16-byte boundaries (Ho*Wo no multiple of 4; a
// kernel of its own, so that the aligned form's registers are not shared with it).
template <int BM, int BN, int BK, bool KLANES, bool STAGED>
__global__ void __maxnreg__(BN == 96 ? 168 : 200)      // (96-channel tiles: 128 threads of 96 accumulators, three CTAs per SM)
conv_f32_tall_kernel(ConvF32Params q) {
  constexpr int THREADS = (BM / 16) * f32_tn(BN);
  constexpr int NPT = BN / f32_tn(BN);                     // channels per thread: 8 or 6
  constexpr int LO = BN == 96 ? 64 : BN / 2;               // channels of the first group (four per thread)
  constexpr int KG = BK / 8;                               // KLANES: groups of eight consecutive k per k-block
  constexpr int NPOS = KLANES ? BK * BM / THREADS / KG : BM / THREADS;   // positions per loader thread
  constexpr int NOFF = KLANES ? KG : BK;                   // offsets per loader thread and k-block
  constexpr int APITCH = KLANES ? BM + 4 : BM;
  constexpr int B_VEC_PER_THREAD = BK * BN / 4 / THREADS;
  static_assert((KLANES ? (THREADS / 32) * NPOS * 4 == BM : BM % THREADS == 0) && (BK * BN / 4) % THREADS == 0, "loader mapping");
  constexpr int STAGES = 3;
  extern __shared__ __align__(16) unsigned char smem_f32[];
  float (*As)[BK][APITCH] = reinterpret_cast<float (*)[BK][APITCH]>(smem_f32);
  float (*Bs)[BK][BN] = reinterpret_cast<float (*)[BK][BN]>(smem_f32 + sizeof(float) * STAGES * BK * APITCH);

  const int tid = threadIdx.x;
  const int tm = tid % (BM / 16);
  const int tn = tid / (BM / 16);
  const int64_t m0 = (int64_t)blockIdx.x * BM;
  const int n0 = blockIdx.y * BN;

  // loader: positions lm + lstep*j; (KLANES) the k's kq + 8 g of every k-block, else all of them
  const int kq = tid & 7;
  const int lm = KLANES ? (tid >> 5) * (NPOS * 4) + ((tid >> 3) & 3) : tid;
  constexpr int lstep = KLANES ? 4 : THREADS;
  const float* abase[NPOS];
  uint32_t lvalid = 0;
#pragma unroll
  for (int j = 0; j < NPOS; ++j) {
    const int64_t lp = m0 + lm + j * lstep;
    abase[j] = q.win;
    if (lp < q.P) {
      int64_t n;
      int r;
      split_position(lp, q, n, r);
      const int ho = r / q.Wo;
      const int wo = r - ho * q.Wo;
      abase[j] += n * q.img_stride + ho * q.strip + (int64_t)wo * q.sKh;
      lvalid |= 1u << j;
    }
  }
  int offreg[NOFF];
  auto load_offsets = [&](int kb) {
#pragma unroll
    for (int i = 0; i < NOFF; ++i) offreg[i] = __ldg(q.koff + kb * BK + (KLANES ? i * 8 + kq : i));
  };
  auto issue_copies = [&](int kb, int buf) {
    const int k0 = kb * BK;
#pragma unroll
    for (int i = 0; i < NOFF; ++i) {
      const int off = offreg[i];
#pragma unroll
      for (int j = 0; j < NPOS; ++j) {
        const bool ok = ((lvalid >> j) & 1u) && off >= 0;
        const float* src = ok ? abase[j] + off : q.win;
        const uint32_t dst = (uint32_t)__cvta_generic_to_shared(&As[buf][KLANES ? i * 8 + kq : i][lm + j * lstep]);
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(ok ? 4 : 0) : "memory");
      }
    }
#pragma unroll
    for (int i = 0; i < B_VEC_PER_THREAD; ++i) {
      const int e = tid + i * THREADS;
      const int kk = e / (BN / 4);
      const int nn = (e - kk * (BN / 4)) * 4;
      const float* src = q.fk + (int64_t)(k0 + kk) * q.Co_pad + n0 + nn;
      const uint32_t dst = (uint32_t)__cvta_generic_to_shared(&Bs[buf][kk][nn]);
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
    }
    if (kb + 1 < q.Kp / BK) load_offsets(kb + 1);
  };
  load_offsets(0);

  unsigned long long acc2[8][NPT];   // acc2[ip][j] = (acc[2 ip][j], acc[2 ip + 1][j]): position pairs
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < NPT; ++j) acc2[i][j] = 0ull;

  const int nkb = q.Kp / BK;
#pragma unroll
  for (int s = 0; s < STAGES - 1; ++s) {
    if (s < nkb) issue_copies(s, s);
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  int buf = 0;
  for (int kb = 0; kb < nkb; ++kb) {
    asm volatile("cp.async.wait_group %0;" ::"n"(STAGES - 2) : "memory");
    __syncthreads();
    {
      const int nk = kb + STAGES - 1;
      int nbuf = buf + STAGES - 1;
      if (nbuf >= STAGES) nbuf -= STAGES;
      if (nk < nkb) issue_copies(nk, nbuf);
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      unsigned long long a[8];
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(&As[buf][kk][g * (BM / 4) + tm * 4]);
        a[2 * g] = v.x; a[2 * g + 1] = v.y;
      }
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[buf][kk][tn * 4]);
      float b[8] = {b0.x, b0.y, b0.z, b0.w, 0.f, 0.f, 0.f, 0.f};
      if (NPT == 8) {
        const float4 b1 = *reinterpret_cast<const float4*>(&Bs[buf][kk][LO + tn * 4]);
        b[4] = b1.x; b[5] = b1.y; b[6] = b1.z; b[7] = b1.w;
      } else {
        const float2 b1 = *reinterpret_cast<const float2*>(&Bs[buf][kk][LO + tn * 2]);
        b[4] = b1.x; b[5] = b1.y;
      }
#pragma unroll
      for (int j = 0; j < NPT; ++j) {
        const unsigned long long bd = dup2(b[j]);
#pragma unroll
        for (int ip = 0; ip < 8; ++ip) ffma2(acc2[ip][j], a[ip], bd);
      }
    }
    if (++buf == STAGES) buf = 0;
  }

  // positions of pair ip: group g = ip / 2, offset (ip % 2) * 2 .. + 1 inside the group's four
  constexpr bool vec_ok = true;        // (STAGED is launched exactly when Ho*Wo is no multiple of 4)
  if (STAGED) {
    // Ho*Wo no multiple of 4: a thread's four positions of one channel do not start on a 16-byte boundary.
    // The tile goes through shared memory (free now) instead, one group of channels at a time, as
    // Cs[channel][position]; every warp then streams whole rows with consecutive lanes on consecutive
    // positions: 128 contiguous bytes per store instruction, whatever the alignment (element-wise stores
    // straight from the registers put 4 bytes at a 16-byte stride: 0.54 against 0.60 of the FFMA peak
    // on two 7x7 stems that differ only in this).
    constexpr int CP = BM + 4;                             // row pitch in floats
    static_assert((size_t)LO * CP <= (size_t)STAGES * BK * (APITCH + BN), "the staged tile fits the operand ring");
    float* Cs = reinterpret_cast<float*>(smem_f32);
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    // this thread's positions while streaming: x = lane + 32 t
    const int lane = tid & 31, wid = tid >> 5;
    int64_t obase[BM / 32];
#pragma unroll
    for (int t = 0; t < BM / 32; ++t) {
      const int64_t pp = m0 + lane + 32 * t;
      obase[t] = -1;
      if (pp < q.P) {
        int64_t n;
        int r;
        split_position(pp, q, n, r);
        obase[t] = n * q.Co * q.HoWo + r;
      }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      constexpr int NJ0 = 4;
      const int nj = h == 0 ? NJ0 : NPT - 4;               // channels of this thread in the group
      const int rows = h == 0 ? LO : BN - LO;              // channels of the group
      __syncthreads();                                     // the ring (or the previous group) has been read
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        if (jj >= nj) break;
        const int j = h * 4 + jj;
        const int c = tn * nj + jj;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          const float2 lo = unpack2(acc2[2 * g][j]), hi = unpack2(acc2[2 * g + 1][j]);
          *reinterpret_cast<float4*>(&Cs[c * CP + g * (BM / 4) + tm * 4]) = make_float4(lo.x, lo.y, hi.x, hi.y);
        }
      }
      __syncthreads();
      const int cbase = n0 + (h == 0 ? 0 : LO);
      for (int c = wid; c < rows; c += THREADS / 32) {
        const int co = cbase + c;
        if (co >= q.Co) break;
#pragma unroll
        for (int t = 0; t < BM / 32; ++t)
          if (obase[t] >= 0) q.y[obase[t] + (int64_t)co * q.HoWo] = Cs[c * CP + lane + 32 * t];
      }
    }
    return;
  }
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    const int64_t p = m0 + g * (BM / 4) + tm * 4;
    if (p >= q.P) continue;
    int64_t n;
    int r;
    split_position(p, q, n, r);
    int64_t nn[4];
    int rr[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      nn[i] = n; rr[i] = r + i;
      while (rr[i] >= q.HoWo) { rr[i] -= q.HoWo; ++nn[i]; }
    }
#pragma unroll
    for (int j = 0; j < NPT; ++j) {
      const int co = j < 4 ? n0 + tn * 4 + j : n0 + LO + tn * (NPT - 4) + (j - 4);
      if (co >= q.Co) continue;
      const float2 lo = unpack2(acc2[2 * g][j]), hi = unpack2(acc2[2 * g + 1][j]);
      const float v[4] = {lo.x, lo.y, hi.x, hi.y};
      if (vec_ok) {
        *reinterpret_cast<float4*>(q.y + (n * q.Co + co) * q.HoWo + r) = make_float4(v[0], v[1], v[2], v[3]);
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (p + i >= q.P) break;
          q.y[(nn[i] * q.Co + co) * q.HoWo + rr[i]] = v[i];
        }
      }
    }
  }
}

}  // namespace

// Tile shape of a layer.  64-channel tiles up to 64 output channels, else 128; 64-position tiles when
// 128-position tiles would leave the last wave badly filled; the k-block is 32 instead of 16 for the
// 64 x 128 tile on reductions of 256 or more (measured there: 2-3.5 % faster, half the barriers per
// FMA; 128 x 128 tiles and the short reductions of the stems are 1-7 % slower with it).
F32Plan plan_f32(const Geometry& g) {
  F32Plan p;
  const bool wide = g.Co > 64;
  // 96-channel tiles where they pad the output channels less than 128-channel tiles do (96, 192, 288, ...)
  const bool bn96 = wide && (g.Co + 95) / 96 * 96 < (g.Co + 127) / 128 * 128;
  p.bn = wide ? (bn96 ? 96 : 128) : 64;
  const int64_t cot = wide ? (g.Co + p.bn - 1) / p.bn : 1;
  auto waves_cost = [&](int bm) {
    const int64_t tiles = (g.P + bm - 1) / bm * cot;
    return (double)((tiles + 147) / 148) * bm;
  };
  bool small_m = waves_cost(64) < 0.9 * waves_cost(128);
  // 128-channel tiles: with four to ten 128-position tiles per SM the partly filled last round of
  // 256-thread CTAs costs more than the 64-position tile's extra filter traffic (measured on 3x3 to
  // 7x7 layers at 28x28 and 10x10: 3-5 % faster; larger grids are 3-4 % faster with 128 positions)
  const int64_t tiles128 = (g.P + 127) / 128 * cot;
  if (wide && tiles128 >= 4 * 148 && tiles128 < 10 * 148) small_m = true;
  if (const char* v = debug_getenv("IM2WIN_F32_BM")) small_m = atoi(v) == 64;   // testing aid
  p.bm = small_m ? 64 : 128;
  p.bk = (wide && small_m && g.K >= 256) ? 32 : 16;
  // k along the lanes of the gather where windows lie 128 bytes or more apart and the reduction is long
  // enough for the per-thread set-up of several positions not to matter (128-position tiles only)
  p.klanes = !small_m && g.s * g.Kh >= 32 && g.K >= 256;
  if (const char* v = debug_getenv("IM2WIN_F32_KLANES")) p.klanes = !small_m && v[0] == '1';   // testing aid
  // 16 x 8 (96-channel tiles: 16 x 6) outputs per thread on 128-position tiles (conv_f32_tall_kernel).  Measured
  // 5-6 % faster there (3x3 on 64 channels at 56x56: 597 -> 567 us; 5x5 on 96 -> 256 channels 0.75 -> 0.79 of
  // the FFMA peak, 3x3 on 64 -> 128 channels at 112x112 0.77 -> 0.815), 1-4 % slower than the 64-position tile with
  // k-blocks of 32 where that one is planned, and slower on a reduction of 27 (two k-blocks per tile); the 11x11
  // stride-4 stems with 96 output channels (k along the lanes, 16 x 6 per thread, three CTAs per SM) 0.60 -> 0.68.
  const bool tall_ok = p.bm == 128 || (p.bn >= 96 && !p.klanes);
  p.tall = tall_ok && p.bm == 128 && g.K >= 128;
  if (const char* v = debug_getenv("IM2WIN_F32_TALL")) p.tall = tall_ok && v[0] == '1';   // testing aid
  if (const char* v = debug_getenv("IM2WIN_F32_BK")) { if (wide && small_m) p.bk = atoi(v) == 32 ? 32 : 16; }   // testing aid
  if (p.tall) p.bk = 16;
  return p;
}

cudaError_t launch_conv_f32(const float* window, float* y, const void* scratch, const Geometry& g,
                            const ScratchLayout& l, cudaStream_t stream) {
  const unsigned char* base = static_cast<const unsigned char*>(scratch);
  ConvF32Params q;
  q.win = window;
  q.fk = reinterpret_cast<const float*>(base + l.filter_off);
  q.koff = reinterpret_cast<const int32_t*>(base + l.koff_off);
  q.y = y;
  q.P = g.P; q.img_stride = g.img_stride; q.strip = g.strip;
  q.HoWo = g.Ho * g.Wo; q.Wo = g.Wo; q.sKh = g.s * g.Kh;
  q.Co = g.Co; q.Co_pad = (int32_t)l.Co_pad; q.Kp = (int32_t)l.Kp;
  const F32Plan p = plan_f32(g);
  if (l.Kp % p.bk != 0) return cudaErrorInvalidValue;       // the filter was packed for another k-block
  const int64_t cot = l.Co_pad / p.bn;
  dim3 grid((unsigned)((g.P + p.bm - 1) / p.bm), (unsigned)cot);
  const int threads = (p.bm / 8) * f32_tn(p.bn);
  const size_t smem = (size_t)3 * p.bk * (p.bm + (p.klanes ? 4 : 0) + p.bn) * 4;
  void (*kernel)(ConvF32Params);
  int which;
  if (p.bn == 96) {
    if (p.bm == 64) { kernel = p.bk == 32 ? conv_f32_kernel<64, 96, 32, false> : conv_f32_kernel<64, 96, 16, false>; which = p.bk == 32 ? 5 : 6; }
    else if (p.klanes) { kernel = conv_f32_kernel<128, 96, 16, true>; which = 8; }
    else { kernel = conv_f32_kernel<128, 96, 16, false>; which = 7; }
  } else if (p.bn == 128) {
    if (p.bm == 64) { kernel = p.bk == 32 ? conv_f32_kernel<64, 128, 32, false> : conv_f32_kernel<64, 128, 16, false>; which = p.bk == 32 ? 0 : 1; }
    else if (p.klanes) { kernel = conv_f32_kernel<128, 128, 16, true>; which = 9; }
    else { kernel = conv_f32_kernel<128, 128, 16, false>; which = 2; }
  } else {
    if (p.bm == 64) { kernel = conv_f32_kernel<64, 64, 16, false>; which = 3; }
    else if (p.klanes) { kernel = conv_f32_kernel<128, 64, 16, true>; which = 10; }
    else { kernel = conv_f32_kernel<128, 64, 16, false>; which = 4; }
  }
  if (smem > 48 * 1024) {
    // per device and tile shape, once: the opt-in to more than 48 KB of dynamic shared memory
    static bool attr_done[64][11] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_done[dev][which]) {
      cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      attr_done[dev][which] = true;
    }
  }
  if (p.tall) {
    void (*tk)(ConvF32Params);
    int tw;
    const bool st = (q.HoWo % 4) != 0;
#define IM2WIN_TALL(BM_, BN_, KL_) (st ? conv_f32_tall_kernel<BM_, BN_, 16, KL_, true> : conv_f32_tall_kernel<BM_, BN_, 16, KL_, false>)
    if (p.klanes) {
      tk = p.bn == 64 ? IM2WIN_TALL(128, 64, true) : (p.bn == 96 ? IM2WIN_TALL(128, 96, true) : IM2WIN_TALL(128, 128, true));
      tw = p.bn == 64 ? 0 : (p.bn == 96 ? 1 : 2);
    } else if (p.bn == 96) {
      tk = p.bm == 64 ? IM2WIN_TALL(64, 96, false) : IM2WIN_TALL(128, 96, false);
      tw = p.bm == 64 ? 3 : 4;
    } else {
      tk = p.bn == 64 ? IM2WIN_TALL(128, 64, false) : (p.bm == 64 ? IM2WIN_TALL(64, 128, false) : IM2WIN_TALL(128, 128, false));
      tw = p.bn == 64 ? 5 : (p.bm == 64 ? 6 : 7);
    }
#undef IM2WIN_TALL
    tw = 2 * tw + (st ? 1 : 0);
    if (smem > 48 * 1024) {
      static bool tall_attr[64][16] = {};
      int dev = 0;
      if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
      if (!tall_attr[dev][tw]) {
        cudaError_t e = cudaFuncSetAttribute(tk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        tall_attr[dev][tw] = true;
      }
    }
    tk<<<grid, (p.bm / 16) * f32_tn(p.bn), smem, stream>>>(q);
    return cudaGetLastError();
  }
  kernel<<<grid, threads, smem, stream>>>(q);
  return cudaGetLastError();
}

}  // namespace im2win
