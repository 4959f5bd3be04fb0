// Group-quantized layer: int8 tensor-core GEMM (tcgen05.mma kind::i8, accumulators in tensor
// memory) whose accumulator is switched at every channel-group boundary, with the per-group
// de-quantizing epilogue
//     Y[t,o] = bias[o] + sw[o] * sum_g s[t,g] * (acc_g[t,o] - Z[t,g] * wsum_g[o])
// (Eq. 1's de-quantizer with the group parameters of Eq. 6) fused in.
//
// CTA = one 128-row output tile x BN columns, persistent over tiles.  Warp roles:
//   warps 0-7   epilogue: lane quarter = warp & 3 (the TMEM lanes a warp may read), column half = warp >> 2
//   warp  8     TMA producer (one lane): A code tile and B weight tile per 128-byte K stage
//   warp  9     MMA issuer (one lane) and TMEM allocator
//   warp  10    output store (one lane): TMA stores of the staged fp16 tile
//   warps 11-15 (4-bit weights only) unpack packed nibbles from global memory into the B stage
// After set-up the data-movement warps hand registers to the epilogue warps (setmaxnreg).
// K runs over 32-code atoms; a stage holds four atoms.  Group segments are multiples of one atom,
// so the issuer moves to the next TMEM accumulator between two atoms, commits the finished one to
// the epilogue and keeps going while the epilogue drains it.
//
// Zero-points: the padding positions of a group carry the code Z on the activation side and
// -wsum_g[o] (spread over the positions) on the weight side, so acc_g already equals
// acc_g - Z wsum_g and the epilogue is one convert and one FMA per element and group.  The
// epilogue only adds a correction for the rare rows whose Z falls outside the code range (the
// stored padding code is then the clamped Z) and for groups whose padding could not hold all of
// wsum (flagged in `res_mask`).
//
// Output: the fp16 tile is staged in shared memory in 64-byte-swizzled panels of 32 columns and
// written with TMA stores, which also clip the ragged last row and column tiles.  The epilogue
// warps only signal "staged" and move on to the next tile; the store warp issues the stores and
// signals "staging free" once they have read the buffer.
// Linear layers: A and B stages are 128-byte-swizzled tiles fetched with one TMA box each.
// 3x3 conv (implicit GEMM): the reduction order is group-major, then filter tap, then channel
// atom; every A atom is its own 32-byte-swizzled 4-D TMA box of the NHWC code tensor shifted by
// the tap, out-of-image rows zero-filled by TMA (exact for zero-centred codes).
#pragma once

#include <type_traits>

#include "weights.cuh"

namespace dgq {

constexpr int GEMM_BM = 128;
constexpr int GEMM_UNPACK_WARPS = 5;
constexpr int GEMM_UNPACK_THREADS = GEMM_UNPACK_WARPS * 32;
// Eight epilogue warps (two aligned groups of four: a warp reads the TMEM lane quarter warp % 4),
// then the producer, issuer and store warps and, for 4-bit weights, the unpack warps; the warp count
// is a multiple of four so that registers can be moved between aligned groups of four warps.
constexpr int GEMM_EPI_WARPS = 8;
constexpr int GEMM_WARP_TMA = GEMM_EPI_WARPS;
constexpr int GEMM_WARP_MMA = GEMM_EPI_WARPS + 1;
constexpr int GEMM_WARP_STORE = GEMM_EPI_WARPS + 2;
constexpr int GEMM_THREADS_W8 = (GEMM_EPI_WARPS + 3) * 32;  // first unpack thread
__host__ __device__ constexpr int gemm_threads(bool w4) { return (w4 ? 16 : 12) * 32; }
// Registers per thread: the kernel starts with `gemm_regs_launch`, the epilogue warps then grow to
// `gemm_regs_epi` with what the other warps give back (8 * epi + rest * other <= warps * launch).
__host__ __device__ constexpr int gemm_regs_launch(bool w4) { return w4 ? 128 : 168; }
__host__ __device__ constexpr int gemm_regs_epi(bool w4) { return w4 ? 192 : 208; }
__host__ __device__ constexpr int gemm_regs_other(bool w4) { return w4 ? 64 : 80; }
static_assert(8 * gemm_regs_epi(true) + 8 * gemm_regs_other(true) <= 16 * gemm_regs_launch(true), "register pool");
static_assert(8 * gemm_regs_epi(false) + 4 * gemm_regs_other(false) <= 12 * gemm_regs_launch(false), "register pool");
constexpr int GEMM_MAX_ATOMS = 1024;           // 32768 reduction positions
constexpr int GEMM_A_STAGE = GEMM_BM * 128;  // bytes
constexpr int GEMM_SMEM_LIMIT = 227 * 1024;

template <int BN, bool W4>
struct GemmCfg {
  // 4-bit weights: ring of packed B stages (BN rows x 64 bytes each) that the unpack warps fill with
  // asynchronous copies PK_AHEAD stages ahead of the stage they expand
  static constexpr int PK_STAGES = W4 ? 4 : 0;
  static constexpr int PK_AHEAD = PK_STAGES - 1;
  static constexpr int PK_STAGE = BN * 64;
  static constexpr int PK_BYTES = PK_STAGES * PK_STAGE;
  static constexpr int B_STAGE = BN * 128;
  static constexpr int STAGE = GEMM_A_STAGE + B_STAGE;
  static constexpr int OUT_BYTES = GEMM_BM * BN * 2;  // fp16 staging of one output tile
  static constexpr int MISC_BYTES = 2048 + (2 + DGQ_MAX_GROUPS) * BN * 4 + GEMM_MAX_ATOMS * 4;  // barriers + sw, bias, wsum of the CTA's columns + conv atom table
  static constexpr int STAGES_RAW = (GEMM_SMEM_LIMIT - 1024 - OUT_BYTES - MISC_BYTES - PK_BYTES) / STAGE;
  static constexpr int STAGES = STAGES_RAW > 8 ? 8 : STAGES_RAW;
  static constexpr int NACC_RAW = 512 / BN;
  static constexpr int NACC = NACC_RAW > 4 ? 4 : NACC_RAW;
  static constexpr int OFF_PK = STAGES * STAGE + OUT_BYTES + MISC_BYTES;
  static constexpr int SMEM = OFF_PK + PK_BYTES + 1024;
  static_assert(MISC_BYTES % 16 == 0, "the packed ring is 16-byte aligned");
  static_assert(BN % 32 == 0 && BN <= 256, "BN must be a multiple of 32 up to 256");
  static_assert(NACC >= 2, "need two accumulators to overlap the epilogue");
  static_assert(NACC * BN <= 512, "tensor memory has 512 columns");
  static_assert(STAGES >= 3, "pipeline too shallow");
};

struct GemmArgs {
  int64_t M;
  int N, N_pad, Kt, G, P;
  int n_tiles_m, n_tiles_n;
  uint32_t idesc;
  int use_zp;                 // 0 for zero-centred codes
  int code_max;               // 2^b - 1
  uint32_t res_mask;          // groups whose padding did not absorb all of wsum
  int per_token;              // 1: scale rows indexed by token, 0: by row_group[token mod P]
  const float* scale;         // [rows][G]
  const int32_t* zp;          // [rows][G]
  const int32_t* row_group;   // [P]
  const float* sw;            // [N_pad]
  const float* wsum;          // [G][N_pad]
  const float* wres;          // [G][N_pad]
  const __half* bias;         // [N] or null
  const uint8_t* w_packed;    // 4-bit weights [N_pad][Kt/2]
  int seg_end[DGQ_MAX_GROUPS];    // end atom of every group segment
  unsigned long long end_mask[GEMM_MAX_ATOMS / 64];  // bit i: atom i is the last of its group
  // conv
  int conv_W, conv_H;
  int grp_atoms[DGQ_MAX_GROUPS];  // channel atoms of every group
  int grp_chan0[DGQ_MAX_GROUPS];  // first padded channel position of every group
};

struct __align__(8) GemmShared {
  uint64_t full[8];
  uint64_t empty[8];
  uint64_t acc_full[4];
  uint64_t acc_empty[4];
  uint64_t out_full;   // all epilogue warps have staged their part of the output tile
  uint64_t out_free;   // the TMA stores of the previous tile have read the staging buffer
  uint32_t tmem_base;
  int abort_flag;
};

template <int BN, bool W4, bool CONV>
__global__ void __maxnreg__(gemm_regs_launch(W4))
gq_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmY, const __grid_constant__ GemmArgs a) {
  using Cfg = GemmCfg<BN, W4>;
  constexpr int STAGES = Cfg::STAGES;
  constexpr int NACC = Cfg::NACC;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) &
                                                         ~uintptr_t(1023));
  unsigned char* smA = smem;
  unsigned char* smB = smem + STAGES * GEMM_A_STAGE;
  unsigned char* smOut = smem + STAGES * Cfg::STAGE;  // 1024-byte aligned: every stage size is
  GemmShared* sh = reinterpret_cast<GemmShared*>(smOut + Cfg::OUT_BYTES);
  // Every tile of this CTA has the same column block (the grid is a multiple of the number of
  // column blocks), so its per-column constants are loaded once.
  float* sw_s = reinterpret_cast<float*>(smOut + Cfg::OUT_BYTES + 2048);  // [BN]
  float* bias_s = sw_s + BN;                                              // [BN]
  float* wsum_s = bias_s + BN;                                            // [G][BN]
  uint32_t* conv_tab = reinterpret_cast<uint32_t*>(wsum_s + DGQ_MAX_GROUPS * BN);  // [atoms] conv: channel | kx << 16 | ky << 18
  const int cta_n0 = ((int)blockIdx.x % a.n_tiles_n) * BN;
  volatile int* abort_flag = &sh->abort_flag;

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int n_atoms = a.Kt >> 5;
  const int n_kstages = (n_atoms + 3) >> 2;
  const int n_tiles = a.n_tiles_m * a.n_tiles_n;

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) {
      mbar_init(&sh->full[i], W4 ? 1 + GEMM_UNPACK_WARPS : 1);
      mbar_init(&sh->empty[i], 1);
    }
    for (int i = 0; i < NACC; ++i) {
      mbar_init(&sh->acc_full[i], 1);
      mbar_init(&sh->acc_empty[i], GEMM_EPI_WARPS);
    }
    mbar_init(&sh->out_full, GEMM_EPI_WARPS);
    mbar_init(&sh->out_free, 1);
    sh->abort_flag = 0;
    fence_barrier_init();
  }
  for (int i = threadIdx.x; i < BN; i += blockDim.x) {
    const int col = cta_n0 + i;
    sw_s[i] = col < a.N_pad ? __ldg(a.sw + col) : 0.f;
    bias_s[i] = (a.bias != nullptr && col < a.N) ? __half2float(a.bias[col]) : 0.f;
  }
  if (a.use_zp)
    for (int i = threadIdx.x; i < a.G * BN; i += blockDim.x) {
      const int g = i / BN, c = i - g * BN;
      wsum_s[i] = cta_n0 + c < a.N_pad ? __ldg(a.wsum + (size_t)g * a.N_pad + cta_n0 + c) : 0.f;
    }
  if (CONV) {
    // Where every A atom of a tile comes from (same for all tiles): first channel position and
    // filter tap.  Built once by all threads, so that the producer lane's chain per copy stays short.
    for (int atom = threadIdx.x; atom < n_atoms; atom += blockDim.x) {
      int g = 0, g_start = 0;
      while (atom >= a.seg_end[g]) {
        g_start = a.seg_end[g];
        ++g;
      }
      const int local = atom - g_start;
      const int tap = local / a.grp_atoms[g];
      const int ca = local - tap * a.grp_atoms[g];
      const int ky = tap / 3, kx = tap - ky * 3;
      conv_tab[atom] = (uint32_t)(a.grp_chan0[g] + ca * 32) | ((uint32_t)kx << 16) | ((uint32_t)ky << 18);
    }
  }
  if (warp == GEMM_WARP_MMA) {
    tmem_alloc(&sh->tmem_base, 512);
    tmem_relinquish();
  }
  // Everything above reads only the layer's constants; codes, scales and zero-points may come from
  // the kernel before this one.
  pdl_wait();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;

  if (warp >= GEMM_EPI_WARPS) {
  // The warps that only move data or issue instructions hand most of their registers to the epilogue.
  reg_dealloc<gemm_regs_other(W4)>();
  if (warp == GEMM_WARP_TMA) {
    // ------------------------------------------------------------ TMA producer
    // Five lanes run the loop together and issue their copies with one instruction: lanes 0-3 an A box each
    // (a conv stage is four boxes, one per atom; a linear stage is one box, lane 0's), lane 4 the B box.
    // Handing a box to the copy engine costs a thread a few hundred cycles of issue time, which one lane
    // alone cannot hide when the boxes are as small as a conv atom's.  The other lanes go straight to the
    // CTA's final barrier.
    if (lane < 5) {
      constexpr uint32_t PROD_MASK = 0x1Fu;
      if (lane == 0) tma_prefetch_desc(&tmA);
      if (!W4 && lane == 4) tma_prefetch_desc(&tmB);
      const uint32_t empty0 = smem_u32(&sh->empty[0]);
      uint32_t s = 0, empty_par = 1;  // fresh barriers pass a wait for parity 1
      for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const int tm = tile / a.n_tiles_n, tn = tile - tm * a.n_tiles_n;
        const int m0 = tm * GEMM_BM, n0 = tn * BN;
        int cw = 0, chh = 0, cn = 0;  // conv: spatial origin of this row tile
        if (CONV) {
          const int hw = a.conv_H * a.conv_W;
          cn = m0 / hw;
          const int rem = m0 - cn * hw;
          chh = rem / a.conv_W;
          cw = rem - chh * a.conv_W;
        }
        for (int ks = 0; ks < n_kstages; ++ks) {
          mbar_wait_lean(empty0 + s * 8u, empty_par, abort_flag);
          const int atoms_here = min(4, n_atoms - ks * 4);
          uint32_t bytes = W4 ? 0u : (uint32_t)Cfg::B_STAGE;
          bytes += CONV ? (uint32_t)(atoms_here * 4096) : (uint32_t)GEMM_A_STAGE;
          if (lane == 0) mbar_arrive_expect_tx(&sh->full[s], bytes);  // before any of the copies below
          __syncwarp(PROD_MASK);
          if (CONV) {
            if (lane < atoms_here) {
              const uint32_t e = conv_tab[ks * 4 + lane];
              tma_load_4d(smA + s * GEMM_A_STAGE + lane * 4096, &tmA, &sh->full[s], (int)(e & 0xFFFFu),
                          cw + (int)((e >> 16) & 3u) - 1, chh + (int)((e >> 18) & 3u) - 1, cn);
            }
          } else if (lane == 0) {
            tma_load_2d(smA + s * GEMM_A_STAGE, &tmA, &sh->full[s], ks * 128, m0);
          }
          if (!W4 && lane == 4) tma_load_2d(smB + s * Cfg::B_STAGE, &tmB, &sh->full[s], ks * 128, n0);
          if (++s == (uint32_t)STAGES) {
            s = 0;
            empty_par ^= 1u;
          }
        }
        if (*abort_flag) break;
      }
    }
    __syncwarp();
  } else if (warp == GEMM_WARP_MMA) {
    // ------------------------------------------------------------ MMA issuer
    // The whole warp runs the loop with uniform control flow; the tcgen05 instructions are issued by
    // one elected lane.  What the issuing path costs per instruction, not the tensor core, bounds short
    // groups: an MMA, a commit and a barrier poll each take tens to hundreds of cycles of this warp's
    // time, whatever the tile width.  So a stage is straight-line code chosen by its pattern of group
    // ends (no per-atom tests), everything that can be is precomputed (descriptor words, barrier
    // addresses, running ring positions and parities).
    {
      constexpr uint32_t A_HI = CONV ? smem_desc_hi(256, 6) : smem_desc_hi(1024, 2);
      constexpr uint32_t B_HI = smem_desc_hi(1024, 2);
      const uint32_t a_lo0 = smem_desc_lo(smem_u32(smA)), b_lo0 = smem_desc_lo(smem_u32(smB));
      const uint32_t idesc = a.idesc;
      const uint32_t full0 = smem_u32(&sh->full[0]), empty0 = smem_u32(&sh->empty[0]);
      const uint32_t accf0 = smem_u32(&sh->acc_full[0]), acce0 = smem_u32(&sh->acc_empty[0]);
      uint32_t s = 0;            // stage slot
      uint32_t full_phase = 0;   // parity of the slot's next "full" phase
      uint32_t ab = 0;           // accumulator of the next group
      uint32_t acc_phase = 1;    // parity to wait for on its "empty" barrier (fresh barriers pass)
      // One stage of four atoms whose group ends are the bits of PAT; `need`: the first atom starts a group.
      auto issue_stage = [&](auto pat_tag, bool need, uint32_t a_lo, uint32_t b_lo) {
        constexpr int PAT = decltype(pat_tag)::value;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const bool starts = (j == 0) ? need : (((PAT >> (j > 0 ? j - 1 : 0)) & 1) != 0);
          if (starts) {
            mbar_wait_lean(acce0 + ab * 8u, acc_phase, abort_flag);
            tc_fence_after();
          }
          if (elect_one()) {
            mma_i8_lohi(tmem_base + ab * (uint32_t)BN, a_lo + (CONV ? j * 256 : j * 2), A_HI, b_lo + j * 2, B_HI, idesc,
                        starts ? 0u : 1u);
            if ((PAT >> j) & 1) mma_commit_addr(accf0 + ab * 8u);  // last atom of the group: hand the accumulator over
          }
          __syncwarp();
          if ((PAT >> j) & 1) {
            if (++ab == (uint32_t)NACC) {
              ab = 0;
              acc_phase ^= 1u;
            }
          }
        }
      };
      for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        bool need = true;      // every tile starts a group
        uint64_t ends = 0;     // bit i: atom (16 * 4) * word + i is the last of its group
        for (int ks = 0; ks < n_kstages; ++ks) {
          if ((ks & 15) == 0) ends = a.end_mask[ks >> 4];
          uint32_t pat = (uint32_t)(ends >> ((ks & 15) * 4)) & 0xFu;
          // A ragged last stage still issues four atoms (the missing ones multiply zero weights); the
          // end of the last group moves to the last atom issued.
          const int atoms_here = n_atoms - ks * 4;
          if (atoms_here < 4) pat = (pat & ~(1u << (atoms_here - 1))) | 8u;
          mbar_wait_lean(full0 + s * 8u, full_phase, abort_flag);
          tc_fence_after();
          const uint32_t a_lo = a_lo0 + s * (uint32_t)(GEMM_A_STAGE >> 4);
          const uint32_t b_lo = b_lo0 + s * (uint32_t)(Cfg::B_STAGE >> 4);
          switch (pat) {
#define DGQ_STAGE_CASE(P) case P: issue_stage(std::integral_constant<int, P>{}, need, a_lo, b_lo); break;
            DGQ_STAGE_CASE(0) DGQ_STAGE_CASE(1) DGQ_STAGE_CASE(2) DGQ_STAGE_CASE(3) DGQ_STAGE_CASE(4) DGQ_STAGE_CASE(5)
            DGQ_STAGE_CASE(6) DGQ_STAGE_CASE(7) DGQ_STAGE_CASE(8) DGQ_STAGE_CASE(9) DGQ_STAGE_CASE(10) DGQ_STAGE_CASE(11)
            DGQ_STAGE_CASE(12) DGQ_STAGE_CASE(13) DGQ_STAGE_CASE(14) DGQ_STAGE_CASE(15)
#undef DGQ_STAGE_CASE
          }
          need = (pat & 8u) != 0;
          if (elect_one()) mma_commit_addr(empty0 + s * 8u);  // stage reusable once these MMAs have read it
          __syncwarp();
          if (++s == (uint32_t)STAGES) {
            s = 0;
            full_phase ^= 1u;
          }
        }
        if (*abort_flag) break;
      }
    }
    __syncwarp();
  } else if (warp == GEMM_WARP_STORE) {
    // ------------------------------------------------------------ output store
    if (lane == 0) {
      tma_prefetch_desc(&tmY);
      const uint32_t out_full_a = smem_u32(&sh->out_full);
      uint32_t tile_it = 0;
      for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tile_it) {
        const int tm = tile / a.n_tiles_n, tn = tile - tm * a.n_tiles_n;
        const int n0 = tn * BN;
        mbar_wait_lean(out_full_a, tile_it & 1u, abort_flag);
        if (*abort_flag) break;
#pragma unroll
        for (int pnl = 0; pnl < BN / 32; ++pnl)
          if (n0 + pnl * 32 < a.N) tma_store_2d(&tmY, smOut + pnl * (GEMM_BM * 64), n0 + pnl * 32, tm * GEMM_BM);
        bulk_commit();
        bulk_wait_read0();
        mbar_arrive(&sh->out_free);
      }
      bulk_wait0();
    }
    __syncwarp();
  } else if (W4 && warp >= GEMM_WARP_STORE + 1) {
    // ------------------------------------------------------------ 4-bit weight unpack into the B stage
    // Every thread owns the same 16-byte pieces of every stage.  It copies them asynchronously from global
    // memory into its slots of the packed ring PK_AHEAD stages before it expands them, one copy group per
    // stage, and reads back only what it copied itself, so the ring needs no barrier: waiting for its own
    // copy groups is enough.  The load latency (L2 or DRAM) is thus spread over PK_AHEAD stages.
    constexpr int ITEMS = (BN * 4 + GEMM_UNPACK_THREADS - 1) / GEMM_UNPACK_THREADS;  // 16-byte pieces per thread
    constexpr int AHEAD = Cfg::PK_AHEAD;
    const int ut = threadIdx.x - GEMM_THREADS_W8;  // 0..GEMM_UNPACK_THREADS-1
    unsigned char* pk_ring = smem + Cfg::OFF_PK;
    uint32_t it = 0;
    bool ok = true;
    const int row_bytes = a.Kt >> 1;
    int f_tile = blockIdx.x, f_ks = 0;  // next stage to request
    uint32_t f_it = 0;
    auto request_next = [&]() {
      if (f_tile < n_tiles) {
        const int n0 = (f_tile % a.n_tiles_n) * BN;
        const uint32_t slot = smem_u32(pk_ring + (f_it % Cfg::PK_STAGES) * Cfg::PK_STAGE);
#pragma unroll
        for (int e = 0; e < ITEMS; ++e) {
          const int item = ut + e * GEMM_UNPACK_THREADS;
          if (item >= BN * 4) continue;
          const int r = item >> 2, qd = item & 3;  // B row, 16-byte packed quarter of the 64-byte row slice
          const int kb = f_ks * 64 + qd * 16;
          const bool in = kb < row_bytes;          // beyond the row: the slot is filled with zeros
          const uint8_t* src = a.w_packed + (size_t)(n0 + r) * row_bytes + (in ? kb : 0);
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(slot + (uint32_t)item * 16u), "l"(src),
                       "r"(in ? 16 : 0)
                       : "memory");
        }
        ++f_it;
        if (++f_ks == n_kstages) {
          f_ks = 0;
          f_tile += gridDim.x;
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");  // one group per call, empty at the end
    };
    // The CTA's whole column block of packed weights (BN rows of Kt / 2 bytes) is asked into L2 up
    // front, so that the copies below find it there.
    if ((int)blockIdx.x < n_tiles) {
      const int n0 = ((int)blockIdx.x % a.n_tiles_n) * BN;
      const int lines_per_row = (row_bytes + 127) >> 7;
      for (int i = ut; i < BN * lines_per_row; i += GEMM_UNPACK_THREADS) {
        const int r = i / lines_per_row, l = i - r * lines_per_row;
        const uint8_t* ptr = a.w_packed + (size_t)(n0 + r) * row_bytes + (size_t)l * 128;
        asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
      }
    }
#pragma unroll
    for (int i = 0; i < AHEAD; ++i) request_next();
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
      for (int ks = 0; ks < n_kstages && ok; ++ks, ++it) {
        // the slot of stage it + AHEAD is the one this thread read in the previous iteration
        request_next();
        asm volatile("cp.async.wait_group %0;" ::"n"(AHEAD) : "memory");  // this thread's pieces of stage `it` have landed
        const int s = it % STAGES;
        ok = __all_sync(0xffffffffu, mbar_wait(&sh->empty[s], ((it / STAGES) & 1) ^ 1, abort_flag));
        if (!ok) break;
        unsigned char* bst = smB + s * Cfg::B_STAGE;
        const unsigned char* pst = pk_ring + (it % Cfg::PK_STAGES) * Cfg::PK_STAGE;
#pragma unroll
        for (int e = 0; e < ITEMS; ++e) {
          const int item = ut + e * GEMM_UNPACK_THREADS;
          if (item >= BN * 4) continue;
          const int r = item >> 2, qd = item & 3;
          const uint4 p4 = *reinterpret_cast<const uint4*>(pst + item * 16);
          const uint4 c0 = make_uint4((p4.x << 4) & 0xF0F0F0F0u, p4.x & 0xF0F0F0F0u, (p4.y << 4) & 0xF0F0F0F0u,
                                      p4.y & 0xF0F0F0F0u);
          const uint4 c1 = make_uint4((p4.z << 4) & 0xF0F0F0F0u, p4.z & 0xF0F0F0F0u, (p4.w << 4) & 0xF0F0F0F0u,
                                      p4.w & 0xF0F0F0F0u);
          // 128-byte swizzle: 16-byte chunk index XOR (row mod 8) inside every 8-row, 1024-byte group
          unsigned char* rowp = bst + (r >> 3) * 1024 + (r & 7) * 128;
          *reinterpret_cast<uint4*>(rowp + (((2 * qd) ^ (r & 7)) << 4)) = c0;
          *reinterpret_cast<uint4*>(rowp + (((2 * qd + 1) ^ (r & 7)) << 4)) = c1;
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh->full[s]);
      }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");  // nothing of this thread's is in flight when the CTA ends
  }
  } else {
    reg_alloc<gemm_regs_epi(W4)>();
    // ------------------------------------------------------------ epilogue
    // The loop is kept lean on purpose: with one convert and half a packed multiply-add per
    // element and group, bookkeeping instructions would otherwise outnumber the arithmetic.
    constexpr int CW = BN / (GEMM_EPI_WARPS / 4);  // columns per thread
    static_assert(CW % 8 == 0, "whole 8-column loads and 16-byte output pieces");
    const int q = warp & 3, sl = warp >> 2;
    const int r_tile = q * 32 + lane;  // row inside the tile = TMEM lane
    const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(sl * CW);
    const uint32_t full0 = smem_u32(&sh->acc_full[0]), empty0 = smem_u32(&sh->acc_empty[0]);
    const uint32_t out_free_a = smem_u32(&sh->out_free), out_full_a = smem_u32(&sh->out_full);
    const int G = a.G;
    const bool use_zp = a.use_zp != 0;
    const uint32_t code_max = (uint32_t)a.code_max, res_mask = a.res_mask;
    uint32_t ab = 0, acc_par = 0, tile_it = 0;  // accumulator of the current group and its "full" parity
    // The first scale / zero-point of the row are fetched one tile ahead, so their latency hides
    // behind the current tile.
    float pre_s = 0.f;
    int pre_z = 0;
    const float* srow = nullptr;
    const int32_t* zrow = nullptr;
    auto prefetch_tile = [&](int tile) {
      const int tm = tile / a.n_tiles_n;
      const int64_t row = (int64_t)tm * GEMM_BM + r_tile;
      const int64_t row_c = row < a.M ? row : a.M - 1;
      const int64_t prow = a.per_token ? row_c : (int64_t)__ldg(a.row_group + row_c % a.P);
      srow = a.scale + prow * G;
      zrow = a.zp + prow * G;
      pre_s = __ldg(srow);
      pre_z = use_zp ? __ldg(zrow) : 0;
    };
    // One group per round: the warp waits for the group's accumulator, brings its CW columns into registers,
    // hands the accumulator back to the issuer and then does the arithmetic, while the other epilogue warp of
    // the scheduler is in another part of its own round.
    uint32_t rb[CW];
    auto load_group = [&](uint32_t taddr) {
#pragma unroll
      for (int k = 0; k < CW / 32; ++k) tmem_ld32(taddr + k * 32, reinterpret_cast<uint32_t(&)[32]>(rb[k * 32]));
      if ((CW % 32) >= 16) tmem_ld16(taddr + (CW / 32) * 32, reinterpret_cast<uint32_t(&)[16]>(rb[(CW / 32) * 32]));
      if (CW % 16) tmem_ld8(taddr + (CW / 16) * 16, reinterpret_cast<uint32_t(&)[8]>(rb[(CW / 16) * 16]));
    };
    if ((int)blockIdx.x < n_tiles) prefetch_tile(blockIdx.x);
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tile_it) {
      const float* srow_t = srow;
      const int32_t* zrow_t = zrow;
      const bool more_tiles = tile + (int)gridDim.x < n_tiles;
      unsigned long long y2[CW / 2];  // packed pairs of fp32 sums
#pragma unroll
      for (int i = 0; i < CW / 2; ++i) y2[i] = 0ull;
      // scale and zero-point of the next group are fetched one group ahead
      float s_next = pre_s;
      int z_next = pre_z;
      for (int g = 0; g < G; ++g) {
        const float s = s_next;
        const int Z = z_next;
        if (g + 1 < G) {
          s_next = __ldg(srow_t + g + 1);
          if (use_zp) z_next = __ldg(zrow_t + g + 1);
        } else if (more_tiles) {
          prefetch_tile(tile + gridDim.x);
        }
        uint32_t nab = ab + 1, npar = acc_par;
        if (nab == (uint32_t)NACC) {
          nab = 0;
          npar ^= 1u;
        }
        const unsigned long long s2 = pack_f32x2(s, s);
        mbar_wait_lean(full0 + ab * 8u, acc_par, abort_flag);
        tc_fence_after();
        load_group(t_lane + ab * (uint32_t)BN);
        tmem_ld_wait();
        // the accumulator goes back to the issuer as soon as its columns are in registers
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_addr(empty0 + ab * 8u);
#pragma unroll
        for (int i = 0; i < CW / 2; ++i) cvt_fma_f32x2(y2[i], s2, rb[2 * i], rb[2 * i + 1]);
        ab = nab;
        acc_par = npar;
        if (use_zp) {
          // rare: Z outside the code range (the stored padding code is the clamped Z), or a group
          // whose padding could not absorb all of wsum
          if (__any_sync(0xffffffffu, (uint32_t)Z > code_max)) {
            const int Zc = min(max(Z, 0), (int)code_max);
            const float c1 = -s * (float)(Z - Zc);
            const unsigned long long c2 = pack_f32x2(c1, c1);
            const ulonglong2* ws = reinterpret_cast<const ulonglong2*>(wsum_s + g * BN + sl * CW);
#pragma unroll
            for (int i = 0; i < CW / 4; ++i) {
              const ulonglong2 u = ws[i];
              y2[2 * i] = fma_f32x2(c2, u.x, y2[2 * i]);
              y2[2 * i + 1] = fma_f32x2(c2, u.y, y2[2 * i + 1]);
            }
          }
          if ((res_mask >> g) & 1u) {
            const float c1 = -s * (float)min(max(Z, 0), (int)code_max);
            const unsigned long long c2 = pack_f32x2(c1, c1);
            const float4* wr = reinterpret_cast<const float4*>(a.wres + (size_t)g * a.N_pad + cta_n0 + sl * CW);
#pragma unroll
            for (int i = 0; i < CW / 4; ++i) {
              const float4 v = __ldg(wr + i);
              y2[2 * i] = fma_f32x2(c2, pack_f32x2(v.x, v.y), y2[2 * i]);
              y2[2 * i + 1] = fma_f32x2(c2, pack_f32x2(v.z, v.w), y2[2 * i + 1]);
            }
          }
        }
      }
      if (*abort_flag) break;  // a wait gave up somewhere in the CTA (same value in every lane)
      // staging buffer: wait until the stores of the previous tile have read it (normally long done)
      mbar_wait_lean(out_free_a, (tile_it & 1u) ^ 1u, abort_flag);
#pragma unroll
      for (int j = 0; j < CW / 8; ++j) {
        const int cl = sl * CW + j * 8;  // first tile column of this 16-byte chunk
        const ulonglong2 s0 = *reinterpret_cast<const ulonglong2*>(sw_s + cl), s1 = *reinterpret_cast<const ulonglong2*>(sw_s + cl + 4);
        const ulonglong2 b0 = *reinterpret_cast<const ulonglong2*>(bias_s + cl), b1 = *reinterpret_cast<const ulonglong2*>(bias_s + cl + 4);
        float f[8];
        unpack_f32x2(fma_f32x2(s0.x, y2[j * 4 + 0], b0.x), f[0], f[1]);
        unpack_f32x2(fma_f32x2(s0.y, y2[j * 4 + 1], b0.y), f[2], f[3]);
        unpack_f32x2(fma_f32x2(s1.x, y2[j * 4 + 2], b1.x), f[4], f[5]);
        unpack_f32x2(fma_f32x2(s1.y, y2[j * 4 + 3], b1.y), f[6], f[7]);
        uint4 o;
        __half2* oh = reinterpret_cast<__half2*>(&o);
        oh[0] = __floats2half2_rn(f[0], f[1]);
        oh[1] = __floats2half2_rn(f[2], f[3]);
        oh[2] = __floats2half2_rn(f[4], f[5]);
        oh[3] = __floats2half2_rn(f[6], f[7]);
        // panel of 32 columns = 64-byte rows, 16-byte chunk index XOR bits 1-2 of the row (64 B swizzle)
        const int panel = cl >> 5, ch = (cl >> 3) & 3;
        *reinterpret_cast<uint4*>(smOut + panel * (GEMM_BM * 64) + r_tile * 64 + ((ch ^ ((r_tile >> 1) & 3)) << 4)) = o;
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive_addr(out_full_a);
    }
  }

  // ------------------------------------------------------------ common exit
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // give copies that may still be in flight time to land before the CTA's shared memory is released
    const long long t0 = clock64();
    while (clock64() - t0 < 200000) {
    }
    __syncthreads();
  }
  if (warp == GEMM_WARP_MMA) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// 4-bit weights -> bytes equal to 16 x the signed code (see pack_int4_words): one 16-byte packed piece
// becomes 32 bytes.  Runs in front of the GEMM on the same stream when the caller provides a workspace;
// the GEMM then reads the bytes like 8-bit weights (from L2) instead of expanding every stage of every
// row tile again.
__global__ void w4_expand_kernel(const uint4* __restrict__ packed, uint4* __restrict__ out, int64_t n_pieces) {
  pdl_launch_dependents();
  pdl_wait();  // the workspace may still be read by the GEMM of the layer before this one
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_pieces; i += (int64_t)gridDim.x * blockDim.x) {
    const uint4 p4 = __ldg(packed + i);
    out[2 * i] = make_uint4((p4.x << 4) & 0xF0F0F0F0u, p4.x & 0xF0F0F0F0u, (p4.y << 4) & 0xF0F0F0F0u, p4.y & 0xF0F0F0F0u);
    out[2 * i + 1] = make_uint4((p4.z << 4) & 0xF0F0F0F0u, p4.z & 0xF0F0F0F0u, (p4.w << 4) & 0xF0F0F0F0u, p4.w & 0xF0F0F0F0u);
  }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

static bool encode_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides,
                       const uint32_t* box, CUtensorMapSwizzle sw,
                       CUtensorMapDataType dtype = CU_TENSOR_MAP_DATA_TYPE_UINT8) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t d[5];
  cuuint64_t st[5];
  cuuint32_t b[5], es[5];
  for (int i = 0; i < rank; ++i) {
    d[i] = dims[i];
    b[i] = box[i];
    es[i] = 1;
  }
  for (int i = 0; i + 1 < rank; ++i) st[i] = strides[i];
  return fn(m, dtype, (cuuint32_t)rank, const_cast<void*>(base), d, st, b, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, bool W4, bool CONV>
static dgq_status launch_gemm(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmY,
                              const GemmArgs& a, int grid, cudaStream_t stream) {
  using Cfg = GemmCfg<BN, W4>;
  static bool attr_set[64] = {false};
  int dev = 0;
  DGQ_CUDA_OK(cudaGetDevice(&dev));
  if (dev >= 64 || !attr_set[dev]) {
    DGQ_CUDA_OK(cudaFuncSetAttribute(gq_gemm_kernel<BN, W4, CONV>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     Cfg::SMEM));
    if (dev < 64) attr_set[dev] = true;
  }
  DGQ_CUDA_OK(launch_pdl(gq_gemm_kernel<BN, W4, CONV>, dim3(grid), dim3(gemm_threads(W4)), (size_t)Cfg::SMEM, stream, tmA,
                         tmB, tmY, a));
  g_launches += 1;
  DGQ_CUDA_OK(cudaGetLastError());
  return DGQ_OK;
}

template <int BN>
static dgq_status launch_gemm_bn(bool w4, bool conv, const CUtensorMap& tmA, const CUtensorMap& tmB,
                                 const CUtensorMap& tmY, const GemmArgs& a, int grid, cudaStream_t stream) {
  if (w4)
    return conv ? launch_gemm<BN, true, true>(tmA, tmB, tmY, a, grid, stream)
                : launch_gemm<BN, true, false>(tmA, tmB, tmY, a, grid, stream);
  return conv ? launch_gemm<BN, false, true>(tmA, tmB, tmY, a, grid, stream)
              : launch_gemm<BN, false, false>(tmA, tmB, tmY, a, grid, stream);
}

}  // namespace dgq

extern "C" dgq_status dgq_linear(const dgq_groups* g, const dgq_weight* w, int timestep, int mode, int layout,
                                 const void* Xq, const float* dyn_scale, const int32_t* dyn_zp, const void* bias,
                                 void* Y, int64_t M, int64_t ldy, const dgq_conv_desc* conv, void* workspace,
                                 size_t workspace_bytes, void* stream) {
  using namespace dgq;
  // 4-bit weights: with a workspace they are expanded once per call in front of the GEMM, without one
  // the GEMM expands them itself, stage by stage
  const size_t ws_need = w && w->w_bits == 4 ? (size_t)w->N_pad * (size_t)w->Kt : 0;
  const bool expand_first = ws_need != 0 && workspace != nullptr;
  if (expand_first) {
    if (workspace_bytes < ws_need) return DGQ_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return DGQ_ERR_ALIGNMENT;
  }
  if (!g || !w || !Xq || !Y || M <= 0) return DGQ_ERR_INVALID_ARG;
  if (mode != DGQ_MODE_STATIC && mode != DGQ_MODE_DYNAMIC_TOKEN) return DGQ_ERR_INVALID_ARG;
  if (layout != DGQ_CODES_U8 && layout != DGQ_CODES_S8_CENTRED) return DGQ_ERR_INVALID_ARG;
  if (timestep < 0 || timestep >= g->T) return DGQ_ERR_INVALID_ARG;
  if (w->C != g->C || w->G != g->G || ldy < w->N) return DGQ_ERR_INVALID_ARG;
  if ((conv != nullptr) != (w->is_conv != 0)) return DGQ_ERR_INVALID_ARG;
  if (!aligned16(Xq) || !aligned16(Y) || (ldy % 8) != 0 || (bias && !aligned16(bias))) return DGQ_ERR_ALIGNMENT;
  if (M > (int64_t)INT32_MAX - 256) return DGQ_ERR_UNSUPPORTED;
  GemmArgs a;
  std::memset(&a, 0, sizeof(a));
  if (mode == DGQ_MODE_STATIC) {
    if (!g->filled[timestep]) return DGQ_ERR_NOT_CALIBRATED;
    const size_t trow = (size_t)timestep * g->R * g->G;
    a.scale = g->d_scale + trow;
    a.zp = g->d_zp + trow;
    a.per_token = 0;
  } else {
    if (!dyn_scale || !dyn_zp) return DGQ_ERR_INVALID_ARG;
    if (layout != DGQ_CODES_U8) return DGQ_ERR_UNSUPPORTED;
    a.scale = dyn_scale;
    a.zp = dyn_zp;
    a.per_token = 1;
  }
  a.M = M;
  a.N = w->N;
  a.N_pad = w->N_pad;
  a.Kt = w->Kt;
  a.G = g->G;
  a.P = g->P;
  a.use_zp = (layout == DGQ_CODES_U8);
  a.code_max = (1 << g->bits) - 1;
  a.res_mask = w->res_mask;
  a.wres = w->d_wres;
  a.row_group = g->d_row_group;
  a.sw = w->d_sw;
  a.wsum = w->d_wsum;
  a.bias = (const __half*)bias;
  a.w_packed = (const uint8_t*)w->d_w;
  if (w->Kt / DGQ_K_ATOM > GEMM_MAX_ATOMS) return DGQ_ERR_UNSUPPORTED;
  for (int k = 0; k < g->G; ++k) a.end_mask[(w->seg_end[k] - 1) >> 6] |= 1ull << ((w->seg_end[k] - 1) & 63);
  for (int k = 0; k < g->G; ++k) {
    a.seg_end[k] = w->seg_end[k];
    a.grp_atoms[k] = (g->group_off[k + 1] - g->group_off[k]) / DGQ_K_ATOM;
    a.grp_chan0[k] = g->group_off[k];
  }
  int BN = 128;
  if (w->N % 160 == 0) BN = 160;
  else if (w->N <= 64) BN = 64;
  // instruction descriptor of kind::i8: int32 accumulator (bits 4-5 = 2), A format bit 7 (0 = u8,
  // 1 = s8), B format bit 10 = 1 (s8), both K-major, N >> 3 at bit 17, M >> 4 at bit 24
  a.idesc = (2u << 4) | ((layout == DGQ_CODES_S8_CENTRED ? 1u : 0u) << 7) | (1u << 10) |
            ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(GEMM_BM >> 4) << 24);
  a.n_tiles_m = (int)((M + GEMM_BM - 1) / GEMM_BM);
  a.n_tiles_n = (w->N + BN - 1) / BN;

  CUtensorMap tmA, tmB, tmY;
  std::memset(&tmA, 0, sizeof(tmA));
  std::memset(&tmB, 0, sizeof(tmB));
  std::memset(&tmY, 0, sizeof(tmY));
  {  // output: panels of 32 fp16 columns x 128 rows, 64-byte swizzle
    const uint64_t dims[2] = {(uint64_t)w->N, (uint64_t)M};
    const uint64_t strides[1] = {(uint64_t)ldy * 2};
    const uint32_t box[2] = {32u, (uint32_t)GEMM_BM};
    if (!encode_map(&tmY, Y, 2, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_DATA_TYPE_FLOAT16))
      return DGQ_ERR_CUDA;
  }
  if (conv) {
    if (layout != DGQ_CODES_S8_CENTRED || mode != DGQ_MODE_STATIC || g->R != 1) return DGQ_ERR_UNSUPPORTED;
    if (conv->c != g->C || (int64_t)conv->n * conv->h * conv->w != M) return DGQ_ERR_INVALID_ARG;
    int bw, bh, bn;
    if (conv->w >= 128) {
      if (conv->w % 128) return DGQ_ERR_UNSUPPORTED;
      bw = 128, bh = 1, bn = 1;
    } else if (128 % conv->w) {
      return DGQ_ERR_UNSUPPORTED;
    } else if (conv->h * conv->w >= 128) {
      bw = conv->w, bh = 128 / conv->w, bn = 1;
      if (conv->h % bh) return DGQ_ERR_UNSUPPORTED;
    } else {
      if (128 % (conv->h * conv->w)) return DGQ_ERR_UNSUPPORTED;
      bw = conv->w, bh = conv->h, bn = 128 / (conv->h * conv->w);
    }
    a.conv_W = conv->w;
    a.conv_H = conv->h;
    const uint64_t Cp = (uint64_t)g->K_pad;
    const uint64_t dims[4] = {Cp, (uint64_t)conv->w, (uint64_t)conv->h, (uint64_t)conv->n};
    const uint64_t strides[3] = {Cp, Cp * conv->w, Cp * conv->w * conv->h};
    const uint32_t box[4] = {32u, (uint32_t)bw, (uint32_t)bh, (uint32_t)bn};
    if (!encode_map(&tmA, Xq, 4, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_32B)) return DGQ_ERR_CUDA;
  } else {
    const uint64_t dims[2] = {(uint64_t)g->K_pad, (uint64_t)M};
    const uint64_t strides[1] = {(uint64_t)g->K_pad};
    const uint32_t box[2] = {128u, (uint32_t)GEMM_BM};
    if (!encode_map(&tmA, Xq, 2, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) return DGQ_ERR_CUDA;
  }
  if (w->w_bits == 8 || expand_first) {
    const void* wb = expand_first ? workspace : (const void*)w->d_w;
    const uint64_t dims[2] = {(uint64_t)w->Kt, (uint64_t)w->N_pad};
    const uint64_t strides[1] = {(uint64_t)w->Kt};
    const uint32_t box[2] = {128u, (uint32_t)BN};
    if (!encode_map(&tmB, wb, 2, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) return DGQ_ERR_CUDA;
  }
  int dev = 0, n_sm = 148;
  DGQ_CUDA_OK(cudaGetDevice(&dev));
  DGQ_CUDA_OK(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
  // a multiple of the number of column blocks, so that every CTA keeps one column block
  if (a.n_tiles_n > n_sm) return DGQ_ERR_UNSUPPORTED;
  const int grid = std::min(a.n_tiles_m, n_sm / a.n_tiles_n) * a.n_tiles_n;
  const bool w4 = (w->w_bits == 4) && !expand_first;
  cudaStream_t st = (cudaStream_t)stream;
  if (expand_first) {
    const int64_t n_pieces = (int64_t)(ws_need / 32);  // 16 packed bytes each
    const int blocks = (int)std::min<int64_t>((n_pieces + 255) / 256, (int64_t)n_sm * 8);
    DGQ_CUDA_OK(launch_pdl(w4_expand_kernel, dim3(blocks), dim3(256), (size_t)0, st, (const uint4*)w->d_w, (uint4*)workspace,
                           n_pieces));
    g_launches += 1;
  }
  if (BN == 160) return launch_gemm_bn<160>(w4, conv != nullptr, tmA, tmB, tmY, a, grid, st);
  if (BN == 64) return launch_gemm_bn<64>(w4, conv != nullptr, tmA, tmB, tmY, a, grid, st);
  return launch_gemm_bn<128>(w4, conv != nullptr, tmA, tmB, tmY, a, grid, st);
}

extern "C" dgq_status dgq_linear_workspace_bytes(const dgq_groups* g, const dgq_weight* w, int64_t M, size_t* bytes) {
  if (!g || !w || !bytes || M <= 0) return DGQ_ERR_INVALID_ARG;
  *bytes = w->w_bits == 4 ? (size_t)w->N_pad * (size_t)w->Kt : 0;
  return DGQ_OK;
}
