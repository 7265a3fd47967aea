// Separable transform on the tensor cores ("Separable spectral decomposition", "Reconstruction"),
// bf16 storage, head_dim 128 or 64 (template parameter CH).  Every axis pass is a batched contraction over "lines" of n grid
// positions along the axis (all other coordinates fixed): out[a][c] = sum_b Mat[a][b] in[b][c].
// A CTA works on tiles of 128 grid positions = 128/n adjacent lines, fetched by one TMA box per
// 64-channel half (a contiguous run of memory for the w axis; 128/n neighbouring w positions per
// axis position for the h and t axes, so that the strided axes also read contiguous pieces).
// One tile is one 128 x 128 x 128 contraction
//     D[j][c] = sum_r A[j][r] * X[r][c],   A = Mat kron I (or I kron Mat) over the lines of the tile
// with A held in tensor memory for the whole launch (loaded once per CTA), X the TMA tile used in place as
// the MN-major B operand, and D in tensor memory with one output position per lane, so that an
// epilogue thread owns a whole 256-byte output row and stores it with 16-byte accesses.
//
// Precision: the transform matrix is split into bf16 hi + lo parts, and so is every intermediate
// between two axis passes (two bf16 grids, hi = bf16(v), lo = bf16(v - hi)); a pass then issues
// C_hi*X_hi + C_lo*X_hi + C_hi*X_lo per k-step.  Intermediates can be far larger than the final
// values (low-frequency content, the constant offset the exchange adds to a whole band), so a
// single bf16 rounding between passes would not meet the output tolerance.
//
// Three-byte intermediates.  Where the three axes run as separate passes, the pair written by the first forward
// pass and the pairs between the inverse passes are stored as the fp32 value rounded to 24 bits: the upper 16
// bits (a bf16 by truncation) in the hi grid and the next 8 bits in a byte grid.  hi and (value - hi) are both
// exact bf16 operands, together they carry 16 significant bits like the bf16 hi/lo pair, and a pass moves 3
// instead of 4 bytes per value.  A launch whose input has the byte form (template parameter LO8) runs four more
// warps that expand the bytes of every arriving tile to the bf16 lo operand in shared memory before the MMAs
// read it (128 channels: in place, the bytes of a row arrive inside the row's own bf16 space).  The expansion
// competes with the epilogue for issue slots; measured per launch at 1M tokens (3 tensor-heads): a middle pass
// 0.55 -> 0.48 ms with byte-form input and output, the band-split pass 0.43 -> 0.67 ms and the last inverse
// pass 0.38 -> 0.42 ms with byte-form input.  So the band-split pass always reads a bf16 pair (the second
// forward pass writes one), and the fused two-axis launches keep bf16 pairs on both sides.
//
// Order of the tiles.  A pass that reads what the previous launch wrote walks its tiles from the last to the
// first (P.reverse), the next one forward again: the end of the previous launch's output is still in L2.
//
//   warp 0      TMA producer (ring of 3-7 stages)
//   warp 1      tcgen05.mma issuer (A from tensor memory), 3 accumulator buffers of 128 TMEM columns
//   warps 2..9  epilogue: tcgen05.ld, convert to hi/lo bf16, store; a thread owns one output position
// Output path (FIRST, MIDDLE, LAST): an epilogue warp's 32 rows are 32 grid positions that form a
// box of the grid, so the warp writes 32 channels of them (64 bytes per row, 64-byte swizzle, no
// bank conflicts) into its own staging area and one lane sends them out with a tensor store; the
// area is reused when that store has read it.  SPLIT scatters rows to band positions: staged the
// same way, then stored by all lanes with four lanes per 64-byte row piece.
// Modes: FIRST  caller's Q/K/V -> hi/lo intermediate
//        MIDDLE hi/lo intermediate -> hi/lo intermediate
//        SPLIT  intermediate -> band-major coefficient buffers (rank evaluated in registers): mid and
//               high band in bf16, low band in fp32 straight from the accumulators (the hi/lo
//               intermediates carry about 16 bits); the router's mid and high band energies are
//               accumulated here from the stored bf16 coefficients (the low band's, few values per
//               channel, by low_energy_kernel from the fp32 coefficients)
//        LAST   intermediate -> the caller's out tensor
#include <cuda.h>

#include <vector>

#include "ff_internal.h"
#include "ff_sm100.cuh"

using namespace sm100;

namespace {

constexpr int CH_MAX = 128;                          // largest head_dim; shared-memory tiles are sized for it
constexpr int TILE_ROWS = 128;
constexpr int TILE_BYTES = TILE_ROWS * CH_MAX * 2; // 32 KB: 128 rows of bf16
constexpr int HALF_BYTES = TILE_BYTES / 2;
constexpr int MAX_STAGE = 8;

#ifdef FF_DCT_PROF
__device__ unsigned long long g_dct_prof[128];
#define PROF_T0(v) const long long v = clock64()
#define PROF_ADD(i, v) atomicAdd(&g_dct_prof[(P.mode * 2 + (LO8 ? 1 : 0)) * 12 + (i)], (unsigned long long)(clock64() - (v)))
#else
#define PROF_T0(v)
#define PROF_ADD(i, v)
#endif
constexpr int NACC = 3;                     // accumulator buffers of 128 tensor-memory columns, behind the matrix (128 columns)
constexpr int IMG_CELLS = 64;               // 32-bit tensor-memory cells per matrix row: two bf16 K elements each
constexpr uint32_t COL_IMG_HI = 0, COL_IMG_LO = 64, COL_ACC = 128;
constexpr int DCT_TC_THREADS = 320;        // TMA warp, MMA warp, 8 epilogue warps
constexpr int DCT_TC_THREADS_LO8 = 448;    // ... and 4 warps that expand a one-byte lo part to the bf16 operand

enum { MODE_FIRST = 0, MODE_MIDDLE = 1, MODE_SPLIT = 2, MODE_LAST = 3 };

struct DctTcParams {
  FFDims dm;
  const uint32_t* image;   // matrix image as the tensor-memory A operand: hi [128][64] cells, then lo
  int n;                   // axis length
  int axis;                // 0 = t, 1 = h, 2 = w
  int mode;
  int group;               // tensor-heads in this launch
  int group_start;         // index of the first one (tensor * BH + bh for the forward, bh for the inverse)
  int in_split;            // input is a hi/lo pair of grids (map0 = hi, map1 = lo)
  int out_lo8;             // the lo part of the output pair is one byte per value (see "Three-byte intermediates")
  int nstage;              // ring depth
  int reverse;             // walk the tiles from the last to the first (what the previous launch wrote last is still in L2)
  __nv_bfloat16* spec_mid; __nv_bfloat16* spec_high;
  float* spec_low;         // MODE_SPLIT: [3 BH][N_low][d] fp32
  double* energy;          // [B][3][128]
  int* status;
};

constexpr int STG_PITCH = 64;                       // bytes per staged row piece; the 16-byte chunks are rotated by row/2 against bank conflicts

struct DctShared {
  uint64_t full[MAX_STAGE], empty[MAX_STAGE], acc_full[NACC], acc_empty[NACC], conv[MAX_STAGE];
  uint32_t tmem_base;
  int abort_flag;
  // per epilogue warp: 32 rows x 64 bytes of hi and of lo, to turn one-row-per-thread registers
  // into stores where four lanes cover a row's 64 contiguous bytes
  alignas(1024) uint8_t stage[8][2][32 * STG_PITCH];
};

// Grid coordinates (w, h, t) of the first position of tile `u` of a tensor-head.  A tile holds
// kf = 128/n lines: kf consecutive h for the w axis, kf consecutive w for the h and t axes.
// (all lengths are powers of two here: lq = log2 of the tiles per row of tiles, H / kf or W / kf)
__device__ __forceinline__ void tile_origin(int axis, int lkf, int lq, int u, int& w, int& h, int& t) {
  const int lo = (u & ((1 << lq) - 1)) << lkf, hi = u >> lq;
  if (axis == 2) { w = 0; h = lo; t = hi; }
  else if (axis == 1) { h = 0; w = lo; t = hi; }
  else { t = 0; w = lo; h = hi; }
}

__device__ __forceinline__ void tma_load_5d(void* smem_dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2,
                                            int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"((uint64_t)map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}

__device__ __forceinline__ void tma_store_5d(const void* smem_src, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                             int c4) {
  asm volatile("cp.async.bulk.tensor.5d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5, %6}], [%1];"
               ::"l"((uint64_t)map), "r"(smem_u32(smem_src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Three source maps (Q, K, V) in MODE_FIRST; otherwise map0 (= hi) and, for split input, map1 (= lo).
// map_oh / map_ol: destination hi / lo grids with the box of one epilogue warp (32 positions x 32
// channels), all modes but SPLIT; MODE_LAST has no lo grid.
template <int CH, bool LO8>
__global__ void __launch_bounds__(LO8 ? DCT_TC_THREADS_LO8 : DCT_TC_THREADS, 1)
dct_tc_kernel(const __grid_constant__ CUtensorMap map0, const __grid_constant__ CUtensorMap map1,
              const __grid_constant__ CUtensorMap map2, const __grid_constant__ CUtensorMap map_oh,
              const __grid_constant__ CUtensorMap map_ol, const DctTcParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const FFDims& dm = P.dm;
  const int n = P.n;
  const int kf = TILE_ROWS / n;                           // lines per tile
  const int lkf = 31 - __clz(kf);
  const int ln = 31 - __clz(n);
  const bool seq = P.axis == 2;                           // lines follow one another (w axis) or interleave
  const int NSTAGE = P.nstage;
  const bool tma_out = P.mode != MODE_SPLIT;
  constexpr int TB = TILE_ROWS * CH * 2;                  // bytes of one data tile (16 KB for 64 channels)
  constexpr int LO8_OFF = CH == 128 ? TB : 2 * TB;         // where a stage takes the lo bytes
  const int STAGE_BYTES = LO8 ? LO8_OFF + TB / 2 + (CH == 128 ? TB / 2 : 0) : (P.in_split ? 2 * TB : TB);   // hi tile, lo tile
  uint8_t* sData = smem;                                  // NSTAGE x STAGE_BYTES
  DctShared& sh = *(DctShared*)(smem + NSTAGE * STAGE_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_per_th = (int)(dm.N / TILE_ROWS);
  const int ltpt = 31 - __clz(tiles_per_th);              // (a power of two)
  const int lq = 31 - __clz((P.axis == 2 ? dm.H : dm.W) >> lkf);
  const int total_tiles = P.group * tiles_per_th;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NSTAGE; ++i) { mbar_init(&sh.full[i], 1); mbar_init(&sh.empty[i], 1); mbar_init(&sh.conv[i], 128); }
    for (int i = 0; i < NACC; ++i) { mbar_init(&sh.acc_full[i], 1); mbar_init(&sh.acc_empty[i], 256); }
    sh.abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(&sh.tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = sh.tmem_base;
  volatile int* abort_flag = &sh.abort_flag;

  if (warp >= 2 && warp < 6) {
    // The matrix (hi and lo bf16 parts) into tensor memory, where it is the A operand of every tile: a thread
    // loads the row of its lane (prepared at plan creation as pairs of bf16 K elements per 32-bit cell).
    const int quarter = warp & 3, row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
#pragma unroll 1
    for (int im = 0; im < 2; ++im) {
      const uint32_t* src = P.image + (size_t)im * TILE_ROWS * IMG_CELLS + (size_t)row * IMG_CELLS;
#pragma unroll
      for (int c0 = 0; c0 < IMG_CELLS; c0 += 32) {
        uint32_t r[32];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const uint4 v = *(const uint4*)(src + c0 + 4 * i);
          r[4 * i] = v.x; r[4 * i + 1] = v.y; r[4 * i + 2] = v.z; r[4 * i + 3] = v.w;
        }
        tmem_st32(tm + lane_addr + im * 64 + c0, r);
      }
    }
    tmem_wait_st();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  if (warp == 0) {
    if (lane == 0) {
      tma_prefetch_desc(&map0);
      unsigned it = 0;
      bool ok = true;
      for (int sl = blockIdx.x; sl < total_tiles && ok; sl += gridDim.x, ++it) {
        const int s = P.reverse ? total_tiles - 1 - sl : sl;
        const int slot = it % NSTAGE;
        PROF_T0(pt);
        if (it >= (unsigned)NSTAGE) ok = mbar_wait(&sh.empty[slot], ((it / NSTAGE) - 1) & 1, abort_flag);
        PROF_ADD(6, pt);
        if (!ok) break;
        uint8_t* dst = sData + slot * STAGE_BYTES;
        const int gi = s >> ltpt, u = s & (tiles_per_th - 1);
        int w, h, t; tile_origin(P.axis, lkf, lq, u, w, h, t);
        const CUtensorMap* map = &map0;
        int slice = gi;
        if (P.mode == MODE_FIRST) {
          const int th = P.group_start + gi;
          const int tensor = (th >= dm.BH) + (th >= 2 * dm.BH);
          map = tensor == 0 ? &map0 : (tensor == 1 ? &map1 : &map2);
          slice = th - tensor * dm.BH;
        }
        mbar_arrive_expect_tx(&sh.full[slot], LO8 ? TB + TB / 2 : STAGE_BYTES);
        tma_load_5d(dst, map, &sh.full[slot], 0, w, h, t, slice);
        if (CH == 128) tma_load_5d(dst + HALF_BYTES, map, &sh.full[slot], 64, w, h, t, slice);
        if (LO8) {
          tma_load_5d(dst + LO8_OFF, &map1, &sh.full[slot], 0, w, h, t, slice);     // the lo bytes: rows of CH bytes
        } else if (P.in_split) {
          tma_load_5d(dst + TB, &map1, &sh.full[slot], 0, w, h, t, slice);
          if (CH == 128) tma_load_5d(dst + TB + HALF_BYTES, &map1, &sh.full[slot], 64, w, h, t, slice);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(TILE_ROWS, CH, /*a_mn_major=*/false, /*b_mn_major=*/true);
      unsigned it = 0;
      bool ok = true;
      for (int sl = blockIdx.x; sl < total_tiles && ok; sl += gridDim.x, ++it) {
        const int slot = it % NSTAGE, ab = it % NACC;
        PROF_T0(pm);
        ok = mbar_wait(LO8 ? &sh.conv[slot] : &sh.full[slot], (it / NSTAGE) & 1, abort_flag);
        PROF_ADD(2, pm);
        PROF_T0(pm2);
        if (ok && it >= NACC) ok = mbar_wait(&sh.acc_empty[ab], ((it / NACC) - 1) & 1, abort_flag);
        PROF_ADD(3, pm2);
        if (!ok) break;
        tc_fence_after();
        const uint32_t dbase = smem_u32(sData + slot * STAGE_BYTES);
        const uint32_t d_tm = tm + COL_ACC + ab * 128;
        const uint64_t xh0 = smem_desc_sw128(dbase, HALF_BYTES, 1024), xl0 = smem_desc_sw128(dbase + TB, HALF_BYTES, 1024);
#pragma unroll
        for (int ks = 0; ks < TILE_ROWS / 16; ++ks) {
          // (a descriptor advances by 2048 bytes = 128 in its address field per 16 rows of K)
          umma_ts(d_tm, tm + COL_IMG_HI + ks * 8, xh0 + (uint64_t)(ks * 128), idesc, ks > 0 ? 1u : 0u);
          umma_ts(d_tm, tm + COL_IMG_LO + ks * 8, xh0 + (uint64_t)(ks * 128), idesc, 1u);
          if (P.in_split) umma_ts(d_tm, tm + COL_IMG_HI + ks * 8, xl0 + (uint64_t)(ks * 128), idesc, 1u);
        }
        umma_commit(&sh.empty[slot]);
        umma_commit(&sh.acc_full[ab]);
      }
    }
  } else if (LO8 && warp >= 10) {
    // ------------------------------------------------------------------ lo bytes -> bf16 lo operand
    // A thread owns a row of the tile.  For every value: v24 = (hi << 16) | (byte << 8) as fp32; lo = v24 - hi,
    // exact in bf16.  The bytes arrive as rows of CH bytes (128-byte swizzle for 128 channels, 64-byte for 64),
    // the bf16 tiles as 64-channel halves of 128-byte rows (128-byte swizzle).
    const int r0 = threadIdx.x - 320;
    unsigned it = 0;
    bool ok = true;
    for (int sl = blockIdx.x; sl < total_tiles && ok; sl += gridDim.x, ++it) {
      const int slot = it % NSTAGE;
      PROF_T0(pc0);
      ok = __all_sync(0xffffffffu, mbar_wait(&sh.full[slot], (it / NSTAGE) & 1, abort_flag));
      if (threadIdx.x == 320) PROF_ADD(0, pc0);
      if (!ok) break;
      PROF_T0(pc1);
      uint8_t* base = sData + slot * STAGE_BYTES;
#pragma unroll 1
      for (int r = r0; r < TILE_ROWS; r += 128) {
      // 128 channels: the bytes arrive where the bf16 lo tile goes, row r's 128 bytes inside the first half of its
      // own bf16 row, so a thread takes them into registers before it writes the row (no other thread touches
      // it).  64 channels: the bytes have their own 8 KB behind the two tiles.
      const uint8_t* lob = base + LO8_OFF + r * CH;
      uint32_t lw[CH / 4];
#pragma unroll
      for (int cc = 0; cc < CH / 16; ++cc) {                 // 16-byte chunk cc of the row (16 channels)
        const int pc = CH == 128 ? (cc ^ (r & 7)) : (cc ^ ((r >> 1) & 3));
        const uint4 lb = *(const uint4*)(lob + (pc << 4));
        lw[4 * cc] = lb.x; lw[4 * cc + 1] = lb.y; lw[4 * cc + 2] = lb.z; lw[4 * cc + 3] = lb.w;
      }
#pragma unroll
      for (int c8 = 0; c8 < CH / 8; ++c8) {                  // 8-channel chunk of the row: one 16-byte chunk of bf16
        const uint32_t off = (uint32_t)(c8 >> 3) * HALF_BYTES + (uint32_t)r * 128 + (uint32_t)(((c8 & 7) ^ (r & 7)) << 4);
        const uint4 hv = *(const uint4*)(base + off);
        const uint32_t hw[4] = {hv.x, hv.y, hv.z, hv.w};
        uint32_t ow[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t by = lw[2 * c8 + (i >> 1)] >> (16 * (i & 1));              // bytes of channels 2i, 2i+1 in the low half
          const uint32_t h0 = hw[i] << 16, h1 = hw[i] & 0xffff0000u;
          const float l0 = __uint_as_float(h0 | ((by & 0xffu) << 8)) - __uint_as_float(h0);
          const float l1 = __uint_as_float(h1 | (by & 0xff00u)) - __uint_as_float(h1);
          const __nv_bfloat162 lp = __floats2bfloat162_rn(l0, l1);
          ow[i] = *(const uint32_t*)&lp;
        }
        *(uint4*)(base + TB + off) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
      }
      }
      fence_proxy_async();
      mbar_arrive(&sh.conv[slot]);
      if (threadIdx.x == 320) PROF_ADD(1, pc1);
    }
  } else {
    const int quarter = warp & 3;
    const int j = quarter * 32 + lane;                    // output position of this thread inside a tile
    const int a = seq ? j & (n - 1) : j >> lkf;           // output index along the axis
    const int l = seq ? j >> ln : j & (kf - 1);           // line of the tile
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const int ew = warp - 2;                              // epilogue warp 0..7: warps 0-3 take channels 0..63, 4-7 channels 64..127
    constexpr int NQ = CH / 64;                           // 32-channel chunks per thread
    const int q_lo = (ew >> 2) * NQ;
    // Grid offset of the warp's first row (tile row 32 quarter) from the tile origin: the warp's 32
    // rows are the box [32 channels] x [these offsets .. + the extents the store map was built with]
    const int j0 = quarter * 32;
    const int a0 = seq ? j0 & (n - 1) : j0 >> lkf, l0 = seq ? j0 >> ln : j0 & (kf - 1);
    const int dw = P.axis == 2 ? a0 : l0, dh = P.axis == 2 ? l0 : (P.axis == 1 ? a0 : 0), dt = P.axis == 0 ? a0 : 0;
    const int Lhw = dm.L[1] * dm.L[2], Mhw = dm.M[1] * dm.M[2];
    // (SPLIT) lane k of a warp accumulates the energies of channels 32 q + 2 (k % 16) + {0, 1} over the
    // warp's rows of parity k / 16: ea = mid + high rows, em = mid rows
    float ea[NQ][2] = {}, em[NQ][2] = {};                 // [chunk of the thread][channel of the pair]
    int e_sample = -1, sample_th = -1, sample_of_th = 0;
    unsigned it = 0;
    bool ok = true;
    auto flush_energy = [&]() {
      if (e_sample >= 0 && P.energy) {
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int c = (q_lo + qi) * 32 + 2 * (lane & 15) + e;
            atomicAdd(P.energy + ((size_t)e_sample * 3 + 1) * CH + c, (double)em[qi][e]);
            atomicAdd(P.energy + ((size_t)e_sample * 3 + 2) * CH + c, (double)(ea[qi][e] - em[qi][e]));
            ea[qi][e] = em[qi][e] = 0.f;
          }
      }
    };
    for (int sl = blockIdx.x; sl < total_tiles && ok; sl += gridDim.x, ++it) {
      const int s = P.reverse ? total_tiles - 1 - sl : sl;
      const int ab = it % NACC;
      PROF_T0(pe0);
      ok = __all_sync(0xffffffffu, mbar_wait(&sh.acc_full[ab], (it / NACC) & 1, abort_flag));
      if (threadIdx.x == 64) PROF_ADD(4, pe0);
      if (!ok) break;
      tc_fence_after();
      PROF_T0(pe1);
      const int gi = s >> ltpt, u = s & (tiles_per_th - 1);
      int w, h, t; tile_origin(P.axis, lkf, lq, u, w, h, t);
      const int th = P.group_start + gi;
      const int tensor = (th >= dm.BH) + (th >= 2 * dm.BH), bh = th - tensor * dm.BH;
      // where this thread's row goes
      __nv_bfloat16* row_hi = nullptr; float* row_f32 = nullptr;
      int band = -1;
      if (P.mode == MODE_SPLIT) {
        if (th != sample_th) { sample_th = th; sample_of_th = bh / dm.heads; }
        const int sample = sample_of_th;
        if (sample != e_sample) { flush_energy(); e_sample = sample; }
        // Band and rank of this row's coefficient: the pass axis supplies index a, the tile origin the
        // other two (lines of a tile are neighbours along w for the t and h passes, along h for the w
        // pass).  The counts of box members below a coefficient are piecewise linear in the coordinates.
        const int kt = P.axis == 0 ? a : t;
        const int h_ = P.axis == 1 ? a : (P.axis == 2 ? h + l : h);
        const int ww = P.axis == 2 ? a : w + l;
        const bool hw_low = h_ < dm.L[1] && ww < dm.L[2], hw_mid = h_ < dm.M[1] && ww < dm.M[2];
        const int offM = (h_ < dm.M[1] ? h_ : dm.M[1]) * dm.M[2] + (h_ < dm.M[1] ? (ww < dm.M[2] ? ww : dm.M[2]) : 0);
        // (axis lengths are at most 128, so every count fits 32 bits)
        const int cm = kt < dm.M[0] ? kt * Mhw + offM : dm.M[0] * Mhw;
        const size_t th_slice = (size_t)tensor * dm.BH + bh;
        long long rk, nband;                                                         // band-local rank, band length
        if (kt < dm.L[0] && hw_low) {
          band = 0;                                                                  // low band: fp32
          rk = (kt * dm.L[1] + h_) * dm.L[2] + ww; nband = dm.Nlow;
          row_f32 = P.spec_low + (th_slice * dm.Nlow + (unsigned)rk) * CH;
        } else if (kt < dm.M[0] && hw_mid) {
          const int offL = (h_ < dm.L[1] ? h_ : dm.L[1]) * dm.L[2] + (h_ < dm.L[1] ? (ww < dm.L[2] ? ww : dm.L[2]) : 0);
          const int cl = kt < dm.L[0] ? kt * Lhw + offL : (int)dm.Nlow;
          band = 1;
          rk = cm - cl; nband = dm.Nmid;
          row_hi = P.spec_mid + (th_slice * dm.Nmid + (unsigned)rk) * CH;
        } else {
          band = 2;
          rk = ((kt * dm.H + h_) * dm.W + ww) - cm; nband = dm.Nhigh;
          row_hi = P.spec_high + (th_slice * dm.Nhigh + (unsigned)rk) * CH;
        }
        // (debug build) the rank must lie inside its band and the coordinates inside the grid
        if (!FF_DBG_OK(kt >= 0 && kt < dm.T && h_ >= 0 && h_ < dm.H && ww >= 0 && ww < dm.W && rk >= 0 && rk < nband &&
                       th_slice < (size_t)3 * dm.BH, P.status, 2)) {
          row_hi = nullptr; row_f32 = nullptr; band = -1;
        }
      }
      // (SPLIT) lane L stores for rows 8 i + L/4 of its warp: fetch those rows' destinations
      __nv_bfloat16* dst_hi[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int src = 8 * i + (lane >> 2);
        dst_hi[i] = (__nv_bfloat16*)__shfl_sync(0xffffffffu, (unsigned long long)row_hi, src);
      }
      const int out_slice = P.mode == MODE_LAST ? th : gi;
      const unsigned nonlow_rows = __ballot_sync(0xffffffffu, band > 0), mid_rows = __ballot_sync(0xffffffffu, band == 1);
      // both 32-channel chunks of the row at once; the accumulator buffer is free as soon as they are read
      uint32_t rr2[NQ][32];
#pragma unroll
      PROF_T0(pl);
      for (int qi = 0; qi < NQ; ++qi) tmem_ld32(tm + lane_addr + COL_ACC + ab * 128 + (q_lo + qi) * 32, rr2[qi]);
      tmem_wait_ld();
      if (threadIdx.x == 64) { PROF_ADD(8, pl); PROF_ADD(9, pe1); }
      tc_fence_before();
      mbar_arrive(&sh.acc_empty[ab]);
#pragma unroll
      for (int qi = 0; qi < NQ; ++qi) {
        const int q = q_lo + qi;
        uint32_t (&r)[32] = rr2[qi];
        if (row_f32) {
#pragma unroll
          for (int i = 0; i < 8; ++i)
            *(uint4*)(row_f32 + q * 32 + i * 4) = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
        }
        {
          const bool want_lo = P.mode == MODE_FIRST || P.mode == MODE_MIDDLE;
          const bool lo8 = want_lo && P.out_lo8;
          uint32_t hi[16], lo[16];
          if (lo8) {
            // three-byte form: the value rounded to 24 bits; hi = its upper 16 bits, lo = the next byte
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] += 0x80u;
#pragma unroll
            for (int i = 0; i < 16; ++i) hi[i] = __byte_perm(r[2 * i], r[2 * i + 1], 0x7632);
#pragma unroll
            for (int i = 0; i < 8; ++i)
              lo[i] = __byte_perm(__byte_perm(r[4 * i], r[4 * i + 1], 0x0051), __byte_perm(r[4 * i + 2], r[4 * i + 3], 0x0051), 0x5410);
          } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const __nv_bfloat162 hp = __floats2bfloat162_rn(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
            hi[i] = *(const uint32_t*)&hp;
          }
          }
          if (want_lo && !lo8) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const __nv_bfloat162 lp = __floats2bfloat162_rn(__uint_as_float(r[2 * i]) - __uint_as_float(hi[i] << 16),
                                                             __uint_as_float(r[2 * i + 1]) - __uint_as_float(hi[i] & 0xffff0000u));
              lo[i] = *(const uint32_t*)&lp;
            }
          }
          uint8_t* st_hi = sh.stage[ew][0];
          uint8_t* st_lo = sh.stage[ew][1];
          if (tma_out) {
            // the previous store of this warp must have read the staging area
            PROF_T0(pw);
            if (lane == 0) bulk_wait_read0();
            __syncwarp();
            if (threadIdx.x == 64) PROF_ADD(7, pw);
          }
          // 16-byte chunk i of row `lane` at chunk position i ^ (lane / 2 % 4): the 64-byte swizzle
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            *(uint4*)(st_hi + lane * STG_PITCH + ((i ^ ((lane >> 1) & 3)) << 4)) = make_uint4(hi[4 * i], hi[4 * i + 1], hi[4 * i + 2], hi[4 * i + 3]);
            if (want_lo && !lo8)
              *(uint4*)(st_lo + lane * STG_PITCH + ((i ^ ((lane >> 1) & 3)) << 4)) = make_uint4(lo[4 * i], lo[4 * i + 1], lo[4 * i + 2], lo[4 * i + 3]);
          }
          if (lo8) {                                        // 32 bytes per row, rows 32 bytes apart (no swizzle)
            *(uint4*)(st_lo + lane * 32) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            *(uint4*)(st_lo + lane * 32 + 16) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
          }
          if (tma_out) {
            PROF_T0(pf);
            fence_proxy_async();
            __syncwarp();
            if (threadIdx.x == 64) PROF_ADD(10, pf);
            if (lane == 0) {
              tma_store_5d(st_hi, &map_oh, q * 32, w + dw, h + dh, t + dt, out_slice);
              if (want_lo) tma_store_5d(st_lo, &map_ol, q * 32, w + dw, h + dh, t + dt, out_slice);
              bulk_commit();
            }
          } else {
            __syncwarp();
            if (P.energy) {
              // Router statistics: channel energies of the staged (bf16) coefficients, summed down the
              // columns of the warp's 32 x 32 block; a lane reads one channel pair of every other row.
              const int par = lane >> 4, cp = lane & 15;
              float a0 = 0.f, a1 = 0.f, m0 = 0.f, m1 = 0.f;
              if (nonlow_rows == 0xffffffffu && (mid_rows == 0u || mid_rows == 0xffffffffu)) {
                // (almost every block: its 32 rows lie in one band, mid or high)
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                  const uint32_t wd = *(const uint32_t*)(st_hi + (2 * i + par) * STG_PITCH + (((cp >> 2) ^ (i & 3)) << 4) + (cp & 3) * 4);
                  const float v0 = __uint_as_float(wd << 16), v1 = __uint_as_float(wd & 0xffff0000u);
                  a0 = fmaf(v0, v0, a0); a1 = fmaf(v1, v1, a1);
                }
                if (mid_rows) { m0 = a0; m1 = a1; }
              } else {
                const unsigned nl = nonlow_rows >> par, md = mid_rows >> par;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                  const uint32_t wd = *(const uint32_t*)(st_hi + (2 * i + par) * STG_PITCH + (((cp >> 2) ^ (i & 3)) << 4) + (cp & 3) * 4);
                  const float v0 = __uint_as_float(wd << 16), v1 = __uint_as_float(wd & 0xffff0000u);
                  const float s0 = v0 * v0, s1 = v1 * v1;
                  if ((nl >> (2 * i)) & 1) { a0 += s0; a1 += s1; }
                  if ((md >> (2 * i)) & 1) { m0 += s0; m1 += s1; }
                }
              }
              ea[qi][0] += a0; ea[qi][1] += a1; em[qi][0] += m0; em[qi][1] += m1;
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int rr = 8 * i + (lane >> 2), piece = lane & 3;      // row of the warp, 16-byte piece of its 64 bytes
              if (dst_hi[i]) *(uint4*)(dst_hi[i] + q * 32 + piece * 8) = *(const uint4*)(st_hi + rr * STG_PITCH + ((piece ^ ((rr >> 1) & 3)) << 4));
            }
            __syncwarp();
          }
        }
      }
      if (threadIdx.x == 64) PROF_ADD(5, pe1);
    }
    if (P.mode == MODE_SPLIT) flush_energy();
    if (tma_out && lane == 0) bulk_wait0();
  }

  tc_fence_before();
  __syncthreads();
  if (sh.abort_flag) {
    if (threadIdx.x == 0) atomicExch(P.status, FF_ERR_TIMEOUT | 0x200);   // low byte: status, next byte: which kernel
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000) { }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tm, 512);
  }
}

// Low-band energy for the router: sum of squares of the fp32 low-band coefficients per channel,
// over Q~, K~, V~ and the heads of a sample.  grid = (row chunks, 3 BH); thread = channel.
__global__ void low_energy_kernel(const float* spec_low, double* energy, FFDims dm) {
  const int th = blockIdx.y, c = threadIdx.x;
  const long long per = (dm.Nlow + gridDim.x - 1) / gridDim.x;
  const long long r0 = (long long)blockIdx.x * per, r1 = r0 + per < dm.Nlow ? r0 + per : dm.Nlow;
  const float* v = spec_low + ((size_t)th * dm.Nlow) * dm.d + c;
  float e0 = 0.f, e1 = 0.f;
  long long r = r0;
  for (; r + 1 < r1; r += 2) {
    const float x0 = v[(size_t)r * dm.d], x1 = v[(size_t)(r + 1) * dm.d];
    e0 = fmaf(x0, x0, e0); e1 = fmaf(x1, x1, e1);
  }
  if (r < r1) { const float x0 = v[(size_t)r * dm.d]; e0 = fmaf(x0, x0, e0); }
  if (r0 < r1) atomicAdd(energy + ((size_t)((th % dm.BH) / dm.heads) * 3) * dm.d + c, (double)(e0 + e1));
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 5-D map over a [slices][T][H][W][128] bf16 grid whose box is one tile of 128 positions for a pass
// along `axis`: 128/n whole lines that are neighbours in memory.
// `bytes`: the grid holds one byte per value (the lo part of the three-byte form); the box then spans all
// channels of a row at once.
bool encode_grid_map(CUtensorMap* map, const void* base, const FFDims& dm, int slices, int axis, bool bytes = false) {
  static EncodeTiledFn enc = nullptr;
  if (!enc) {
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", (void**)&enc, cudaEnableDefault, &qr) != cudaSuccess || !enc)
      return false;
  }
  const cuuint64_t CH = (cuuint64_t)dm.d, eb = bytes ? 1 : 2;
  cuuint64_t dims[5] = {CH, (cuuint64_t)dm.W, (cuuint64_t)dm.H, (cuuint64_t)dm.T, (cuuint64_t)slices};
  cuuint64_t strides[4] = {CH * eb, (cuuint64_t)dm.W * CH * eb, (cuuint64_t)dm.H * dm.W * CH * eb,
                           (cuuint64_t)dm.N * CH * eb};
  const int n = axis == 2 ? dm.W : (axis == 1 ? dm.H : dm.T);
  const int kf = TILE_ROWS / n;
  cuuint32_t box[5] = {bytes ? (cuuint32_t)dm.d : 64u, 1, 1, 1, 1};
  box[1 + (2 - axis)] = (cuuint32_t)n;
  if (axis == 2) box[2] = (cuuint32_t)kf; else box[1] = (cuuint32_t)kf;
  cuuint32_t es[5] = {1, 1, 1, 1, 1};
  return enc(map, bytes ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims,
             strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
             bytes && dm.d == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Store map over the same kind of grid: the box is what one epilogue warp holds, 32 channels of the
// 32 positions of a quarter tile (tile rows 32 q .. 32 q + 31 of a pass along `axis`), 64-byte swizzle.
bool encode_store_map(CUtensorMap* map, const void* base, const FFDims& dm, int slices, int axis, bool bytes = false) {
  static EncodeTiledFn enc = nullptr;
  if (!enc) {
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", (void**)&enc, cudaEnableDefault, &qr) != cudaSuccess || !enc)
      return false;
  }
  const cuuint64_t CH = (cuuint64_t)dm.d, eb = bytes ? 1 : 2;
  cuuint64_t dims[5] = {CH, (cuuint64_t)dm.W, (cuuint64_t)dm.H, (cuuint64_t)dm.T, (cuuint64_t)slices};
  cuuint64_t strides[4] = {CH * eb, (cuuint64_t)dm.W * CH * eb, (cuuint64_t)dm.H * dm.W * CH * eb,
                           (cuuint64_t)dm.N * CH * eb};
  const int n = axis == 2 ? dm.W : (axis == 1 ? dm.H : dm.T);
  const int kf = TILE_ROWS / n;
  cuuint32_t box[5] = {32, 1, 1, 1, 1};
  if (axis == 2) {                       // rows = line * n + a: 32 consecutive rows
    box[1] = (cuuint32_t)(n < 32 ? n : 32);
    box[2] = (cuuint32_t)(n < 32 ? 32 / n : 1);
  } else {                               // rows = a * kf + line: 32 consecutive rows
    box[1] = (cuuint32_t)(kf < 32 ? kf : 32);
    box[1 + (2 - axis)] = (cuuint32_t)(kf < 32 ? 32 / kf : 1);
  }
  cuuint32_t es[5] = {1, 1, 1, 1, 1};
  return enc(map, bytes ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims,
             strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, bytes ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_64B,
             CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// `in_lo8`: the input pair's lo grid is the byte form (m1 = its byte map).
cudaError_t launch_pass(ff_plan* p, const CUtensorMap& m0, const CUtensorMap& m1, const CUtensorMap& m2,
                        const CUtensorMap& moh, const CUtensorMap& mol, DctTcParams& P, bool in_lo8, cudaStream_t st) {
  const size_t tile = (size_t)TILE_ROWS * P.dm.d * 2;
  const size_t stage = in_lo8 ? (P.dm.d == 128 ? 2 * tile : 2 * tile + tile / 2) : (size_t)(P.in_split ? 2 : 1) * tile;
  const size_t fixed = sizeof(DctShared) + 1024;
  int nstage = (int)((232448 - 256 - fixed) / stage);   // 227 KB of shared memory per CTA
  if (nstage > MAX_STAGE) nstage = MAX_STAGE;
  P.nstage = nstage;
  const size_t smem = nstage * stage + fixed;
  cudaError_t e = cudaSuccess;
  const int stages = (int)(P.group * (P.dm.N / TILE_ROWS));
  const int grid = stages < p->sm_count ? stages : p->sm_count;
#define FF_DCT(D, L)                                                                                              \
  do {                                                                                                            \
    e = cudaFuncSetAttribute(dct_tc_kernel<D, L>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);        \
    if (e == cudaSuccess)                                                                                         \
      dct_tc_kernel<D, L><<<grid, L ? DCT_TC_THREADS_LO8 : DCT_TC_THREADS, smem, st>>>(m0, m1, m2, moh, mol, P);  \
  } while (0)
  if (P.dm.d == 128) { if (in_lo8) FF_DCT(128, true); else FF_DCT(128, false); }
  else { if (in_lo8) FF_DCT(64, true); else FF_DCT(64, false); }
#undef FF_DCT
  if (e != cudaSuccess) return e;
  p->launches += 1;
  return cudaGetLastError();
}

#ifdef FF_DCT_PROF
}  // namespace
extern "C" void ff_debug_dct_prof(unsigned long long* out64, int reset) {
  cudaDeviceSynchronize();
  cudaMemcpyFromSymbol(out64, g_dct_prof, sizeof(unsigned long long) * 128);
  if (reset) { unsigned long long z[128] = {}; cudaMemcpyToSymbol(g_dct_prof, z, sizeof(z)); }
}
namespace {
#endif

bool axis_ok(int n) { return n == 16 || n == 32 || n == 64 || n == 128; }

}  // namespace

// bf16, head_dim 128 or 64, power-of-two axis lengths 16..128.
bool ffk_dct_tc_supported(const FFDims& dm) {
  if (dm.fp32 || (dm.d != 128 && dm.d != 64) || !axis_ok(dm.T) || !axis_ok(dm.H) || !axis_ok(dm.W)) return false;
  // a tile groups 128/n lines: consecutive h for the w pass, consecutive w for the h and t passes
  return dm.H % (TILE_ROWS / dm.W) == 0 && dm.W % (TILE_ROWS / dm.H) == 0 && dm.W % (TILE_ROWS / dm.T) == 0;
}

// The matrix of axis `axis` (0 = t, 1 = h, 2 = w), forward or inverse, as the tensor-memory operand image the
// plan holds (built at plan creation by ffk_dct2_build_image: w lines follow one another, A = I kron Mat;
// h and t lines interleave, A = Mat kron I).
static const uint32_t* matrix_image(const ff_plan* p, int axis, int inverse) {
  return p->dct2_images + (size_t)((inverse ? 3 : 0) + axis) * 2 * TILE_ROWS * IMG_CELLS;
}

// Scratch: two hi/lo pairs of bf16 grids for `group` tensor-heads.
size_t ffk_dct_tc_scratch_bytes(const FFDims& dm, int group) {
  const size_t grid = (size_t)group * dm.N * dm.d * 2;
  return 4 * ((grid + 255) / 256 * 256);
}

namespace {
struct Scratch { __nv_bfloat16 *a_hi, *a_lo, *b_hi, *b_lo; };
Scratch carve(ff_plan* p) {
  const size_t grid_bytes = ((size_t)p->dct_group * p->dm.N * p->dm.d * 2 + 255) / 256 * 256;
  char* base = (char*)p->buf.scratchA;
  Scratch s;
  s.a_hi = (__nv_bfloat16*)base; s.a_lo = (__nv_bfloat16*)(base + grid_bytes);
  s.b_hi = (__nv_bfloat16*)(base + 2 * grid_bytes); s.b_lo = (__nv_bfloat16*)(base + 3 * grid_bytes);
  return s;
}
}  // namespace

cudaError_t ffk_forward_transform_tc(ff_plan* p, const void* Q, const void* K, const void* V, bool want_energy,
                                     cudaStream_t st) {
  const FFDims& dm = p->dm;
  const int G = p->dct_group;
  const Scratch sc = carve(p);
  // Default: w and the shorter of h, t in one launch (intermediate on chip), then the band-split pass
  // along the remaining axis.  Kernel-select bit 4: the three axes as separate passes w, h, t.
  const bool fused = p->dct2_ok && !(p->attn_impl & 4);
  const int last_axis = fused ? (p->dct2_axis2 == 1 ? 0 : 1) : 0;
  const int last_n = last_axis == 0 ? dm.T : dm.H;
  // Between the launches the hi/lo pair has the three-byte form (the lo grids hold bytes).
  // mXh/mXl: load maps of a pass's input pair; oXh/oXl: store maps of a pass's output pair (the box
  // follows the axis of the pass that uses the map)
  const bool mid8 = false;        // (measured: the band-split pass is slower with a byte-form input)
  CUtensorMap mq, mk, mv, m1h, m1l, m2h, m2l, o0h, o0l, o1h, o1l, m3h, m3l;
  if (!encode_grid_map(&mq, Q, dm, dm.BH, 2) || !encode_grid_map(&mk, K, dm, dm.BH, 2) ||
      !encode_grid_map(&mv, V, dm, dm.BH, 2) || !encode_grid_map(&m1h, sc.a_hi, dm, G, 1) ||
      !encode_grid_map(&m1l, sc.a_lo, dm, G, 1, true) || !encode_grid_map(&m2h, sc.b_hi, dm, G, 0) ||
      !encode_grid_map(&m2l, sc.b_lo, dm, G, 0, mid8) || !encode_store_map(&o0h, sc.a_hi, dm, G, 2) ||
      !encode_store_map(&o0l, sc.a_lo, dm, G, 2, true) || !encode_store_map(&o1h, sc.b_hi, dm, G, 1) ||
      !encode_store_map(&o1l, sc.b_lo, dm, G, 1, mid8) || !encode_grid_map(&m3h, sc.a_hi, dm, G, last_axis) ||
      !encode_grid_map(&m3l, sc.a_lo, dm, G, last_axis))
    return cudaErrorInvalidValue;
  const int total = 3 * dm.BH;
  DctTcParams P{};
  P.dm = dm; P.status = p->buf.status;
  P.spec_mid = (__nv_bfloat16*)p->buf.spec_mid; P.spec_high = (__nv_bfloat16*)p->buf.spec_high;
  P.energy = want_energy ? p->buf.energy : nullptr;
  P.spec_low = p->buf.spec_low;
  for (int g0 = 0; g0 < total; g0 += G) {
    const int g = total - g0 < G ? total - g0 : G;
    P.group = g; P.group_start = g0;
    cudaError_t e;
    if (p->pipe_in) {                              // host-buffer entry point: this group's copy must have landed
      e = cudaStreamWaitEvent(st, p->ev_copy[g0 / G], 0);
      if (e != cudaSuccess) return e;
    }
    if (fused) {
      e = ffk_dct2_forward(p, Q, K, V, g0, g, sc.a_hi, sc.a_lo, st);
      if (e != cudaSuccess) return e;
      P.in_split = 1; P.out_lo8 = 0; P.reverse = 1;
      P.mode = MODE_SPLIT; P.axis = last_axis; P.n = last_n; P.image = matrix_image(p, last_axis, 0);
      e = launch_pass(p, m3h, m3l, m3l, m3h, m3l, P, false, st);    // (no tensor stores in this mode)
      if (e != cudaSuccess) return e;
      continue;
    }
    P.mode = MODE_FIRST; P.in_split = 0; P.out_lo8 = 1; P.reverse = 0; P.axis = 2; P.n = dm.W; P.image = matrix_image(p, 2, 0);
    e = launch_pass(p, mq, mk, mv, o0h, o0l, P, false, st);
    if (e != cudaSuccess) return e;
    P.mode = MODE_MIDDLE; P.in_split = 1; P.out_lo8 = mid8 ? 1 : 0; P.reverse = 1; P.axis = 1; P.n = dm.H; P.image = matrix_image(p, 1, 0);
    e = launch_pass(p, m1h, m1l, m1l, o1h, o1l, P, true, st);
    if (e != cudaSuccess) return e;
    P.in_split = 1; P.out_lo8 = 0; P.reverse = 0;
    P.mode = MODE_SPLIT; P.axis = 0; P.n = dm.T; P.image = matrix_image(p, 0, 0);
    e = launch_pass(p, m2h, m2l, m2l, m2h, m2l, P, mid8, st);    // (no tensor stores in this mode)
    if (e != cudaSuccess) return e;
  }
  if (want_energy) {
    long long chunks = (dm.Nlow + 511) / 512;             // about 512 rows per block
    if (chunks > 256) chunks = 256;
    low_energy_kernel<<<dim3((unsigned)chunks, (unsigned)total), dm.d, 0, st>>>(p->buf.spec_low, p->buf.energy, dm);
    p->launches += 1;
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// Inverse transform of `g` recombined grids (three-byte form in the first scratch pair, written by the
// exchange) into out[h0 .. h0+g).
cudaError_t ffk_inverse_transform_tc(ff_plan* p, int h0, int g, void* out, cudaStream_t st) {
  const FFDims& dm = p->dm;
  const int G = p->dct_group;
  const Scratch sc = carve(p);
  const bool fused = p->dct2_ok && !(p->attn_impl & 4);
  const int first_axis = fused ? (p->dct2_axis2 == 1 ? 0 : 1) : 0;       // the axis the fused launch leaves out
  const int first_n = first_axis == 0 ? dm.T : dm.H;
  // The first pass reads the exchange's output, which has the three-byte form.  With three passes the pairs
  // between them have it too; the fused launch takes a bf16 pair.
  const bool b8 = !fused;
  const bool inv8 = true;
  CUtensorMap m_in, m_inl, mbh, mbl, mah, mal, obh, obl, oah, oal, mout;
  if (!encode_grid_map(&m_in, sc.a_hi, dm, G, first_axis) || !encode_grid_map(&m_inl, sc.a_lo, dm, G, first_axis, true) ||
      !encode_grid_map(&mbh, sc.b_hi, dm, G, 1) ||
      !encode_grid_map(&mbl, sc.b_lo, dm, G, 1, true) || !encode_grid_map(&mah, sc.a_hi, dm, G, 2) ||
      !encode_grid_map(&mal, sc.a_lo, dm, G, 2, inv8) || !encode_store_map(&obh, sc.b_hi, dm, G, first_axis) ||
      !encode_store_map(&obl, sc.b_lo, dm, G, first_axis, b8) || !encode_store_map(&oah, sc.a_hi, dm, G, 1) ||
      !encode_store_map(&oal, sc.a_lo, dm, G, 1, inv8) || !encode_store_map(&mout, out, dm, dm.BH, 2))
    return cudaErrorInvalidValue;
  DctTcParams P{};
  P.dm = dm; P.status = p->buf.status; P.group = g; P.group_start = h0;
  P.mode = MODE_MIDDLE; P.in_split = 1; P.out_lo8 = b8 ? 1 : 0; P.reverse = 1; P.axis = first_axis; P.n = first_n;
  P.image = matrix_image(p, first_axis, 1);
  cudaError_t e = launch_pass(p, m_in, m_inl, m_inl, obh, obl, P, true, st);
  if (e != cudaSuccess) return e;
  if (fused) return ffk_dct2_inverse(p, sc.b_hi, sc.b_lo, h0, g, out, st);
  P.in_split = 1; P.out_lo8 = inv8 ? 1 : 0; P.reverse = 0; P.axis = 1; P.n = dm.H; P.image = matrix_image(p, 1, 1);
  e = launch_pass(p, mbh, mbl, mbl, oah, oal, P, true, st);
  if (e != cudaSuccess) return e;
  P.mode = MODE_LAST; P.out_lo8 = 0; P.reverse = 1; P.axis = 2; P.n = dm.W; P.image = matrix_image(p, 2, 1);
  return launch_pass(p, mah, mal, mal, mout, mout, P, inv8, st);
}
