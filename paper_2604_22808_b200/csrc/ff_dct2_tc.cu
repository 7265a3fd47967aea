// Two axis passes of the separable transform in one launch ("Separable spectral decomposition",
// "Reconstruction"): the w axis and a second axis (h or t, whichever is shorter), with the
// intermediate between them kept in shared memory.  bf16 storage, 32 channels per work item.
//
// A work item is one plane of the grid (all positions of the two axes at one coordinate of the third
// axis) of one tensor-head, for one chunk of 32 channels.  A thread-block cluster of CS CTAs owns the
// item: the plane's intermediate (hi/lo bf16, 4 bytes per value) is spread over the CTAs' shared
// memory, 128 KB or less each.
//   phase 1  every CTA transforms its share of the plane's w lines (tiles of 128 positions = 128/W
//            lines, fetched by TMA) and scatters each result row, as a hi/lo bf16 pair, into the
//            shared memory of the CTA that owns the row's w coefficient (st.shared::cluster); the
//            rows land in the operand layout of phase 2
//   phase 2  every CTA transforms the second axis for its share of the w coefficients (tiles of
//            128/n2 neighbouring coefficients x all n2 positions), straight from its part of the
//            buffer, and stores the result with tensor stores (hi/lo grids, or the caller's tensor)
// Both contractions are D[j][c] = sum_r A[j][r] X[r][c] over tiles of 128 positions x 32 channels
// with the matrix A = I kron Mat (w lines follow one another) or Mat kron I (lines of the second
// axis interleave) held in TENSOR MEMORY as the A operand (hi and lo bf16 parts, 64 columns each),
// so that a tile costs no shared-memory traffic for the matrix; the data tile is the MN-major B
// operand in place (64-byte rows, 64-byte swizzle); four tiles share one instruction (N = 128: an
// instruction takes the same time for any N up to 128).
//
//   warp 0        TMA producer (ring of 8 tiles, or 4 hi/lo pairs)
//   warp 1        tcgen05.mma issuer of phase 1; owns the tensor-memory allocation
//   warp 2        tells the cluster when this CTA has finished reading its part of the buffer
//   warp 3        tcgen05.mma issuer of phase 2
//   warps 4..11   phase-1 epilogue (a thread owns one position of a tile; the first four warps take
//                 the first tile of a pair, the next four the second)
//   warps 12..19  phase-2 epilogue
// so that phase 1 of the next item runs while phase 2 of the current one drains.
// Hand-shakes across the cluster use mbarriers with remote arrivals; every wait is bounded.
#include <cuda.h>

#include <vector>

#include "ff_internal.h"
#include "ff_sm100.cuh"

using namespace sm100;

namespace {

constexpr int CHK = 32;                       // channels per work item
constexpr int ROWS = 128;                     // positions per tile
constexpr int TILE_B = ROWS * CHK * 2;        // 8 KB: one bf16 tile
constexpr int NSTG = 8;                       // input ring: at most 8 tiles (64 KB: 8 bf16 tiles or 4 hi/lo pairs)
constexpr int RING_B = NSTG * TILE_B;
constexpr int MAX_TPC = 8;                    // tiles per CTA and item (128 KB of hi/lo buffer)
constexpr int D2_THREADS = 640;                 // TMA, MMA 1, release, MMA 2, 8 phase-1 and 8 phase-2 epilogue warps
constexpr int NA1 = 1, NA2 = 1;               // accumulator buffers (batches of 128 columns) of the two phases
constexpr int IMG_CELLS = 64;                 // 32-bit tensor-memory cells per matrix row: two bf16 K elements each
constexpr int STG_ROW = 64;                   // bytes per staged row (32 channels)

struct Dct2Params {
  FFDims dm;
  const uint32_t* img1;    // w-axis matrix: hi [128][64] cells, then lo
  const uint32_t* img2;    // second-axis matrix: hi, then lo
  int axis2;               // 1 = h, 0 = t
  int n1, n2, n3;          // W, length of the second axis, length of the remaining axis
  int in_split;            // input is a hi/lo pair of grids (map0 = hi, map1 = lo); otherwise Q, K, V
  int last;                // output is the caller's tensor (bf16, no lo part)
  int group, group_start;
  int nchunk;              // head_dim / 32
  int tpc;                 // tiles per CTA and item
  int cs;                  // CTAs per cluster
  int* status;
};

#ifdef FF_D2_PROF
__device__ unsigned long long g_d2_prof[32];
#define PROF_T0(v) const long long v = clock64()
#define PROF_ADD(i, v) atomicAdd(&g_d2_prof[i], (unsigned long long)(clock64() - (v)))
#else
#define PROF_T0(v)
#define PROF_ADD(i, v)
#endif

struct D2Shared {
  uint64_t in_full[NSTG], in_empty[NSTG], acc1_full[NA1], acc1_empty[NA1], acc2_full[NA2], acc2_empty[NA2];
  // The plane buffer has one slot of 8 tiles or two of 4 (items alternate): phase 1 of the next item fills one
  // slot while phase 2 of the current item reads the other.
  uint64_t buf_full[2];    // all rows of the item have landed in this CTA's slot (arrivals from every CTA's warps)
  uint64_t buf_half[2];    // (one CTA per plane) the rows of the first half of the second axis have landed
  uint64_t half_free[2];   // (one CTA per plane) phase 2 has finished reading those rows (its k-steps 0..3 of every batch)
  uint64_t buf_free[2];    // every CTA of the cluster has finished reading the slot (phase 2 of the item)
  uint64_t mma2_done[2];   // this CTA's phase-2 instructions of the item (by slot) have completed
  uint32_t tmem_base;
  int abort_flag;
};

// Shared-memory descriptor of an MN-major operand stored as 64-byte rows (32 bf16) with the 64-byte
// swizzle: 8-row groups 512 bytes apart (SBO); `lbo` = distance between 32-element chunks along N.
__device__ __forceinline__ uint64_t smem_desc_sw64(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)4 << 61;   // SWIZZLE_64B
  return d;
}

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_id_x() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_count_x() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t mapa(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_cluster_v4(uint32_t addr, uint4 v) {
  asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
               : "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint4 v) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait on a barrier whose arrivals come from other CTAs of the cluster.
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait_cluster(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > kWaitLimitCycles) { *abort_flag = 1; return false; }
  }
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

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

// Item `it` of the launch: chunk fastest (clusters that run side by side read neighbouring 64-byte
// pieces of the same rows), then the coordinate of the remaining axis, then the tensor-head.
__device__ __forceinline__ void decode_item(const Dct2Params& P, int it, int& gi, int& a3, int& chunk) {
  chunk = it % P.nchunk;
  const int rest = it / P.nchunk;
  a3 = rest % P.n3;
  gi = rest / P.n3;
}

// fp32 accumulators of one row (32 channels) -> bf16 hi and lo words (two channels per word)
__device__ __forceinline__ void split_hi_lo(const uint32_t (&r)[32], uint32_t (&hi)[16], uint32_t (&lo)[16], bool want_lo) {
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const __nv_bfloat162 hp = __floats2bfloat162_rn(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
    hi[i] = *(const uint32_t*)&hp;
  }
  if (want_lo) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const __nv_bfloat162 lp = __floats2bfloat162_rn(__uint_as_float(r[2 * i]) - __uint_as_float(hi[i] << 16),
                                                     __uint_as_float(r[2 * i + 1]) - __uint_as_float(hi[i] & 0xffff0000u));
      lo[i] = *(const uint32_t*)&lp;
    }
  }
}

// map0..map2: sources (Q, K, V; or hi, lo, -).  map_oh / map_ol: destinations (hi / lo grids, or the
// caller's tensor in map_oh), box = the 32 positions x 32 channels an epilogue warp holds.
__global__ void __launch_bounds__(D2_THREADS, 1)
dct2_tc_kernel(const __grid_constant__ CUtensorMap map0, const __grid_constant__ CUtensorMap map1,
               const __grid_constant__ CUtensorMap map2, const __grid_constant__ CUtensorMap map_oh,
               const __grid_constant__ CUtensorMap map_ol, const Dct2Params P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const FFDims& dm = P.dm;
  const int tpc = P.tpc;
  const int STAGE_B = P.in_split ? 2 * TILE_B : TILE_B;            // hi tile, then lo tile
  uint8_t* sBuf = smem;                                            // tpc x (hi 8 KB, lo 8 KB): the plane's intermediate
  uint8_t* sStage = smem + MAX_TPC * 2 * TILE_B;                   // 8 phase-2 warps x (hi 2 KB, lo 2 KB), 1024-byte aligned
  uint8_t* sIn = sStage + 8 * 2 * 32 * STG_ROW;                    // NSTG x STAGE_B
  D2Shared& sh = *(D2Shared*)(sIn + RING_B);
  const int nslot = RING_B / STAGE_B;                              // ring slots: 8 tiles, or 4 hi/lo pairs
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int cs = P.cs;
  const int n1 = P.n1, n2 = P.n2;
  const int ln1 = 31 - __clz(n1);
  const int kf1 = ROWS / n1, kf2 = ROWS / n2;
  const int lkf2 = 31 - __clz(kf2);
  const int ltpc = 31 - __clz(tpc);
  const int total = P.group * P.n3 * P.nchunk;
  const int nsl = tpc <= MAX_TPC / 2 ? 2 : 1;                      // slots of the plane buffer
  const int bt = tpc < 4 ? tpc : 4;                                // tiles per instruction batch (N = 32 bt columns): an
  const int nb = tpc / bt;                                         // instruction costs the same for any N up to 128
  // One CTA per plane and an even number of batches: the first half of the phase-1 batches holds the first half
  // of the second axis, i.e. rows 0..63 of every phase-2 tile = its k-steps 0..3.  Phase 2 of the item's first
  // batch starts on those while phase 1 still works on the second half.
  const bool half_start = cs == 1 && nb >= 2 && (nb & 1) == 0;
  // ... and phase 1 of the next item may overwrite those rows as soon as phase 2 has read them (forward launch:
  // measured slower for the inverse, whose phase 1 issues half as many instructions again)
  const bool half_release = half_start && !P.in_split;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NSTG; ++i) { mbar_init(&sh.in_full[i], 1); mbar_init(&sh.in_empty[i], 1); }
    for (int i = 0; i < NA1; ++i) { mbar_init(&sh.acc1_full[i], 1); mbar_init(&sh.acc1_empty[i], 256); }
    for (int i = 0; i < NA2; ++i) { mbar_init(&sh.acc2_full[i], 1); mbar_init(&sh.acc2_empty[i], 256); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sh.buf_full[i], 8 * cs); mbar_init(&sh.buf_free[i], cs); mbar_init(&sh.buf_half[i], 8); }
    mbar_init(&sh.mma2_done[0], 1); mbar_init(&sh.mma2_done[1], 1);
    mbar_init(&sh.half_free[0], 1); mbar_init(&sh.half_free[1], 1);
    sh.abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(&sh.tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  // every CTA's barriers exist before any peer arrives at them
  cluster_arrive();
  cluster_wait();
  tc_fence_after();
  const uint32_t tm = sh.tmem_base;
  volatile int* abort_flag = &sh.abort_flag;
  // tensor-memory columns: matrix images [0,256): w hi, w lo, second axis hi, lo; phase-1 accumulators
  // (NA1 batches of 128 columns) from 256; phase-2 accumulators (NA2 batches) behind them
  constexpr uint32_t COL_A1H = 0, COL_A1L = 64, COL_A2H = 128, COL_A2L = 192, COL_ACC1 = 256, COL_ACC2 = 256 + NA1 * 128;
  static_assert(COL_ACC2 + NA2 * 128 <= 512, "tensor memory has 512 columns");

  if (warp >= 4 && warp < 8) {
    // the four matrix images into tensor memory: a thread loads the row of its lane
    const int quarter = warp & 3, row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
#pragma unroll 1
    for (int im = 0; im < 4; ++im) {
      const uint32_t* src = (im < 2 ? P.img1 : P.img2) + (size_t)(im & 1) * ROWS * IMG_CELLS + (size_t)row * IMG_CELLS;
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

  const int cid = (int)cluster_id_x(), ncl = (int)cluster_count_x();
  PROF_T0(t_all);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&map0);
      unsigned n = 0;
      bool ok = true;
      for (int it = cid; it < total && ok; it += ncl) {
        int gi, a3, chunk; decode_item(P, it, gi, a3, chunk);
        const CUtensorMap* map = &map0;
        int slice = gi;
        if (!P.in_split) {
          const int th = P.group_start + gi;
          const int tensor = th / dm.BH;
          map = tensor == 0 ? &map0 : (tensor == 1 ? &map1 : &map2);
          slice = th % dm.BH;
        }
        for (int k = 0; k < tpc && ok; ++k, ++n) {
          const int slot = n % nslot;
          PROF_T0(tp0);
          if (n >= (unsigned)nslot) ok = mbar_wait(&sh.in_empty[slot], ((n / nslot) - 1) & 1, abort_flag);
          PROF_ADD(12, tp0);
          if (!ok) break;
          uint8_t* dst = sIn + slot * STAGE_B;
          const int u1 = (int)rank * tpc + k;                      // tile of the plane: lines u1 kf1 .. + kf1
          const int b0 = u1 * kf1;
          const int ch = P.axis2 == 1 ? b0 : a3, ct = P.axis2 == 1 ? a3 : b0;
          mbar_arrive_expect_tx(&sh.in_full[slot], STAGE_B);
          tma_load_5d(dst, map, &sh.in_full[slot], chunk * CHK, 0, ch, ct, slice);
          if (P.in_split) tma_load_5d(dst + TILE_B, &map1, &sh.in_full[slot], chunk * CHK, 0, ch, ct, slice);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer, phase 1
    // batches of bt input tiles (neighbouring slots of the ring), N = 32 bt.  A descriptor advances by
    // 1024 bytes (64 in its address field) per 16 rows of K.
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(ROWS, bt * CHK, /*a_mn_major=*/false, /*b_mn_major=*/true);
      const uint32_t in_base = smem_u32(sIn);
      unsigned n1b = 0;
      bool ok = true;
      for (int it = cid; it < total && ok; it += ncl) {
        for (int kb = 0; kb < nb && ok; ++kb, ++n1b) {
          const int ab = n1b % NA1;
          const unsigned nt = bt * n1b;                            // index of the batch's first tile in the ring sequence
          PROF_T0(tm0);
          for (int i = 0; i < bt && ok; ++i) ok = mbar_wait(&sh.in_full[(nt + i) % nslot], ((nt + i) / nslot) & 1, abort_flag);
          PROF_ADD(7, tm0);
          PROF_T0(tm1);
          if (ok && n1b >= (unsigned)NA1) ok = mbar_wait(&sh.acc1_empty[ab], ((n1b / NA1) - 1) & 1, abort_flag);
          PROF_ADD(8, tm1);
          if (!ok) break;
          tc_fence_after();
          const uint32_t x0 = in_base + (uint32_t)(nt % nslot) * STAGE_B;
          const uint64_t xh = smem_desc_sw64(x0, STAGE_B, 512), xl = smem_desc_sw64(x0 + TILE_B, STAGE_B, 512);
          const uint32_t d_tm = tm + COL_ACC1 + ab * 128;
          if (P.in_split) {
#pragma unroll
            for (int ks = 0; ks < ROWS / 16; ++ks) {
              umma_ts(d_tm, tm + COL_A1H + ks * 8, xh + (uint64_t)(ks * 64), idesc, ks > 0 ? 1u : 0u);
              umma_ts(d_tm, tm + COL_A1L + ks * 8, xh + (uint64_t)(ks * 64), idesc, 1u);
              umma_ts(d_tm, tm + COL_A1H + ks * 8, xl + (uint64_t)(ks * 64), idesc, 1u);
            }
          } else {
#pragma unroll
            for (int ks = 0; ks < ROWS / 16; ++ks) {
              umma_ts(d_tm, tm + COL_A1H + ks * 8, xh + (uint64_t)(ks * 64), idesc, ks > 0 ? 1u : 0u);
              umma_ts(d_tm, tm + COL_A1L + ks * 8, xh + (uint64_t)(ks * 64), idesc, 1u);
            }
          }
          for (int i = 0; i < bt; ++i) umma_commit(&sh.in_empty[(nt + i) % nslot]);
          umma_commit(&sh.acc1_full[ab]);
        }
      }
    }
  } else if (warp == 3) {
    // ------------------------------------------------------------------ MMA issuer, phase 2
    // (a thread of its own: phase 2 of an item waits for the whole cluster, phase 1 of the next item does not)
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(ROWS, bt * CHK, /*a_mn_major=*/false, /*b_mn_major=*/true);
      const uint32_t buf_base = smem_u32(sBuf);
      unsigned n2b = 0, ni = 0;
      bool ok = true;
      for (int it = cid; it < total && ok; it += ncl, ++ni) {
        // the plane's rows have landed in this CTA's buffer
        PROF_T0(tm2);
        const int sl = (int)(ni % nsl);                             // the item's slot of the plane buffer
        ok = half_start ? mbar_wait(&sh.buf_half[sl], (ni / nsl) & 1, abort_flag)
                        : mbar_wait_cluster(&sh.buf_full[sl], (ni / nsl) & 1, abort_flag);
        PROF_ADD(9, tm2);
        if (!ok) break;
        fence_proxy_async_all();
        for (int kb = 0; kb < nb && ok; ++kb, ++n2b) {
          const int ab = n2b % NA2;
          PROF_T0(tm3);
          if (n2b >= (unsigned)NA2) ok = mbar_wait(&sh.acc2_empty[ab], ((n2b / NA2) - 1) & 1, abort_flag);
          PROF_ADD(10, tm3);
          if (!ok) break;
          tc_fence_after();
          const uint32_t x0 = buf_base + (uint32_t)(sl * tpc + bt * kb) * 2 * TILE_B;   // tiles bt kb ..: hi, lo of each in turn
          const uint64_t xh = smem_desc_sw64(x0, 2 * TILE_B, 512), xl = smem_desc_sw64(x0 + TILE_B, 2 * TILE_B, 512);
          const uint32_t d_tm = tm + COL_ACC2 + ab * 128;
#pragma unroll
          for (int ks = 0; ks < ROWS / 16; ++ks) {
            if (ks == ROWS / 32 && kb == 0 && half_start) {          // the second half of the rows
              PROF_T0(tm4);
              ok = mbar_wait_cluster(&sh.buf_full[sl], (ni / nsl) & 1, abort_flag);
              PROF_ADD(11, tm4);
              if (!ok) break;
              fence_proxy_async_all();
              tc_fence_after();
            }
            umma_ts(d_tm, tm + COL_A2H + ks * 8, xh + (uint64_t)(ks * 64), idesc, ks > 0 ? 1u : 0u);
            umma_ts(d_tm, tm + COL_A2L + ks * 8, xh + (uint64_t)(ks * 64), idesc, 1u);
            umma_ts(d_tm, tm + COL_A2H + ks * 8, xl + (uint64_t)(ks * 64), idesc, 1u);
            // rows 0..63 of every tile have been read once the last batch's k-step 3 is done: phase 1 of the next
            // item may overwrite them
            if (ks == ROWS / 32 - 1 && kb == nb - 1 && half_release) umma_commit(&sh.half_free[sl]);
          }
          if (!ok) break;
          umma_commit(&sh.acc2_full[ab]);
        }
        umma_commit(&sh.mma2_done[sl]);
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ buffer release
    if (lane == 0) {
      unsigned ni = 0;
      bool ok = true;
      for (int it = cid; it < total && ok; it += ncl, ++ni) {
        ok = mbar_wait(&sh.mma2_done[ni % nsl], (ni / nsl) & 1, abort_flag);
        if (!ok) break;
        for (int rk = 0; rk < cs; ++rk) mbar_arrive_cluster(mapa(smem_u32(&sh.buf_free[ni % nsl]), (uint32_t)rk));
      }
    }
  } else if (warp >= 4 && warp < 12) {
    // ------------------------------------------------------------------ phase-1 epilogue
    // accumulators -> hi/lo rows in the owners' buffers.  A thread owns row (line l1, w coefficient a1)
    // of its tile and sends it as four 16-byte pieces of hi and four of lo, straight from registers.
    const int ew = warp - 4;                               // 0..7
    const int half = ew >> 2;                              // which tile of a pair
    const int quarter = warp & 3;
    const int j = quarter * 32 + lane;                     // position of this thread inside a tile
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const uint32_t buf_base = smem_u32(sBuf);
    const int l1 = j >> ln1, a1 = j & (n1 - 1);
    const int u2 = a1 >> lkf2;                             // phase-2 tile of the plane that takes coefficient a1
    const uint32_t owner = (uint32_t)(u2 >> ltpc);
    const int u2l = u2 & (tpc - 1);
    // Eight neighbouring lanes store at once; their rows are kf2 per tile, and rows of different tiles
    // that share (row / 2) % 4 would meet in the same banks: the lanes of tile t of the eight start
    // their four pieces at piece `rot` instead of 0, which spreads them over the banks.
    const int rot = (kf2 >= 8 ? 0 : ((lane & 7) >> lkf2) * (kf2 == 4 ? 2 : 1)) & 3;
    unsigned n1b = 0, ni = 0;
    bool ok = true;
    for (int it = cid; it < total && ok; it += ncl, ++ni) {
      PROF_T0(te0);
      const int sl = (int)(ni % nsl);                         // the item's slot: free once phase 2 of item ni - nsl is done
      if (ni >= (unsigned)nsl) {
        // (half_release: the first half of the batches writes rows phase 2 releases earlier; the rest waits below)
        ok = half_release ? __all_sync(0xffffffffu, mbar_wait(&sh.half_free[sl], ((ni / nsl) - 1) & 1, abort_flag))
                        : __all_sync(0xffffffffu, mbar_wait_cluster(&sh.buf_free[sl], ((ni / nsl) - 1) & 1, abort_flag));
        if (!ok) break;
      }
      if (threadIdx.x == 128) PROF_ADD(1, te0);
      for (int kb = 0; kb < nb && ok; ++kb, ++n1b) {
        if (half_release && kb == nb / 2 && ni >= (unsigned)nsl) {
          ok = __all_sync(0xffffffffu, mbar_wait_cluster(&sh.buf_free[sl], ((ni / nsl) - 1) & 1, abort_flag));
          if (!ok) break;
        }
        const int ab = n1b % NA1;
        PROF_T0(te1);
        ok = __all_sync(0xffffffffu, mbar_wait(&sh.acc1_full[ab], (n1b / NA1) & 1, abort_flag));
        if (!ok) break;
        if (threadIdx.x == 128) PROF_ADD(0, te1);
        PROF_T0(te2);
        tc_fence_after();
        for (int tb = half; tb < bt; tb += 2) {            // this warp's tiles of the batch
        uint32_t r[32];
        tmem_ld32(tm + lane_addr + COL_ACC1 + ab * 128 + tb * 32, r);
        tmem_wait_ld();
        if (tb + 2 >= bt) {                                // the accumulators are free once the warp's last tile is read
          tc_fence_before();
          mbar_arrive(&sh.acc1_empty[ab]);
        }
        uint32_t hi[16], lo[16];
        split_hi_lo(r, hi, lo, true);
        // where the row goes: position b of the second axis, row b kf2 + (a1 mod kf2) of tile u2l of `owner`
        const int u1 = (int)rank * tpc + bt * kb + tb;
        const int b = u1 * kf1 + l1;
        const int drow = (b << lkf2) | (a1 & (kf2 - 1));
        const uint32_t laddr = buf_base + (uint32_t)(sl * tpc + u2l) * 2 * TILE_B + (uint32_t)drow * STG_ROW;
        const uint32_t daddr = cs == 1 ? laddr : mapa(laddr, owner);
        const int swz = (drow >> 1) & 3;
        // (debug build) the row lies inside a tile of the owner's buffer
        if (!FF_DBG_OK(drow >= 0 && drow < ROWS && u2l >= 0 && u2l < tpc && owner < (uint32_t)cs && b < n2, P.status, 4)) continue;
        // rotate the pieces by `rot` (two conditional swaps), then piece i of the registers is piece (i + rot) % 4 of the row
        if (rot & 1) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint32_t h0 = hi[q], l0 = lo[q];
            hi[q] = hi[4 + q]; hi[4 + q] = hi[8 + q]; hi[8 + q] = hi[12 + q]; hi[12 + q] = h0;
            lo[q] = lo[4 + q]; lo[4 + q] = lo[8 + q]; lo[8 + q] = lo[12 + q]; lo[12 + q] = l0;
          }
        }
        if (rot & 2) {
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const uint32_t h0 = hi[q], l0 = lo[q];
            hi[q] = hi[8 + q]; hi[8 + q] = h0;
            lo[q] = lo[8 + q]; lo[8 + q] = l0;
          }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t dst = daddr + (uint32_t)((((i + rot) & 3) ^ swz) << 4);
          if (cs == 1) {                                    // the whole plane is this CTA's: plain shared-memory stores
            st_shared_v4(dst, make_uint4(hi[4 * i], hi[4 * i + 1], hi[4 * i + 2], hi[4 * i + 3]));
            st_shared_v4(dst + TILE_B, make_uint4(lo[4 * i], lo[4 * i + 1], lo[4 * i + 2], lo[4 * i + 3]));
          } else {
            st_cluster_v4(dst, make_uint4(hi[4 * i], hi[4 * i + 1], hi[4 * i + 2], hi[4 * i + 3]));
            st_cluster_v4(dst + TILE_B, make_uint4(lo[4 * i], lo[4 * i + 1], lo[4 * i + 2], lo[4 * i + 3]));
          }
        }
        }
        if (threadIdx.x == 128) PROF_ADD(2, te2);
        if (half_start && kb == nb / 2 - 1) {               // this warp's rows of the first half are written
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh.buf_half[sl]);
        }
      }
      if (!ok) break;
      // this warp's rows of the item are written: tell every CTA of the cluster
      PROF_T0(te4);
      if (cs == 1) {
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.buf_full[sl]);
      } else {
        fence_proxy_async_all();
        __syncwarp();
        if (lane < cs) mbar_arrive_cluster(mapa(smem_u32(&sh.buf_full[sl]), (uint32_t)lane));
      }
      if (threadIdx.x == 128) PROF_ADD(6, te4);
    }
  } else if (warp >= 12) {
    // ------------------------------------------------------------------ phase-2 epilogue
    // accumulators -> destination grids.  Rows 32 quarter .. + 31 of a tile are the box [a2 = a0 .., w = l0 ..]
    // of the store map; the warp stages them (64-byte swizzle) and one lane issues the tensor stores.
    const int ew = warp - 12;                              // 0..7
    const int half = ew >> 2;
    const int quarter = warp & 3;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    uint8_t* st_hi = sStage + ew * 2 * 32 * STG_ROW;
    uint8_t* st_lo = st_hi + 32 * STG_ROW;
    const int j0 = quarter * 32;
    const int a0 = j0 >> lkf2, l0 = j0 & (kf2 - 1);
    unsigned n2b = 0;
    bool ok = true;
    for (int it = cid; it < total && ok; it += ncl) {
      int gi, a3, chunk; decode_item(P, it, gi, a3, chunk);
      const int out_slice = P.last ? P.group_start + gi : gi;
      for (int kb = 0; kb < nb && ok; ++kb, ++n2b) {
        const int ab = n2b % NA2;
        PROF_T0(te5);
        ok = __all_sync(0xffffffffu, mbar_wait(&sh.acc2_full[ab], (n2b / NA2) & 1, abort_flag));
        if (!ok) break;
        if (threadIdx.x == 384) PROF_ADD(3, te5);
        PROF_T0(te6);
        tc_fence_after();
        for (int tb = half; tb < bt; tb += 2) {            // this warp's tiles of the batch
        uint32_t r[32];
        tmem_ld32(tm + lane_addr + COL_ACC2 + ab * 128 + tb * 32, r);
        tmem_wait_ld();
        if (tb + 2 >= bt) {
          tc_fence_before();
          mbar_arrive(&sh.acc2_empty[ab]);
        }
        uint32_t hi[16], lo[16];
        split_hi_lo(r, hi, lo, !P.last);
        // the previous tensor store of this warp must have read the staging area
        PROF_T0(te7);
        if (lane == 0) bulk_wait_read0();
        __syncwarp();
        if (threadIdx.x == 384) PROF_ADD(4, te7);
        // 16-byte chunk i of row `lane` at chunk position i ^ (lane / 2 % 4): the 64-byte swizzle
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int so = lane * STG_ROW + ((i ^ ((lane >> 1) & 3)) << 4);
          *(uint4*)(st_hi + so) = make_uint4(hi[4 * i], hi[4 * i + 1], hi[4 * i + 2], hi[4 * i + 3]);
          if (!P.last) *(uint4*)(st_lo + so) = make_uint4(lo[4 * i], lo[4 * i + 1], lo[4 * i + 2], lo[4 * i + 3]);
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
          const int u2g = (int)rank * tpc + bt * kb + tb;        // tile of the plane: w coefficients u2g kf2 .. + kf2
          const int cw = u2g * kf2 + l0;
          const int ch = P.axis2 == 1 ? a0 : a3, ct = P.axis2 == 1 ? a3 : a0;
          tma_store_5d(st_hi, &map_oh, chunk * CHK, cw, ch, ct, out_slice);
          if (!P.last) tma_store_5d(st_lo, &map_ol, chunk * CHK, cw, ch, ct, out_slice);
          bulk_commit();
        }
        }
        if (threadIdx.x == 384) PROF_ADD(5, te6);
      }
    }
    if (lane == 0) bulk_wait0();
  }

  // ------------------------------------------------------------------ teardown
  if (threadIdx.x == 128) PROF_ADD(15, t_all);
  tc_fence_before();
  __syncthreads();
  if (sh.abort_flag) {
    if (threadIdx.x == 0) atomicExch(P.status, FF_ERR_TIMEOUT | 0x400);   // low byte: status, next byte: which kernel
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000) { }
    __syncthreads();
  }
  // no CTA leaves while a peer may still write into its shared memory or arrive at its barriers
  cluster_arrive();
  cluster_wait();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tm, 512);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encoder() {
  static EncodeTiledFn enc = nullptr;
  if (!enc) {
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", (void**)&enc, cudaEnableDefault, &qr) != cudaSuccess) enc = nullptr;
  }
  return enc;
}

// 5-D map over a [slices][T][H][W][d] bf16 grid.  Load box: one phase-1 tile, 32 channels of 128/W
// whole w lines that are neighbours along the second axis.
bool encode_in_map(CUtensorMap* map, const void* base, const FFDims& dm, int slices, int axis2) {
  EncodeTiledFn enc = encoder();
  if (!enc) return false;
  const cuuint64_t CH = (cuuint64_t)dm.d;
  cuuint64_t dims[5] = {CH, (cuuint64_t)dm.W, (cuuint64_t)dm.H, (cuuint64_t)dm.T, (cuuint64_t)slices};
  cuuint64_t strides[4] = {CH * 2, (cuuint64_t)dm.W * CH * 2, (cuuint64_t)dm.H * dm.W * CH * 2, (cuuint64_t)dm.N * CH * 2};
  cuuint32_t box[5] = {CHK, (cuuint32_t)dm.W, 1, 1, 1};
  box[axis2 == 1 ? 2 : 3] = (cuuint32_t)(ROWS / dm.W);
  cuuint32_t es[5] = {1, 1, 1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Store box: what one epilogue warp holds after phase 2, 32 channels of tile rows 32 q .. 32 q + 31,
// row = (position along the second axis) * kf2 + (w coefficient inside the tile).
bool encode_out_map(CUtensorMap* map, const void* base, const FFDims& dm, int slices, int axis2) {
  EncodeTiledFn enc = encoder();
  if (!enc) return false;
  const cuuint64_t CH = (cuuint64_t)dm.d;
  cuuint64_t dims[5] = {CH, (cuuint64_t)dm.W, (cuuint64_t)dm.H, (cuuint64_t)dm.T, (cuuint64_t)slices};
  cuuint64_t strides[4] = {CH * 2, (cuuint64_t)dm.W * CH * 2, (cuuint64_t)dm.H * dm.W * CH * 2, (cuuint64_t)dm.N * CH * 2};
  const int n2 = axis2 == 1 ? dm.H : dm.T;
  const int kf2 = ROWS / n2;                       // at most 8
  cuuint32_t box[5] = {CHK, (cuuint32_t)kf2, 1, 1, 1};
  box[axis2 == 1 ? 2 : 3] = (cuuint32_t)(32 / kf2);
  cuuint32_t es[5] = {1, 1, 1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// (the staging areas of the tensor stores sit 1024-byte aligned: their 64-byte swizzle is a function of the address)
constexpr size_t D2_SMEM = 1024 + (size_t)MAX_TPC * 2 * TILE_B + (size_t)8 * 2 * 32 * STG_ROW + (size_t)RING_B + sizeof(D2Shared) + 64;

bool axis_ok(int n) { return n == 16 || n == 32 || n == 64 || n == 128; }

cudaError_t launch(ff_plan* p, const CUtensorMap& m0, const CUtensorMap& m1, const CUtensorMap& m2, const CUtensorMap& moh,
                   const CUtensorMap& mol, Dct2Params& P, cudaStream_t st) {
  cudaError_t e = cudaFuncSetAttribute(dct2_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)D2_SMEM);
  if (e != cudaSuccess) return e;
  const int items = P.group * P.n3 * P.nchunk;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)P.cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  cfg.blockDim = dim3(D2_THREADS); cfg.dynamicSmemBytes = D2_SMEM; cfg.stream = st;
  int clusters = p->dct2_clusters;
  if (clusters <= 0) {
    // how many clusters of this size the device runs at once
    cfg.gridDim = dim3((unsigned)(p->sm_count / P.cs * P.cs));
    int n = 0;
    e = cudaOccupancyMaxActiveClusters(&n, dct2_tc_kernel, &cfg);
    if (e != cudaSuccess || n < 1) { (void)cudaGetLastError(); n = P.cs == 1 ? p->sm_count : p->sm_count / P.cs / 2; }
    if (n < 1) n = 1;
    clusters = p->dct2_clusters = n;
  }
  if (clusters > items) clusters = items;
  cfg.gridDim = dim3((unsigned)(clusters * P.cs));
  e = cudaLaunchKernelEx(&cfg, dct2_tc_kernel, m0, m1, m2, moh, mol, P);
  if (e != cudaSuccess) return e;
  p->launches += 1;
  return cudaGetLastError();
}

}  // namespace

// Which second axis the fused launch takes and how many CTAs share a plane: the shorter of h and t
// (smaller planes need fewer CTAs), an even number of tiles per CTA.  The kernel runs clusters of up to
// eight CTAs, but it is used only where one or two CTAs hold the plane (W x n2 <= 2048 positions):
// measured on B200, the launch beats the separate passes by 23% at T=16, W=64 (one CTA per plane) and by
// 6% at T=32 (two), and loses from four CTAs on (the remote stores of phase 1 and their cluster-scope
// release cost more than the saved DRAM round trip).
constexpr int MAX_CLUSTER_USED = 2;

bool ffk_dct2_supported(const FFDims& dm, int* axis2, int* cs) {
  if (dm.fp32 || dm.d % CHK != 0 || (dm.d != 128 && dm.d != 64) || !axis_ok(dm.T) || !axis_ok(dm.H) || !axis_ok(dm.W)) return false;
  const int a2 = dm.T < dm.H ? 0 : 1;
  const int n2 = a2 == 1 ? dm.H : dm.T;
  const int tiles = dm.W * n2 / ROWS;
  int c = 1;
  while (tiles / c > MAX_TPC) c *= 2;
  if (c > MAX_CLUSTER_USED || tiles % c != 0 || (tiles / c) % 2 != 0) return false;
  if (axis2) *axis2 = a2;
  if (cs) *cs = c;
  return true;
}

// Matrix image of one axis and direction as the tensor-memory A operand: row j = output position
// of a tile, cell c = the bf16 pair (A[j][2c], A[j][2c+1]); hi part [128][64], then lo part.
// w axis: lines follow one another, A = I kron Mat (index = line*n + a); h, t: A = Mat kron I
// (index = a*kf + line).  `mat` is the host matrix [n][n], out[a] = sum_b mat[a][b] in[b].
bool ffk_dct2_build_image(ff_plan* p, int axis, int inverse, const float* mat, int n) {
  const size_t per = (size_t)2 * ROWS * IMG_CELLS;      // cells of one image (hi + lo)
  if (!p->dct2_images && cudaMalloc((void**)&p->dct2_images, 6 * per * sizeof(uint32_t)) != cudaSuccess) return false;
  const int kf = ROWS / n;
  const bool seq = axis == 2;
  std::vector<uint32_t> img(per);
  for (int j = 0; j < ROWS; ++j)
    for (int r = 0; r < ROWS; ++r) {
      float v;
      if (seq) v = (j / n == r / n) ? mat[(j % n) * n + (r % n)] : 0.f;
      else v = (j % kf == r % kf) ? mat[(j / kf) * n + (r / kf)] : 0.f;
      const __nv_bfloat16 hi = __float2bfloat16_rn(v);
      const __nv_bfloat16 lo = __float2bfloat16_rn(v - __bfloat162float(hi));
      const uint32_t hb = *(const uint16_t*)&hi, lb = *(const uint16_t*)&lo;
      const size_t cell = (size_t)j * IMG_CELLS + (r >> 1);
      if (r & 1) { img[cell] |= hb << 16; img[(size_t)ROWS * IMG_CELLS + cell] |= lb << 16; }
      else { img[cell] = hb; img[(size_t)ROWS * IMG_CELLS + cell] = lb; }
    }
  const int slot = (inverse ? 3 : 0) + axis;
  return cudaMemcpy(p->dct2_images + slot * per, img.data(), per * sizeof(uint32_t), cudaMemcpyHostToDevice) == cudaSuccess;
}

// Forward: Q, K, V of tensor-heads [g0, g0 + g) -> w and second-axis transform -> hi/lo grids.
cudaError_t ffk_dct2_forward(ff_plan* p, const void* Q, const void* K, const void* V, int g0, int g, void* out_hi, void* out_lo,
                             cudaStream_t st) {
  const FFDims& dm = p->dm;
  const int G = p->dct_group;
  int axis2, cs;
  if (!ffk_dct2_supported(dm, &axis2, &cs)) return cudaErrorInvalidValue;
  CUtensorMap mq, mk, mv, oh, ol;
  if (!encode_in_map(&mq, Q, dm, dm.BH, axis2) || !encode_in_map(&mk, K, dm, dm.BH, axis2) ||
      !encode_in_map(&mv, V, dm, dm.BH, axis2) || !encode_out_map(&oh, out_hi, dm, G, axis2) ||
      !encode_out_map(&ol, out_lo, dm, G, axis2))
    return cudaErrorInvalidValue;
  const size_t per = (size_t)2 * ROWS * IMG_CELLS;
  Dct2Params P{};
  P.dm = dm; P.status = p->buf.status;
  P.img1 = p->dct2_images + (size_t)(0 + 2) * per; P.img2 = p->dct2_images + (size_t)(0 + axis2) * per;
  P.axis2 = axis2; P.n1 = dm.W; P.n2 = axis2 == 1 ? dm.H : dm.T; P.n3 = axis2 == 1 ? dm.T : dm.H;
  P.in_split = 0; P.last = 0; P.group = g; P.group_start = g0; P.nchunk = dm.d / CHK;
  P.cs = cs; P.tpc = dm.W * P.n2 / ROWS / cs;
  return launch(p, mq, mk, mv, oh, ol, P, st);
}

// Inverse: hi/lo grids of heads [h0, h0 + g) -> w and second-axis inverse transform -> out.
cudaError_t ffk_dct2_inverse(ff_plan* p, const void* in_hi, const void* in_lo, int h0, int g, void* out, cudaStream_t st) {
  const FFDims& dm = p->dm;
  const int G = p->dct_group;
  int axis2, cs;
  if (!ffk_dct2_supported(dm, &axis2, &cs)) return cudaErrorInvalidValue;
  CUtensorMap mh, ml, mo;
  if (!encode_in_map(&mh, in_hi, dm, G, axis2) || !encode_in_map(&ml, in_lo, dm, G, axis2) ||
      !encode_out_map(&mo, out, dm, dm.BH, axis2))
    return cudaErrorInvalidValue;
  const size_t per = (size_t)2 * ROWS * IMG_CELLS;
  Dct2Params P{};
  P.dm = dm; P.status = p->buf.status;
  P.img1 = p->dct2_images + (size_t)(3 + 2) * per; P.img2 = p->dct2_images + (size_t)(3 + axis2) * per;
  P.axis2 = axis2; P.n1 = dm.W; P.n2 = axis2 == 1 ? dm.H : dm.T; P.n3 = axis2 == 1 ? dm.T : dm.H;
  P.in_split = 1; P.last = 1; P.group = g; P.group_start = h0; P.nchunk = dm.d / CHK;
  P.cs = cs; P.tpc = dm.W * P.n2 / ROWS / cs;
  return launch(p, mh, ml, ml, mo, mo, P, st);
}

#ifdef FF_D2_PROF
extern "C" void ff_debug_d2_prof(unsigned long long* out32, int reset) {
  cudaDeviceSynchronize();
  cudaMemcpyFromSymbol(out32, g_d2_prof, sizeof(unsigned long long) * 32);
  if (reset) { unsigned long long z[32] = {}; cudaMemcpyToSymbol(g_d2_prof, z, sizeof(z)); }
}
#endif
