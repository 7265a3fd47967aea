// Linear projections around the attention path ("Setup and notation": per-head Q_h, K_h, V_h are linear
// projections of the layer input; "Reconstruction": the head outputs are concatenated and projected), as one
// tcgen05 GEMM kernel, bf16 operands, fp32 accumulation:
//   QKV mode   [Q | K | V] = X [W_q | W_k | W_v],  X [B][N][D] token-major, D = heads * d, each W [D][D] with
//              y = x W; the epilogue writes the result straight into the per-head layout the transform reads,
//              Q/K/V [B][heads][N][d]
//   OUT mode   out = concat_h(O_h) W_o: the A operand is gathered from the per-head attention output
//              [B][heads][N][d] (K runs over (head, channel)), the result is token-major [B][N][D]
// Tiles of 128 tokens x 256 output columns, K in chunks of 64: A tile K-major (128-byte swizzle), B tile
// MN-major (four 64-column pieces), a ring of four stages filled by TMA, two accumulator buffers of 256
// tensor-memory columns so that the epilogue of one tile overlaps the main loop of the next.
//   warp 0      TMA producer          warp 1      tcgen05.mma issuer (owns the tensor memory)
//   warps 2..5  epilogue: tcgen05.ld, bf16, 16-byte stores; a thread owns one token of the tile
#include <cuda.h>

#include "ff_internal.h"
#include "ff_sm100.cuh"

using namespace sm100;

namespace {

constexpr int PM = 128, PN = 256, PK = 64;
constexpr int A_BYTES = PM * PK * 2;             // 16 KB
constexpr int B_PIECE = PK * 64 * 2;             // 8 KB: 64 K-rows x 64 columns
constexpr int B_BYTES = 4 * B_PIECE;             // 32 KB
constexpr int P_STAGE = A_BYTES + B_BYTES;
constexpr int P_NSTAGE = 4;
constexpr int P_THREADS = 192;

struct ProjParams {
  int mode;                // 0 = QKV, 1 = OUT
  int B, heads, d;         // batch, heads, head_dim
  long long N;             // tokens per sample
  int D;                   // heads * d: K extent, and the output width of one matrix
  int n_out;               // output columns in total: 3 D (QKV) or D (OUT)
  __nv_bfloat16* dst[3];   // QKV: Q, K, V [B][heads][N][d];  OUT: dst[0] = out [B][N][D]
  int* status;
};

struct ProjShared {
  uint64_t full[P_NSTAGE], empty[P_NSTAGE], acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

__global__ void __launch_bounds__(P_THREADS, 1)
proj_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const ProjParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  ProjShared& sh = *(ProjShared*)(smem + P_NSTAGE * P_STAGE);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m_tiles = (int)(P.N / PM), n_tiles = P.n_out / PN;
  const long long tiles = (long long)P.B * m_tiles * n_tiles;
  const int kchunks = P.D / PK;
  const int cpd = P.d / PK;                       // K chunks per head (OUT mode)

  if (threadIdx.x == 0) {
    for (int i = 0; i < P_NSTAGE; ++i) { mbar_init(&sh.full[i], 1); mbar_init(&sh.empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sh.acc_full[i], 1); mbar_init(&sh.acc_empty[i], 128); }
    sh.abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(&sh.tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = sh.tmem_base;
  volatile int* abort_flag = &sh.abort_flag;

  if (warp == 0) {
    if (lane == 0) {
      tma_prefetch_desc(&map_a); tma_prefetch_desc(&map_b);
      unsigned n = 0;
      bool ok = true;
      for (long long t = blockIdx.x; t < tiles && ok; t += gridDim.x) {
        const int nt = (int)(t % n_tiles);
        const long long mt = t / n_tiles;
        const int b = (int)(mt / m_tiles), m0 = (int)(mt % m_tiles) * PM;
        const int col0 = nt * PN;                 // first output column of the tile
        const int mat = col0 / P.D, ncol = col0 % P.D;   // which matrix (QKV: q, k, v) and its first column
        for (int kc = 0; kc < kchunks && ok; ++kc, ++n) {
          const int slot = n % P_NSTAGE;
          if (n >= (unsigned)P_NSTAGE) ok = mbar_wait(&sh.empty[slot], ((n / P_NSTAGE) - 1) & 1, abort_flag);
          if (!ok) break;
          uint8_t* dst = smem + slot * P_STAGE;
          mbar_arrive_expect_tx(&sh.full[slot], P_STAGE);
          if (P.mode == 0) tma_load_3d(dst, &map_a, &sh.full[slot], kc * PK, m0, b);
          else tma_load_3d(dst, &map_a, &sh.full[slot], (kc % cpd) * PK, m0, b * P.heads + kc / cpd);
#pragma unroll
          for (int c = 0; c < 4; ++c) tma_load_3d(dst + A_BYTES + c * B_PIECE, &map_b, &sh.full[slot], ncol + c * 64, kc * PK, mat);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(PM, PN, /*a_mn_major=*/false, /*b_mn_major=*/true);
      unsigned n = 0, nt = 0;
      bool ok = true;
      for (long long t = blockIdx.x; t < tiles && ok; t += gridDim.x, ++nt) {
        const int ab = nt & 1;
        if (nt >= 2) ok = mbar_wait(&sh.acc_empty[ab], ((nt >> 1) - 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        for (int kc = 0; kc < kchunks && ok; ++kc, ++n) {
          const int slot = n % P_NSTAGE;
          ok = mbar_wait(&sh.full[slot], (n / P_NSTAGE) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t abase = smem_u32(smem + slot * P_STAGE), bbase = abase + A_BYTES;
#pragma unroll
          for (int ks = 0; ks < PK / 16; ++ks)
            umma_ss(tm + ab * PN, smem_desc_sw128(abase + ks * 32, 16, 1024), smem_desc_sw128(bbase + ks * 2048, B_PIECE, 1024),
                    idesc, (kc > 0 || ks > 0) ? 1u : 0u);
          umma_commit(&sh.empty[slot]);
        }
        umma_commit(&sh.acc_full[ab]);
      }
    }
  } else {
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    unsigned nt = 0;
    bool ok = true;
    for (long long t = blockIdx.x; t < tiles && ok; t += gridDim.x, ++nt) {
      const int ab = nt & 1;
      const int ntile = (int)(t % n_tiles);
      const long long mt = t / n_tiles;
      const int b = (int)(mt / m_tiles);
      const long long m = (mt % m_tiles) * PM + row;          // token of this thread
      const int col0 = ntile * PN;
      ok = __all_sync(0xffffffffu, mbar_wait(&sh.acc_full[ab], (nt >> 1) & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
#pragma unroll 1
      for (int q = 0; q < PN / 32; ++q) {
        uint32_t r[32];
        tmem_ld32(tm + lane_addr + ab * PN + q * 32, r);
        tmem_wait_ld();
        const int col = col0 + q * 32;
        __nv_bfloat16* dst;
        if (P.mode == 0) {
          const int mat = col / P.D, c = col % P.D;
          dst = P.dst[mat] + (((size_t)b * P.heads + c / P.d) * P.N + m) * P.d + c % P.d;
        } else {
          dst = P.dst[0] + ((size_t)b * P.N + m) * P.D + col;
        }
#pragma unroll
        for (int v4 = 0; v4 < 4; ++v4) {
          uint32_t w[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(r[v4 * 8 + 2 * i]), __uint_as_float(r[v4 * 8 + 2 * i + 1]));
            w[i] = *(const uint32_t*)&v;
          }
          *(uint4*)(dst + v4 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
      tc_fence_before();
      mbar_arrive(&sh.acc_empty[ab]);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (sh.abort_flag) {
    if (threadIdx.x == 0) atomicExch(P.status, FF_ERR_TIMEOUT | 0x600);   // low byte: status, next byte: which kernel
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000) { }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tm, 512);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 3-D map over [slices][rows][cols] bf16 with a box of `box_rows` rows x 64 columns, 128-byte swizzle.
bool encode_map(CUtensorMap* map, const void* base, long long cols, long long rows, long long slices, int box_rows) {
  static EncodeTiledFn enc = nullptr;
  if (!enc) {
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", (void**)&enc, cudaEnableDefault, &qr) != cudaSuccess || !enc)
      return false;
  }
  cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)slices};
  cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)rows * cols * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t es[3] = {1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaError_t launch_proj(ff_plan* p, const CUtensorMap& ma, const CUtensorMap& mb, const ProjParams& P, cudaStream_t st) {
  const size_t smem = (size_t)P_NSTAGE * P_STAGE + sizeof(ProjShared) + 1024;
  cudaError_t e = cudaFuncSetAttribute(proj_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const long long tiles = (long long)P.B * (P.N / PM) * (P.n_out / PN);
  const int grid = tiles < p->sm_count ? (int)tiles : p->sm_count;
  proj_tc_kernel<<<grid, P_THREADS, smem, st>>>(ma, mb, P);
  p->launches += 1;
  return cudaGetLastError();
}

}  // namespace

// bf16 storage, head_dim 64 or 128, token count a multiple of 128, model width a multiple of 256.
bool ffk_proj_supported(const FFDims& dm) {
  return !dm.fp32 && (dm.d == 64 || dm.d == 128) && dm.N % PM == 0 && ((long long)dm.heads * dm.d) % PN == 0;
}

// Q, K, V [B][heads][N][d] = X [B][N][D] (W_q | W_k | W_v), Wqkv [3][D][D].
cudaError_t ffk_project_qkv(ff_plan* p, const void* X, const void* Wqkv, void* Q, void* K, void* V, cudaStream_t st) {
  const FFDims& dm = p->dm;
  const int D = dm.heads * dm.d;
  CUtensorMap ma, mb;
  if (!encode_map(&ma, X, D, dm.N, dm.B, PM) || !encode_map(&mb, Wqkv, D, D, 3, PK)) return cudaErrorInvalidValue;
  ProjParams P{};
  P.mode = 0; P.B = dm.B; P.heads = dm.heads; P.d = dm.d; P.N = dm.N; P.D = D; P.n_out = 3 * D;
  P.dst[0] = (__nv_bfloat16*)Q; P.dst[1] = (__nv_bfloat16*)K; P.dst[2] = (__nv_bfloat16*)V; P.status = p->buf.status;
  return launch_proj(p, ma, mb, P, st);
}

// out [B][N][D] = concat_h(O_h) W_o, O [B][heads][N][d], Wo [D][D].
cudaError_t ffk_project_out(ff_plan* p, const void* O, const void* Wo, void* out, cudaStream_t st) {
  const FFDims& dm = p->dm;
  const int D = dm.heads * dm.d;
  CUtensorMap ma, mb;
  if (!encode_map(&ma, O, dm.d, dm.N, dm.BH, PM) || !encode_map(&mb, Wo, D, D, 1, PK)) return cudaErrorInvalidValue;
  ProjParams P{};
  P.mode = 1; P.B = dm.B; P.heads = dm.heads; P.d = dm.d; P.N = dm.N; P.D = D; P.n_out = D;
  P.dst[0] = (__nv_bfloat16*)out; P.status = p->buf.status;
  return launch_proj(p, ma, mb, P, st);
}
