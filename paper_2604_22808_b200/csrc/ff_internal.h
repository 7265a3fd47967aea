// Internal declarations shared by the host API and the kernel translation units.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stddef.h>
#include <stdint.h>

#include "freqformer.h"

#if defined(__CUDACC__)
#define FF_HD __host__ __device__ __forceinline__
#else
#define FF_HD inline
#endif

// Debug build (-DFF_DEBUG): every computed band rank, row offset and tile coordinate is range-checked on
// the device before it is used; a value out of range is not used for the access (the store or copy is
// skipped) and FF_ERR_INVALID_ARG together with the kernel's id is raised in the plan's status word, where
// ff_plan_device_status reports it.  The release build compiles the checks away.
#if defined(FF_DEBUG) && defined(__CUDACC__)
#define FF_DBG_OK(cond, status_ptr, kernel_id) \
  ((cond) ? true : (atomicExch((status_ptr), FF_ERR_INVALID_ARG | ((kernel_id) << 8)), false))
#else
#define FF_DBG_OK(cond, status_ptr, kernel_id) (true)
#endif

// Problem sizes derived from ff_config_t ("Frequency band partitioning": N_low + N_mid + N_high = N).
struct FFDims {
  int B, T, H, W, heads, d, BH;
  int L[3], M[3];
  int r, b, s, R, m, hid, dt;
  int fp32;              // storage type of Q,K,V,out and of the mid/high band buffers
  int pattern;           // mid-band sparse pattern: FF_MID_STRIDED or FF_MID_ANCHOR
  long long N, Nlow, Nbar, Nmid, Nhigh;
  long long nb;          // number of mid blocks
};

// Number of members of the box A = [0,A_t) x [0,A_h) x [0,A_w) whose flat index is below that of k.
FF_HD long long ff_box_count_below(int At, int Ah, int Aw, int kt, int kh, int kw) {
  long long c = (long long)(kt < At ? kt : At) * Ah * Aw;
  if (kt < At) {
    c += (long long)(kh < Ah ? kh : Ah) * Aw;
    if (kh < Ah) c += (kw < Aw ? kw : Aw);
  }
  return c;
}

// Band (0 low, 1 mid, 2 high) and band-local rank of coefficient (kt,kh,kw): nested boxes, band
// order = increasing flat index.
FF_HD int ff_band_rank_of(const FFDims& dm, int kt, int kh, int kw, long long* rank) {
  const long long cl = ff_box_count_below(dm.L[0], dm.L[1], dm.L[2], kt, kh, kw);
  const long long cm = ff_box_count_below(dm.M[0], dm.M[1], dm.M[2], kt, kh, kw);
  const bool in_low = kt < dm.L[0] && kh < dm.L[1] && kw < dm.L[2];
  const bool in_mid = kt < dm.M[0] && kh < dm.M[1] && kw < dm.M[2];
  if (in_low) { *rank = cl; return 0; }
  if (in_mid) { *rank = cm - cl; return 1; }
  *rank = ((long long)kt * dm.H + kh) * dm.W + kw - cm;
  return 2;
}

// Device buffers inside the caller's workspace.
struct FFBuffers {
  float* spec_low;   // [3][BH][Nlow][d]
  void* spec_mid;    // st [3][BH][Nmid][d]
  void* spec_high;   // st [3][BH][Nhigh][d]
  float* pooled;     // [3][BH][Nbar][d]
  __nv_bfloat16* pooled_bf;  // the same values as bf16, operands of the tensor-core low branch (NULL if unused)
  float* y_low;      // [BH][Nbar][d]
  void* y_mid;       // st [BH][Nmid][d]
  void* y_high;      // st [BH][Nhigh][d]
  float* summary;    // [BH][3][m][d]
  double* energy;    // [B][3][d]
  uint8_t* alloc;    // [BH]
  float* pi;         // [B][3]
  float* timestep;   // [B]
  int* status;       // device status word
  int* work;         // worklist of the tensor-core attention kernel
  float* scratchA;   // [G][N][d]
  float* scratchB;   // [G][N][d]
  void* stage_q;     // host-call staging (st [BH][N][d]) or NULL
  void* stage_k;
  void* stage_v;
  void* stage_out;
};

struct FFLayout {
  size_t off[24];
  size_t total;
  int group;         // G: tensor-heads processed per generic transform launch
  int tc_group;      // tensor-heads per tensor-core transform launch
  int tc_group_pipe; // ... when the launches are pipelined with host copies (host-buffer entry point)
};

constexpr int FF_COPY_EVENTS = 64;

struct ff_plan {
  ff_config_t cfg;
  FFDims dm;
  int device;
  // device tables owned by the plan
  float* basis[3];    // C_T, C_H, C_W  [n][n], C[k][i]
  float* basis_t[3];  // transposes
  float* W1; float* b1; float* W2; float* b2; float* U;
  bool has_router;
  int identity_u;     // no summary projections were given: U_l = I
  // workspace
  void* ws; size_t ws_bytes;
  FFBuffers buf;
  FFLayout lay;
  bool ws_has_staging;
  int attn_impl;
  int sm_count;
  bool tc_ok;                                  // tensor-core attention usable with this plan + workspace
  bool dct_tc_ok;                              // tensor-core transform usable
  int dct_group;                               // tensor-heads per tensor-core transform launch
  bool xtc_ok;                                 // tensor-core exchange usable
  int* pos_table;                              // rank -> flat coefficient index of the mid, then the high band (plan-owned)
  alignas(64) unsigned char tmap_x[4][128];    // CUtensorMaps of the exchange kernel (Y / V~ of the mid and high bands)
  uint32_t* dct2_images;                       // 6 x (hi, lo) transform matrices as tensor-memory operand images (plan-owned)
  bool dct2_ok;                                // the fused two-axis launch covers this configuration
  int dct2_axis2;                              // its second axis (1 = h, 0 = t); the remaining axis gets a pass of its own
  int dct2_clusters;                           // clusters of that launch the device runs at once (0 = not yet asked)
  alignas(64) unsigned char tmap_mid[128];     // CUtensorMap over the mid-band / high-band coefficient buffers
  alignas(64) unsigned char tmap_high[128];
  alignas(64) unsigned char tmap_low[128];     // ... over the pooled low band (bf16 copy), when low_tc_ok
  bool low_tc_ok;                              // the low branch runs in the tensor-core attention launch
  long long launches;
  // ff_forward_host on the tensor-core path: copies run on a second stream, one event per launch
  // group of the forward transform (host -> device) and of the inverse transform (device -> host)
  cudaStream_t copy_stream;
  cudaEvent_t ev_copy[2 * FF_COPY_EVENTS + 1];   // [0,64) input groups, [64,128) output groups, [128] start
  bool pipe_in, pipe_out;                      // set for the duration of one ff_forward_host
  void* pipe_out_host;                         // host destination of `out`
  size_t pipe_head_bytes;                      // bytes of one (batch, head) slice of Q / K / V / out
  bool profiling;
  cudaEvent_t ev[FF_STAGE_COUNT + 1];
  long long stage_launches[FF_STAGE_COUNT];
  char err[512];
};

// Records `msg` as the calling thread's plan-less error (what ff_last_error(NULL) returns).
void ff_set_thread_error(const char* msg);

void ff_compute_layout(const FFDims& dm, bool with_staging, FFLayout* lay);

// ---- kernel launchers (ff_simt.cu).  Each returns the cudaError_t of its launches. --------------
cudaError_t ffk_forward_transform(ff_plan* p, const void* Q, const void* K, const void* V, cudaStream_t st);
cudaError_t ffk_band_energy(ff_plan* p, cudaStream_t st);
cudaError_t ffk_router(ff_plan* p, uint8_t* alloc_out, cudaStream_t st);
cudaError_t ffk_pool_low(ff_plan* p, cudaStream_t st);
cudaError_t ffk_attention_simt(ff_plan* p, int band_bits, cudaStream_t st);   // band_bits: which bands to run
// ---- tensor-core attention (ff_attn_tc.cu) -------------------------------------------------------
size_t ffk_tc_work_bytes();
bool ffk_tc_supported(const FFDims& dm);
bool ffk_tc_prepare(ff_plan* p);               // builds the tensor maps over the workspace
cudaError_t ffk_attention_tc(ff_plan* p, cudaStream_t st);
// ---- tensor-core exchange (ff_exchange_tc.cu) -----------------------------------------------------
bool ffk_exchange_tc_supported(const FFDims& dm);
bool ffk_exchange_tc_build_tables(ff_plan* p);
bool ffk_exchange_tc_prepare(ff_plan* p);
cudaError_t ffk_exchange_tc(ff_plan* p, int h0, int g, void* grid_hi, void* grid_lo, cudaStream_t st);
// ---- tensor-core transform (ff_dct_tc.cu) --------------------------------------------------------
bool ffk_dct_tc_supported(const FFDims& dm);
size_t ffk_dct_tc_scratch_bytes(const FFDims& dm, int group);
cudaError_t ffk_forward_transform_tc(ff_plan* p, const void* Q, const void* K, const void* V, bool want_energy,
                                     cudaStream_t st);
cudaError_t ffk_inverse_transform_tc(ff_plan* p, int h0, int g, void* out, cudaStream_t st);
// ---- two axis passes in one launch, intermediate in shared memory (ff_dct2_tc.cu) --------------------
bool ffk_dct2_supported(const FFDims& dm, int* axis2, int* cs);
bool ffk_dct2_build_image(ff_plan* p, int axis, int inverse, const float* mat_host, int n);
cudaError_t ffk_dct2_forward(ff_plan* p, const void* Q, const void* K, const void* V, int g0, int g, void* out_hi, void* out_lo,
                             cudaStream_t st);
cudaError_t ffk_dct2_inverse(ff_plan* p, const void* in_hi, const void* in_lo, int h0, int g, void* out, cudaStream_t st);
// ---- projections around the path (ff_proj_tc.cu) -------------------------------------------------------
bool ffk_proj_supported(const FFDims& dm);
cudaError_t ffk_project_qkv(ff_plan* p, const void* X, const void* Wqkv, void* Q, void* K, void* V, cudaStream_t st);
cudaError_t ffk_project_out(ff_plan* p, const void* O, const void* Wo, void* out, cudaStream_t st);
cudaError_t ffk_summaries(ff_plan* p, cudaStream_t st);
cudaError_t ffk_exchange_inverse(ff_plan* p, void* out, cudaStream_t st);
