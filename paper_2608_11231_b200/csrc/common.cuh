// Shared device/host helpers of the lkv CUDA library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/lkv.h"

namespace lkv {

// First 256 bytes of every workspace: word 0 is the device status (0 = fine).
constexpr size_t kWsHeaderBytes = 256;
// Status values written by kernels whose bounded waits ran out.
constexpr int kDevTimeout = 1;

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

template <typename T>
__device__ __forceinline__ float to_f32(T x);
template <>
__device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__device__ __forceinline__ T from_f32(float x);
template <>
__device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Final-state store of the scans: element idx of S_T as fp32, or rounded to bf16 when the caller asked for that.
__device__ __forceinline__ void store_state(float *S_T, int st_bf16, size_t idx, float v) {
    if (st_bf16) reinterpret_cast<__nv_bfloat16 *>(S_T)[idx] = __float2bfloat16_rn(v);
    else S_T[idx] = v;
}

// Small host-checked index arrays travel to the device inside the kernel parameters
// (no copy, no extra stream operation); lists longer than CAP are copied into the
// caller's workspace instead and reached through `ptr`.
template <int CAP>
struct IndexBlock {
    const int32_t *ptr;  // device copy, or nullptr when the inline array is used
    int32_t v[CAP];
    __device__ __forceinline__ int32_t operator[](int i) const { return ptr ? ptr[i] : v[i]; }
};
constexpr int kInitIdxCap = 4000;  // ints: cu_k | sel | ids
constexpr int kScanIdxCap = 1000;  // ints: cu_seqlens[n_seq + 1] | launch order[n_seq]

// Launch-side records shared by the entry points and the kernels.  Passed by value as
// __grid_constant__ kernel parameters.
struct InitArgs {
    const void *states;        // pool
    const float *transitions;  // pool (log-decay or dense)
    float *S0;                 // [n_req, H, d_k, d_v]
    int32_t n_req, H, d_k, d_v, n_chunks;
    int32_t off_sel;           // offset of sel[n_req] in idx, or -1 (= last block)
    int32_t off_ids;           // offset of ids[total_K] in idx; cu_k[n_req + 1] sits at 0
    int32_t *status;           // device status word
    IndexBlock<kInitIdxCap> idx;
    __device__ __forceinline__ int cu_k(int r) const { return idx[r]; }
    __device__ __forceinline__ int id(int i) const { return idx[off_ids + i]; }
    __device__ __forceinline__ int sel(int r, int K) const { return off_sel < 0 ? K - 1 : idx[off_sel + r]; }
};

struct GdnArgs {
    const void *q, *k, *v;
    const float *g, *beta, *S0;
    void *o;
    float *S_T;                  // final states, fp32 or (st_bf16) bf16 behind the same pointer
    const float *S_add;          // added to every final state before it is stored (Eq. 5: S_out = T_C S_in + S_local), or nullptr
    int32_t st_bf16;
    int32_t n_seq, T_total, H_k, H_v, d_k, d_v;
    float scale;
    int32_t s0_identity;         // start every sequence from S = I (d_k == d_v) instead of S0; with v == nullptr (read
                                 // as zeros) the final state is then the sequence's accumulated transition; o may be nullptr
    // Sequences tr_first .. n_seq-1 are "transition sequences": they run in that mode (S = I, v = 0, no outputs) whatever
    // the call's own mode is, over the token range of sequence (seq - tr_first + tr_src0).  cu has n_ranges + 1 entries
    // (the ranges of sequences 0 .. tr_first-1); a plain call has n_ranges = tr_first = n_seq.
    int32_t n_ranges, tr_first, tr_src0;
    float *tr_out;               // where transition sequence tr_first + i stores its final state (index i), or nullptr: S_T like the others
    int32_t *status;
    IndexBlock<kScanIdxCap> cu;  // cu_seqlens[n_seq + 1], then the launch order: sequence of grid row y at [n_seq + 1 + y]
};

struct SsdArgs {
    const void *x, *B, *C;
    const float *dt, *A, *S0;
    void *y;
    float *S_T;                  // final states, fp32 or (st_bf16) bf16 behind the same pointer
    int32_t st_bf16;
    int32_t n_seq, T_total, H, P, N, G;
    int32_t *status;
    IndexBlock<kScanIdxCap> cu;  // cu_seqlens[n_seq + 1]
};

// Kernel launchers (one translation unit each); all return a cudaError_t from the launch.
cudaError_t launch_init_single(const InitArgs &a, bool pool_bf16, cudaStream_t s);
cudaError_t launch_init_mamba_exact(const InitArgs &a, bool pool_bf16, cudaStream_t s);
// persistent streaming variant (head size a multiple of 16 KB of pool values); same results bit for bit
bool init_mamba_stream_supported(const InitArgs &a, bool pool_bf16);
cudaError_t launch_init_mamba_exact_stream(const InitArgs &a, bool pool_bf16, cudaStream_t s);
cudaError_t launch_init_gdn_exact_fp32(const InitArgs &a, bool pool_bf16, cudaStream_t s);
bool init_gdn_exact_tensor_supported(const InitArgs &a, bool pool_bf16);
cudaError_t launch_init_gdn_exact_tensor(const InitArgs &a, bool pool_bf16, cudaStream_t s);

bool gdn_scan_fp32_supported(int d_k, int d_v);
cudaError_t launch_gdn_scan_fp32(const GdnArgs &a, bool io_bf16, cudaStream_t s);
bool gdn_scan_tensor_supported(const GdnArgs &a, bool io_bf16);
cudaError_t launch_gdn_scan_tensor(const GdnArgs &a, cudaStream_t s);

bool ssd_scan_fp32_supported(int N, int P);
cudaError_t launch_ssd_scan_fp32(const SsdArgs &a, bool io_bf16, cudaStream_t s);
bool ssd_scan_tensor_supported(const SsdArgs &a, bool io_bf16);
cudaError_t launch_ssd_scan_tensor(const SsdArgs &a, cudaStream_t s);
// lambda[c][h] = A[h] * sum of dt over sequence c (cu in the parameter block of `a`; only dt, A, H, n_seq, cu are read)
cudaError_t launch_mamba_logdecay(const SsdArgs &a, float *logdecay, cudaStream_t s);
// rel_err[i] = ||x_i - r_i|| / ||r_i|| over n_states runs of `elems` floats; parts = CTAs per state, partial sums
// (2 floats per CTA) in `partials`
int state_err_parts(size_t elems);
cudaError_t launch_state_rel_error(const float *x, const float *r, float *rel_err, int n_states, size_t elems,
                                   float *partials, cudaStream_t s);

// one CTA waits on an mbarrier nobody arrives on, with the kernels' own bounded wait and a small poll limit
cudaError_t launch_selftest_bounded_wait(uint32_t poll_limit, int32_t *status, cudaStream_t s);

}  // namespace lkv
