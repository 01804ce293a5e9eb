// Shared host/device helpers of the pd library (sm_100a only).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "pd.h"

namespace pd {

// First bytes of every workspace: words the device latches errors into.
//   word 0: status (0 = ok, else a pd_status value), word 1: detail (bad id, or stage that timed out)
constexpr size_t kStatusBytes = 256;

extern std::atomic<int64_t> g_launches;

inline void count_launch(int n = 1) { g_launches.fetch_add(n, std::memory_order_relaxed); }

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned256(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline pd_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? PD_OK : PD_ERR_CUDA; }

// Per-device host state: a process may drive several GPUs from several threads.
constexpr int kMaxDevices = 64;

inline int current_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
    return dev;
}

// SM count of the current device.
inline int sm_count() {
    static std::atomic<int> cached[kMaxDevices];
    const int dev = current_device();
    int n = cached[dev].load(std::memory_order_relaxed);
    if (n > 0) return n;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev].store(n, std::memory_order_relaxed);
    return n;
}

// Opts a kernel into `bytes` of dynamic shared memory on the current device, once per device.  The attribute
// is per device; `done` is the caller's array of kMaxDevices flags for this kernel (one per instantiation).
template <typename Kernel>
inline bool ensure_dynamic_smem(Kernel kernel, int bytes, std::atomic<bool> *done) {
    const int dev = current_device();
    if (done[dev].load(std::memory_order_acquire)) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    done[dev].store(true, std::memory_order_release);  // setting it twice from two threads is harmless
    return true;
}

__device__ __forceinline__ void latch_error(uint32_t *status, uint32_t code, uint32_t detail) {
    if (atomicCAS(status, 0u, code) == 0u) status[1] = detail;
}

// --- launchers implemented in the .cu files (all enqueue on `stream`, none synchronises) ---
// Weights and activations are 16-bit values passed as __half pointers; `bf16` says that the bits are bfloat16
// (the scale vectors are binary16 either way).
size_t pack_scratch_bytes(int64_t d_out, int64_t d_in);  // the sums; zero on entry, zero again on return
pd_status launch_pack(const __half *w_f, const __half *w_b, int64_t d_out, int64_t d_in, uint32_t *mask,
                      __half *v_row, __half *v_col, unsigned long long *sums, bool bf16, cudaStream_t stream);
pd_status launch_merge(const __half *w_b, const uint32_t *mask, const __half *v, int axis, int64_t d_out,
                       int64_t d_in, __half *w_hat, bool bf16, cudaStream_t stream);

// What the decode kernels need from the caller's workspace.
struct GemvScratch {
    uint32_t *status;        // device status words
    bool weights_resident;   // PD_LINEAR_WEIGHTS_RESIDENT: the weight stream may start before the previous kernel has finished
    bool bf16;               // x, W_b and y are bfloat16
};

// M <= 16 tokens (mask == nullptr: base weights only).  With group_offsets != nullptr the tokens are
// rows row_index[group_offsets[group] .. group_offsets[group+1]) of x / y (any count, read on the device).
// scratch carries the status words and the call's switches.
pd_status launch_gemv(const __half *x, int M, int64_t ldx, const __half *w_b, const uint32_t *mask,
                      const __half *v, int axis, int64_t d_out, int64_t d_in, __half *y, int64_t ldy,
                      const int *row_index, const int *group_offsets, int group, const GemvScratch *scratch,
                      cudaStream_t stream);

// M > 16 tokens on the tcgen05 tensor cores (needs d_in % 8 == 0; tails in M, d_out and d_in are handled).
// With few tokens the k loop is dealt to several tiles (split-K): `partial` then holds gemm_partial_bytes() of fp32
// partial sums (0 bytes when the call does not split; nullptr is fine then).
size_t gemm_partial_bytes(int64_t M, int64_t d_out, int64_t d_in);
int pair_split_steps(int64_t d_in, int splits);
pd_status launch_gemm(const __half *x, int64_t M, int64_t ldx, const __half *w_b, const uint32_t *mask,
                      const __half *v, int axis, int64_t d_out, int64_t d_in, __half *y, int64_t ldy,
                      float *partial, uint32_t *status, bool bf16, cudaStream_t stream);

// Multi-variant prefill: x_sorted holds the token rows in bucket order (contiguous, pitch d_in); token tile
// i of tile_table is {variant (V = base only), first sorted row, rows (<= token_tile), 0}; token_tile is 64, 128
// or 256 (grouped_token_tile picks it from the average bucket size).
constexpr int kGroupedMinTokenTile = 64;
inline int grouped_token_tile(int64_t M, int V) {
    const int64_t avg = M / (V > 0 ? V : 1);
    return avg <= 48 ? 64 : (avg <= 100 ? 128 : 256);
}
// Layers with at least 256 output rows run on CTA pairs (256-row tiles); smaller ones on one CTA per 128-row tile.
bool gemm_pair_enabled();
// Token tile the multi-variant path cuts buckets into: 256 when the pair kernel takes them.
inline int grouped_token_tile_for(int64_t M, int V, int64_t d_out) {
    return (gemm_pair_enabled() && d_out >= 256) ? 256 : grouped_token_tile(M, V);
}
pd_status launch_gemm_grouped(const __half *x_sorted, int64_t M, const __half *w_b, const uint32_t *masks,
                              int64_t mask_stride, const __half *vs, int64_t v_stride, unsigned long long col_axis_bits,
                              int V, int64_t d_out, int64_t d_in, __half *y, int64_t ldy, const int4 *tile_table,
                              const int *n_token_tiles, int max_token_tiles, int token_tile, const int *row_index,
                              uint32_t *status, bool bf16, cudaStream_t stream);

// Multi-variant decode: at most kMvDecodeMaxTokens token rows, d_in a multiple of 128.  One launch, one pass over
// W_b; the kernel buckets the rows by variant id itself (ids outside [-1, V) latch PD_ERR_BAD_VARIANT).
constexpr int kMvDecodeMaxTokens = 64;
size_t mv_decode_scratch_bytes(int64_t M, int32_t V, int64_t d_in);  // x and col-axis scales in the kernel's own layout
pd_status launch_mv_decode(const __half *x, int M, int64_t ldx, const int32_t *ids, const __half *w_b, const uint32_t *masks,
                           int64_t mask_stride, const __half *vs, int64_t v_stride, unsigned long long col_axis_bits, int V,
                           int64_t d_out, int64_t d_in, __half *y, int64_t ldy, unsigned char *scratch, uint32_t *status,
                           bool bf16, cudaStream_t stream);

// Stable bucket sort of token rows by variant id: offsets[g] .. offsets[g+1] index row_index for
// variant g (g = 0..V-1), offsets[V] .. offsets[V+1] the rows with id -1.  Other ids latch an error.
// With tile_table != nullptr it also cuts every bucket into token tiles of at most token_tile rows
// (tile_table, *n_token_tiles), and with x_sorted != nullptr a second kernel gathers the rows of x.
pd_status launch_group_rows(const int32_t *ids, int M, int V, int *offsets, int *row_index, uint32_t *status,
                            int4 *tile_table, int *n_token_tiles, int token_tile, const __half *x, int64_t ldx,
                            int64_t d_in, __half *x_sorted, cudaStream_t stream);


// Scale fitting (pd_fit.cu).  v, gradients and optimiser state are fp32; axis may also be PD_AXIS_SCALAR.
size_t fit_scratch_bytes(int64_t M, int64_t d_out, int64_t d_in);
size_t fit_layer_scratch_bytes(int64_t m_batch, int64_t m_val, int64_t d_out, int64_t d_in);
pd_status launch_transpose_mask(const uint32_t *mask, int64_t d_out, int64_t d_in, uint32_t *mask_t, cudaStream_t stream);
pd_status launch_fit_loss_grad(const __half *x, const __half *y, int64_t M, const __half *w_b, const uint32_t *mask,
                               const uint32_t *mask_t, const float *v, int axis, int64_t d_out, int64_t d_in, float *loss,
                               float *grad, unsigned char *scratch, uint32_t *status, cudaStream_t stream);
pd_status launch_fit_adamw(float *v, float *m1, float *m2, const float *g, int64_t len, int64_t t, float lr, float b1, float b2,
                           float eps, float wd, __half *v16, cudaStream_t stream);
pd_status launch_fit_layer(const __half *x_tr, const __half *y_tr, int64_t m_tr, const __half *x_val, const __half *y_val,
                           int64_t m_val, const __half *w_b, const uint32_t *mask, const __half *v_row0, const __half *v_col0,
                           int64_t d_out, int64_t d_in, int epochs, int64_t batch, const pd_adamw &opt, int cosine, __half *v_out,
                           int32_t *axis_out, float *val_loss, unsigned char *scratch, uint32_t *status, cudaStream_t stream);

}  // namespace pd
