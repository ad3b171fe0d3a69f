// Shared host/device helpers of the astraea library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "../../include/astraea.h"

namespace astraea {

constexpr int kMaxSMs = 256;            // upper bound for per-SM host tables (a full B200 has 2 dies x 74 = 148)
constexpr int kMaxDevices = 64;         // per-device host state is kept for device ordinals below this
constexpr int kErrTimeout = 1;          // values of the device-side error word
constexpr int kErrBadIndex = 2;

// SMs of the current device (cudaDevAttrMultiProcessorCount, read once per device; a part with SMs fused off
// reports fewer than 148 and every grid is sized from this).  148 if the query fails.
int sm_count();

// Runs `f` once per device (the current one) and remembers the devices on which it returned cudaSuccess:
// cudaFuncSetAttribute and the like apply to the current device only.  Thread-safe.
class PerDeviceOnce {
public:
    template <class F> cudaError_t run(F &&f) {
        int dev = -1;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= kMaxDevices) return f();            // no slot: just do it every time
        if (__atomic_load_n(&done_[dev], __ATOMIC_ACQUIRE)) return cudaSuccess;
        e = f();                                                   // idempotent: two racing threads may both run it
        if (e == cudaSuccess) __atomic_store_n(&done_[dev], 1, __ATOMIC_RELEASE);
        return e;
    }
private:
    int done_[kMaxDevices] = {};
};

// cuTensorMapEncodeTiled from the driver (looked up once, thread-safe); nullptr if the driver does not have it
void *tensor_map_encoder();

// thread-local text of the last failure
void set_error(const char *fmt, ...);
int32_t fail(int32_t code, const char *fmt, ...);
int32_t check_launch(const char *what);

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// kernel launchers (one per .cu file)
int32_t launch_score(const void *x_cur, const void *x_ref, const float *lse, const int32_t *n_skip,
                     float *score, int B, int N, int N_sel, int D, int H, float w_alpha, float w_beta,
                     int delta_mode, int lse_mode, cudaStream_t stream, float *part = nullptr);
int32_t launch_score_combine(const float *part, const int32_t *n_skip, float *score, int B, int N_sel, int D, int H,
                             int has_lse, float w_alpha, float w_beta, cudaStream_t stream);
int32_t launch_select(const float *score, int B, int N_sel, int k, int n_always, int32_t *idx_sel,
                      int32_t *idx_rem, int32_t *n_skip, void *workspace, cudaStream_t stream);
size_t select_workspace_bytes(int B, int N_sel);
int32_t launch_scatter(void *cache, const void *rows, const int32_t *idx, int B, int N, int M,
                       int row_elems, uint32_t flags, int *err_word, cudaStream_t stream, int pitch_elems = 0);   // pitch 0: rows are dense

size_t linear_workspace_bytes();
int32_t launch_gathered_linear(const void *x, const int32_t *idx, int M, const void *w, const void *bias, void *y,
                               int B, int N, int K, int N_out, uint32_t flags, int *err_word, cudaStream_t stream,
                               const void *residual = nullptr, const void *gate = nullptr);
int32_t launch_layernorm_modulate(const void *x, const int32_t *idx, int M, const void *scale, const void *shift, void *y,
                                  int B, int N, int D, float eps, uint32_t flags, int *err_word, cudaStream_t stream);

struct AttnArgs {
    const void *q, *k, *v;
    int64_t q_sb, q_sh, q_sn, k_sb, k_sh, k_sn, v_sb, v_sh, v_sn;
    const int32_t *q_idx;
    int M;
    void *out;
    float *lse_out;
    int B, H, N, d;          // N: keys
    int N_tok;               // tokens of q / out / lse_out
    float scale;
    uint32_t flags;
    int *err_word;
    int head_begin = 0, head_count = 0;   // a sub-range of the H heads (head_count 0: all); strides and H stay those of the full tensors
    // room for the key shares of a split last round of CTAs (256-byte aligned; NULL: the launch is never split).  Two
    // launches that may run at the same time must not share it.
    void *split_ws = nullptr;
    size_t split_ws_bytes = 0;
};
int32_t launch_sparse_attn(const AttnArgs &a, cudaStream_t stream);
// the schedule launch_sparse_attn would pick (host logic only; uses B, H / head_count, N, M, d, flags, split_ws, split_ws_bytes)
void attn_plan(const AttnArgs &a, int *small_ctas, int *split_units, int *split);
size_t attn_workspace_bytes(int B, int H, int N, int M, int d);
int32_t launch_wait_selftest(int *err_word, uint64_t limit_ns, int *gave_up, cudaStream_t stream);
int32_t noalloc_scratch_address(void **scratch_out);   // device address of the library's built-in scratch array on the current device
size_t attn_kv_workspace_bytes(int B, int H, int M_kv, int d);
int32_t launch_sparse_attn_kv(AttnArgs a, const int32_t *kv_idx, int M_kv, void *workspace, cudaStream_t stream);   // gathers the listed K/V rows into the workspace first

}  // namespace astraea
