// Host-side launchers of the stage kernels.  Every launcher only enqueues work on `st`.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <atomic>

#include "common.cuh"

namespace ast {

struct ConvGeom {
    int n, hi, wi, ci, ho, wo, co, k, stride, pad;
};

// Kernel kinds, for launch counting and the optional per-launch event trace.
enum KernelKind {
    K_CONV_FWD = 0, K_CONV_BWD_DATA, K_CONV_BWD_WEIGHT, K_REDUCE_SPLITS, K_DW_FWD, K_DW_BWD_DATA, K_DW_BWD_WEIGHT,
    K_DW_BWD_WEIGHT_FINISH, K_BN_STATS, K_BN_STATS_FINISH, K_BN_BWD_REDUCE, K_BN_BWD_FINISH, K_EW_ADD, K_EW_MASK, K_EW_SUM,
    K_GAP_FWD, K_GAP_BWD, K_ACCUMULATE, K_SGD_STEP, K_REFRESH, K_LOSS_MSE, K_LOSS_XENT, K_PW_FWD_TC, K_PW_BWD_DATA_TC, K_PW_BWD_WEIGHT_TC, K_CONV3_FWD_TC, K_CONV3_BWD_DATA_TC, K_CONV3_BWD_WEIGHT_TC, K_DW_BWD_FUSED, K_IM2COL, K_COL_AUX, K_SILU, K_SE, K_KINDS
};
const char* kernel_name(int kind);

// Launches `kernel` on `st` with programmatic stream serialization allowed (the kernel must open
// with pdl_wait()).
template <typename... KArgs, typename... Args>
inline void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Raises a kernel's dynamic shared-memory limit once per device (the attribute is per device; TAG makes the bookkeeping
// unique per call site).
template <int TAG, typename K> inline void smem_limit_once(K* kernel, int bytes) {
    static std::atomic<unsigned long long> done{0};
    int dev = 0;
    cudaGetDevice(&dev);
    const unsigned long long bit = 1ull << (dev & 63);
    if (!(done.load(std::memory_order_acquire) & bit)) {
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        done.fetch_or(bit, std::memory_order_release);
    }
}

// Brackets one kernel launch: counts it and, while a trace is active, records a CUDA event on
// `st` before and after it together with the bytes the kernel must move (each tensor once)
// and its floating-point operations.
struct LaunchScope {
    LaunchScope(int kind, double alg_bytes, double flops, cudaStream_t st);
    ~LaunchScope();
    int slot;
    cudaStream_t st;
};
uint64_t launches();
// number of multiprocessors of the calling thread's current device (queried once per device)
int sm_count();
// true while a per-launch event trace is being recorded
bool tracing();
// records `msg` as the calling thread's last error and returns `code`
int report_error(int code, const char* msg);

// BatchNorm-backward reduction fused into the kernel that writes the gradient dy of a conv->BN->activation unit's
// output: z is that unit's raw conv output, scale/shift/mean/rstd its forward statistics, act its activation.
struct BnRed {
    const void* z;
    const float *scale, *shift, *mean, *rstd;
    int act;
    float* partial;          // [blocks][2][c]
    size_t partial_floats;
};

// ---- dense convolution as implicit GEMM (plain FFMA tiles; float and bfloat16 storage) ----
// z[n,ho,wo,ko] = sum_{r,s,c} x[n,ho*st-pad+r,wo*st-pad+s,c] * w[ko][r][s][c]  (+ bias[ko])
void conv_fwd(int dtype, const ConvGeom& g, const ValSrc& x, const float* w, const float* bias, void* z, cudaStream_t st);
// dx[n,hi,wi,c] = sum_{r,s,ko} dz[n,(hi+pad-r)/st,(wi+pad-s)/st,ko] * wt[c][r][s][ko]  (+ addend)
void conv_bwd_data(int dtype, const ConvGeom& g, const GradSrc& dz, const float* wt, const void* addend, void* dx, cudaStream_t st);
// gw[ko][r][s][c] = sum_{n,ho,wo} dz[n,ho,wo,ko] * x[n,ho*st-pad+r,wo*st-pad+s,c]; split over pixels, partials in scratch
void conv_bwd_weight(int dtype, const ConvGeom& g, const GradSrc& dz, const ValSrc& x, float* scratch, size_t scratch_floats,
                     float* gw, cudaStream_t st);

// ---- dense conv with a short reduction (k*k*c_in <= 64, e.g. the 3-channel stem) in bfloat16 mode: explicit im2col,
// then the pointwise tensor-core kernels over col[pixels][Kp] with weights padded to [co][Kp] ----
void conv_im2col(const ConvGeom& g, const ValSrc& x, int Kp, void* col, cudaStream_t st);
void conv_pad_weights(const float* w, int co, int K, int Kp, __nv_bfloat16* wpad, cudaStream_t st);
void conv_unpad_grad(const float* gpad, int co, int K, int Kp, float* gw, cudaStream_t st);

// ---- pointwise conv on tcgen05 tensor cores (bf16 storage, channel counts multiples of 8) ----
bool pw_tc_supported(int dtype, const ConvGeom& g, bool bwd_data);
// wb: bf16 weights [co][ci]; wtb: bf16 transposed weights [ci][co]; err: device error word
// With `pivot` and `partial` given, the pipelined kernel also writes the BatchNorm statistics partials of its output,
// partial[cta][2][co] = sums of (z - pivot[c]) and (z - pivot[c])^2 over the CTA's pixels (z as stored, after rounding),
// and returns the number of CTAs (for bn_stats_finish_partials); 0 = no partials written, statistics need their own pass.
int pw_fwd_tc(const ConvGeom& g, const ValSrc& x, const __nv_bfloat16* wb, const float* bias, void* z, const float* pivot, float* partial,
              size_t partial_floats, int* err, cudaStream_t st);
// With `red` given, the pipelined kernel also writes the BatchNorm-backward partial sums of the gradient it produces,
// partial[cta][2][ci] = sums over the CTA's pixels of dpre = dx * [pre inside the activation's linear region] and of
// dpre * xhat (dx as stored, after rounding and after the addend), where pre / xhat come from red->z, the raw output
// of the unit that produced this conv's input.  Returns the number of CTAs (for bn_bwd_finish_partials); 0 = none written.
int pw_bwd_data_tc(const ConvGeom& g, const GradSrc& dz, const __nv_bfloat16* wtb, const void* addend, void* dx, const BnRed* red, int* err,
                   cudaStream_t st);
// streaming form (pw_stream.cu) for stride-1 layers with more than 256 channels on a side (channel counts multiples of 64): forward
// (bwd == false: x [P][K], w = [N][K]) or backward-data (bwd == true: dz [P][K], w = transposed weights [N][K]); false = does not fit
bool pw_stream(bool bwd, int P, int K, int N, const ValSrc& x, const GradSrc& dz, const __nv_bfloat16* w, const void* addend, void* out, int* err,
               int kind, double bytes, cudaStream_t st);
// gw[co][ci]; per-CTA partial sums in scratch, summed in fixed order by a second kernel
void pw_bwd_weight_tc(const ConvGeom& g, const GradSrc& dz, const ValSrc& x, float* scratch, size_t scratch_floats, float* gw, int* err,
                      cudaStream_t st);

// ---- dense 3x3 conv (stride 1, pad 1, channels multiples of 64) on tcgen05 ----
bool conv3_tc_supported(int dtype, const ConvGeom& g);
// wb: bf16 weights [co][3][3][ci]; wtb: bf16 derived weights [ci][3][3][co].  useful_flops > 0 replaces the operation count the
// trace records (a stride-2 layer evaluated on its input grid executes four times the multiply-adds of its definition).
void conv3_fwd_tc(const ConvGeom& g, const ValSrc& x, const __nv_bfloat16* wb, void* z, int* err, cudaStream_t st, double useful_flops = 0);
void conv3_bwd_data_tc(const ConvGeom& g, const GradSrc& dz, const __nv_bfloat16* wtb, const void* addend, void* dx, int* err, cudaStream_t st,
                       double useful_flops = 0);
// out[i] = sum over k < splits of partial[k][i] in a fixed order; n a multiple of 4, both pointers 16-byte aligned (conv3_tc.cu)
void reduce_splits_f4(const float* partial, int splits, size_t n, float* out, cudaStream_t st);
// pipelined form (conv3_pipe.cu) for up to 128 reduction channels: forward (bwd == false: x, w = [c_out][9][c_in], C = c_in,
// N = c_out) or backward-data (bwd == true: dz, w = [c_in][9][c_out], C = c_out, N = c_in); false = layer does not fit, nothing launched
bool conv3_pipe(bool bwd, int n_img, int H, int W, int C, int N, const ValSrc& x, const GradSrc& dz, const __nv_bfloat16* w, const void* addend,
                void* out, int* err, int kind, double bytes, double flops, cudaStream_t st);
// pipelined weight gradient (conv3_wgrad_pipe.cu): writes per-CTA partials [ctas][c_out][9][c_in] and returns ctas, or 0 if the
// layer does not fit (nothing launched)
int conv3_wgrad_pipe(int n_img, int H, int W, int CI, int CO, const GradSrc& dz, const ValSrc& x, float* partial, size_t partial_floats, int* err,
                     double bytes, double flops, cudaStream_t st);
bool conv3_wgrad_tc_supported(int dtype, const ConvGeom& g);
void conv3_bwd_weight_tc(const ConvGeom& g, const GradSrc& dz, const ValSrc& x, float* scratch, size_t scratch_floats, float* gw, int* err,
                         cudaStream_t st, double useful_flops = 0);

// ---- depthwise 3x3 (weights tap-major: w9c[r*3+s][c]) ----
// With `pivot` and `partial` given, the stride-1 kernel also writes the BatchNorm statistics partials of its output
// (layout and meaning as for pw_fwd_tc) and returns the number of blocks that wrote them; 0 = none.
int dw_fwd(int dtype, const ConvGeom& g, const ValSrc& x, const float* w9c, void* z, const float* pivot, float* partial, size_t partial_floats,
           cudaStream_t st);
void dw_bwd_data(int dtype, const ConvGeom& g, const GradSrc& dz, const float* w9c, const void* addend, void* dx, cudaStream_t st);
// stride-1 bf16 layers with enough image columns: input gradient and weight gradient in one pass; false = not applicable
bool dw_bwd_fused(int dtype, const ConvGeom& g, const GradSrc& dz, const ValSrc& x, const float* w9c, const void* addend, void* dx,
                  float* scratch, size_t scratch_floats, float* gw, cudaStream_t st);
// gw[c][r][s]
void dw_bwd_weight(int dtype, const ConvGeom& g, const GradSrc& dz, const ValSrc& x, float* scratch, size_t scratch_floats,
                   float* gw, cudaStream_t st);

// ---- BatchNorm statistics and backward reductions over a [pixels][c] tensor ----
struct BnFwdOut {
    float *mean, *rstd, *scale, *shift, *run_mean, *run_var;
};
void bn_stats(int dtype, const void* z, size_t pixels, int c, const float* gamma, const float* beta, float eps, float momentum,
              float* scratch, size_t scratch_floats, const BnFwdOut& o, cudaStream_t st);
// finishing step alone, for statistics partials written by the producing kernel; the pivot is the running mean
// as it stood before this call (the value the producer read)
void bn_stats_finish_partials(const float* partial, int blocks, size_t pixels, int c, const float* gamma, const float* beta, float eps,
                              float momentum, const BnFwdOut& o, cudaStream_t st);
struct BnBwdOut {
    float *dgamma, *dbeta, *k1, *k2, *k3;   // dgamma/k* null: only dbeta = sum of dpre (bias gradient)
};
void bn_bwd_reduce(int dtype, const void* dy, const void* z, size_t pixels, int c, const float* scale, const float* shift, int act,
                   const float* mean, const float* rstd, const float* gamma, float* scratch, size_t scratch_floats,
                   const BnBwdOut& o, cudaStream_t st);

// finishing step alone, for partial sums written by the kernel that produced dy
void bn_bwd_finish_partials(const float* partial, int blocks, size_t pixels, int c, const float* mean, const float* rstd, const float* gamma,
                            const BnBwdOut& o, cudaStream_t st);

// ---- elementwise over [pixels][c] ----
void ew_add(int dtype, const ValSrc& a, const ValSrc& b, int act, size_t pixels, int c, void* out, void* out2, cudaStream_t st);
void ew_apply(int dtype, const ValSrc& a, size_t pixels, int c, void* out, cudaStream_t st);
void ew_relu_mask(int dtype, const void* d, const void* out_val, size_t n, void* dst, cudaStream_t st);
// the same, fused with the BatchNorm-backward sums (and finishing step) of the operand branch whose raw conv output is z and whose
// BatchNorm has no activation: dst's sums are that BatchNorm's; false = channel count not a whole number of vectors, nothing launched
bool ew_relu_mask_bn_sums(int dtype, const void* d, const void* out_val, const void* z, size_t pixels, int c, const float* mean, const float* rstd,
                          const float* gamma, void* dst, float* scratch, size_t scratch_floats, const BnBwdOut& o, cudaStream_t st);
void ew_sum(int dtype, const void* a, const void* b, size_t n, void* dst, cudaStream_t st);
// bfloat16, channel counts multiples of 8: zero-inserted gradient / subsampled output of a stride-2 3x3 conv (see conv3_s2_tc_supported)
void ew_upsample2_grad(const GradSrc& d, int n, int hi, int wi, int ho, int wo, int c, void* up, cudaStream_t st);
void ew_subsample2(const void* full, int n, int hi, int wi, int ho, int wo, int c, void* z, cudaStream_t st);
void gap_fwd(int dtype, const ValSrc& x, int n, int hw, int c, void* out, cudaStream_t st);
void gap_bwd(int dtype, const void* da, int n, int hw, int c, const void* addend, void* dx, cudaStream_t st);

// ---- EfficientNet MBConv pieces (mbconv.cu) ----
// SiLU as a materialising unit: out = silu(value(x)); dx = dy * silu'(value(x)) (+ addend)
void silu_fwd(int dtype, const ValSrc& x, size_t pixels, int c, void* out, void* out2, cudaStream_t st);
void silu_bwd(int dtype, const void* dy, const ValSrc& x, const void* addend, size_t pixels, int c, void* dx, cudaStream_t st);
// squeeze-excite over [n][hw][c] with k hidden units; s [n][c], p1 [n][k], gate [n][c] are float vectors kept for the backward pass;
// work: >= n*(2c+k) floats; scratch: partials of the pixel-split reductions (any size >= n*c floats; more allows more splits)
void se_forward(int dtype, const ValSrc& x, int n, int hw, int c, int k, const float* w1, const float* b1, const float* w2, const float* b2,
                float* s, float* p1, float* gate, float* scratch, size_t scratch_floats, void* out, void* out2, cudaStream_t st);
void se_backward(int dtype, const void* dout, const ValSrc& x, int n, int hw, int c, int k, const float* w1, const float* w2, const float* s,
                 const float* p1, const float* gate, float* work, float* scratch, size_t scratch_floats, const void* addend, void* dx, float* gw1, float* gb1,
                 float* gw2, float* gb2, cudaStream_t st);
// depthwise conv of odd kernel size k <= 7, pad (k-1)/2, stride 1 or 2; weights tap-major wkc[r*k+s][c]; gw[c][k][k]
void dwk_fwd(int dtype, const ConvGeom& g, const ValSrc& x, const float* wkc, void* z, cudaStream_t st);
void dwk_bwd_data(int dtype, const ConvGeom& g, const GradSrc& dz, const float* wkc, const void* addend, void* dx, cudaStream_t st);
void dwk_bwd_weight(int dtype, const ConvGeom& g, const GradSrc& dz, const ValSrc& x, float* scratch, size_t scratch_floats, float* gw, cudaStream_t st);

// ---- parameters ----
void accumulate(float* G, const float* g, size_t n, cudaStream_t st);
void sgd_step(float* w, float* v, float* G, size_t n, float inv_m, float lr, float mu, cudaStream_t st);
// derived[i] = w[perm[i]]; wb[i] = bf16(w[i]); wtb[i] = bf16(w[perm[i]])  (wb/wtb may be null)
void refresh_derived(const float* w, const int32_t* perm, float* derived, __nv_bfloat16* wb, __nv_bfloat16* wtb, size_t n, cudaStream_t st);

// ---- losses (scratch: >= 1024 floats + 1 counter word) ----
void loss_mse(int dtype, const void* y, const void* t, size_t n, void* dy, float* loss, float* scratch, cudaStream_t st);
void loss_xent(int dtype, const void* logits, const int32_t* labels, int rows, int classes, void* dlogits, float* loss,
               float* scratch, cudaStream_t st);

// one warp waits `limit` polls on an mbarrier nobody arrives at; sets *err = 1 when the wait gave up
void launch_bounded_wait_probe(int* err, unsigned limit, cudaStream_t st);

}  // namespace ast
