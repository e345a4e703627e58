// Internal declarations shared by the translation units of libeoq (not part of the public ABI).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "eoq.h"

namespace eoq {

constexpr int kMaxTaps = 64;        // kh * kw of any supported filter
constexpr int kTileM = 128;         // GEMM rows per CTA tile (TMEM lanes)
constexpr int kEpilogueWarps = 16;  // implicit GEMM: four epilogue warps per scheduler hide the latency of the integer chain
constexpr int kGemmThreads = 128 + 32 * kEpilogueWarps;  // warps 0, 2, 3: TMA, warp 1: MMA + TMEM owner, then the epilogue
constexpr int kWgradThreads = 256;  // weight gradient: warps 0, 2, 3 TMA, warp 1 MMA, warps 4..7 epilogue
constexpr uint32_t kSpinLimit = 1u << 22;  // polls before a wait gives up (normal waits end within microseconds)

// Device state a handle owns.
struct DeviceState {
    unsigned status;       // EOQ_DEV_* bits
    unsigned absmax_u32;   // reduction cell for |.| maxima (int32 sources, float bit patterns)
    unsigned long long absmax_u64;
    long long sum0, sum1;  // reduction cells for integer sums
    unsigned long long absmax2_u64;  // second maximum of a call that also serves its consumer's error head (masked |.|)
    long long sum2;                  // third sum of such a call
    unsigned tensor_absmax[256];  // per-tensor maxima of the multi-tensor update
    unsigned ticket;       // blocks of the kernel that consumes the cells last count themselves here (see last_block_done)
    unsigned arrivals;     // grid-wide barrier of the one-kernel error head (cooperative launch)
    unsigned long long probe_cycles;  // eoq_probe_mma_i8: longest issue loop of the last launch, in SM clock cycles
};
// Invariant: absmax_u32, absmax_u64, absmax2_u64, sum0, sum1, sum2, ticket and arrivals are zero whenever no call is in flight on the handle.
// The kernel that reads a call's reductions last puts the cells it used back to zero (its last block does), so
// no call starts with a memset.  A kernel that gave up on a wait (EOQ_DEV_TIMEOUT) may leave them dirty:
// eoq_last_status clears them again when it reports that bit.

// eoq_set_reduce_hook: called on the host between the kernel that forms a value reduced over the batch and the kernel
// that consumes it; it enqueues an all-reduce of the device buffer on the stream (no-op when no hook is set).
// The error head of the layer that consumes an error tensor, fused into the second pass of the kernel that produces it
// (eoq_conv_dgrad_head, eoq_aux_join_head, eoq_aux_maxpool_bwd_head).
struct NextHeadArgs {
    const uint8_t *mask;      // that layer's ReLU mask bits
    const int16_t *x2;        // its x2, or null
    const int32_t *gamma;     // its gamma code (device)
    int8_t *e3;
    int32_t *e3_exp;
    long long *sum_e1, *sum_e1x2;
};

// The first pass of an error join (its two maxima) riding on the Q_e pass that writes the join's first operand
// (eoq_conv_dgrad_join_head): operand b with its exponent and gate bits, and the consumer's mask for the masked maximum.
struct JoinStatArgs {
    const int8_t *b;
    const int32_t *b_exp;
    const uint8_t *mask_b;     // gate bits of b, or null
    const uint8_t *next_mask;  // ReLU mask of the layer that consumes the joined error, or null
};

struct ReduceHook {
    eoq_reduce_fn fn;
    void *user;
    void operator()(void *ptr, size_t count, int dtype, int op, cudaStream_t s) const
    {
        if (fn) fn(user, ptr, count, dtype, op, reinterpret_cast<void *>(s));
    }
};

constexpr int kClassBranches = 3;

struct ProfRecord {
    int kind;
    cudaEvent_t begin, end;
};

struct Handle {
    int device;
    int sm_count;
    int last_cuda_error;
    DeviceState *dev;
    unsigned long long launches;  // kernels launched through this handle
    bool profiling;
    ReduceHook hook;              // all-reduce between the phases of every batch-wide reduction (data-parallel replicas)
    bool gemm_only;               // timing aid: dgrad and wgrad calls launch their GEMM kernel only (eoq_profile_gemm_only)
    bool force_timeout;           // self-test: the next error-head call makes its grid-wide wait run out
    int num_records;
    ProfRecord *records;          // kMaxProfRecords entries, allocated on first eoq_profile_start
    // Fork and join events of the calls that issue independent kernels on the class_branch streams (null branch
    // streams: everything stays on the caller's stream).  Under stream capture they become graph edges.
    int gemm_ctas;                // most CTAs a GEMM launch of this handle may use (eoq_set_gemm_ctas; default: one per SM)
    cudaEvent_t fork_ev, join_ev;
    // further branch streams: the per-class GEMMs of a strided error back-propagation write disjoint pixels and
    // run side by side, each with its share of the CTAs
    cudaStream_t class_branch[kClassBranches];
    cudaEvent_t class_join[kClassBranches];
};
constexpr int kMaxProfRecords = 8192;
int static_path_last_cuda_error();  // last cudaError_t of eoq_conv_dgrad_static (eoq_static.cu)

// Counts `n` kernel launches on the handle.
inline void count_launches(Handle *h, int n) { h->launches += (unsigned long long)n; }

// ---------------------------------------------------------------------------------------------
// Implicit-GEMM kernel used by the forward pass and by error back-propagation.
//   D[m, j] = sum over sub-tiles s of  A_s[m, 0..kc) . B_s[j, 0..kc)
// A_s is fetched by TMA in im2col mode from an NHWC int8 tensor (tap offset + channel chunk),
// B_s by a tiled TMA from a [rows][taps][channels] int8 tensor.
// ---------------------------------------------------------------------------------------------
enum EpilogueKind { kEpiForward = 0, kEpiDgrad = 1 };

struct IgemmParams {
    // GEMM extent
    int M;              // rows: n_img * hq * wq
    int N;              // columns (multiple of 16)
    int hq, wq;         // pixel grid per image walked by the rows
    int tile_n;         // columns per CTA tile (multiple of 16, <= 256)
    int num_m_tiles, num_n_tiles;
    // K structure
    int kc;             // channel bytes per sub-tile: 16, 32, 64 or 128 (= TMA swizzle span, 16 = none)
    int chunks_per_tap; // source channels / kc
    int num_sub;        // taps * chunks_per_tap (padded to even when kc == 16)
    int real_sub;       // sub-tiles that carry data
    int subs_per_stage;
    int num_stages;
    int src_stride;     // TMA traversal stride in source pixels (rows)
    int src_stride_w;   // same along a row (1 when the map's W axis already steps by the convolution stride)
    int base_h, base_w; // source coordinate of tap offset (0,0) for pixel (0,0)
    unsigned char tap_dh[kMaxTaps], tap_dw[kMaxTaps];  // im2col offsets of each tap
    unsigned char tap_b[kMaxTaps];                     // tap coordinate of each tap in the B tensor
    int ntaps;
    // output mapping: GEMM row (n, y, x) -> pixel (n, y*out_step + out_off_h, x*out_step + out_off_w)
    int out_h, out_w, out_step, out_off_h, out_off_w;
    int epilogue;       // EpilogueKind
    // forward epilogue
    const int32_t *x_exp;     // device exponent of the input or null
    int32_t b1_c, gamma_c, b2_c;
    const int32_t *scal_dev;  // device {b1_c, gamma_c, b2_c} replacing the three host values, or null
    const uint8_t *next_mask; // dgrad: ReLU mask bits of the layer that consumes the error (its head rides on Q_e), or null
    int k_total;              // taps * input channels: bounds the accumulator when b1 is only known on the device
    const int32_t *b1_table;  // [classes][N] tap-validity sums of the weights (null when b1_c == 0)
    int b1_nlo_h, b1_nhi_h, b1_nrc, b1_nlo_w, b1_nhi_w, b1_ncc;
    const int8_t *shortcut;
    int relu;
    int8_t *x5;
    int16_t *x2;
    uint8_t *relu_mask;
    int32_t *acc_out;         // forward: optional dump; dgrad: the int32 scratch (required)
    DeviceState *dev;
    // B operand read MN-major (patch kernel, error back-propagation): the weights stay [c_out][tap][c_in], a sub-tile
    // is [kc reduction rows][tile_n columns] made of tile_n / b_row atoms of b_row-byte rows, kc * b_row bytes apart
    int b_mn;
    int b_row;
};

// Patch variant of the implicit GEMM for stride-1 filters (eoq_igemm_patch.cu): an M tile is `r_rows` output rows
// of one image in the raster of a patch that is (kdim - 1) pixels wider than the output row; the patch of source
// pixels is loaded once and every filter tap reads it through a descriptor started (a * pw + b) rows further.
struct PatchPlan {
    int n_img;
    int kdim;           // square filter size
    int pad;            // tap (a, b) reads source pixel (y + a - pad, x + b - pad)
    int pw;             // patch width = wq + kdim - 1
    int r_rows;         // output rows per tile
    int tiles_per_img;
    int chunks;         // source channels / kc
    int a_bytes;        // bytes of one patch buffer (multiple of 1024)
    int a_box_bytes;    // bytes one patch load delivers
    int num_a, num_b;   // ring depths (patches, weight sub-tiles)
    int b_resident;     // all weight sub-tiles of the layer stay in shared memory
};
constexpr int kPatchThreads = 128 + 32 * kEpilogueWarps;  // warps: 0 patch loads, 1 MMA + TMEM, 2 weight loads, 3 idle, then the epilogue

size_t igemm_patch_smem_bytes(const IgemmParams &p, const PatchPlan &pl);
cudaError_t launch_igemm_patch(const IgemmParams &p, const PatchPlan &pl, const CUtensorMap &map_a,
                               const CUtensorMap &map_b, int grid, cudaStream_t stream);

size_t igemm_smem_bytes(const IgemmParams &p);
cudaError_t launch_igemm(const IgemmParams &p, const CUtensorMap &map_a, const CUtensorMap &map_b, int grid,
                         cudaStream_t stream);

// ---------------------------------------------------------------------------------------------
// Weight-gradient kernel: D[(tap, ic), oc] = sum over pixels of x1[pixel + tap, ic] * e3[pixel, oc]
// ---------------------------------------------------------------------------------------------
struct WgradParams {
    int P;               // reduction length: n * ho * wo error pixels
    int ho, wo;
    int c_in, c_out;
    int ntaps;
    int kc;              // c_in bytes per A sub-tile (16..128)
    int nc;              // c_out bytes per B sub-tile (16..128)
    int chunks_per_tap;  // c_in / kc
    int rows_total;      // ntaps * c_in (GEMM M)
    int subs_per_mtile;  // 128 / kc
    int tile_n;          // c_out columns per CTA (multiple of 16, <= 256)
    int num_m_tiles, num_n_tiles, num_k_splits;
    int mtiles_per_cta;  // M tiles one CTA accumulates side by side in TMEM (they share the error tile of a stage)
    int num_m_groups;    // ceil(num_m_tiles / mtiles_per_cta)
    int pixels_per_stage;   // 64
    int stages_per_split;   // pipeline iterations each CTA runs
    int num_stages;
    int src_stride, src_stride_w, base_h, base_w;
    int row_window_kw;   // 0, or the filter width when an M tile is one filter row of 8 x 16 bytes (7 real taps of 8)
    unsigned char tap_dh[kMaxTaps], tap_dw[kMaxTaps];
    long long *acc;      // [c_out][taps][c_in] int64, zeroed before launch
    DeviceState *dev;
};

// Patch variant of the weight gradient for stride-1 filters (eoq_wgrad_patch.cu).  A pixel block is `r_rows`
// output rows of one image; the error patch [r_rows x pw pixels] (zero in the pw - wo extra columns) and the
// activation patch [(r_rows + k - 1) x pw] are loaded once, and the activation operand of tap (a, b) is the same
// patch read (a * pw + b) rows further.  One CTA = one group (output-channel tile, input-channel chunk, a set of
// filter rows) x one range of pixel blocks; it leaves int32 partial sums in its own slice (no atomics).
struct WgradPatchPlan {
    int n_img, ho, wo;
    int c_in, c_out;
    int kdim, pad;
    int pw;              // patch width = wo + kdim - 1
    int r_rows;          // output rows per pixel block
    int blocks_per_img;
    int kp;              // reduction rows per block, r_rows * pw rounded up to 32
    int kc, chunks;      // activation channel bytes per chunk (32/64/128), chunks
    int apa;             // taps per accumulator: 128 / kc adjacent taps of one filter row share an MMA
    int accs_per_row;    // accumulators per filter row
    int rows_per_group, row_groups;  // filter rows one CTA handles, groups of them
    int tile_n, n_tiles; // output-channel columns per CTA (32/64/128)
    int num_groups;      // n_tiles * chunks * row_groups
    int num_splits;      // pixel-block ranges
    int blocks_per_split;
    int x_bytes, e_bytes;  // bytes of one stage's activation / error buffer (multiples of 1024)
    int x_box_bytes, e_box_bytes;
    int num_stages;
    int rows_total;      // taps * c_in
    int32_t *partials;   // [num_splits][c_out][taps][c_in]
    DeviceState *dev;
};
constexpr int kWgradPatchThreads = 192;  // warp 0 loads, warp 1 MMA + TMEM, warps 2..5 epilogue
constexpr int kWgradTargetCtas = 148;    // CTAs the split count aims at (one per SM of a 148-SM part; shared memory allows one)

size_t wgrad_patch_smem_bytes(const WgradPatchPlan &pl);
cudaError_t launch_wgrad_patch(const WgradPatchPlan &pl, const CUtensorMap &map_x, const CUtensorMap &map_e,
                               cudaStream_t stream);

size_t wgrad_smem_bytes(const WgradParams &p);
cudaError_t launch_wgrad(const WgradParams &p, const CUtensorMap &map_x, const CUtensorMap &map_e, cudaStream_t stream);

// Issue-rate measurement of tcgen05.mma kind::i8 (eoq_probe.cu): `grid` CTAs, each `iters` x 4 MMAs of 128 x n_cols x 32.
cudaError_t launch_probe_mma_i8(int n_cols, int iters, int grid, DeviceState *dev, unsigned long long *cycles_out,
                                cudaStream_t s);

// ---------------------------------------------------------------------------------------------
// Elementwise / reduction kernels
// ---------------------------------------------------------------------------------------------
cudaError_t launch_reset_cells(DeviceState *dev, cudaStream_t s);
cudaError_t launch_quantize_image(const float *src, int n, int h, int w, int c_src, int c_dst, int wmargin, int8_t *dst,
                                  int32_t *dst_exp, DeviceState *dev, int sm_count, cudaStream_t s, const ReduceHook &hook);
// w[oc][kh][kw][16] -> wp[oc][kh][8][16], zero in the taps kw..7 (weights of the filter-row path)
cudaError_t launch_weight_pad_rows(const int8_t *w, int8_t *wp, int c_out, int kh, int kw, int c_in, cudaStream_t s);
cudaError_t launch_quantize_f32(int mode, const float *src, size_t n, void *dst, int32_t *dst_exp, DeviceState *dev,
                                int sm_count, cudaStream_t s, const ReduceHook &hook);
cudaError_t launch_sq_i32(const int32_t *src, const int32_t *src_exp, int exp_bias, size_t n, int8_t *dst,
                          int32_t *dst_exp, long long *sum_codes, bool max_already_reduced, DeviceState *dev,
                          int sm_count, cudaStream_t s, const ReduceHook &hook, const NextHeadArgs *next = nullptr,
                          const JoinStatArgs *join = nullptr);
// Q_g of the exact sums.  `src` holds int64 sums; when `parts` is given the sums are first formed from
// `num_parts` int32 slices of n elements each (and written to src).
cudaError_t launch_sq_i32_scatter(const int32_t *src, const int32_t *src_exp, int exp_bias, int n_img, int hh, int ww, int c,
                                  int stride, int hq, int wq, int8_t *dst, int32_t *dst_exp, long long *sum_codes,
                                  DeviceState *dev, int sm_count, cudaStream_t s, const ReduceHook &hook);
// b1 is b1_c, or the code at b1_dev when that is given.  Two kernels: slice sum + b1 term + max, then Q_g; the maximum
// travels through the handle's absmax_u64 cell, which the second kernel puts back to zero.
// tap_sums: kTapReplicas copies, `replica_stride` elements apart, whose sum is the b1 error sum per (oc, tap).
cudaError_t launch_sq_i64(const long long *src, const int32_t *src_exp, int exp_bias, size_t n, int8_t *dst,
                          int32_t *dst_exp, long long *copy_out, const long long *tap_sums, size_t replica_stride,
                          int32_t b1_c, const int32_t *b1_dev, int c_in, const int32_t *parts, int num_parts,
                          DeviceState *dev, int sm_count, cudaStream_t s, const ReduceHook &hook);
// gamma is gamma_c, or the code at gamma_dev when that is given.  force_timeout: self-test of the bounded wait.
cudaError_t launch_err_prescale(const int8_t *e0, const int32_t *e0_exp, const uint8_t *mask, const int16_t *x2,
                                size_t n_el, int32_t gamma_c, const int32_t *gamma_dev, int8_t *e3, int32_t *e3_exp,
                                long long *sum_e1, long long *sum_e1x2, DeviceState *dev, int sm_count, cudaStream_t s,
                                int *kernels, bool force_timeout, const ReduceHook &hook);
struct UpdateTensor {
    int8_t *w;
    const int8_t *g;
    const int32_t *g_exp;
    unsigned long long n;
    int32_t *master;  // wide update only: the k_m-bit master codes (w then receives Q_w of them)
};
// step_dev (device, optional): the step counter is read from it and it is incremented behind the update.
cudaError_t launch_update(const UpdateTensor *t, int num, int32_t lr_mant, int32_t lr_exp, int stochastic,
                          uint64_t seed, uint64_t step, unsigned long long *step_dev, DeviceState *dev, int sm_count,
                          cudaStream_t s);
// The same update with a k_u-bit update quantizer on k_m-bit master codes (t[i].master); t[i].w receives Q_w(master).
cudaError_t launch_update_wide(const UpdateTensor *t, int num, int32_t lr_mant, int32_t lr_exp, int k_u, int k_m, int stochastic,
                               uint64_t seed, uint64_t step, unsigned long long *step_dev, DeviceState *dev, cudaStream_t s);
cudaError_t launch_layout_convert(const int8_t *src, int8_t *dst, int n, int c, int h, int w, int to_nhwc,
                                  cudaStream_t s);
cudaError_t launch_weight_transpose(const int8_t *w, int8_t *wt, int c_out, int taps, int c_in, cudaStream_t s);
// b1 support: class tables of weight sums (forward) and of error sums (weight gradient)
struct BorderClasses {
    int nlo_h, nhi_h, nrc, nlo_w, nhi_w, ncc;
};
cudaError_t launch_b1_weight_table(const int8_t *w, int32_t *table, const eoq_conv_desc_t &d, const BorderClasses &bc,
                                   cudaStream_t s);
constexpr int kTapReplicas = 4;  // copies of the b1 error sums the blocks spread their atomics over
cudaError_t launch_b1_error_sums(const int8_t *e3, long long *tap_sums, size_t replica_stride, const eoq_conv_desc_t &d, int ho,
                                 int wo, const BorderClasses &bc, int sm_count, cudaStream_t s);
constexpr int kMaxBorderClasses = 64;  // classes (rows x columns) the b1 kernels keep in shared memory

// eoq_weight_prep: one launch derives the b1 tables (and the row-padded first-layer weights) of up to kPrepChunk layers
struct PrepItem {
    const int8_t *w;
    int32_t *table;   // [classes][c_out]
    int8_t *w_rows;   // [c_out][kh][8][c_in] or null
    eoq_conv_desc_t d;
    int ho, wo;
    BorderClasses bc;
};
constexpr int kPrepChunk = 32;
struct PrepBatch {
    PrepItem item[kPrepChunk];
    int first_block[kPrepChunk + 1];
    int num;
};
cudaError_t launch_weight_prep(const PrepBatch &b, cudaStream_t s);


// ---------------------------------------------------------------------------------------------
// Network glue (eoq_aux.cu)
// ---------------------------------------------------------------------------------------------
cudaError_t launch_maxpool_fwd(const int8_t *x, int n, int h, int w, int c, int k, int s, int p, int8_t *y, uint8_t *arg,
                               int sm_count, cudaStream_t st);
cudaError_t launch_maxpool_bwd(const int8_t *e, const int32_t *e_exp, const uint8_t *arg, int n, int h, int w, int c, int k, int s,
                               int p, int8_t *e_in, int32_t *e_in_exp, const uint8_t *next_mask, const int32_t *next_gamma, int8_t *e3,
                               int32_t *e3_exp, long long *sum_e1, DeviceState *dev, int sm_count, cudaStream_t st,
                               const ReduceHook &hook);
cudaError_t launch_avgpool_sum(const int8_t *x, int n, int hw, int c, int32_t *sums, cudaStream_t st);
cudaError_t launch_join(const int8_t *a, const int32_t *a_exp, const int8_t *b, const int32_t *b_exp, const uint8_t *mask_b,
                        size_t n_el, int8_t *out, int32_t *out_exp, long long *sum_out, const uint8_t *next_mask,
                        const int16_t *next_x2, const int32_t *next_gamma, int8_t *e3, int32_t *e3_exp, long long *sum_e1,
                        long long *sum_e1x2, DeviceState *dev, int sm_count, cudaStream_t st, const ReduceHook &hook);
// the second pass of launch_join alone: the maxima are already in the handle's cells (see JoinStatArgs)
cudaError_t launch_join_second(const int8_t *a, const int32_t *a_exp, const int8_t *b, const int32_t *b_exp, const uint8_t *mask_b,
                               size_t n_el, int8_t *out, int32_t *out_exp, long long *sum_out, const NextHeadArgs *next,
                               DeviceState *dev, int sm_count, cudaStream_t st);
cudaError_t launch_head(const int32_t *sums, int n, int c, int hw, int classes, float *W, float *bias, const int32_t *labels,
                        float lr, float *loss_out, float *dpooled, float *logits, float *pooled, float *dl, double *loss_n,
                        cudaStream_t st);
cudaError_t launch_head_update(const float *dl, const float *pooled, int n, int c, int classes, float lr, float *W, float *bias,
                               cudaStream_t st);
cudaError_t launch_head_error(const float *dpooled, int n, int c, int hw, float *ef, int8_t *e, int32_t *e_exp, DeviceState *dev,
                              int sm_count, cudaStream_t st, const ReduceHook &hook);
struct ScalarItem {
    int32_t *theta;          // the code to update (device)
    int32_t *mirror;         // a second place that receives the new code, or null
    const long long *total;  // exact sum behind the gradient (device)
    const int32_t *exp;      // its exponent (device) ...
    int exp_bias;            // ... plus this constant
    int tensor_id;           // counter of the rounding hash
    int32_t *grad_out;       // receives {code, exponent} of Q_g(total), or null
};
constexpr int kScalarChunk = 64;
struct ScalarBatch {
    ScalarItem item[kScalarChunk];
    int num;
};
// Finish of the weight gradients of many layers in a few launches (eoq_wgrad_finish): per layer the b1 error sums,
// the sum of the split-K slices plus the b1 term, and Q_g.  One item per layer; blocks find their item by their index.
constexpr int kFinishChunk = 16;
struct FinishItem {
    const int8_t *e3;
    const int32_t *e3_exp;
    const int32_t *b1_dev;         // null: no b1 term (then the tap sums are neither formed nor read)
    long long *tap_sums;           // kTapReplicas copies, tap_stride elements apart; zeroed by the finish itself
    unsigned long long *max_cell;  // max |sum| of the layer (in the spare bytes behind the tap sums)
    long long *acc;                // exact sums [oc][tap][ic]
    const int32_t *parts;          // int32 split-K slices, or null when the GEMM added into acc
    int8_t *g;
    int32_t *g_exp;
    unsigned long long n;          // weights
    unsigned long long tap_stride, zero_bytes;
    unsigned long long pixels;
    eoq_conv_desc_t d;
    BorderClasses bc;
    int ho, wo, pixels_per_block, tap_grid_x, tap_grid_y;
    int num_parts, groups, fin_blocks, sq_blocks;
};
struct FinishBatch {
    int num;
    int tap_first[kFinishChunk + 1], fin_first[kFinishChunk + 1], sq_first[kFinishChunk + 1];
    FinishItem item[kFinishChunk];
};
// fills the launch geometry of an item (tap grid, block counts) from its sizes
void plan_finish_item(FinishItem &it, int sm_count);
cudaError_t launch_wgrad_finish(const FinishBatch &b, unsigned *status, cudaStream_t s);

// Batch normalisation behind the convolution (comparison case, eoq_bn.cu): per-channel record in the workspace
struct BnChannel {
    long long s1, shh, shl, sll;   // sum of A; sum of A^2 in three parts (A = h * 2^16 + l): h*h, h*l, l*l
    long long d1, d2;              // backward: sum of E * mask, sum of E * mask * A
    double mu, inv;                // mean in units of A; 1 / sqrt(var + eps)
    float scale, shift;            // y = fma((float)A, scale, shift)
    float ca, cb, cc, pad;         // da = fma(ca, E * mask, fma(cb, (float)A, cc))
};
size_t bn_workspace_bytes(int c);   // records + per-block partial sums
cudaError_t launch_bn_fwd(const int32_t *acc, int p, size_t pixels, int c, const float *gamma, const float *beta, float eps,
                          int8_t *x5, uint8_t *relu_mask, BnChannel *ch, int sm_count, cudaStream_t st);
cudaError_t launch_bn_bwd(const int8_t *e, const int32_t *e_exp, const uint8_t *relu_mask, const int32_t *acc, int p, size_t pixels,
                          int c, const float *gamma, BnChannel *ch, float *da, float *dgamma, float *dbeta, int sm_count,
                          cudaStream_t st);

cudaError_t launch_scalar_update(const ScalarBatch &b, int32_t lr_mant, int32_t lr_exp, int stochastic, uint64_t seed,
                                 const unsigned long long *step_dev, uint64_t step, cudaStream_t st);

}  // namespace eoq
