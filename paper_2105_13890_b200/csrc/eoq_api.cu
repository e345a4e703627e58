// C ABI of libeoq: argument checks, TMA descriptors, launch plans.  Declarations and their contract: eoq.h.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include "eoq_internal.h"

using namespace eoq;

namespace {

// --------------------------------------------------------------------------------- driver entry points

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const int *, const int *, cuuint32_t, cuuint32_t,
                                   const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn g_encode_tiled = nullptr;
EncodeIm2colFn g_encode_im2col = nullptr;

bool load_driver_entry_points()
{
    if (g_encode_tiled && g_encode_im2col) return true;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn) return false;
    g_encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
    fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn) return false;
    g_encode_im2col = reinterpret_cast<EncodeIm2colFn>(fn);
    return true;
}

CUtensorMapSwizzle swizzle_for(int row_bytes)
{
    switch (row_bytes) {
        case 128: return CU_TENSOR_MAP_SWIZZLE_128B;
        case 64: return CU_TENSOR_MAP_SWIZZLE_64B;
        case 32: return CU_TENSOR_MAP_SWIZZLE_32B;
        default: return CU_TENSOR_MAP_SWIZZLE_NONE;
    }
}

// Widest of 128/64/32/16 channel bytes that divides c (c is a multiple of 16).
int chunk_bytes(int c)
{
    for (int k = 128; k > 16; k >>= 1)
        if (c % k == 0) return k;
    return 16;
}

// im2col view of an NHWC int8 tensor [n][h][w][c]: `pixels` consecutive positions of the walk that starts at
// (lower_w, lower_h) and advances by `stride`, `box_c` channels each.  count_w/h = positions per row/column.
// View for the filter-row path: the pixel of the walk is a 128-byte window of 8 adjacent 16-channel pixels that
// starts at memory column (first_col + k * stride) of a row w_mem pixels long, so consecutive windows overlap
// (the W stride of the view is smaller than its inner extent).  Rows are walked with zero fill above and below.
bool make_row_window_map(CUtensorMap *map, const void *ptr, int n, int h, int w_mem, int c, int first_col, int count_w,
                         int count_h, int stride, int pad_h, int pixels)
{
    const cuuint64_t window = 8u * c;  // bytes of 8 adjacent pixels
    cuuint64_t dims[4] = {window, (cuuint64_t)count_w, (cuuint64_t)h, (cuuint64_t)n};
    cuuint64_t strides[3] = {(cuuint64_t)stride * c, (cuuint64_t)w_mem * c, (cuuint64_t)w_mem * c * h};
    int lower[2] = {0, -pad_h};
    int upper[2] = {0, (count_h - 1) * stride + 1 - pad_h - h};
    if (upper[1] < -128 || upper[1] > 127 || pad_h > 128) return false;
    cuuint32_t estr[4] = {1, 1, (cuuint32_t)stride, 1};
    const char *base = static_cast<const char *>(ptr) + (long long)first_col * c;
    return g_encode_im2col(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<char *>(base), dims, strides, lower, upper,
                           (cuuint32_t)window, (cuuint32_t)pixels, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           swizzle_for((int)window), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_im2col_map(CUtensorMap *map, const void *ptr, int n, int h, int w, int c, int lower_w, int lower_h,
                     int count_w, int count_h, int stride, int box_c, int pixels)
{
    cuuint64_t dims[4] = {(cuuint64_t)c, (cuuint64_t)w, (cuuint64_t)h, (cuuint64_t)n};
    cuuint64_t strides[3] = {(cuuint64_t)c, (cuuint64_t)c * w, (cuuint64_t)c * w * h};
    int lower[2] = {lower_w, lower_h};
    // the walk covers count positions: (extent + upper - lower - 1) / stride + 1 = count
    int upper[2] = {(count_w - 1) * stride + 1 + lower_w - w, (count_h - 1) * stride + 1 + lower_h - h};
    for (int i = 0; i < 2; ++i)
        if (lower[i] < -128 || lower[i] > 127 || upper[i] < -128 || upper[i] > 127) return false;
    cuuint32_t estr[4] = {1, (cuuint32_t)stride, (cuuint32_t)stride, 1};
    return g_encode_im2col(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(ptr), dims, strides, lower, upper,
                           (cuuint32_t)box_c, (cuuint32_t)pixels, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           swizzle_for(box_c), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tiled view of an NHWC int8 tensor with a (box_c, box_w, box_h, 1) box: one patch of pixels, halo included.
bool make_patch_map(CUtensorMap *map, const void *ptr, int n, int h, int w, int c, int box_c, int box_w, int box_h)
{
    if (box_w > 256 || box_h > 256) return false;
    cuuint64_t dims[4] = {(cuuint64_t)c, (cuuint64_t)w, (cuuint64_t)h, (cuuint64_t)n};
    cuuint64_t strides[3] = {(cuuint64_t)c, (cuuint64_t)c * w, (cuuint64_t)c * w * h};
    cuuint32_t box[4] = {(cuuint32_t)box_c, (cuuint32_t)box_w, (cuuint32_t)box_h, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(ptr), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(box_c), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tiled view of a [rows][taps][c] int8 tensor with a (box_c, 1, box_rows) box.
bool make_weight_map(CUtensorMap *map, const void *ptr, int rows, int taps, int c, int box_c, int box_rows)
{
    cuuint64_t dims[3] = {(cuuint64_t)c, (cuuint64_t)taps, (cuuint64_t)rows};
    cuuint64_t strides[2] = {(cuuint64_t)c, (cuuint64_t)c * taps};
    cuuint32_t box[3] = {(cuuint32_t)box_c, 1, (cuuint32_t)box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    return g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void *>(ptr), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(box_c), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tiled view of a [rows][c] int8 matrix with a (box_c, box_rows) box.
bool make_matrix_map(CUtensorMap *map, const void *ptr, size_t rows, int c, int box_c, int box_rows)
{
    cuuint64_t dims[2] = {(cuuint64_t)c, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)c};
    cuuint32_t box[2] = {(cuuint32_t)box_c, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(ptr), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(box_c), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// --------------------------------------------------------------------------------- checks and geometry

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
inline size_t round256(size_t v) { return (v + 255) & ~(size_t)255; }

struct Geometry {
    int ho, wo, taps;
    size_t in_elems, out_elems, w_elems;
};

int check_desc(const eoq_conv_desc_t *d, Geometry *g)
{
    if (!d) return EOQ_ERR_BAD_ARG;
    if (d->n <= 0 || d->h <= 0 || d->w <= 0 || d->c_in <= 0 || d->c_out <= 0 || d->kh <= 0 || d->kw <= 0 ||
        d->stride <= 0 || d->pad < 0)
        return EOQ_ERR_BAD_ARG;
    if (d->h + 2 * d->pad < d->kh || d->w + 2 * d->pad < d->kw) return EOQ_ERR_BAD_ARG;
    if ((d->c_in % 16 && d->c_in != 8) || d->c_out % 16) return EOQ_ERR_ALIGNMENT;  // 8: the filter-row path only
    if (d->x_wmargin < 0 || d->x_wmargin > 64) return EOQ_ERR_BAD_ARG;
    if (d->kh * d->kw > kMaxTaps || d->kh > 16 || d->kw > 16 || d->stride > 8 || d->pad > 64) return EOQ_ERR_UNSUPPORTED;
    g->ho = (d->h + 2 * d->pad - d->kh) / d->stride + 1;
    g->wo = (d->w + 2 * d->pad - d->kw) / d->stride + 1;
    g->taps = d->kh * d->kw;
    g->in_elems = (size_t)d->n * d->h * d->w * d->c_in;
    g->out_elems = (size_t)d->n * g->ho * g->wo * d->c_out;
    g->w_elems = (size_t)d->c_out * g->taps * d->c_in;
    if ((size_t)d->n * d->h * d->w >= (1u << 31) || (size_t)d->n * g->ho * g->wo >= (1u << 31)) return EOQ_ERR_UNSUPPORTED;
    return EOQ_OK;
}

// Rows (or columns) whose filter window leaves the image at the low / high end.
void border_counts(int extent_in, int extent_out, int k, int stride, int pad, int *nlo, int *nhi, int *ncls)
{
    int lo = 0, hi = 0;
    for (int y = 0; y < extent_out; ++y) {
        if (y * stride - pad < 0) ++lo;
        if (y * stride - pad + k - 1 > extent_in - 1) ++hi;
    }
    *nlo = lo;
    *nhi = hi;
    *ncls = (lo + hi + 1 >= extent_out) ? extent_out : lo + hi + 1;
}

BorderClasses border_classes(const eoq_conv_desc_t &d, const Geometry &g)
{
    BorderClasses bc;
    border_counts(d.h, g.ho, d.kh, d.stride, d.pad, &bc.nlo_h, &bc.nhi_h, &bc.nrc);
    border_counts(d.w, g.wo, d.kw, d.stride, d.pad, &bc.nlo_w, &bc.nhi_w, &bc.ncc);
    return bc;
}

int record(Handle *h, cudaError_t e)
{
    if (e == cudaSuccess) return EOQ_OK;
    h->last_cuda_error = (int)e;
    return EOQ_ERR_CUDA;
}

// 16- or 8-channel inputs under filters 5 to 8 taps wide (the 7x7 first layer) stored with wide enough zero margins
// take the filter-row path: a filter row is 8 adjacent pixels, one 128- or 64-byte K sub-tile, instead of one TMA
// row per tap.  The window of an output pixel starts (stride * c_in) bytes after its neighbour's and the first one
// (x_wmargin - pad) pixels into the row: both must be multiples of 16 bytes, which 8 channels meet for even strides
// and an even distance between margin and padding.
inline bool use_row_window(const eoq_conv_desc_t &d, int wo)
{
    if ((d.c_in != 16 && d.c_in != 8) || d.kw < 5 || d.kw > 8) return false;
    if (d.c_in == 8 && ((d.stride & 1) || ((d.x_wmargin - d.pad) & 1) || (d.w & 1))) return false;
    const int need_right = (wo - 1) * d.stride - d.pad + 8 - d.w;
    return d.x_wmargin >= d.pad && d.x_wmargin >= need_right;
}

// CTAs of a persistent GEMM over `tiles` tiles.  The kernel lasts as long as its busiest CTA, ceil(tiles / SMs)
// tiles; spreading the tiles evenly over the fewest CTAs that keep that maximum costs nothing and leaves the other
// SMs to kernels of other streams (448 tiles on 148 SMs: 112 CTAs of 4 tiles instead of 148 of 3 or 4).
inline int persistent_grid(int tiles, int sm_count)
{
    if (tiles <= sm_count) return tiles < 1 ? 1 : tiles;
    const int per_cta = (tiles + sm_count - 1) / sm_count;
    return (tiles + per_cta - 1) / per_cta;
}

// Shared tiling choices of the implicit GEMM: K sub-tiles, pipeline depth, column tile.
void plan_igemm(IgemmParams &p, int src_channels, int ntaps, int sm_count)
{
    p.kc = chunk_bytes(src_channels);
    p.chunks_per_tap = src_channels / p.kc;
    p.ntaps = ntaps;
    p.real_sub = ntaps * p.chunks_per_tap;
    p.num_sub = (p.kc == 16 && (p.real_sub & 1)) ? p.real_sub + 1 : p.real_sub;
    p.subs_per_stage = 128 / p.kc;
    if (p.subs_per_stage > p.num_sub) p.subs_per_stage = p.num_sub;
    p.num_m_tiles = (p.M + kTileM - 1) / kTileM;
    // An MMA costs at least ~57 cycles whatever its width and reaches the tensor peak only from 128 columns
    // up, so tiles stay 128 wide even when that leaves some SMs without one; 256 when there are tiles to spare.
    int tn = p.N < 256 ? p.N : 256;
    if (tn == 256 && (long long)p.num_m_tiles * ((p.N + 255) / 256) < 2LL * sm_count) tn = 128;
    p.tile_n = tn;
    p.num_n_tiles = (p.N + tn - 1) / tn;
    const size_t stage = (size_t)p.subs_per_stage * (kTileM + tn) * p.kc;
    int stages = (int)((200 * 1024) / stage);
    p.num_stages = stages > 8 ? 8 : (stages < 2 ? 2 : stages);
}

// Plan of the patch variant for a stride-1 k x k correlation over a source [n][hs][ws][c_src] producing a
// [n][hq][wq] grid with n_cols columns.  Returns false when the geometry does not suit it (then the per-tap
// path is used): strided or 1x1 filters, fewer than 32 channels, rows too wide for a tile, or tiles that would
// be mostly padding.
bool plan_patch(IgemmParams &p, PatchPlan &pl, int n_img, int c_src, int hq, int wq, int k, int pad_src, int n_cols,
                int sm_count)
{
    if (k < 2 || c_src % 32 || pad_src < 0 || pad_src > k - 1) return false;
    const int pw = wq + k - 1;
    if (pw > kTileM) return false;
    int r = kTileM / pw;
    if (r > hq) r = hq;
    const int tiles_per_img = (hq + r - 1) / r;
    if ((double)hq * wq < 0.6 * (double)tiles_per_img * kTileM) return false;
    pl.n_img = n_img;
    pl.kdim = k;
    pl.pad = pad_src;
    pl.pw = pw;
    pl.r_rows = r;
    pl.tiles_per_img = tiles_per_img;
    p.kc = chunk_bytes(c_src);
    pl.chunks = c_src / p.kc;
    p.chunks_per_tap = pl.chunks;
    p.ntaps = k * k;
    const int patch_rows = r + k - 1;
    pl.a_box_bytes = p.kc * pw * patch_rows;
    const int rows_read = (k - 1) * (pw + 1) + kTileM;  // the last tap's tile ends here
    const int rows = pw * patch_rows > rows_read ? pw * patch_rows : rows_read;
    pl.a_bytes = (int)((((size_t)rows * p.kc) + 1023) & ~(size_t)1023);
    p.M = n_img * hq * wq;
    p.N = n_cols;
    p.hq = hq;
    p.wq = wq;
    p.num_m_tiles = n_img * tiles_per_img;
    int tn = n_cols < 256 ? n_cols : 256;
    if (tn == 256 && (long long)p.num_m_tiles * ((n_cols + 255) / 256) < 2LL * sm_count) tn = 128;
    p.tile_n = tn;
    p.num_n_tiles = (n_cols + tn - 1) / tn;
    const size_t budget = 200 * 1024;
    const size_t b_sub = (size_t)tn * p.kc;
    const size_t b_all = b_sub * pl.chunks * p.ntaps;
    pl.b_resident = (p.num_n_tiles == 1 && b_all + 2 * (size_t)pl.a_bytes <= budget && b_all < (1u << 20)) ? 1 : 0;
    if (pl.b_resident) {
        size_t na = (budget - b_all) / pl.a_bytes;
        pl.num_a = na > 4 ? 4 : (int)na;
        pl.num_b = 1;
    } else {
        pl.num_a = pl.chunks > 1 ? 3 : 2;
        if ((size_t)pl.num_a * pl.a_bytes + 2 * b_sub > budget) return false;
        size_t nb = (budget - (size_t)pl.num_a * pl.a_bytes) / b_sub;
        pl.num_b = nb > 8 ? 8 : (int)nb;
    }
    return pl.num_a >= 2 || (pl.b_resident && pl.num_a >= 1);
}

// Plan of the patch variant of the weight gradient; false when the geometry does not suit it.
bool plan_wgrad_patch(WgradPatchPlan &pl, const eoq_conv_desc_t &d, int ho, int wo, int target_ctas = kWgradTargetCtas)
{
    if (d.stride != 1 || d.kh != d.kw || d.kh < 2 || d.x_wmargin != 0 || d.c_in % 32 || d.c_out % 32) return false;
    if (d.pad > d.kh - 1) return false;
    memset(&pl, 0, sizeof(pl));
    pl.n_img = d.n; pl.ho = ho; pl.wo = wo; pl.c_in = d.c_in; pl.c_out = d.c_out;
    pl.kdim = d.kh; pl.pad = d.pad;
    pl.pw = wo + d.kh - 1;
    if (pl.pw > 256) return false;
    pl.kc = chunk_bytes(d.c_in);
    pl.chunks = d.c_in / pl.kc;
    pl.apa = 128 / pl.kc;
    pl.accs_per_row = (d.kh + pl.apa - 1) / pl.apa;
    pl.tile_n = chunk_bytes(d.c_out);
    pl.n_tiles = d.c_out / pl.tile_n;
    int rpg = 512 / (pl.tile_n * pl.accs_per_row);
    if (rpg * pl.accs_per_row > 8) rpg = 8 / pl.accs_per_row;
    if (rpg > d.kh) rpg = d.kh;
    if (rpg < 1) return false;
    pl.rows_per_group = rpg;
    pl.row_groups = (d.kh + rpg - 1) / rpg;
    pl.num_groups = pl.n_tiles * pl.chunks * pl.row_groups;
    pl.rows_total = d.kh * d.kw * d.c_in;
    // rows per pixel block: as many as keep one stage near 64 KB (three stages in flight)
    int r = ho < 32 ? ho : 32;
    for (; r >= 1; --r) {
        const int kp = (r * pl.pw + 31) / 32 * 32;
        int x_rows = (r + d.kh - 1) * pl.pw;
        const int x_read = (d.kh - 1) * (pl.pw + 1) + pl.apa + kp;
        if (x_read > x_rows) x_rows = x_read;
        pl.x_bytes = (x_rows * pl.kc + 1023) / 1024 * 1024;
        pl.e_bytes = (kp * pl.tile_n + 1023) / 1024 * 1024;
        pl.kp = kp;
        if (pl.x_bytes + pl.e_bytes <= 66 * 1024) break;
    }
    if (r < 1) return false;
    pl.r_rows = r;
    pl.blocks_per_img = (ho + r - 1) / r;
    pl.x_box_bytes = pl.kc * pl.pw * (r + d.kh - 1);
    pl.e_box_bytes = pl.tile_n * pl.pw * r;
    int stages = (200 * 1024) / (pl.x_bytes + pl.e_bytes);
    pl.num_stages = stages > 4 ? 4 : stages;
    if (pl.num_stages < 2) return false;
    const int total_blocks = d.n * pl.blocks_per_img;
    int splits = target_ctas / pl.num_groups;  // rounded down: a few CTAs beyond one wave would double the kernel's time
    if (splits > total_blocks) splits = total_blocks;
    if (splits < 1) splits = 1;
    int per = (total_blocks + splits - 1) / splits;
    const int max_per = 130000 / pl.kp;  // keeps a CTA's int32 partial sums exact: rows * 127 * 128 < 2^31
    if (max_per < 1) return false;
    if (per > max_per) per = max_per;
    pl.blocks_per_split = per;
    pl.num_splits = (total_blocks + per - 1) / per;
    return true;
}

}  // namespace

// ================================================================================= handle

extern "C" int eoq_create(eoq_handle_t *handle, int device)
{
    if (!handle) return EOQ_ERR_BAD_ARG;
    *handle = nullptr;
    if (cudaSetDevice(device) != cudaSuccess) return EOQ_ERR_CUDA;
    if (!load_driver_entry_points()) return EOQ_ERR_CUDA;
    Handle *h = new (std::nothrow) Handle();
    if (!h) return EOQ_ERR_BAD_ARG;
    h->device = device;
    h->last_cuda_error = 0;
    h->dev = nullptr;
    h->launches = 0;
    h->profiling = false;
    h->force_timeout = false;
    h->gemm_only = false;
    h->hook = ReduceHook{nullptr, nullptr};
    h->num_records = 0;
    h->records = nullptr;
    h->fork_ev = h->join_ev = nullptr;
    for (int k = 0; k < kClassBranches; ++k) {
        h->class_branch[k] = nullptr;
        h->class_join[k] = nullptr;
    }
    cudaDeviceProp prop;
    cudaError_t e = cudaGetDeviceProperties(&prop, device);
    if (e == cudaSuccess) {
        h->sm_count = prop.multiProcessorCount;
        h->gemm_ctas = h->sm_count;
        if (prop.major != 10) {
            delete h;
            return EOQ_ERR_UNSUPPORTED;  // the kernels are sm_100a only
        }
        e = cudaMalloc(reinterpret_cast<void **>(&h->dev), sizeof(DeviceState));
    }
    if (e == cudaSuccess) e = cudaMemset(h->dev, 0, sizeof(DeviceState));
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->fork_ev, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->join_ev, cudaEventDisableTiming);
    for (int k = 0; k < kClassBranches && e == cudaSuccess; ++k) {
        e = cudaStreamCreateWithFlags(&h->class_branch[k], cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->class_join[k], cudaEventDisableTiming);
    }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        for (int k = 0; k < kClassBranches; ++k) {
            if (h->class_join[k]) cudaEventDestroy(h->class_join[k]);
            if (h->class_branch[k]) cudaStreamDestroy(h->class_branch[k]);
        }
        if (h->join_ev) cudaEventDestroy(h->join_ev);
        if (h->fork_ev) cudaEventDestroy(h->fork_ev);
        if (h->dev) cudaFree(h->dev);
        delete h;
        return EOQ_ERR_CUDA;
    }
    *handle = reinterpret_cast<eoq_handle_t>(h);
    return EOQ_OK;
}

extern "C" int eoq_destroy(eoq_handle_t handle)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h) return EOQ_ERR_BAD_ARG;
    cudaSetDevice(h->device);
    cudaDeviceSynchronize();
    for (int k = 0; k < kClassBranches; ++k) {
        if (h->class_join[k]) cudaEventDestroy(h->class_join[k]);
        if (h->class_branch[k]) cudaStreamDestroy(h->class_branch[k]);
    }
    if (h->join_ev) cudaEventDestroy(h->join_ev);
    if (h->fork_ev) cudaEventDestroy(h->fork_ev);
    if (h->dev) cudaFree(h->dev);
    if (h->records) {
        for (int i = 0; i < h->num_records; ++i) {
            cudaEventDestroy(h->records[i].begin);
            cudaEventDestroy(h->records[i].end);
        }
        delete[] h->records;
    }
    delete h;
    return EOQ_OK;
}

extern "C" int eoq_profile_start(eoq_handle_t handle)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h) return EOQ_ERR_BAD_ARG;
    if (!h->records) {
        h->records = new (std::nothrow) ProfRecord[kMaxProfRecords];
        if (!h->records) return EOQ_ERR_BAD_ARG;
    }
    for (int i = 0; i < h->num_records; ++i) {
        cudaEventDestroy(h->records[i].begin);
        cudaEventDestroy(h->records[i].end);
    }
    h->num_records = 0;
    h->profiling = true;
    return EOQ_OK;
}

extern "C" int eoq_profile_stop(eoq_handle_t handle, int launches[EOQ_PROF_KINDS], double milliseconds[EOQ_PROF_KINDS])
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || !launches || !milliseconds) return EOQ_ERR_BAD_ARG;
    h->profiling = false;
    cudaError_t e = cudaDeviceSynchronize();
    for (int k = 0; k < EOQ_PROF_KINDS; ++k) {
        launches[k] = 0;
        milliseconds[k] = 0.0;
    }
    for (int i = 0; i < h->num_records && e == cudaSuccess; ++i) {
        float ms = 0.f;
        e = cudaEventElapsedTime(&ms, h->records[i].begin, h->records[i].end);
        launches[h->records[i].kind] += 1;
        milliseconds[h->records[i].kind] += ms;
    }
    return record(h, e);
}

extern "C" int eoq_profile_gemm_only(eoq_handle_t handle, int on)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h) return EOQ_ERR_BAD_ARG;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess && h->gemm_only && !on) {
        // the GEMMs that ran without their consumers left maxima in the reduction cells
        e = launch_reset_cells(h->dev, nullptr);
        if (e == cudaSuccess) e = cudaDeviceSynchronize();
    }
    h->gemm_only = on != 0;
    return record(h, e);
}

extern "C" int eoq_set_reduce_hook(eoq_handle_t handle, eoq_reduce_fn fn, void *user)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h) return EOQ_ERR_BAD_ARG;
    h->hook = ReduceHook{fn, user};
    return EOQ_OK;
}

extern "C" int eoq_set_gemm_ctas(eoq_handle_t handle, int ctas)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || ctas < 0) return EOQ_ERR_BAD_ARG;
    h->gemm_ctas = (ctas == 0 || ctas > h->sm_count) ? h->sm_count : ctas;
    return EOQ_OK;
}

extern "C" unsigned long long eoq_launch_count(eoq_handle_t handle)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    return h ? h->launches : 0ull;
}

namespace {

// Brackets one tensor-core kernel launch with events while profiling is on.
struct ProfScope {
    Handle *h;
    cudaStream_t s;
    ProfRecord *r;
    ProfScope(Handle *h_, int kind, cudaStream_t s_) : h(h_), s(s_), r(nullptr)
    {
        if (!h->profiling || h->num_records >= kMaxProfRecords) return;
        ProfRecord *c = &h->records[h->num_records];
        if (cudaEventCreate(&c->begin) != cudaSuccess) return;
        if (cudaEventCreate(&c->end) != cudaSuccess) {
            cudaEventDestroy(c->begin);
            return;
        }
        c->kind = kind;
        ++h->num_records;
        r = c;
        cudaEventRecord(r->begin, s);
    }
    ~ProfScope()
    {
        if (r) cudaEventRecord(r->end, s);
    }
};

}  // namespace

extern "C" int eoq_last_status(eoq_handle_t handle, void *stream, unsigned *bits)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || !bits) return EOQ_ERR_BAD_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    unsigned v = 0;
    cudaError_t e = cudaMemcpyAsync(&v, &h->dev->status, sizeof(unsigned), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(&h->dev->status, 0, sizeof(unsigned), s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e == cudaSuccess && (v & EOQ_DEV_TIMEOUT)) {
        // a kernel that gave up may not have put the reduction cells back to zero
        e = launch_reset_cells(h->dev, s);
        if (e == cudaSuccess) e = cudaMemsetAsync(&h->dev->ticket, 0, 2 * sizeof(unsigned), s);  // ticket and arrivals
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    }
    *bits = v;
    return record(h, e);
}

extern "C" int eoq_last_cuda_error(eoq_handle_t handle)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    return h ? h->last_cuda_error : static_path_last_cuda_error();
}

extern "C" const char *eoq_status_string(int status)
{
    switch (status) {
        case EOQ_OK: return "ok";
        case EOQ_ERR_BAD_ARG: return "bad argument";
        case EOQ_ERR_ALIGNMENT: return "alignment (16-byte pointers, channels in multiples of 16)";
        case EOQ_ERR_UNSUPPORTED: return "unsupported geometry or device";
        case EOQ_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case EOQ_ERR_RANGE: return "scalar code out of range";
        case EOQ_ERR_CUDA: return "CUDA error";
        default: return "unknown status";
    }
}

// ================================================================================= workspace

extern "C" int eoq_workspace_size(const eoq_conv_desc_t *desc, int pass, size_t *bytes)
{
    Geometry g;
    if (!bytes) return EOQ_ERR_BAD_ARG;
    int st = check_desc(desc, &g);
    if (st != EOQ_OK) return st;
    const BorderClasses bc = border_classes(*desc, g);
    switch (pass) {
        case EOQ_PASS_FWD:  // b1 table, then the row-padded weights of the filter-row path
            *bytes = round256((size_t)bc.nrc * bc.ncc * desc->c_out * sizeof(int32_t)) +
                     (use_row_window(*desc, g.wo) ? round256((size_t)desc->c_out * desc->kh * 8 * desc->c_in) : 0);
            return EOQ_OK;
        case EOQ_PASS_DGRAD:  // transposed weights + int32 sums
            *bytes = round256(g.w_elems) + round256(g.in_elems * sizeof(int32_t));
            return EOQ_OK;
        case EOQ_PASS_WGRAD: {  // per-tap error sums, reduction cell, int64 sums, split-K slices
            WgradPatchPlan wp;
            const size_t slices = plan_wgrad_patch(wp, *desc, g.ho, g.wo) ? (size_t)wp.num_splits * g.w_elems * sizeof(int32_t) : 0;
            *bytes = kTapReplicas * round256((size_t)desc->c_out * g.taps * sizeof(long long)) + 256 +
                     round256(g.w_elems * sizeof(long long)) + round256(slices);
            return EOQ_OK;
        }
        default: return EOQ_ERR_BAD_ARG;
    }
}

static int check_workspace(const eoq_conv_desc_t *desc, int pass, const void *ws, size_t ws_bytes)
{
    size_t need = 0;
    int st = eoq_workspace_size(desc, pass, &need);
    if (st != EOQ_OK) return st;
    if (need == 0) return EOQ_OK;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) || ws_bytes < need) return EOQ_ERR_WORKSPACE;
    return EOQ_OK;
}

// ================================================================================= forward

// Forward chain behind eoq_conv_fwd and eoq_conv_fwd_dev.  The scalars are the three host codes, or the device
// array `scal_dev`.  `prep` holds what eoq_weight_prep derives from the weights; when it is null the call derives it
// itself into `workspace` (two more kernels on the forward chain).
static int conv_fwd_impl(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *x, const int32_t *x_exp,
                         int32_t b1_c, int32_t gamma_c, int32_t b2_c, const int32_t *scal_dev, const int8_t *w,
                         const void *prep, const int8_t *shortcut, int relu, int8_t *x5, int16_t *x2, uint8_t *relu_mask,
                         int32_t *acc_dump, void *workspace, size_t workspace_bytes, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    Geometry g;
    if (!h || !x || !w || !x5) return EOQ_ERR_BAD_ARG;
    int st = check_desc(desc, &g);
    if (st != EOQ_OK) return st;
    if (!aligned16(x) || !aligned16(w) || !aligned16(x5) || !aligned16(shortcut) || !aligned16(x2) ||
        !aligned16(relu_mask) || !aligned16(acc_dump))
        return EOQ_ERR_ALIGNMENT;
    if (b1_c < -32768 || b1_c > 32767 || gamma_c < -32768 || gamma_c > 32767 || b2_c < -32768 || b2_c > 32767)
        return EOQ_ERR_RANGE;
    const eoq_conv_desc_t &d = *desc;
    // the accumulator with its b1 term must fit int32: taps * c_in * (127 + |b1|) * 127 < 2^31
    if ((double)g.taps * d.c_in * (127.0 + (b1_c < 0 ? -b1_c : b1_c)) * 127.0 >= 2147483647.0 - 16777216.0) return EOQ_ERR_RANGE;
    const bool row_window = use_row_window(d, g.wo);
    if (d.c_in == 8 && !row_window) return EOQ_ERR_UNSUPPORTED;
    // with device scalars b1 is unknown here: the table is applied whenever prepared weights are at hand
    const bool use_b1 = scal_dev ? prep != nullptr : b1_c != 0;
    if (scal_dev && !prep && row_window) return EOQ_ERR_BAD_ARG;
    if (!prep && (use_b1 || row_window) && (st = check_workspace(desc, EOQ_PASS_FWD, workspace, workspace_bytes)) != EOQ_OK) return st;
    if (prep && (reinterpret_cast<uintptr_t>(prep) & 255)) return EOQ_ERR_ALIGNMENT;
    char *prep_base = prep ? static_cast<char *>(const_cast<void *>(prep)) : static_cast<char *>(workspace);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const int w_mem = d.w + 2 * d.x_wmargin;

    IgemmParams p;
    memset(&p, 0, sizeof(p));
    PatchPlan pl;
    memset(&pl, 0, sizeof(pl));
    const bool patch = d.stride == 1 && d.kh == d.kw && d.x_wmargin == 0 && !x_exp &&
                       plan_patch(p, pl, d.n, d.c_in, g.ho, g.wo, d.kh, d.pad, d.c_out, h->sm_count);
    p.M = d.n * g.ho * g.wo;
    p.N = d.c_out;
    p.hq = g.ho;
    p.wq = g.wo;
    p.src_stride = d.stride;
    p.base_h = -d.pad;
    int8_t *w_rows = nullptr;
    if (patch) {
        for (int t = 0; t < g.taps; ++t) p.tap_b[t] = (unsigned char)t;
    } else if (row_window) {
        // K sub-tile = one filter row (8 pixels x c_in channels); the map's W axis already steps by the stride
        plan_igemm(p, 8 * d.c_in, d.kh, h->sm_count);
        p.src_stride_w = 1;
        p.base_w = 0;
        for (int t = 0; t < d.kh; ++t) {
            p.tap_dh[t] = (unsigned char)t;
            p.tap_dw[t] = 0;
            p.tap_b[t] = (unsigned char)t;
        }
        const BorderClasses bc0 = border_classes(d, g);
        w_rows = reinterpret_cast<int8_t *>(prep_base) + round256((size_t)bc0.nrc * bc0.ncc * d.c_out * sizeof(int32_t));
        if (!prep) {
            ProfScope prof(h, EOQ_PROF_FWD_AUX, s);
            cudaError_t e = launch_weight_pad_rows(w, w_rows, d.c_out, d.kh, d.kw, d.c_in, s);
            if (e != cudaSuccess) return record(h, e);
            count_launches(h, 1);
        }
    } else {
        plan_igemm(p, d.c_in, g.taps, h->sm_count);
        p.src_stride_w = d.stride;
        p.base_w = d.x_wmargin - d.pad;
        for (int t = 0; t < g.taps; ++t) {
            p.tap_dh[t] = (unsigned char)(t / d.kw);
            p.tap_dw[t] = (unsigned char)(t % d.kw);
            p.tap_b[t] = (unsigned char)t;
        }
    }
    p.out_h = g.ho;
    p.out_w = g.wo;
    p.out_step = 1;
    p.epilogue = kEpiForward;
    p.x_exp = x_exp;
    p.b1_c = b1_c;
    p.gamma_c = gamma_c;
    p.b2_c = b2_c;
    p.scal_dev = scal_dev;
    p.k_total = g.taps * d.c_in;
    p.shortcut = shortcut;
    p.relu = relu ? 1 : 0;
    p.x5 = x5;
    p.x2 = x2;
    p.relu_mask = relu_mask;
    p.acc_out = acc_dump;
    p.dev = h->dev;
    if (use_b1) {
        const BorderClasses bc = border_classes(d, g);
        if (bc.nrc * bc.ncc > kMaxBorderClasses) return EOQ_ERR_UNSUPPORTED;
        p.b1_table = reinterpret_cast<const int32_t *>(prep_base);
        p.b1_nlo_h = bc.nlo_h; p.b1_nhi_h = bc.nhi_h; p.b1_nrc = bc.nrc;
        p.b1_nlo_w = bc.nlo_w; p.b1_nhi_w = bc.nhi_w; p.b1_ncc = bc.ncc;
        if (!prep) {
            ProfScope prof(h, EOQ_PROF_FWD_AUX, s);
            cudaError_t e = launch_b1_weight_table(w, reinterpret_cast<int32_t *>(prep_base), d, bc, s);
            if (e != cudaSuccess) return record(h, e);
            count_launches(h, 1);
        }
    }
    CUtensorMap map_a, map_b;
    if (patch) {
        if (!make_patch_map(&map_a, x, d.n, d.h, d.w, d.c_in, p.kc, pl.pw, pl.r_rows + d.kh - 1) ||
            !make_weight_map(&map_b, w, d.c_out, g.taps, d.c_in, p.kc, p.tile_n))
            return EOQ_ERR_UNSUPPORTED;
        const int ptiles = p.num_m_tiles * p.num_n_tiles;
        count_launches(h, 1);
        ProfScope prof(h, EOQ_PROF_IGEMM_FWD, s);
        return record(h, launch_igemm_patch(p, pl, map_a, map_b, persistent_grid(ptiles, h->gemm_ctas), s));
    }
    if (row_window) {
        if (!make_row_window_map(&map_a, x, d.n, d.h, w_mem, d.c_in, d.x_wmargin - d.pad, g.wo, g.ho, d.stride, d.pad, kTileM) ||
            !make_weight_map(&map_b, w_rows, d.c_out, d.kh, 8 * d.c_in, 8 * d.c_in, p.tile_n))
            return EOQ_ERR_UNSUPPORTED;
    } else if (!make_im2col_map(&map_a, x, d.n, d.h, w_mem, d.c_in, d.x_wmargin - d.pad, -d.pad, g.wo, g.ho, d.stride, p.kc,
                                kTileM) ||
               !make_weight_map(&map_b, w, d.c_out, g.taps, d.c_in, p.kc, p.tile_n)) {
        return EOQ_ERR_UNSUPPORTED;
    }
    const int tiles = p.num_m_tiles * p.num_n_tiles;
    count_launches(h, 1);
    ProfScope prof(h, EOQ_PROF_IGEMM_FWD, s);
    return record(h, launch_igemm(p, map_a, map_b, persistent_grid(tiles, h->gemm_ctas), s));
}

extern "C" int eoq_conv_fwd(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *x, const int32_t *x_exp,
                            int32_t b1_c, const int8_t *w, int32_t gamma_c, int32_t b2_c, const int8_t *shortcut,
                            int relu, int8_t *x5, int16_t *x2, uint8_t *relu_mask, int32_t *acc_dump, void *workspace,
                            size_t workspace_bytes, void *stream)
{
    return conv_fwd_impl(handle, desc, x, x_exp, b1_c, gamma_c, b2_c, nullptr, w, nullptr, shortcut, relu, x5, x2, relu_mask,
                         acc_dump, workspace, workspace_bytes, stream);
}

extern "C" int eoq_conv_fwd_dev(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *x, const int32_t *x_exp,
                                const int32_t *scalars, const int8_t *w, const void *w_prep, const int8_t *shortcut,
                                int relu, int8_t *x5, int16_t *x2, uint8_t *relu_mask, void *stream)
{
    if (!scalars || (reinterpret_cast<uintptr_t>(scalars) & 3)) return EOQ_ERR_BAD_ARG;
    return conv_fwd_impl(handle, desc, x, x_exp, 0, 128, 0, scalars, w, w_prep, shortcut, relu, x5, x2, relu_mask, nullptr,
                         nullptr, 0, stream);
}

extern "C" int eoq_weight_prep_size(const eoq_conv_desc_t *desc, size_t *bytes)
{
    return eoq_workspace_size(desc, EOQ_PASS_FWD, bytes);
}

extern "C" int eoq_weight_prep(eoq_handle_t handle, int num, const eoq_conv_desc_t *descs, const int8_t *const *w,
                               void *const *prep, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || num <= 0 || !descs || !w || !prep) return EOQ_ERR_BAD_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    // every argument is checked before the first launch
    for (int i = 0; i < num; ++i) {
        Geometry g;
        int st = check_desc(&descs[i], &g);
        if (st != EOQ_OK) return st;
        if (!w[i] || !prep[i]) return EOQ_ERR_BAD_ARG;
        if (!aligned16(w[i]) || (reinterpret_cast<uintptr_t>(prep[i]) & 255)) return EOQ_ERR_ALIGNMENT;
        const BorderClasses bc = border_classes(descs[i], g);
        if (bc.nrc * bc.ncc > kMaxBorderClasses) return EOQ_ERR_UNSUPPORTED;
    }
    for (int base = 0; base < num; base += kPrepChunk) {
        PrepBatch b;
        memset(&b, 0, sizeof(b));
        b.num = num - base < kPrepChunk ? num - base : kPrepChunk;
        int blocks = 0;
        for (int k = 0; k < b.num; ++k) {
            const eoq_conv_desc_t &d = descs[base + k];
            Geometry g;
            check_desc(&d, &g);
            PrepItem &it = b.item[k];
            it.w = w[base + k];
            it.table = static_cast<int32_t *>(prep[base + k]);
            it.d = d;
            it.ho = g.ho;
            it.wo = g.wo;
            it.bc = border_classes(d, g);
            it.w_rows = use_row_window(d, g.wo)
                            ? static_cast<int8_t *>(prep[base + k]) + round256((size_t)it.bc.nrc * it.bc.ncc * d.c_out * sizeof(int32_t))
                            : nullptr;
            b.first_block[k] = blocks;
            blocks += d.c_out;
        }
        b.first_block[b.num] = blocks;
        ProfScope prof(h, EOQ_PROF_FWD_AUX, s);
        cudaError_t e = launch_weight_prep(b, s);
        if (e != cudaSuccess) return record(h, e);
        count_launches(h, 1);
    }
    return EOQ_OK;
}

// ================================================================================= error back-propagation

// The error join that takes e4 as its first operand, run behind the dgrad (eoq_conv_dgrad_join_head): the join's first
// pass rides on Q_e, its second pass follows; `next` there is the head of the layer that consumes the joined error.
struct JoinCall {
    const int8_t *b;
    const int32_t *b_exp;
    const uint8_t *mask_b;
    int8_t *out;
    int32_t *out_exp;
    long long *sum_out;
    const NextHeadArgs *next;
};

// `next`: the error head of the layer that consumes e4, fused into Q_e (null for the plain call); `jc`: see JoinCall
static int conv_dgrad_impl(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *e3, const int32_t *e3_exp,
                           const int8_t *w, int8_t *e4, int32_t *e4_exp, int64_t *sum_e4, int32_t *acc_dump,
                           const NextHeadArgs *next, void *workspace, size_t workspace_bytes, void *stream,
                           const JoinCall *jc = nullptr)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    Geometry g;
    if (!h || !e3 || !e3_exp || !w || !e4 || !e4_exp) return EOQ_ERR_BAD_ARG;
    int st = check_desc(desc, &g);
    if (st != EOQ_OK) return st;
    if (!aligned16(e3) || !aligned16(w) || !aligned16(e4) || !aligned16(acc_dump)) return EOQ_ERR_ALIGNMENT;
    if (desc->c_in % 16) return EOQ_ERR_UNSUPPORTED;  // 8 channels exist for the network input, which takes no error
    if (next) {
        if (!next->mask || !next->gamma || !next->e3 || !next->e3_exp) return EOQ_ERR_BAD_ARG;
        if (!aligned16(next->e3) || (next->x2 && !aligned16(next->x2)) || (reinterpret_cast<uintptr_t>(next->mask) & 1))
            return EOQ_ERR_ALIGNMENT;
        // the compact sums of a strided 1x1 filter are not laid out like the error tensor
        if (desc->kh == 1 && desc->kw == 1 && desc->pad == 0 && desc->stride > 1) return EOQ_ERR_UNSUPPORTED;
    }
    JoinStatArgs jstat{};
    const JoinStatArgs *jstat_p = nullptr;
    if (jc) {
        if (!jc->b || !jc->b_exp || !jc->out || !jc->out_exp || (g.in_elems % 16)) return EOQ_ERR_BAD_ARG;
        if (!aligned16(jc->b) || !aligned16(jc->out) || (reinterpret_cast<uintptr_t>(jc->mask_b) & 1)) return EOQ_ERR_ALIGNMENT;
        if (jc->next) {
            if (!jc->next->mask || !jc->next->gamma || !jc->next->e3 || !jc->next->e3_exp) return EOQ_ERR_BAD_ARG;
            if (!aligned16(jc->next->e3) || (jc->next->x2 && !aligned16(jc->next->x2)) ||
                (reinterpret_cast<uintptr_t>(jc->next->mask) & 1))
                return EOQ_ERR_ALIGNMENT;
        }
        if (desc->kh == 1 && desc->kw == 1 && desc->pad == 0 && desc->stride > 1) return EOQ_ERR_UNSUPPORTED;
        if (!h->hook.fn) {   // with replicas the join runs as its own two passes, each followed by its exchange
            jstat = JoinStatArgs{jc->b, jc->b_exp, jc->mask_b, jc->next ? jc->next->mask : nullptr};
            jstat_p = &jstat;
        }
    }
    // what follows Q_e when a join was asked for
    auto join_after = [&](cudaError_t e, cudaStream_t st) -> int {
        if (e != cudaSuccess || !jc) return record(h, e);
        ProfScope prof(h, EOQ_PROF_GLUE, st);
        if (jstat_p) {
            count_launches(h, 1);
            return record(h, launch_join_second(e4, e4_exp, jc->b, jc->b_exp, jc->mask_b, g.in_elems, jc->out, jc->out_exp, jc->sum_out,
                                                jc->next, h->dev, h->sm_count, st));
        }
        count_launches(h, 2);
        const NextHeadArgs *n = jc->next;
        return record(h, launch_join(e4, e4_exp, jc->b, jc->b_exp, jc->mask_b, g.in_elems, jc->out, jc->out_exp, jc->sum_out,
                                     n ? n->mask : nullptr, n ? n->x2 : nullptr, n ? n->gamma : nullptr, n ? n->e3 : nullptr,
                                     n ? n->e3_exp : nullptr, n ? n->sum_e1 : nullptr, n ? n->sum_e1x2 : nullptr, h->dev, h->sm_count,
                                     st, h->hook));
    };
    if ((st = check_workspace(desc, EOQ_PASS_DGRAD, workspace, workspace_bytes)) != EOQ_OK) return st;
    const eoq_conv_desc_t &d = *desc;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);

    int8_t *wt = reinterpret_cast<int8_t *>(workspace);
    int32_t *sums = acc_dump ? acc_dump : reinterpret_cast<int32_t *>(reinterpret_cast<char *>(workspace) + round256(g.w_elems));
    cudaError_t e;

    // One GEMM per residue class (y mod stride, x mod stride) of the input pixels: within a class the taps
    // kh with (y + pad - kh) divisible by the stride form a unit-stride correlation over e3.
    if (d.stride == 1 && d.kh == d.kw && d.kh - 1 - d.pad >= 0) {
        // stride 1: one correlation of e3 with the flipped filter, padding k - 1 - pad
        IgemmParams p;
        memset(&p, 0, sizeof(p));
        PatchPlan pl;
        memset(&pl, 0, sizeof(pl));
        if (plan_patch(p, pl, d.n, d.c_out, d.h, d.w, d.kh, d.kh - 1 - d.pad, d.c_in, h->sm_count)) {
            for (int a = 0; a < d.kh; ++a)
                for (int b = 0; b < d.kw; ++b) p.tap_b[a * d.kw + b] = (unsigned char)((d.kh - 1 - a) * d.kw + (d.kw - 1 - b));
            p.out_h = d.h;
            p.out_w = d.w;
            p.out_step = 1;
            p.epilogue = kEpiDgrad;
            p.acc_out = sums;
            p.dev = h->dev;
            p.next_mask = next ? next->mask : nullptr;
            // the weights are read where they are, [c_out][tap][c_in]: the reduction (c_out) is their slow axis, so
            // they reach the MMA as MN-major atoms of b_row input channels
            p.b_mn = 1;
            p.b_row = chunk_bytes(p.tile_n);
            CUtensorMap map_a, map_b;
            if (!make_patch_map(&map_a, e3, d.n, g.ho, g.wo, d.c_out, p.kc, pl.pw, pl.r_rows + d.kh - 1) ||
                !make_weight_map(&map_b, w, d.c_out, g.taps, d.c_in, p.b_row, p.kc))
                return EOQ_ERR_UNSUPPORTED;
            const int ptiles = p.num_m_tiles * p.num_n_tiles;
            count_launches(h, 1);
            {
                ProfScope prof(h, EOQ_PROF_IGEMM_DGRAD, s);
                e = launch_igemm_patch(p, pl, map_a, map_b, persistent_grid(ptiles, h->gemm_ctas), s);
            }
            if (e != cudaSuccess || h->gemm_only) return record(h, e);
            {
                ProfScope prof(h, EOQ_PROF_DGRAD_AUX, s);
                e = launch_sq_i32(sums, e3_exp, -7, g.in_elems, e4, e4_exp, reinterpret_cast<long long *>(sum_e4), true,
                                  h->dev, h->sm_count, s, h->hook, next, jstat_p);
            }
            count_launches(h, 1);
            return join_after(e, s);
        }
    }
    // With at least 32 output channels per K chunk the per-class GEMMs read the weights in place as MN-major atoms
    // (as the patch kernel does); narrower layers read a K-major transposed copy [c_in][tap][c_out].
    const bool weights_in_place = d.c_out % 32 == 0;
    if (!weights_in_place) {
        {
            ProfScope prof(h, EOQ_PROF_DGRAD_AUX, s);
            e = launch_weight_transpose(w, wt, d.c_out, g.taps, d.c_in, s);
        }
        if (e != cudaSuccess) return record(h, e);
        count_launches(h, 1);
    }
    // a class no tap reaches (e.g. the odd pixels of a strided 1x1 filter) keeps zero sums: clear first
    bool any_empty = false;
    for (int r = 0; r < d.stride; ++r) {
        bool hit_h = false, hit_w = false;
        for (int kh = 0; kh < d.kh; ++kh) hit_h |= (r + d.pad - kh) % d.stride == 0;
        for (int kw = 0; kw < d.kw; ++kw) hit_w |= (r + d.pad - kw) % d.stride == 0;
        any_empty |= (r < d.h && !hit_h) || (r < d.w && !hit_w);
    }
    // A strided 1x1 filter without padding reaches only the pixels on the stride grid: its one GEMM leaves compact
    // sums [n][hq][wq][c_in] and Q_e scatters them into the full tensor (zeros elsewhere), so nothing is cleared.
    const bool compact = d.kh == 1 && d.kw == 1 && d.pad == 0 && d.stride > 1 && !acc_dump &&
                         (size_t)d.n * d.h * d.w * (d.c_in / 16) <= 0xffffffffull;
    if (any_empty && !compact) {
        e = cudaMemsetAsync(sums, 0, g.in_elems * sizeof(int32_t), s);
        if (e != cudaSuccess) return record(h, e);
    }
    // The classes write disjoint pixels, so their GEMMs are independent: with more than one class and branch streams
    // at hand they are issued side by side (fork on `s`, one stream per class, joins before Q_e), each with a
    // share of the CTAs in proportion to its taps, instead of one after the other at full width.
    int total_taps = 0, live_classes = 0;
    for (int py = 0; py < d.stride && py < d.h; ++py)
        for (int px = 0; px < d.stride && px < d.w; ++px) {
            int nh = 0, nw = 0;
            for (int kh = 0; kh < d.kh; ++kh) nh += (py + d.pad - kh) % d.stride == 0;
            for (int kw = 0; kw < d.kw; ++kw) nw += (px + d.pad - kw) % d.stride == 0;
            total_taps += nh * nw;
            live_classes += nh * nw > 0;
        }
    // (worth it only while a class alone cannot keep the device busy for more than a wave of tiles)
    const long long class_tiles = ((long long)d.n * ((d.h + d.stride - 1) / d.stride) * ((d.w + d.stride - 1) / d.stride) +
                                   kTileM - 1) / kTileM * ((d.c_in + 255) / 256);
    const bool side_by_side = live_classes > 1 && h->class_branch[0] != nullptr && class_tiles <= h->gemm_ctas;
    // timed as one group on `s` (fork to join): the brackets of kernels that run side by side would overlap
    ProfScope *group = side_by_side ? new (std::nothrow) ProfScope(h, EOQ_PROF_IGEMM_DGRAD, s) : nullptr;
    struct GroupEnd {
        ProfScope *&g;
        ~GroupEnd() { delete g; }
    } group_end{group};
    if (side_by_side) {
        e = cudaEventRecord(h->fork_ev, s);
        if (e != cudaSuccess) return record(h, e);
    }
    int class_no = 0;
    unsigned joins = 0;
    for (int py = 0; py < d.stride && py < d.h; ++py)
        for (int px = 0; px < d.stride && px < d.w; ++px) {
            IgemmParams p;
            memset(&p, 0, sizeof(p));
            int dh[16], dw[16], kh_of[16], kw_of[16], nh = 0, nw = 0, min_h = 0, min_w = 0;
            for (int kh = 0; kh < d.kh; ++kh)
                if ((py + d.pad - kh) % d.stride == 0) {
                    // floor division is exact here; negative quotients are rows above the image
                    dh[nh] = (py + d.pad - kh) / d.stride;
                    kh_of[nh] = kh;
                    if (dh[nh] < min_h) min_h = dh[nh];
                    ++nh;
                }
            for (int kw = 0; kw < d.kw; ++kw)
                if ((px + d.pad - kw) % d.stride == 0) {
                    dw[nw] = (px + d.pad - kw) / d.stride;
                    kw_of[nw] = kw;
                    if (dw[nw] < min_w) min_w = dw[nw];
                    ++nw;
                }
            const int hq = (d.h - py + d.stride - 1) / d.stride, wq = (d.w - px + d.stride - 1) / d.stride;
            if (nh == 0 || nw == 0) continue;  // no tap reaches this class: its sums stay zero
            p.M = d.n * hq * wq;
            p.N = d.c_in;
            p.hq = hq;
            p.wq = wq;
            plan_igemm(p, d.c_out, nh * nw, h->sm_count);
            p.src_stride = 1;
            p.src_stride_w = 1;
            p.base_h = min_h;
            p.base_w = min_w;
            for (int a = 0; a < nh; ++a)
                for (int b = 0; b < nw; ++b) {
                    const int t = a * nw + b;
                    if (dh[a] - min_h > 255 || dw[b] - min_w > 255) return EOQ_ERR_UNSUPPORTED;
                    p.tap_dh[t] = (unsigned char)(dh[a] - min_h);
                    p.tap_dw[t] = (unsigned char)(dw[b] - min_w);
                    p.tap_b[t] = (unsigned char)(kh_of[a] * d.kw + kw_of[b]);
                }
            p.out_h = compact ? hq : d.h;
            p.out_w = compact ? wq : d.w;
            p.out_step = compact ? 1 : d.stride;
            p.out_off_h = py;
            p.out_off_w = px;
            p.epilogue = kEpiDgrad;
            p.acc_out = sums;
            p.dev = h->dev;
            p.next_mask = next ? next->mask : nullptr;
            CUtensorMap map_a, map_b;
            if (weights_in_place) {
                p.b_mn = 1;
                p.b_row = chunk_bytes(p.tile_n);
            }
            if (!make_im2col_map(&map_a, e3, d.n, g.ho, g.wo, d.c_out, min_w, min_h, wq, hq, 1, p.kc, kTileM) ||
                !(weights_in_place ? make_weight_map(&map_b, w, d.c_out, g.taps, d.c_in, p.b_row, p.kc)
                                   : make_weight_map(&map_b, wt, d.c_in, g.taps, d.c_out, p.kc, p.tile_n)))
                return EOQ_ERR_UNSUPPORTED;
            const int tiles = p.num_m_tiles * p.num_n_tiles;
            count_launches(h, 1);
            cudaStream_t cs = s;
            int ctas = h->gemm_ctas;
            if (side_by_side) {
                ctas = (int)((long long)h->gemm_ctas * (nh * nw) / total_taps);
                if (ctas < 1) ctas = 1;
                if (class_no > 0) {
                    const int k = (class_no - 1) % kClassBranches;
                    cs = h->class_branch[k];
                    // a stream that already carries a class of this call simply queues the next one behind it
                    if (!(joins & (1u << k))) e = cudaStreamWaitEvent(cs, h->fork_ev, 0);
                    if (e != cudaSuccess) return record(h, e);
                    joins |= 1u << k;
                }
            }
            ++class_no;
            if (side_by_side) {
                e = launch_igemm(p, map_a, map_b, persistent_grid(tiles, ctas), cs);
            } else {
                ProfScope prof(h, EOQ_PROF_IGEMM_DGRAD, cs);
                e = launch_igemm(p, map_a, map_b, persistent_grid(tiles, ctas), cs);
            }
            if (e != cudaSuccess) {
                launch_reset_cells(h->dev, s);  // GEMMs already queued have touched the maximum cell
                return record(h, e);
            }
        }
    for (int k = 0; k < kClassBranches; ++k)
        if (joins & (1u << k)) {
            e = cudaEventRecord(h->class_join[k], h->class_branch[k]);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(s, h->class_join[k], 0);
            if (e != cudaSuccess) return record(h, e);
        }
    delete group;  // closes the group's bracket on `s`, behind the joins
    group = nullptr;
    if (h->gemm_only) return EOQ_OK;
    // Q_e over the whole tensor: the maximum is complete only now
    {
        ProfScope prof(h, EOQ_PROF_DGRAD_AUX, s);
        if (compact)
            e = launch_sq_i32_scatter(sums, e3_exp, -7, d.n, d.h, d.w, d.c_in, d.stride, (d.h + d.stride - 1) / d.stride,
                                      (d.w + d.stride - 1) / d.stride, e4, e4_exp, reinterpret_cast<long long *>(sum_e4),
                                      h->dev, h->sm_count, s, h->hook);
        else
            e = launch_sq_i32(sums, e3_exp, -7, g.in_elems, e4, e4_exp, reinterpret_cast<long long *>(sum_e4), true, h->dev,
                              h->sm_count, s, h->hook, next, jstat_p);
    }
    count_launches(h, 1);
    return join_after(e, s);
}

extern "C" int eoq_conv_dgrad(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *e3,
                              const int32_t *e3_exp, const int8_t *w, int8_t *e4, int32_t *e4_exp, int64_t *sum_e4,
                              int32_t *acc_dump, void *workspace, size_t workspace_bytes, void *stream)
{
    return conv_dgrad_impl(handle, desc, e3, e3_exp, w, e4, e4_exp, sum_e4, acc_dump, nullptr, workspace, workspace_bytes, stream);
}

extern "C" int eoq_conv_dgrad_join_head(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *e3, const int32_t *e3_exp,
                                        const int8_t *w, int8_t *e4, int32_t *e4_exp, int64_t *sum_e4, const int8_t *b,
                                        const int32_t *b_exp, const uint8_t *mask_b, int8_t *out, int32_t *out_exp, int64_t *sum_out,
                                        const uint8_t *next_relu_mask, const int16_t *next_x2, const int32_t *next_gamma,
                                        int8_t *next_e3, int32_t *next_e3_exp, int64_t *next_sum_e1, int64_t *next_sum_e1x2,
                                        void *workspace, size_t workspace_bytes, void *stream)
{
    const NextHeadArgs next{next_relu_mask, next_x2, next_gamma, next_e3, next_e3_exp, reinterpret_cast<long long *>(next_sum_e1),
                            reinterpret_cast<long long *>(next_sum_e1x2)};
    const JoinCall jc{b, b_exp, mask_b, out, out_exp, reinterpret_cast<long long *>(sum_out), next_relu_mask ? &next : nullptr};
    return conv_dgrad_impl(handle, desc, e3, e3_exp, w, e4, e4_exp, sum_e4, nullptr, nullptr, workspace, workspace_bytes, stream, &jc);
}

extern "C" int eoq_conv_dgrad_head(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *e3, const int32_t *e3_exp,
                                   const int8_t *w, int8_t *e4, int32_t *e4_exp, int64_t *sum_e4, const uint8_t *next_relu_mask,
                                   const int16_t *next_x2, const int32_t *next_gamma, int8_t *next_e3, int32_t *next_e3_exp,
                                   int64_t *next_sum_e1, int64_t *next_sum_e1x2, void *workspace, size_t workspace_bytes,
                                   void *stream)
{
    const NextHeadArgs next{next_relu_mask, next_x2, next_gamma, next_e3, next_e3_exp, reinterpret_cast<long long *>(next_sum_e1),
                            reinterpret_cast<long long *>(next_sum_e1x2)};
    return conv_dgrad_impl(handle, desc, e3, e3_exp, w, e4, e4_exp, sum_e4, nullptr, &next, workspace, workspace_bytes, stream);
}

// ================================================================================= weight gradient

// The b1 tap sums (one pass over e3), in front of the weight-gradient GEMM on the same stream.  (Issued on a second
// stream "beside" the GEMM they gain nothing: a GEMM CTA fills its SM, so the blocks of this kernel only start as
// the GEMM's CTAs leave, and the call pays for a fork and a join on top.)
static cudaError_t launch_tap_sums(Handle *h, const int8_t *e3, long long *tap_sums, size_t tap_bytes,
                                   const eoq_conv_desc_t &d, int ho, int wo, const BorderClasses &bc, cudaStream_t s)
{
    const size_t tap_stride = tap_bytes / kTapReplicas / sizeof(long long);
    count_launches(h, 1);
    ProfScope prof(h, EOQ_PROF_WGRAD_TAPS, s);
    cudaError_t e = cudaMemsetAsync(tap_sums, 0, tap_bytes, s);  // the kernel adds into them
    return e != cudaSuccess ? e : launch_b1_error_sums(e3, tap_sums, tap_stride, d, ho, wo, bc, h->sm_count, s);
}

// Weight gradient behind eoq_conv_wgrad and eoq_conv_wgrad_dev: b1 is the host code b1_c, or the code at b1_dev.
// num_parts_out (eoq_conv_wgrad_gemm): the GEMM alone; the sums stay in the workspace for eoq_wgrad_finish and
// *num_parts_out tells it how many int32 slices there are (0: the GEMM added into the int64 sums).
static int conv_wgrad_impl(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *e3, const int32_t *e3_exp,
                           const int8_t *x, int32_t b1_c, const int32_t *b1_dev, int8_t *gq, int32_t *g_exp,
                           int64_t *acc_dump, void *workspace, size_t workspace_bytes, void *stream, int *num_parts_out = nullptr)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    Geometry g;
    const bool gemm_only = num_parts_out != nullptr || (h && h->gemm_only);
    if (!h || !e3 || !e3_exp || !x || (!num_parts_out && (!gq || !g_exp))) return EOQ_ERR_BAD_ARG;
    int st = check_desc(desc, &g);
    if (st != EOQ_OK) return st;
    if (!aligned16(e3) || !aligned16(x) || !aligned16(gq) || !aligned16(acc_dump)) return EOQ_ERR_ALIGNMENT;
    if (b1_c < -32768 || b1_c > 32767) return EOQ_ERR_RANGE;
    if ((st = check_workspace(desc, EOQ_PASS_WGRAD, workspace, workspace_bytes)) != EOQ_OK) return st;
    const eoq_conv_desc_t &d = *desc;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);

    // workspace: [tap sums][256 spare bytes][int64 sums][split-K slices]
    const BorderClasses bc = border_classes(d, g);
    const bool use_b1 = b1_dev != nullptr || b1_c != 0;  // a device-resident b1 may be anything: its term is always formed
    if (use_b1 && bc.nrc * bc.ncc > kMaxBorderClasses) return EOQ_ERR_UNSUPPORTED;
    char *ws = reinterpret_cast<char *>(workspace);
    long long *tap_sums = reinterpret_cast<long long *>(ws);
    const size_t tap_stride = round256((size_t)d.c_out * g.taps * sizeof(long long)) / sizeof(long long);  // one copy, in elements
    const size_t tap_bytes = kTapReplicas * tap_stride * sizeof(long long);
    long long *acc = reinterpret_cast<long long *>(ws + tap_bytes + 256);
    const size_t acc_bytes = round256(g.w_elems * sizeof(long long));

    WgradPatchPlan wp;
    if (plan_wgrad_patch(wp, d, g.ho, g.wo, h->gemm_ctas < kWgradTargetCtas ? h->gemm_ctas : kWgradTargetCtas)) {
        wp.partials = reinterpret_cast<int32_t *>(ws + tap_bytes + 256 + acc_bytes);
        wp.dev = h->dev;
        cudaError_t e;
        if (gemm_only) {
            CUtensorMap mx, me;
            if (!make_patch_map(&mx, x, d.n, d.h, d.w, d.c_in, wp.kc, wp.pw, wp.r_rows + d.kh - 1) ||
                !make_patch_map(&me, e3, d.n, g.ho, g.wo, d.c_out, wp.tile_n, wp.pw, wp.r_rows))
                return EOQ_ERR_UNSUPPORTED;
            count_launches(h, 1);
            if (num_parts_out) *num_parts_out = wp.num_splits;
            ProfScope prof(h, EOQ_PROF_WGRAD, s);
            return record(h, launch_wgrad_patch(wp, mx, me, s));
        }
        e = use_b1 ? launch_tap_sums(h, e3, tap_sums, tap_bytes, d, g.ho, g.wo, bc, s) : cudaSuccess;
        if (e != cudaSuccess) return record(h, e);
        CUtensorMap map_x, map_e;
        if (!make_patch_map(&map_x, x, d.n, d.h, d.w, d.c_in, wp.kc, wp.pw, wp.r_rows + d.kh - 1) ||
            !make_patch_map(&map_e, e3, d.n, g.ho, g.wo, d.c_out, wp.tile_n, wp.pw, wp.r_rows))
            return EOQ_ERR_UNSUPPORTED;
        count_launches(h, 1);
        {
            ProfScope prof(h, EOQ_PROF_WGRAD, s);
            e = launch_wgrad_patch(wp, map_x, map_e, s);
        }
        if (e != cudaSuccess) return record(h, e);
        ProfScope prof_q(h, EOQ_PROF_WGRAD_AUX, s);
        e = launch_sq_i64(acc, e3_exp, -7, g.w_elems, gq, g_exp, reinterpret_cast<long long *>(acc_dump),
                          use_b1 ? tap_sums : nullptr, tap_stride, b1_c, b1_dev, d.c_in, wp.partials, wp.num_splits, h->dev, h->sm_count, s, h->hook);
        count_launches(h, 2);
        return record(h, e);
    }

    WgradParams p;
    memset(&p, 0, sizeof(p));
    p.P = d.n * g.ho * g.wo;
    p.ho = g.ho;
    p.wo = g.wo;
    p.c_in = d.c_in;
    p.c_out = d.c_out;
    p.ntaps = g.taps;
    const bool row_window = use_row_window(d, g.wo);
    if (d.c_in == 8 && !row_window) return EOQ_ERR_UNSUPPORTED;
    const int w_mem = d.w + 2 * d.x_wmargin;
    p.kc = row_window ? 8 * d.c_in : chunk_bytes(d.c_in);
    p.nc = chunk_bytes(d.c_out);
    p.chunks_per_tap = row_window ? 1 : d.c_in / p.kc;
    p.rows_total = g.taps * d.c_in;
    p.subs_per_mtile = kTileM / p.kc;
    // filter-row path: a filter row is 8 taps x c_in rows, 128 / (8 c_in) filter rows per M tile
    p.num_m_tiles = row_window ? (d.kh * p.kc + kTileM - 1) / kTileM : (p.rows_total + kTileM - 1) / kTileM;
    if (row_window) {
        p.ntaps = d.kh;
        p.row_window_kw = d.kw;
    }
    p.tile_n = d.c_out < 256 ? d.c_out : 256;
    if (p.tile_n % p.nc) p.tile_n = (p.tile_n / p.nc) * p.nc;
    p.num_n_tiles = (d.c_out + p.tile_n - 1) / p.tile_n;
    p.pixels_per_stage = 64;
    // M tiles accumulated side by side by one CTA share the stage's error tile (fewer TMA rows per MMA): as many
    // as tensor memory (512 columns) and three pipeline stages of shared memory allow
    {
        int mpc = 512 / p.tile_n;
        const size_t a_mtile = (size_t)p.subs_per_mtile * p.pixels_per_stage * p.kc, b_tile = (size_t)p.tile_n * p.pixels_per_stage;
        while (mpc > 1 && 3 * (mpc * a_mtile + b_tile) > 200 * 1024) --mpc;
        if (mpc > p.num_m_tiles) mpc = p.num_m_tiles;
        p.mtiles_per_cta = mpc < 1 ? 1 : mpc;
        p.num_m_groups = (p.num_m_tiles + p.mtiles_per_cta - 1) / p.mtiles_per_cta;
    }
    const int total_stages = (p.P + p.pixels_per_stage - 1) / p.pixels_per_stage;
    // a 64-pixel stage adds at most 64 * 127 * 255 to an int32 partial sum: cap the stages one CTA runs
    const int max_stages_exact = 1024;
    const int tiles = p.num_m_groups * p.num_n_tiles;
    int splits = (2 * h->gemm_ctas + tiles - 1) / tiles;
    const int max_splits = (total_stages + 7) / 8;  // at least 8 stages of work per CTA
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
    int per = (total_stages + splits - 1) / splits;
    if (per > max_stages_exact) per = max_stages_exact;
    splits = (total_stages + per - 1) / per;
    p.stages_per_split = per;
    p.num_k_splits = splits;
    const size_t stage_bytes = (size_t)p.mtiles_per_cta * p.subs_per_mtile * p.pixels_per_stage * p.kc +
                               (size_t)p.tile_n * p.pixels_per_stage;
    int stages = (int)((200 * 1024) / stage_bytes);
    p.num_stages = stages > 8 ? 8 : (stages < 2 ? 2 : stages);
    p.src_stride = d.stride;
    p.base_h = -d.pad;
    if (row_window) {
        p.src_stride_w = 1;
        p.base_w = 0;
        for (int t = 0; t < d.kh; ++t) {
            p.tap_dh[t] = (unsigned char)t;
            p.tap_dw[t] = 0;
        }
    } else {
        p.src_stride_w = d.stride;
        p.base_w = d.x_wmargin - d.pad;
        for (int t = 0; t < g.taps; ++t) {
            p.tap_dh[t] = (unsigned char)(t / d.kw);
            p.tap_dw[t] = (unsigned char)(t % d.kw);
        }
    }
    p.acc = acc;
    p.dev = h->dev;

    cudaError_t e = cudaSuccess;
    if (!h->gemm_only) {
        ProfScope aux(h, EOQ_PROF_WGRAD_AUX, s);
        e = cudaMemsetAsync(acc, 0, acc_bytes, s);  // the GEMM adds into the int64 sums with atomics
    }
    if (e == cudaSuccess && use_b1 && !gemm_only) e = launch_tap_sums(h, e3, tap_sums, tap_bytes, d, g.ho, g.wo, bc, s);
    if (e != cudaSuccess) return record(h, e);
    CUtensorMap map_x, map_e;
    if (!make_matrix_map(&map_e, e3, (size_t)p.P, d.c_out, p.nc, p.pixels_per_stage)) return EOQ_ERR_UNSUPPORTED;
    if (row_window ? !make_row_window_map(&map_x, x, d.n, d.h, w_mem, d.c_in, d.x_wmargin - d.pad, g.wo, g.ho, d.stride, d.pad,
                                          p.pixels_per_stage)
                   : !make_im2col_map(&map_x, x, d.n, d.h, w_mem, d.c_in, d.x_wmargin - d.pad, -d.pad, g.wo, g.ho, d.stride,
                                      p.kc, p.pixels_per_stage))
        return EOQ_ERR_UNSUPPORTED;
    count_launches(h, 1);
    {
        ProfScope prof(h, EOQ_PROF_WGRAD, s);
        e = launch_wgrad(p, map_x, map_e, s);
    }
    if (num_parts_out) *num_parts_out = 0;
    if (e != cudaSuccess || gemm_only) return record(h, e);
    // the kernel leaves sums as [oc][tap][ic], which is the layout of g
    ProfScope prof_q(h, EOQ_PROF_WGRAD_AUX, s);
    e = launch_sq_i64(acc, e3_exp, -7, g.w_elems, gq, g_exp, reinterpret_cast<long long *>(acc_dump),
                      use_b1 ? tap_sums : nullptr, tap_stride, b1_c, b1_dev, d.c_in, nullptr, 0, h->dev, h->sm_count, s, h->hook);
    count_launches(h, 2);
    return record(h, e);
}

extern "C" int eoq_conv_wgrad(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *e3,
                              const int32_t *e3_exp, const int8_t *x, int32_t b1_c, int8_t *gq, int32_t *g_exp,
                              int64_t *acc_dump, void *workspace, size_t workspace_bytes, void *stream)
{
    return conv_wgrad_impl(handle, desc, e3, e3_exp, x, b1_c, nullptr, gq, g_exp, acc_dump, workspace, workspace_bytes, stream);
}

extern "C" int eoq_conv_wgrad_dev(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *e3,
                                  const int32_t *e3_exp, const int8_t *x, const int32_t *b1_c, int8_t *gq, int32_t *g_exp,
                                  void *workspace, size_t workspace_bytes, void *stream)
{
    // b1_c null: the layer has no bias in front of its convolution (the first layer of a network)
    return conv_wgrad_impl(handle, desc, e3, e3_exp, x, 0, b1_c, gq, g_exp, nullptr, workspace, workspace_bytes, stream);
}

extern "C" int eoq_conv_wgrad_gemm(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *e3, const int32_t *e3_exp,
                                   const int8_t *x, void *workspace, size_t workspace_bytes, int *num_parts, void *stream)
{
    if (!num_parts) return EOQ_ERR_BAD_ARG;
    return conv_wgrad_impl(handle, desc, e3, e3_exp, x, 0, nullptr, nullptr, nullptr, nullptr, workspace, workspace_bytes, stream,
                           num_parts);
}

extern "C" int eoq_wgrad_finish(eoq_handle_t handle, int num, const eoq_conv_desc_t *descs, const int8_t *const *e3,
                                const int32_t *const *e3_exp, const int32_t *const *b1_c, int8_t *const *gq, int32_t *const *g_exp,
                                void *const *workspace, const size_t *workspace_bytes, const int *num_parts, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || num <= 0 || !descs || !e3 || !e3_exp || !b1_c || !gq || !g_exp || !workspace || !workspace_bytes || !num_parts)
        return EOQ_ERR_BAD_ARG;
    if (h->hook.fn) return EOQ_ERR_UNSUPPORTED;  // replicas exchange per layer: eoq_conv_wgrad_dev
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    for (int i = 0; i < num; ++i) {
        Geometry g;
        int st = check_desc(&descs[i], &g);
        if (st != EOQ_OK) return st;
        if (!e3[i] || !e3_exp[i] || !gq[i] || !g_exp[i] || num_parts[i] < 0) return EOQ_ERR_BAD_ARG;
        if (!aligned16(e3[i]) || !aligned16(gq[i])) return EOQ_ERR_ALIGNMENT;
        if ((st = check_workspace(&descs[i], EOQ_PASS_WGRAD, workspace[i], workspace_bytes[i])) != EOQ_OK) return st;
        const BorderClasses bc = border_classes(descs[i], g);
        if (b1_c[i] && bc.nrc * bc.ncc > kMaxBorderClasses) return EOQ_ERR_UNSUPPORTED;
    }
    for (int base = 0; base < num; base += kFinishChunk) {
        FinishBatch b;
        memset(&b, 0, sizeof(b));
        b.num = num - base < kFinishChunk ? num - base : kFinishChunk;
        for (int k = 0; k < b.num; ++k) {
            const eoq_conv_desc_t &d = descs[base + k];
            Geometry g;
            check_desc(&d, &g);
            FinishItem &it = b.item[k];
            // the workspace as eoq_conv_wgrad_gemm laid it out: [tap sums][256 spare bytes][int64 sums][split-K slices]
            char *ws = reinterpret_cast<char *>(workspace[base + k]);
            const size_t tap_stride = round256((size_t)d.c_out * g.taps * sizeof(long long)) / sizeof(long long);
            const size_t tap_bytes = kTapReplicas * tap_stride * sizeof(long long);
            const size_t acc_bytes = round256(g.w_elems * sizeof(long long));
            it.e3 = e3[base + k];
            it.e3_exp = e3_exp[base + k];
            it.b1_dev = b1_c[base + k];
            it.tap_sums = reinterpret_cast<long long *>(ws);
            it.tap_stride = tap_stride;
            it.zero_bytes = tap_bytes + 256;
            it.max_cell = reinterpret_cast<unsigned long long *>(ws + tap_bytes);
            it.acc = reinterpret_cast<long long *>(ws + tap_bytes + 256);
            it.num_parts = num_parts[base + k];
            it.parts = it.num_parts > 0 ? reinterpret_cast<const int32_t *>(ws + tap_bytes + 256 + acc_bytes) : nullptr;
            it.g = gq[base + k];
            it.g_exp = g_exp[base + k];
            it.n = g.w_elems;
            it.pixels = (unsigned long long)d.n * g.ho * g.wo;
            it.d = d;
            it.bc = border_classes(d, g);
            it.ho = g.ho;
            it.wo = g.wo;
            plan_finish_item(it, h->sm_count);
            b.tap_first[k + 1] = b.tap_first[k] + it.tap_grid_x * it.tap_grid_y;
            b.fin_first[k + 1] = b.fin_first[k] + it.fin_blocks;
            b.sq_first[k + 1] = b.sq_first[k] + it.sq_blocks;
        }
        ProfScope prof(h, EOQ_PROF_WGRAD_AUX, s);
        const cudaError_t e = launch_wgrad_finish(b, &h->dev->status, s);
        count_launches(h, 4);
        if (e != cudaSuccess) return record(h, e);
    }
    return EOQ_OK;
}

// ================================================================================= tensor-pipe probe

extern "C" int eoq_probe_mma_i8(eoq_handle_t handle, int n_cols, int iters, int launches, double *tops,
                                double *cycles_per_mma, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || !tops || n_cols < 16 || n_cols > 256 || (n_cols % 16) || iters < 1 || iters > (1 << 20) || launches < 1 ||
        launches > 100000)
        return EOQ_ERR_BAD_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    cudaEvent_t a = nullptr, b = nullptr;
    cudaError_t e = cudaEventCreate(&a);
    if (e == cudaSuccess) e = cudaEventCreate(&b);
    unsigned long long *cyc = &h->dev->probe_cycles;
    if (e == cudaSuccess) e = launch_probe_mma_i8(n_cols, iters, h->sm_count, h->dev, cyc, s);  // warm-up
    if (e == cudaSuccess) e = cudaMemsetAsync(cyc, 0, sizeof(unsigned long long), s);
    if (e == cudaSuccess) e = cudaEventRecord(a, s);
    for (int i = 0; i < launches && e == cudaSuccess; ++i) e = launch_probe_mma_i8(n_cols, iters, h->sm_count, h->dev, cyc, s);
    if (e == cudaSuccess) e = cudaEventRecord(b, s);
    if (e == cudaSuccess) e = cudaEventSynchronize(b);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, a, b);
    unsigned long long cycles = 0;
    if (e == cudaSuccess) e = cudaMemcpy(&cycles, cyc, sizeof(cycles), cudaMemcpyDeviceToHost);
    if (a) cudaEventDestroy(a);
    if (b) cudaEventDestroy(b);
    if (e != cudaSuccess) return record(h, e);
    count_launches(h, launches + 1);
    const double ops = 2.0 * kTileM * n_cols * 32.0 * 4.0 * iters * (double)h->sm_count * launches;
    *tops = ms > 0.f ? ops / (ms * 1e-3) / 1e12 : 0.0;
    if (cycles_per_mma) *cycles_per_mma = (double)cycles / (4.0 * iters);
    return EOQ_OK;
}

// ================================================================================= plan report

extern "C" int eoq_describe_plan(eoq_handle_t handle, const eoq_conv_desc_t *desc, int pass, char *buf, size_t buf_bytes)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    Geometry g;
    if (!h || !buf || buf_bytes == 0) return EOQ_ERR_BAD_ARG;
    int st = check_desc(desc, &g);
    if (st != EOQ_OK) return st;
    const eoq_conv_desc_t &d = *desc;
    IgemmParams p;
    memset(&p, 0, sizeof(p));
    PatchPlan pl;
    memset(&pl, 0, sizeof(pl));
    buf[0] = 0;
    if (pass == EOQ_PASS_FWD) {
        if (d.stride == 1 && d.kh == d.kw && d.x_wmargin == 0 &&
            plan_patch(p, pl, d.n, d.c_in, g.ho, g.wo, d.kh, d.pad, d.c_out, h->sm_count)) {
            snprintf(buf, buf_bytes, "kernel=igemm_patch tile_n=%d accumulators=%d m_tiles=%d n_tiles=%d weights=%s", p.tile_n,
                     p.tile_n <= 128 ? 2 : 1, p.num_m_tiles, p.num_n_tiles, pl.b_resident ? "resident" : "streamed");
            return EOQ_OK;
        }
        p.M = d.n * g.ho * g.wo;
        p.N = d.c_out;
        const bool rw = use_row_window(d, g.wo);
        plan_igemm(p, rw ? 8 * d.c_in : d.c_in, rw ? d.kh : g.taps, h->sm_count);
        snprintf(buf, buf_bytes, "kernel=igemm%s tile_n=%d m_tiles=%d n_tiles=%d kc=%d stages=%d", rw ? "_filter_rows" : "",
                 p.tile_n, p.num_m_tiles, p.num_n_tiles, p.kc, p.num_stages);
        return EOQ_OK;
    }
    if (pass == EOQ_PASS_DGRAD) {
        if (d.stride == 1 && d.kh == d.kw && d.kh - 1 - d.pad >= 0 &&
            plan_patch(p, pl, d.n, d.c_out, d.h, d.w, d.kh, d.kh - 1 - d.pad, d.c_in, h->sm_count)) {
            snprintf(buf, buf_bytes, "kernel=igemm_patch tile_n=%d accumulators=%d m_tiles=%d n_tiles=%d weights=%s", p.tile_n,
                     p.tile_n <= 128 ? 2 : 1, p.num_m_tiles, p.num_n_tiles, pl.b_resident ? "resident" : "streamed");
            return EOQ_OK;
        }
        const int hq = (d.h + d.stride - 1) / d.stride, wq = (d.w + d.stride - 1) / d.stride;
        p.M = d.n * hq * wq;
        p.N = d.c_in;
        plan_igemm(p, d.c_out, ((d.kh + d.stride - 1) / d.stride) * ((d.kw + d.stride - 1) / d.stride), h->sm_count);
        snprintf(buf, buf_bytes, "kernel=igemm classes=%d tile_n=%d m_tiles=%d n_tiles=%d kc=%d", d.stride * d.stride, p.tile_n,
                 p.num_m_tiles, p.num_n_tiles, p.kc);
        return EOQ_OK;
    }
    if (pass == EOQ_PASS_WGRAD) {
        WgradPatchPlan wp;
        if (plan_wgrad_patch(wp, d, g.ho, g.wo, h->gemm_ctas < kWgradTargetCtas ? h->gemm_ctas : kWgradTargetCtas))
            snprintf(buf, buf_bytes, "kernel=wgrad_patch groups=%d splits=%d tile_n=%d kc=%d", wp.num_groups, wp.num_splits, wp.tile_n,
                     wp.kc);
        else
            snprintf(buf, buf_bytes, "kernel=wgrad%s", use_row_window(d, g.wo) ? "_filter_rows" : "");
        return EOQ_OK;
    }
    return EOQ_ERR_BAD_ARG;
}

// ================================================================================= elementwise entry points

extern "C" int eoq_quantize(eoq_handle_t handle, int mode, const void *src, int src_is_float, const int32_t *src_exp,
                            size_t n, void *dst, int32_t *dst_exp, void *workspace, size_t workspace_bytes,
                            void *stream)
{
    (void)workspace;
    (void)workspace_bytes;
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || !src || !dst || n == 0) return EOQ_ERR_BAD_ARG;
    if (mode != EOQ_Q && mode != EOQ_CQ && mode != EOQ_SQ) return EOQ_ERR_BAD_ARG;
    if (mode == EOQ_SQ && !dst_exp) return EOQ_ERR_BAD_ARG;
    if (!aligned16(src) || !aligned16(dst)) return EOQ_ERR_ALIGNMENT;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    count_launches(h, mode == EOQ_SQ ? 2 : 1);
    ProfScope prof(h, EOQ_PROF_OTHER, s);
    if (src_is_float)
        return record(h, launch_quantize_f32(mode, reinterpret_cast<const float *>(src), n, dst, dst_exp, h->dev, h->sm_count, s, h->hook));
    if (mode != EOQ_SQ || !src_exp) return EOQ_ERR_UNSUPPORTED;
    return record(h, launch_sq_i32(reinterpret_cast<const int32_t *>(src), src_exp, 0, n, reinterpret_cast<int8_t *>(dst),
                                   dst_exp, nullptr, false, h->dev, h->sm_count, s, h->hook));
}

static int err_prescale_impl(eoq_handle_t handle, const int8_t *e0, const int32_t *e0_exp, const uint8_t *relu_mask,
                             const int16_t *x2, size_t n_el, int32_t gamma_c, const int32_t *gamma_dev, int8_t *e3,
                             int32_t *e3_exp, int64_t *sum_e1, int64_t *sum_e1x2, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || !e0 || !e0_exp || !e3 || !e3_exp || n_el == 0 || (n_el % 16)) return EOQ_ERR_BAD_ARG;
    if (!aligned16(e0) || !aligned16(e3) || !aligned16(x2) || (reinterpret_cast<uintptr_t>(relu_mask) & 1)) return EOQ_ERR_ALIGNMENT;
    if (gamma_c < -32768 || gamma_c > 32767) return EOQ_ERR_RANGE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    ProfScope prof(h, EOQ_PROF_ERR_HEAD, s);
    int kernels = 0;
    const bool force_timeout = h->force_timeout;
    h->force_timeout = false;
    const cudaError_t e = launch_err_prescale(e0, e0_exp, relu_mask, x2, n_el, gamma_c, gamma_dev, e3, e3_exp,
                                              reinterpret_cast<long long *>(sum_e1), reinterpret_cast<long long *>(sum_e1x2),
                                              h->dev, h->sm_count, s, &kernels, force_timeout, h->hook);
    count_launches(h, kernels);
    return record(h, e);
}

extern "C" int eoq_err_prescale(eoq_handle_t handle, const int8_t *e0, const int32_t *e0_exp, const uint8_t *relu_mask,
                                const int16_t *x2, size_t n_el, int32_t gamma_c, int8_t *e3, int32_t *e3_exp,
                                int64_t *sum_e1, int64_t *sum_e1x2, void *stream)
{
    return err_prescale_impl(handle, e0, e0_exp, relu_mask, x2, n_el, gamma_c, nullptr, e3, e3_exp, sum_e1, sum_e1x2, stream);
}

extern "C" int eoq_err_prescale_dev(eoq_handle_t handle, const int8_t *e0, const int32_t *e0_exp, const uint8_t *relu_mask,
                                    const int16_t *x2, size_t n_el, const int32_t *gamma_c, int8_t *e3, int32_t *e3_exp,
                                    int64_t *sum_e1, int64_t *sum_e1x2, void *stream)
{
    if (!gamma_c) return EOQ_ERR_BAD_ARG;
    return err_prescale_impl(handle, e0, e0_exp, relu_mask, x2, n_el, 128, gamma_c, e3, e3_exp, sum_e1, sum_e1x2, stream);
}

extern "C" int eoq_debug_force_wait_timeout(eoq_handle_t handle)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h) return EOQ_ERR_BAD_ARG;
    h->force_timeout = true;
    return EOQ_OK;
}

static int update_impl(eoq_handle_t handle, int num, int8_t *const *w, const int8_t *const *g,
                       const int32_t *const *g_exp, const size_t *n, int32_t lr_mant, int32_t lr_exp, int round_mode,
                       uint64_t seed, uint64_t step, uint64_t *step_dev, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || num <= 0 || !w || !g || !g_exp || !n) return EOQ_ERR_BAD_ARG;
    if (num > 256) return EOQ_ERR_UNSUPPORTED;
    if (lr_mant < 1 || lr_mant > 255 || lr_exp < -64 || lr_exp > 64) return EOQ_ERR_RANGE;
    if (round_mode != EOQ_ROUND_RNE && round_mode != EOQ_ROUND_STOCHASTIC) return EOQ_ERR_BAD_ARG;
    UpdateTensor t[256];
    for (int i = 0; i < num; ++i) {
        if (!w[i] || !g[i] || !g_exp[i] || n[i] == 0) return EOQ_ERR_BAD_ARG;
        t[i].w = w[i];
        t[i].g = g[i];
        t[i].g_exp = g_exp[i];
        t[i].n = n[i];
        t[i].master = nullptr;
    }
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    count_launches(h, 2 * ((num + 63) / 64) + (step_dev ? 1 : 0));
    ProfScope prof(h, EOQ_PROF_UPDATE, s);
    return record(h, launch_update(t, num, lr_mant, lr_exp, round_mode == EOQ_ROUND_STOCHASTIC, seed, step,
                                   reinterpret_cast<unsigned long long *>(step_dev), h->dev, h->sm_count, s));
}

extern "C" int eoq_update(eoq_handle_t handle, int num, int8_t *const *w, const int8_t *const *g,
                          const int32_t *const *g_exp, const size_t *n, int32_t lr_mant, int32_t lr_exp,
                          int round_mode, uint64_t seed, uint64_t step, void *stream)
{
    return update_impl(handle, num, w, g, g_exp, n, lr_mant, lr_exp, round_mode, seed, step, nullptr, stream);
}

extern "C" int eoq_update_dev(eoq_handle_t handle, int num, int8_t *const *w, const int8_t *const *g,
                              const int32_t *const *g_exp, const size_t *n, int32_t lr_mant, int32_t lr_exp,
                              int round_mode, uint64_t seed, uint64_t *step, void *stream)
{
    if (!step || (reinterpret_cast<uintptr_t>(step) & 7)) return EOQ_ERR_BAD_ARG;
    return update_impl(handle, num, w, g, g_exp, n, lr_mant, lr_exp, round_mode, seed, 0, step, stream);
}

extern "C" int eoq_update_wide(eoq_handle_t handle, int num, int32_t *const *master, int8_t *const *w, const int8_t *const *g,
                               const int32_t *const *g_exp, const size_t *n, int32_t lr_mant, int32_t lr_exp, int k_u, int k_m,
                               int round_mode, uint64_t seed, uint64_t step, uint64_t *step_dev, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || num <= 0 || !master || !w || !g || !g_exp || !n) return EOQ_ERR_BAD_ARG;
    if (num > 256) return EOQ_ERR_UNSUPPORTED;
    if (lr_mant < 1 || lr_mant > 255 || lr_exp < -64 || lr_exp > 64) return EOQ_ERR_RANGE;
    if (k_u < 2 || k_u > 24 || k_m < 8 || k_m > 24) return EOQ_ERR_UNSUPPORTED;
    if (round_mode != EOQ_ROUND_RNE && round_mode != EOQ_ROUND_STOCHASTIC) return EOQ_ERR_BAD_ARG;
    if (step_dev && (reinterpret_cast<uintptr_t>(step_dev) & 7)) return EOQ_ERR_BAD_ARG;
    UpdateTensor t[256];
    for (int i = 0; i < num; ++i) {
        if (!master[i] || !w[i] || !g[i] || !g_exp[i] || n[i] == 0) return EOQ_ERR_BAD_ARG;
        t[i].w = w[i];
        t[i].g = g[i];
        t[i].g_exp = g_exp[i];
        t[i].n = n[i];
        t[i].master = master[i];
    }
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    count_launches(h, 2 * ((num + 63) / 64) + (step_dev ? 1 : 0));
    ProfScope prof(h, EOQ_PROF_UPDATE, s);
    return record(h, launch_update_wide(t, num, lr_mant, lr_exp, k_u, k_m, round_mode == EOQ_ROUND_STOCHASTIC, seed, step,
                                        reinterpret_cast<unsigned long long *>(step_dev), h->dev, s));
}

extern "C" int eoq_layout_convert(eoq_handle_t handle, const int8_t *src, int8_t *dst, int n, int c, int hh, int ww,
                                  int to_nhwc, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || !src || !dst || n <= 0 || c <= 0 || hh <= 0 || ww <= 0 || n > 65535) return EOQ_ERR_BAD_ARG;
    count_launches(h, 1);
    return record(h, launch_layout_convert(src, dst, n, c, hh, ww, to_nhwc, reinterpret_cast<cudaStream_t>(stream)));
}

extern "C" int eoq_quantize_image(eoq_handle_t handle, const float *src, int n, int hh, int ww, int c_src, int c_dst,
                                  int wmargin, int8_t *dst, int32_t *dst_exp, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || !src || !dst || !dst_exp || n <= 0 || hh <= 0 || ww <= 0 || c_src <= 0 || c_dst < c_src || wmargin < 0 ||
        wmargin > 64)
        return EOQ_ERR_BAD_ARG;
    if ((c_dst % 16 && c_dst != 8) || c_dst > 64 || !aligned16(src) || !aligned16(dst)) return EOQ_ERR_ALIGNMENT;
    count_launches(h, 2);
    ProfScope prof(h, EOQ_PROF_INPUT_Q, reinterpret_cast<cudaStream_t>(stream));
    return record(h, launch_quantize_image(src, n, hh, ww, c_src, c_dst, wmargin, dst, dst_exp, h->dev, h->sm_count,
                                           reinterpret_cast<cudaStream_t>(stream), h->hook));
}

// ================================================================================= network glue

extern "C" int eoq_aux_maxpool_fwd(eoq_handle_t handle, const int8_t *x, int n, int hh, int ww, int c, int k, int stride, int pad,
                                   int8_t *y, uint8_t *arg, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || !x || !y || !arg || n <= 0 || hh <= 0 || ww <= 0 || c <= 0 || k <= 0 || k > 15 || stride <= 0 || pad < 0 || pad >= k)
        return EOQ_ERR_BAD_ARG;
    if (c % 16 || !aligned16(x) || !aligned16(y) || !aligned16(arg)) return EOQ_ERR_ALIGNMENT;
    if ((size_t)n * hh * ww * (c / 16) > 0xffffffffull) return EOQ_ERR_UNSUPPORTED;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    count_launches(h, 1);
    ProfScope prof(h, EOQ_PROF_GLUE, s);
    return record(h, launch_maxpool_fwd(x, n, hh, ww, c, k, stride, pad, y, arg, h->sm_count, s));
}

extern "C" int eoq_aux_maxpool_bwd(eoq_handle_t handle, const int8_t *e, const int32_t *e_exp, const uint8_t *arg, int n, int hh,
                                   int ww, int c, int k, int stride, int pad, int8_t *e_in, int32_t *e_in_exp, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || !e || !e_exp || !arg || !e_in || !e_in_exp || n <= 0 || hh <= 0 || ww <= 0 || c <= 0 || k <= 0 || k > 15 ||
        stride <= 0 || pad < 0 || pad >= k)
        return EOQ_ERR_BAD_ARG;
    if (c % 16 || !aligned16(e) || !aligned16(arg) || !aligned16(e_in)) return EOQ_ERR_ALIGNMENT;
    if ((size_t)n * hh * ww * (c / 16) > 0x7fffffffull) return EOQ_ERR_UNSUPPORTED;   // 32-bit item index in the kernel
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    count_launches(h, 2);
    ProfScope prof(h, EOQ_PROF_GLUE, s);
    return record(h, launch_maxpool_bwd(e, e_exp, arg, n, hh, ww, c, k, stride, pad, e_in, e_in_exp, nullptr, nullptr, nullptr, nullptr,
                                        nullptr, h->dev, h->sm_count, s, h->hook));
}

extern "C" int eoq_aux_maxpool_bwd_head(eoq_handle_t handle, const int8_t *e, const int32_t *e_exp, const uint8_t *arg, int n, int hh,
                                        int ww, int c, int k, int stride, int pad, int8_t *e_in, int32_t *e_in_exp,
                                        const uint8_t *relu_mask, const int32_t *gamma, int8_t *e3, int32_t *e3_exp, int64_t *sum_e1,
                                        void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || !e || !e_exp || !arg || !relu_mask || !gamma || !e3 || !e3_exp || n <= 0 || hh <= 0 || ww <= 0 || c <= 0 || k <= 0 ||
        k > 15 || stride <= 0 || pad < 0 || pad >= k)
        return EOQ_ERR_BAD_ARG;
    if (c % 16 || !aligned16(e) || !aligned16(arg) || !aligned16(e3) || (e_in && !aligned16(e_in)) ||
        (reinterpret_cast<uintptr_t>(relu_mask) & 1))
        return EOQ_ERR_ALIGNMENT;
    if ((size_t)n * hh * ww * (c / 16) > 0x7fffffffull) return EOQ_ERR_UNSUPPORTED;   // 32-bit item index in the kernel
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    count_launches(h, 2);
    ProfScope prof(h, EOQ_PROF_GLUE, s);
    return record(h, launch_maxpool_bwd(e, e_exp, arg, n, hh, ww, c, k, stride, pad, e_in, e_in_exp, relu_mask, gamma, e3, e3_exp,
                                        reinterpret_cast<long long *>(sum_e1), h->dev, h->sm_count, s, h->hook));
}

extern "C" int eoq_bn_workspace_size(int c, size_t *bytes)
{
    if (!bytes || c <= 0) return EOQ_ERR_BAD_ARG;
    *bytes = (bn_workspace_bytes(c) + 255) & ~(size_t)255;
    return EOQ_OK;
}

static int bn_check(Handle *h, size_t pixels, int c, const void *ws, size_t ws_bytes)
{
    if (!h || !ws || pixels == 0 || c <= 0) return EOQ_ERR_BAD_ARG;
    if (c % 16 || !aligned16(ws)) return EOQ_ERR_ALIGNMENT;
    if (c > 1024 || pixels > 0x7fffffffull) return EOQ_ERR_UNSUPPORTED;
    if (ws_bytes < bn_workspace_bytes(c)) return EOQ_ERR_WORKSPACE;
    return EOQ_OK;
}

extern "C" int eoq_bn_fwd(eoq_handle_t handle, const int32_t *acc, int acc_exp, size_t pixels, int c, const float *gamma,
                          const float *beta, float eps, int8_t *x5, uint8_t *relu_mask, void *workspace, size_t workspace_bytes,
                          void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!acc || !gamma || !beta || !x5 || !relu_mask || !(eps >= 0.0f) || acc_exp < -60 || acc_exp > 60) return EOQ_ERR_BAD_ARG;
    const int chk = bn_check(h, pixels, c, workspace, workspace_bytes);
    if (chk != EOQ_OK) return chk;
    if (!aligned16(acc) || !aligned16(x5) || (reinterpret_cast<uintptr_t>(relu_mask) & 1)) return EOQ_ERR_ALIGNMENT;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    count_launches(h, 3);
    ProfScope prof(h, EOQ_PROF_OTHER, s);
    return record(h, launch_bn_fwd(acc, acc_exp, pixels, c, gamma, beta, eps, x5, relu_mask, reinterpret_cast<BnChannel *>(workspace),
                                   h->sm_count, s));
}

extern "C" int eoq_bn_bwd(eoq_handle_t handle, const int8_t *e, const int32_t *e_exp, const uint8_t *relu_mask, const int32_t *acc,
                          int acc_exp, size_t pixels, int c, const float *gamma, void *workspace, size_t workspace_bytes, float *da,
                          float *dgamma, float *dbeta, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!e || !e_exp || !relu_mask || !acc || !gamma || !da || !dgamma || !dbeta || acc_exp < -60 || acc_exp > 60)
        return EOQ_ERR_BAD_ARG;
    const int chk = bn_check(h, pixels, c, workspace, workspace_bytes);
    if (chk != EOQ_OK) return chk;
    if (!aligned16(acc) || !aligned16(e) || !aligned16(da) || (reinterpret_cast<uintptr_t>(relu_mask) & 1)) return EOQ_ERR_ALIGNMENT;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    count_launches(h, 3);
    ProfScope prof(h, EOQ_PROF_OTHER, s);
    return record(h, launch_bn_bwd(e, e_exp, relu_mask, acc, acc_exp, pixels, c, gamma, reinterpret_cast<BnChannel *>(workspace), da,
                                   dgamma, dbeta, h->sm_count, s));
}

extern "C" int eoq_aux_avgpool_sum(eoq_handle_t handle, const int8_t *x, int n, int hw, int c, int32_t *sums, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || !x || !sums || n <= 0 || hw <= 0 || c <= 0 || hw > (1 << 23)) return EOQ_ERR_BAD_ARG;
    if (c % 16 || !aligned16(x)) return EOQ_ERR_ALIGNMENT;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    count_launches(h, 1);
    ProfScope prof(h, EOQ_PROF_GLUE, s);
    return record(h, launch_avgpool_sum(x, n, hw, c, sums, s));
}

extern "C" int eoq_aux_join(eoq_handle_t handle, const int8_t *a, const int32_t *a_exp, const int8_t *b, const int32_t *b_exp,
                            const uint8_t *mask_b, size_t n_el, int8_t *out, int32_t *out_exp, int64_t *sum_out, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || !a || !a_exp || !b || !b_exp || !out || !out_exp || n_el == 0 || (n_el % 16)) return EOQ_ERR_BAD_ARG;
    if (!aligned16(a) || !aligned16(b) || !aligned16(out) || (reinterpret_cast<uintptr_t>(mask_b) & 1)) return EOQ_ERR_ALIGNMENT;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    count_launches(h, 2);
    ProfScope prof(h, EOQ_PROF_GLUE, s);
    return record(h, launch_join(a, a_exp, b, b_exp, mask_b, n_el, out, out_exp, reinterpret_cast<long long *>(sum_out), nullptr, nullptr,
                                 nullptr, nullptr, nullptr, nullptr, nullptr, h->dev, h->sm_count, s, h->hook));
}

extern "C" int eoq_aux_join_head(eoq_handle_t handle, const int8_t *a, const int32_t *a_exp, const int8_t *b, const int32_t *b_exp,
                                 const uint8_t *mask_b, size_t n_el, int8_t *out, int32_t *out_exp, int64_t *sum_out,
                                 const uint8_t *relu_mask, const int16_t *x2, const int32_t *gamma, int8_t *e3, int32_t *e3_exp,
                                 int64_t *sum_e1, int64_t *sum_e1x2, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || !a || !a_exp || !b || !b_exp || !out || !out_exp || !relu_mask || !gamma || !e3 || !e3_exp || n_el == 0 || (n_el % 16))
        return EOQ_ERR_BAD_ARG;
    if (!aligned16(a) || !aligned16(b) || !aligned16(out) || !aligned16(e3) || (x2 && !aligned16(x2)) ||
        (reinterpret_cast<uintptr_t>(mask_b) & 1) || (reinterpret_cast<uintptr_t>(relu_mask) & 1))
        return EOQ_ERR_ALIGNMENT;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    count_launches(h, 2);
    ProfScope prof(h, EOQ_PROF_GLUE, s);
    return record(h, launch_join(a, a_exp, b, b_exp, mask_b, n_el, out, out_exp, reinterpret_cast<long long *>(sum_out), relu_mask, x2, gamma,
                                 e3, e3_exp, reinterpret_cast<long long *>(sum_e1), reinterpret_cast<long long *>(sum_e1x2), h->dev,
                                 h->sm_count, s, h->hook));
}

extern "C" int eoq_aux_head_workspace_size(int n, int c, int classes, size_t *bytes)
{
    if (!bytes || n <= 0 || c <= 0 || classes <= 0) return EOQ_ERR_BAD_ARG;
    *bytes = round256((size_t)n * c * sizeof(float)) * 2 + round256((size_t)n * classes * sizeof(float)) + round256((size_t)n * sizeof(double));
    return EOQ_OK;
}

extern "C" int eoq_aux_head(eoq_handle_t handle, const int32_t *sums, int n, int c, int hw, int classes, float *W, float *bias,
                            const int32_t *labels, float lr, float *loss, float *dpooled, float *logits, void *workspace,
                            size_t workspace_bytes, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || !sums || !W || !bias || !labels || !dpooled || !logits || n <= 0 || c <= 0 || hw <= 0 || classes <= 0)
        return EOQ_ERR_BAD_ARG;
    if (c > 1536) return EOQ_ERR_UNSUPPORTED;  // the pooled activations of 32 samples are kept in shared memory
    size_t need = 0;
    eoq_aux_head_workspace_size(n, c, classes, &need);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < need) return EOQ_ERR_WORKSPACE;
    char *ws = static_cast<char *>(workspace);
    float *pooled = reinterpret_cast<float *>(ws);
    float *dl = reinterpret_cast<float *>(ws + 2 * round256((size_t)n * c * sizeof(float)));
    double *loss_n = reinterpret_cast<double *>(ws + 2 * round256((size_t)n * c * sizeof(float)) + round256((size_t)n * classes * sizeof(float)));
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    count_launches(h, lr != 0.0f ? 5 : 4);
    ProfScope prof(h, EOQ_PROF_GLUE, s);
    return record(h, launch_head(sums, n, c, hw, classes, W, bias, labels, lr, loss, dpooled, logits, pooled, dl, loss_n, s));
}

extern "C" int eoq_aux_head_update(eoq_handle_t handle, int n, int c, int classes, float *W, float *bias, float lr, const void *workspace,
                                   size_t workspace_bytes, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || !W || !bias || n <= 0 || c <= 0 || classes <= 0) return EOQ_ERR_BAD_ARG;
    size_t need = 0;
    eoq_aux_head_workspace_size(n, c, classes, &need);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < need) return EOQ_ERR_WORKSPACE;
    const char *ws = static_cast<const char *>(workspace);
    const float *pooled = reinterpret_cast<const float *>(ws);
    const float *dl = reinterpret_cast<const float *>(ws + 2 * round256((size_t)n * c * sizeof(float)));
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    count_launches(h, 1);
    ProfScope prof(h, EOQ_PROF_GLUE, s);
    return record(h, launch_head_update(dl, pooled, n, c, classes, lr, W, bias, s));
}

extern "C" int eoq_aux_head_error(eoq_handle_t handle, const float *dpooled, int n, int c, int hw, int8_t *e, int32_t *e_exp,
                                  void *workspace, size_t workspace_bytes, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || !dpooled || !e || !e_exp || n <= 0 || c <= 0 || hw <= 0) return EOQ_ERR_BAD_ARG;
    if (c % 16 || !aligned16(e)) return EOQ_ERR_ALIGNMENT;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < (size_t)n * c * sizeof(float)) return EOQ_ERR_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    count_launches(h, 2);
    ProfScope prof(h, EOQ_PROF_GLUE, s);
    return record(h, launch_head_error(dpooled, n, c, hw, static_cast<float *>(workspace), e, e_exp, h->dev, h->sm_count, s, h->hook));
}

extern "C" int eoq_aux_scalar_update(eoq_handle_t handle, int num, int32_t *const *theta, int32_t *const *mirror,
                                     const int64_t *const *total, const int32_t *const *total_exp, const int *exp_bias,
                                     const int *tensor_id, int32_t *const *grad_out, int32_t lr_mant, int32_t lr_exp,
                                     int round_mode, uint64_t seed, const uint64_t *step, void *stream)
{
    Handle *h = reinterpret_cast<Handle *>(handle);
    if (!h || num <= 0 || !theta || !total || !total_exp || !exp_bias || !tensor_id) return EOQ_ERR_BAD_ARG;
    if (lr_mant < 1 || lr_mant > 255 || lr_exp < -64 || lr_exp > 64) return EOQ_ERR_RANGE;
    if (round_mode != EOQ_ROUND_RNE && round_mode != EOQ_ROUND_STOCHASTIC) return EOQ_ERR_BAD_ARG;
    for (int i = 0; i < num; ++i)
        if (!theta[i] || !total[i] || !total_exp[i]) return EOQ_ERR_BAD_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    ProfScope prof(h, EOQ_PROF_GLUE, s);
    for (int base = 0; base < num; base += kScalarChunk) {
        ScalarBatch b;
        memset(&b, 0, sizeof(b));
        b.num = num - base < kScalarChunk ? num - base : kScalarChunk;
        for (int k = 0; k < b.num; ++k) {
            ScalarItem &it = b.item[k];
            it.theta = theta[base + k];
            it.mirror = mirror ? mirror[base + k] : nullptr;
            it.total = reinterpret_cast<const long long *>(total[base + k]);
            it.exp = total_exp[base + k];
            it.exp_bias = exp_bias[base + k];
            it.tensor_id = tensor_id[base + k];
            it.grad_out = grad_out ? grad_out[base + k] : nullptr;
        }
        cudaError_t e = launch_scalar_update(b, lr_mant, lr_exp, round_mode == EOQ_ROUND_STOCHASTIC, seed,
                                             reinterpret_cast<const unsigned long long *>(step), 0, s);
        if (e != cudaSuccess) return record(h, e);
        count_launches(h, 1);
    }
    return EOQ_OK;
}
