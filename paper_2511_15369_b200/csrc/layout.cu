// Token re-ordering for windowed attention (Swin-style blocks): window partition with cyclic shift and padding,
// its inverse, and the 2x2 patch merge are all "destination row i = concatenation of some source rows", with the
// source row numbers in a table built once on the host.  Pure data movement, 16 bytes per thread per step.
#include <algorithm>

#include "iptq_common.cuh"

namespace iptq {

__global__ void __launch_bounds__(256)
gather_rows_kernel(const int4* __restrict__ src, int4* __restrict__ dst, const int32_t* __restrict__ index,
                   int64_t n_dst, int parts, int vec_per_part)
{
    grid_dep_launch();
    grid_dep_wait();
    const int vec_per_row = parts * vec_per_part;
    const int64_t total = n_dst * vec_per_row;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int64_t row = i / vec_per_row;
        const int v = (int)(i - row * vec_per_row);
        const int part = v / vec_per_part;
        const int s = __ldg(index + row * parts + part);
        int4 val = make_int4(0, 0, 0, 0);
        if (s >= 0) val = __ldg(src + (int64_t)s * vec_per_part + (v - part * vec_per_part));
        dst[i] = val;
    }
}

// Image -> patch rows: out[(b, py, px), (c, dy, dx)] = img[b, c, py P + dy, px P + dx].  One 16-byte piece of a
// patch line per thread per step; P is a multiple of 16, so every piece is aligned on both sides.
__global__ void __launch_bounds__(256)
patchify_kernel(const int4* __restrict__ img, int4* __restrict__ out, int64_t B, int C, int H, int W, int P)
{
    grid_dep_launch();
    grid_dep_wait();
    const int gw = W / P, gh = H / P, vp = P / 16;          // grid of patches, 16-byte pieces per patch line
    const int vec_per_row = C * P * vp;
    const int64_t total = B * gh * gw * vec_per_row;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int64_t row = i / vec_per_row;
        int v = (int)(i - row * vec_per_row);
        const int piece = v % vp; v /= vp;
        const int dy = v % P;
        const int c = v / P;
        const int px = (int)(row % gw);
        const int py = (int)((row / gw) % gh);
        const int64_t b = row / ((int64_t)gw * gh);
        const int64_t src = (((b * C + c) * H + (int64_t)py * P + dy) * W + (int64_t)px * P) / 16 + piece;
        out[i] = __ldg(img + src);
    }
}

}  // namespace iptq

using namespace iptq;

extern "C" int iptq_patchify(const int8_t* img, int8_t* out, int64_t B, int C, int H, int W, int P,
                             iptq_stream_t stream)
{
    if (B < 0 || C < 1 || P < 16 || (P & 15) || H < P || W < P || H % P || W % P) return IPTQ_ERR_SHAPE;
    if (B == 0) return IPTQ_OK;
    if (!img || !out) return IPTQ_ERR_NULL;
    if (!aligned16(img) || !aligned16(out)) return IPTQ_ERR_ALIGN;
    const int64_t total = B * (H / P) * (W / P) * C * P * (P / 16);
    const int grid = (int)std::min<int64_t>((total + 255) / 256, (int64_t)sm_count() * 16);
    if (launch_kernel(patchify_kernel, grid, 256, 0, stream, reinterpret_cast<const int4*>(img),
                      reinterpret_cast<int4*>(out), B, C, H, W, P) != cudaSuccess)
        return IPTQ_ERR_CUDA;
    note_launch();
    return last_launch_status();
}

extern "C" int iptq_gather_rows(const int8_t* src, int8_t* dst, const int32_t* index, int64_t n_dst, int parts,
                                int row_bytes, iptq_stream_t stream)
{
    if (n_dst < 0 || parts < 1 || row_bytes < 16 || (row_bytes & 15)) return IPTQ_ERR_SHAPE;
    if (n_dst == 0) return IPTQ_OK;
    if (!src || !dst || !index) return IPTQ_ERR_NULL;
    if (!aligned16(src) || !aligned16(dst) || (reinterpret_cast<uintptr_t>(index) & 3u)) return IPTQ_ERR_ALIGN;
    const int vec_per_part = row_bytes / 16;
    const int64_t total = n_dst * parts * vec_per_part;
    const int grid = (int)std::min<int64_t>((total + 255) / 256, (int64_t)sm_count() * 16);
    if (launch_kernel(gather_rows_kernel, grid, 256, 0, stream, reinterpret_cast<const int4*>(src),
                      reinterpret_cast<int4*>(dst), index, n_dst, parts, vec_per_part) != cudaSuccess)
        return IPTQ_ERR_CUDA;
    note_launch();
    return last_launch_status();
}
