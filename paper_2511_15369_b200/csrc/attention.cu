// Host side of the fused integer attention: argument checks, tile geometry, tensor maps, dispatch to the
// per-variant kernel files.
#include "attention_window.cuh"
#include "iptq_internal.cuh"

namespace iptq {

int attention_launch_variant0(int dh, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                              const AttnParams& p, int smem_bytes, cudaStream_t st);
int attention_launch_variant1(int dh, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                              const AttnParams& p, int smem_bytes, cudaStream_t st);
int attention_launch_variant2(int dh, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                              const AttnParams& p, int smem_bytes, cudaStream_t st);
int attention_launch_variant3(int dh, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                              const AttnParams& p, int smem_bytes, cudaStream_t st);
int window_launch_variant0(int dh, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                           const AttnParams& p, int smem_bytes, cudaStream_t st);
int window_launch_variant1(int dh, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                           const AttnParams& p, int smem_bytes, cudaStream_t st);
int window_launch_variant2(int dh, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                           const AttnParams& p, int smem_bytes, cudaStream_t st);
int window_launch_variant3(int dh, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                           const AttnParams& p, int smem_bytes, cudaStream_t st);

// Bytes of the re-laid-out bias the window kernel (N <= 64) reads: [H][ceil(N/4) column quads][64 rows] x 4 int32.
static size_t attention_bias_t_bytes(int H, int N) { return N <= 64 ? (size_t)H * (size_t)((N + 3) / 4) * 64 * 16 : 0; }

// out[h][c4][r] = bias[h][r][4 c4 .. 4 c4 + 3] (0 past column N): one 16-byte load gives a thread four columns of
// its row, and the 32 rows of a warp are 512 contiguous bytes.
__global__ void __launch_bounds__(256)
bias_relayout_kernel(const int32_t* __restrict__ bias, int4* __restrict__ out, int H, int N)
{
    grid_dep_launch();
    grid_dep_wait();
    const int C4 = (N + 3) / 4;
    const int total = H * C4 * N;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        const int r = i % N, c4 = (i / N) % C4, h = i / (N * C4);
        const int32_t* src = bias + ((size_t)h * N + r) * N + 4 * c4;
        int4 q;
        q.x = __ldg(src);
        q.y = 4 * c4 + 1 < N ? __ldg(src + 1) : 0;
        q.z = 4 * c4 + 2 < N ? __ldg(src + 2) : 0;
        q.w = 4 * c4 + 3 < N ? __ldg(src + 3) : 0;
        out[((size_t)h * C4 + c4) * 64 + r] = q;
    }
}

static int launch_attn_v(bool window, int dh, int variant, const CUtensorMap& mq, const CUtensorMap& mk,
                         const CUtensorMap& mv, const AttnParams& p, int smem_bytes, cudaStream_t st)
{
    switch (variant) {
        case IPTQ_SM_BITEXP: return window ? window_launch_variant0(dh, mq, mk, mv, p, smem_bytes, st)
                                           : attention_launch_variant0(dh, mq, mk, mv, p, smem_bytes, st);
        case IPTQ_SM_SHIFTMAX: return window ? window_launch_variant1(dh, mq, mk, mv, p, smem_bytes, st)
                                             : attention_launch_variant1(dh, mq, mk, mv, p, smem_bytes, st);
        case IPTQ_SM_POLY: return window ? window_launch_variant2(dh, mq, mk, mv, p, smem_bytes, st)
                                         : attention_launch_variant2(dh, mq, mk, mv, p, smem_bytes, st);
        case IPTQ_SM_LOG2: return window ? window_launch_variant3(dh, mq, mk, mv, p, smem_bytes, st)
                                         : attention_launch_variant3(dh, mq, mk, mv, p, smem_bytes, st);
        default: return IPTQ_ERR_VARIANT;
    }
}

// Host-side argument checks alone: nothing is enqueued.
static int attention_check(const AttnArgs& a)
{
    if (!a.sm || !a.out_rq) return IPTQ_ERR_NULL;
    if (a.B < 0 || a.B > (1 << 24) || a.H < 1 || a.H > 1024 || a.N < 1 || a.N > 256) return IPTQ_ERR_SHAPE;
    if (a.dh != 32 && a.dh != 64) return IPTQ_ERR_SHAPE;
    if (a.sm->row_len != a.N) return IPTQ_ERR_SHAPE;
    if (a.sm->out_bits < 4 || a.sm->out_bits > 8) return IPTQ_ERR_BITS;
    if (a.sm->x0 < 8 || a.sm->M < 31 || a.sm->M > 40) return IPTQ_ERR_SCALE_RANGE;
    int rc = check_requant(a.out_rq);
    if (rc != IPTQ_OK) return rc;
    if (!a.status) return IPTQ_ERR_WORKSPACE;
    if (a.B == 0) return IPTQ_OK;
    if (!a.q || !a.k || !a.v || !a.out) return IPTQ_ERR_NULL;
    if (!aligned16(a.q) || !aligned16(a.k) || !aligned16(a.v) || !aligned16(a.out) ||
        (a.bias && (reinterpret_cast<uintptr_t>(a.bias) & 3u)) || (a.bias_t && !aligned16(a.bias_t)) ||
        (a.tok_stride & 15) || (a.head_stride & 15) || (a.batch_stride & 15))
        return IPTQ_ERR_ALIGN;
    if (a.B * a.H * ((a.N + 127) / 128) > (int64_t)1 << 30) return IPTQ_ERR_SHAPE;
    return IPTQ_OK;
}

int attention_launch(const AttnArgs& a, cudaStream_t st)
{
    int rc = attention_check(a);
    if (rc != IPTQ_OK || a.B == 0) return rc;

    AttnParams p;
    p.B = (int)a.B; p.H = a.H; p.N = a.N; p.dh = a.dh;
    p.mtiles = (a.N + 127) / 128;
    p.items = p.B * p.H * p.mtiles;
    p.full_items = p.B * p.H * (a.N / 128);
    // Problems of at most 64 tokens (Swin windows) go two per item through the window kernel
    const bool window = a.N <= 64 && a.B * a.H >= 2;
    int smem_bytes;
    p.lut_n = 0;
    if (window) {
        const WinGeom w = window_geometry(a.dh, a.sm->variant);
        p.mtiles = 1;
        p.items = (int)((a.B * a.H + 1) / 2);
        p.full_items = 0;
        p.npad_s = 128; p.kpad = 128; p.o_col = 128;
        p.q_bytes = p.k_bytes = p.v_bytes = 128 * a.dh;
        p.stage_bytes = w.stage_bytes;
        p.stages = w.stages;
        p.p_plane = 16384;
        p.p_bytes = w.p_bytes;
        p.p_off = w.stages * w.stage_bytes;
        p.xch_off = p.lut_off = p.p_off + w.groups * w.p_bytes;
        if (const int64_t n = exp_table_entries(*a.sm)) {
            const int64_t bytes = (2 * (n + 1) + 255) & ~(int64_t)255;
            if (p.lut_off + bytes + 512 + 1024 <= 227 * 1024) p.lut_n = (int)n;
        }
        const int lut_bytes = p.lut_n ? (int)((2 * ((int64_t)p.lut_n + 1) + 255) & ~255) : 0;
        p.bar_off = p.lut_off + lut_bytes;
        smem_bytes = p.bar_off + 512 + 1024;
        p.tmem_cols = 32;
        while ((int)p.tmem_cols < w.groups * w.gcols) p.tmem_cols <<= 1;
    } else {
        p.npad_s = (a.N + 15) & ~15;
        p.kpad = (a.N + 31) & ~31;
        auto up1k = [](int v) { return (v + 1023) & ~1023; };
        p.q_bytes = up1k(128 * a.dh);
        p.k_bytes = up1k(p.npad_s * a.dh);
        p.v_bytes = up1k(p.kpad * a.dh);
        p.stage_bytes = p.q_bytes + p.k_bytes + p.v_bytes;
        p.p_plane = ((p.kpad + 127) / 128) * 16384;
        p.p_bytes = (a.sm->variant == IPTQ_SM_LOG2 ? 2 : 1) * p.p_plane;
        // Exponential table (shift-based variants with values below 2^16), where it fits beside 3 or 2 operand stages.
        p.stages = ATT_STAGES;
        const int fixed = 2 * p.p_bytes + 2 * 4 * 128 * 4 + 256 + 1024;
        if (const int64_t n = exp_table_entries(*a.sm)) {
            const int64_t bytes = (2 * (n + 1) + 255) & ~(int64_t)255;
            if (fixed + 3 * p.stage_bytes + bytes <= 227 * 1024) { p.lut_n = (int)n; }
            else if (fixed + 2 * p.stage_bytes + bytes <= 227 * 1024) { p.lut_n = (int)n; p.stages = 2; }
        }
        // two operand planes per P buffer (logarithm candidate) leave room for a ring of two only
        if (fixed + p.stages * p.stage_bytes > 226 * 1024) p.stages = 2;
        const int lut_bytes = p.lut_n ? (int)((2 * ((int64_t)p.lut_n + 1) + 255) & ~255) : 0;
        p.p_off = p.stages * p.stage_bytes;
        p.xch_off = p.p_off + 2 * p.p_bytes;
        p.lut_off = p.xch_off + 2 * 4 * 128 * 4;
        p.bar_off = p.lut_off + lut_bytes;
        smem_bytes = p.bar_off + 256 + 1024;
        p.o_col = (p.npad_s + 31) & ~31;                     // O sits behind S in TMEM
        p.tmem_cols = 32;
        while ((int)p.tmem_cols < p.o_col + (a.sm->variant == IPTQ_SM_LOG2 ? 2 : 1) * a.dh) p.tmem_cols <<= 1;
    }
    p.lut_src = (p.lut_n && a.sm->table && a.sm->table_n == p.lut_n) ? a.sm->table : nullptr;
    p.bias = a.bias; p.mask_id = a.mask_id; p.out = a.out;
    p.bias_q = (window && a.bias && a.bias_t) ? reinterpret_cast<const int4*>(a.bias_t) : nullptr;
    p.ex = to_dev_exp(*a.sm);
    p.M = a.sm->M; p.f_shl = a.sm->f_shl; p.p_shr = a.sm->p_shr;
    p.orq = to_dev(*a.out_rq);
    p.status = a.status;

    // q/k/v as 4-D tensors (dh, N, H, B); rows past N read as zero, which is what the padding needs.
    CUtensorMap mq, mk, mv;
    const uint64_t dims[4] = {(uint64_t)a.dh, (uint64_t)a.N, (uint64_t)a.H, (uint64_t)a.B};
    const uint64_t str[3] = {(uint64_t)a.tok_stride, (uint64_t)a.head_stride, (uint64_t)a.batch_stride};
    const uint32_t box_q[4] = {(uint32_t)a.dh, window ? 64u : 128u, 1u, 1u};
    const uint32_t box_k[4] = {(uint32_t)a.dh, window ? 64u : (uint32_t)p.npad_s, 1u, 1u};
    const uint32_t box_v[4] = {(uint32_t)a.dh, window ? 64u : (uint32_t)p.kpad, 1u, 1u};
    if ((rc = make_tensor_map_u8(&mq, a.q, 4, dims, str, box_q, a.dh)) != IPTQ_OK) return rc;
    if ((rc = make_tensor_map_u8(&mk, a.k, 4, dims, str, box_k, a.dh)) != IPTQ_OK) return rc;
    if ((rc = make_tensor_map_u8(&mv, a.v, 4, dims, str, box_v, a.dh)) != IPTQ_OK) return rc;
    return launch_attn_v(window, a.dh, a.sm->variant, mq, mk, mv, p, smem_bytes, st);
}

}  // namespace iptq

using namespace iptq;

extern "C" {

size_t iptq_attention_workspace_bytes(int64_t, int, int, int) { return kStatusBytes; }

size_t iptq_attention_bias_bytes(int H, int N) { return (H < 1 || N < 1) ? 0 : attention_bias_t_bytes(H, N); }

int iptq_attention_bias_prepare(const int32_t* bias, int32_t* bias_t, int H, int N, iptq_stream_t stream)
{
    if (H < 1 || H > 1024 || N < 1 || N > 256) return IPTQ_ERR_SHAPE;
    if (attention_bias_t_bytes(H, N) == 0) return IPTQ_OK;          // N > 64: the row-major bias is what the kernel reads
    if (!bias || !bias_t) return IPTQ_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(bias) & 3u) || !aligned16(bias_t)) return IPTQ_ERR_ALIGN;
    const int total = H * ((N + 3) / 4) * N;
    launch_kernel(bias_relayout_kernel, std::min((total + 255) / 256, 4 * sm_count()), 256, 0, stream, bias,
                  reinterpret_cast<int4*>(bias_t), H, N);
    note_launch();
    return last_launch_status();
}

int iptq_attention_block(const int8_t* q, const int8_t* k, const int8_t* v, int8_t* out, int64_t B, int H,
                         int N, int dh, const int32_t* bias, const int32_t* bias_t, const uint8_t* mask_id,
                         const iptq_softmax_consts* sm, const iptq_requant* out_rq, void* ws, size_t ws_bytes,
                         iptq_stream_t stream)
{
    if (!ws || ws_bytes < kStatusBytes) return IPTQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return IPTQ_ERR_ALIGN;
    AttnArgs a{q, k, v, (int64_t)dh, (int64_t)N * dh, (int64_t)H * N * dh, out, B, H, N, dh, bias, mask_id, sm, out_rq,
               static_cast<StatusBlock*>(ws), bias_t};
    return attention_launch(a, stream);
}

}  // extern "C"
