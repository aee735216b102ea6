// One integer encoder block as a chain of the library's kernels on the caller's stream:
// LN1 -> QKV GEMM -> fused attention (reads heads straight out of the QKV activation) -> proj GEMM
// (+ residual) -> LN2 -> FC1 GEMM with GELU epilogue -> FC2 GEMM (+ residual).  Each layer runs the
// approximation variant its constants name (the per-layer table of Sec. 3.2).
#include "iptq_internal.cuh"

namespace iptq {

static size_t a256(size_t v) { return (v + 255) & ~size_t(255); }

struct BlockLayout {
    size_t h1, qkv, att, x1, h2, hid, w_qkv, w_proj, w_fc1, w_fc2, total;
};

static BlockLayout block_layout(const iptq_block_params* p)
{
    BlockLayout l;
    const size_t T = (size_t)p->B * (size_t)p->N, D = (size_t)p->D, Dh = (size_t)p->Dh;
    size_t off = kStatusBytes;
    auto take = [&](size_t bytes) { size_t o = off; off += a256(bytes); return o; };
    l.h1 = take(T * D);
    l.qkv = take(T * 3 * D);
    l.att = take(T * D);
    l.x1 = take(T * D);
    l.h2 = take(T * D);
    l.hid = take(T * Dh);
    l.w_qkv = l.w_proj = l.w_fc1 = l.w_fc2 = 0;
    if (p->w_bits == 4) {
        l.w_qkv = take(3 * D * D);
        l.w_proj = take(D * D);
        l.w_fc1 = take(Dh * D);
        l.w_fc2 = take(D * Dh);
    }
    l.total = off;
    return l;
}

static int check_block(const iptq_block_params* p)
{
    if (!p) return IPTQ_ERR_NULL;
    if (p->B < 0 || p->N < 1 || p->D < 16 || p->H < 1 || p->Dh < 16) return IPTQ_ERR_SHAPE;
    if (p->H * p->dh != p->D) return IPTQ_ERR_SHAPE;
    if (p->w_bits != 8 && p->w_bits != 4) return IPTQ_ERR_BITS;
    if (!p->ln1 || !p->ln2 || !p->sm || !p->pv_rq || !p->gelu || !p->res1_rq || !p->res2_rq) return IPTQ_ERR_NULL;
    if (!p->w_qkv || !p->w_proj || !p->w_fc1 || !p->w_fc2) return IPTQ_ERR_NULL;
    if (p->table.sm != p->sm->variant || p->table.gelu != p->gelu->variant || p->table.ln1 != p->ln1->variant ||
        p->table.ln2 != p->ln2->variant)
        return IPTQ_ERR_VARIANT;
    return IPTQ_OK;
}

}  // namespace iptq

using namespace iptq;

extern "C" {

size_t iptq_encoder_block_workspace_bytes(const iptq_block_params* p)
{
    if (check_block(p) != IPTQ_OK) return 0;
    return block_layout(p).total;
}

static int encoder_block_run(const int8_t* x, int8_t* y, const iptq_block_params* p, void* ws, size_t ws_bytes,
                             cudaStream_t stream, cudaEvent_t* ev)
{
    int rc = check_block(p);
    if (rc != IPTQ_OK) return rc;
    if (!ws) return IPTQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return IPTQ_ERR_ALIGN;
    const BlockLayout l = block_layout(p);
    if (ws_bytes < l.total) return IPTQ_ERR_WORKSPACE;
    if (p->B == 0) return IPTQ_OK;
    if (!x || !y) return IPTQ_ERR_NULL;
    uint8_t* base = static_cast<uint8_t*>(ws);
    StatusBlock* status = reinterpret_cast<StatusBlock*>(base);
    int8_t* h1 = reinterpret_cast<int8_t*>(base + l.h1);
    int8_t* qkv = reinterpret_cast<int8_t*>(base + l.qkv);
    int8_t* att = reinterpret_cast<int8_t*>(base + l.att);
    int8_t* x1 = reinterpret_cast<int8_t*>(base + l.x1);
    int8_t* h2 = reinterpret_cast<int8_t*>(base + l.h2);
    int8_t* hid = reinterpret_cast<int8_t*>(base + l.hid);
    const int64_t T = p->B * p->N;
    const int D = p->D, Dh = p->Dh;
    int stage = 0;
    auto mark = [&]() -> int {                     // stage boundary: record the caller's event, if any
        if (!ev) return IPTQ_OK;
        return cuda_status(cudaEventRecord(ev[stage++], stream));
    };
    if ((rc = mark()) != IPTQ_OK) return rc;

    const int8_t *wq = static_cast<const int8_t*>(p->w_qkv), *wp = static_cast<const int8_t*>(p->w_proj),
                 *w1 = static_cast<const int8_t*>(p->w_fc1), *w2 = static_cast<const int8_t*>(p->w_fc2);
    if (p->w_bits == 4) {
        struct { const void* src; size_t off; int64_t n; const int8_t** dst; } u[4] = {
            {p->w_qkv, l.w_qkv, (int64_t)3 * D * D, &wq}, {p->w_proj, l.w_proj, (int64_t)D * D, &wp},
            {p->w_fc1, l.w_fc1, (int64_t)Dh * D, &w1}, {p->w_fc2, l.w_fc2, (int64_t)D * Dh, &w2}};
        const void* srcs[4];
        int8_t* dsts[4];
        int64_t ns[4];
        for (int i = 0; i < 4; ++i) {
            srcs[i] = u[i].src;
            dsts[i] = reinterpret_cast<int8_t*>(base + u[i].off);
            ns[i] = u[i].n;
            *u[i].dst = dsts[i];
        }
        if ((rc = unpack_int4_multi_launch(srcs, dsts, ns, 4, stream)) != IPTQ_OK) return rc;   // one launch for the four matrices
    }

    if ((rc = layernorm_launch(x, h1, T, D, p->ln1_gamma, p->ln1_beta, p->ln1_ptf, p->ln1, stream)) != IPTQ_OK) return rc;
    if ((rc = mark()) != IPTQ_OK) return rc;
    const int ab = p->act_bits ? p->act_bits : 8;            // width of the QKV / proj / FC2 outputs
    if (ab < 4 || ab > 8) return IPTQ_ERR_BITS;
    LinearArgs lq{h1, wq, p->b_qkv, p->m_qkv, p->s_qkv, 0, nullptr, nullptr, nullptr, qkv, T, 3 * D, D, status, ab};
    if ((rc = linear_launch(lq, stream)) != IPTQ_OK) return rc;
    if ((rc = mark()) != IPTQ_OK) return rc;
    // a row of qkv is [q | k | v]; head h occupies columns h*dh .. of each third
    AttnArgs aa{qkv, qkv + D, qkv + 2 * D, (int64_t)3 * D, (int64_t)p->dh, (int64_t)p->N * 3 * D, att, p->B, p->H, p->N,
                p->dh, p->attn_bias, p->mask_id, p->sm, p->pv_rq, status, p->attn_bias_t};
    if ((rc = attention_launch(aa, stream)) != IPTQ_OK) return rc;
    if ((rc = mark()) != IPTQ_OK) return rc;
    LinearArgs lp{att, wp, p->b_proj, p->m_proj, p->s_proj, p->proj_zp, x, p->res1_rq, nullptr, x1, T, D, D, status, ab};
    if ((rc = linear_launch(lp, stream)) != IPTQ_OK) return rc;
    if ((rc = mark()) != IPTQ_OK) return rc;
    if ((rc = layernorm_launch(x1, h2, T, D, p->ln2_gamma, p->ln2_beta, p->ln2_ptf, p->ln2, stream)) != IPTQ_OK) return rc;
    if ((rc = mark()) != IPTQ_OK) return rc;
    LinearArgs l1{h2, w1, p->b_fc1, p->m_fc1, p->s_fc1, 0, nullptr, nullptr, p->gelu, hid, T, Dh, D, status};
    if ((rc = linear_launch(l1, stream)) != IPTQ_OK) return rc;
    if ((rc = mark()) != IPTQ_OK) return rc;
    LinearArgs l2{hid, w2, p->b_fc2, p->m_fc2, p->s_fc2, p->fc2_zp, x1, p->res2_rq, nullptr, y, T, D, Dh, status, ab};
    if ((rc = linear_launch(l2, stream)) != IPTQ_OK) return rc;
    return mark();
}

int iptq_encoder_block(const int8_t* x, int8_t* y, const iptq_block_params* p, void* ws, size_t ws_bytes,
                       iptq_stream_t stream)
{
    return encoder_block_run(x, y, p, ws, ws_bytes, stream, nullptr);
}

int iptq_encoder_block_profiled(const int8_t* x, int8_t* y, const iptq_block_params* p, void* ws, size_t ws_bytes,
                                iptq_stream_t stream, void* const* events, int n_events)
{
    if (!events) return IPTQ_ERR_NULL;
    if (n_events != IPTQ_BLOCK_STAGES + 1) return IPTQ_ERR_SHAPE;
    for (int i = 0; i < n_events; ++i)
        if (!events[i]) return IPTQ_ERR_NULL;
    cudaEvent_t ev[IPTQ_BLOCK_STAGES + 1];
    for (int i = 0; i < n_events; ++i) ev[i] = static_cast<cudaEvent_t>(events[i]);
    return encoder_block_run(x, y, p, ws, ws_bytes, stream, ev);
}

}  // extern "C"
