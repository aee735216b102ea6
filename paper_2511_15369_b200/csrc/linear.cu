// INT8 x INT8 -> INT32 GEMM on the 5th-generation tensor cores (tcgen05.mma.kind::i8, TMEM accumulators,
// TMA-fed shared-memory pipeline) with the integer epilogues of the path applied straight out of TMEM:
//   - per-channel dyadic requantisation (QKV, proj, FC2), optionally with the int8 residual branch;
//   - FC1: requantise to the GELU input scale, integer GELU (Sec. 3.3, Eqs. (3), (5)), requantise to int8.
// No int32 intermediate is written to HBM.
//
// One persistent CTA per SM, 18 warps: warp 0 = TMA producer, warp 1 = MMA issuer (owns TMEM), warps 2..17 =
// epilogue.  The accumulator is double-buffered in TMEM so that the epilogue of tile i overlaps the mainloop of
// tile i+1.
#include <algorithm>
#include <climits>
#include <mutex>

#include "tc_common.cuh"
#include "iptq_internal.cuh"

namespace iptq {

// ---------------------------------------------------------------- host: tensor map encoding
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

int make_tensor_map_u8(CUtensorMap* map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides,
                       const uint32_t* box, int swizzle_bytes)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return IPTQ_ERR_CUDA;
    cuuint64_t gdim[5], gstr[5];
    cuuint32_t bx[5], estr[5];
    for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bx[i] = box[i]; estr[i] = 1; }
    for (int i = 0; i + 1 < rank; ++i) {
        gstr[i] = strides[i];
        if (strides[i] & 15u) return IPTQ_ERR_ALIGN;
    }
    if (reinterpret_cast<uintptr_t>(base) & 15u) return IPTQ_ERR_ALIGN;
    CUtensorMapSwizzle sw = swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                          : swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                          : swizzle_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE;
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstr, bx, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? IPTQ_OK : IPTQ_ERR_CUDA;
}

// ---------------------------------------------------------------- kernel
// The product is computed transposed, D^T[channel, token] = W X^T: the weight tile is the A operand (128 output
// channels = the 128 TMEM lanes), the activation tile the B operand (TN tokens = TMEM columns).  A thread of the
// epilogue then owns ONE output channel, so the per-channel requantisation constants (bias, multiplier, shift,
// rounding constant) are four registers instead of per-column vectors, and nothing but the accumulator is read
// from TMEM.  The outputs of a warp (32 channels x TN/4 tokens) go through a shared-memory block in the row-major
// [token][channel] order of y and leave with one TMA store, which also clips at M and N.
enum { EPI_REQUANT = 0, EPI_RESIDUAL = 1, EPI_GELU = 2, EPI_GELU_TAB = 3 };

constexpr int BK = 128;                  // bytes of K per ring stage = one 128-byte swizzle row = 4 MMA k-steps
constexpr int CT = 128;                  // output channels per tile = TMEM lanes
constexpr int W_BYTES = CT * BK;         // weight tile of one stage
constexpr int MAX_STAGES = 8;
constexpr int EPI_WARPS = 16;            // 4 TMEM lane quadrants x 4 token quarters
constexpr int GEMM_THREADS = 32 * (2 + EPI_WARPS);
constexpr int ACC_COLS = 256;            // TMEM columns between the two accumulators
constexpr uint32_t TMEM_COLS = 512;
constexpr int SMEM_LIMIT = 227 * 1024;

struct GemmParams {
    int M, N, K;                                      // tokens, output channels, reduction length
    int TN;                                           // tokens per tile: 64, 128, 192 or 256
    int n_ct, n_tt;                                   // channel tiles, token tiles
    int stages, stage_bytes;                          // TMA ring
    int epi_bufs;                                     // staging buffers of the epilogue (output, residual): 1 or 2
    int off_res, off_tab, off_bar, off_ring;          // shared-memory layout (the output blocks start at 0)
    const int32_t* bias; const int32_t* mult; const int8_t* shift;
    int out_zp;
    int qmin, qmax;                                   // output range
    int res_mult, res_rnd, res_shift, res_off;        // residual branch: ((res << 16) - res_off) through R
    GeluDev gelu;
    const int8_t* gelu_tab;                           // device table of the integer GELU (EPI_GELU_TAB)
    StatusBlock* status;
    int acc_floor;                                    // INT_MIN, as a value the compiler cannot see (epilogue, bias add)
};

// The tiles of this CTA, round by round: tiles are numbered with the channel tile fastest, so that CTAs running side by side
// share an activation tile in L2.  A CTA pair takes two neighbouring channel tiles of one token tile (the odd CTA's
// may lie past N when the number of channel tiles is odd: its weight rows then read as zeros and nothing is stored).
// Rounds alternate in direction: CTA j of S takes tile r S + j in even rounds and r S + (S - 1 - j) in odd ones.  The
// ragged last token tile is narrower and its tiles come last, so the few tiles of a final, partly filled round then
// go to the CTAs whose previous tile was a short one too, instead of to those that have only had full ones
// (ViT-Base proj 22.1 -> 21.4 us, FC2 48.6 -> 47.9 us, DeiT-Small FC2 12.1 -> 11.3 us).  ALTERNATE = false keeps every
// round in the same direction: the tabulated-GELU kernel on single CTAs is 7-10 % slower with the longer walk state.
template <bool PAIR, bool ALTERNATE>
struct TileWalk {
    int tt, ct;                  // the current tile: token tile, channel tile
    int c, nc, rank;             // channel unit (tile, or pair of tiles), units per row of tiles
    int dtt0, dc0, dtt1, dc1;    // step to the next round's tile after an even and after an odd round
    int odd;                     // parity of the current round
    __device__ __forceinline__ void start(const GemmParams& p, uint32_t rank_)
    {
        rank = (int)rank_;
        nc = PAIR ? (p.n_ct + 1) >> 1 : p.n_ct;
        const int first = PAIR ? (int)cluster_id_x() : (int)blockIdx.x;
        const int stride = PAIR ? (int)cluster_count_x() : (int)gridDim.x;
        tt = first / nc; c = first - tt * nc;
        const int s0 = ALTERNATE ? 2 * (stride - 1 - first) + 1 : stride, s1 = ALTERNATE ? 2 * first + 1 : stride;
        dtt0 = s0 / nc; dc0 = s0 - dtt0 * nc;
        dtt1 = s1 / nc; dc1 = s1 - dtt1 * nc;
        odd = 0;
        ct = PAIR ? 2 * c + rank : c;
    }
    // one round further (no division in the roles' loops)
    __device__ __forceinline__ void next()
    {
        if (ALTERNATE) { tt += odd ? dtt1 : dtt0; c += odd ? dc1 : dc0; odd ^= 1; }
        else { tt += dtt0; c += dc0; }
        if (c >= nc) { c -= nc; ++tt; }
        ct = PAIR ? 2 * c + rank : c;
    }
    __device__ __forceinline__ bool valid(const GemmParams& p) const { return tt < p.n_tt; }
};

// Tokens the MMAs of token tile tt cover: all TN, or, for the ragged last tile, what is left of M rounded up to 32
// (the MMA's N).  The last round of tiles is usually made of such tiles; they then cost their share of a full one.
__device__ __forceinline__ int tile_tokens(const GemmParams& p, int tt)
{
    return min(p.TN, (p.M - tt * p.TN + 31) & ~31);
}

// PAIR: two CTAs of a cluster compute 256 channels x TN tokens with one MMA stream (cta_group::2).  Each stages its
// own 128 weight rows and HALF of the activation tile (TN / 2 tokens), which lowers the operand traffic per SM from
// (128 + TN) to (128 + TN / 2) rows per 128-byte block of K; each receives its 128 channels x TN tokens in its own
// TMEM, so the epilogue is the same as without pairs.  The even CTA issues the MMAs: its `full` barriers count the
// bytes of both CTAs' copies, its `acc_empty` barriers the epilogue warps of both, and its commits signal the
// `empty` and `acc_full` barriers of both.
template <int EPI, int GELU_VARIANT, bool PAIR>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_i8_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
               const __grid_constant__ CUtensorMap map_y, const __grid_constant__ CUtensorMap map_res,
               const GemmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* ring = smem + p.off_ring;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + p.off_bar);
    uint64_t* empty_bar = full_bar + MAX_STAGES;
    uint64_t* acc_full = empty_bar + MAX_STAGES;  // [2]
    uint64_t* acc_empty = acc_full + 2;           // [2]
    uint64_t* res_bar = acc_empty + 2;            // [EPI_WARPS][2]: one per warp and staging buffer
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(res_bar + 2 * EPI_WARPS);
    CtaControl* ctl = reinterpret_cast<CtaControl*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int kblocks = (p.K + BK - 1) / BK;
    const int stages = p.stages;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;

    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], PAIR ? 2 * EPI_WARPS : EPI_WARPS); }
        for (int w = 0; w < 2 * EPI_WARPS; ++w) mbar_init(&res_bar[w], 1);
        ctl->abort = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_w);
        prefetch_tensormap(&map_x);
        prefetch_tensormap(&map_y);
        if (EPI == EPI_RESIDUAL) prefetch_tensormap(&map_res);
    }
    if (warp == 1) {
        if (PAIR) { tmem_alloc_pair(tmem_slot, TMEM_COLS); tmem_relinquish_pair(); }
        else { tmem_alloc(tmem_slot, TMEM_COLS); tmem_relinquish(); }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (PAIR) cluster_sync();                                  // the peer's barriers exist before anything signals them
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    grid_dep_launch();

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (elect_one()) {
            grid_dep_wait();                                   // the activations (and unpacked weights) come from earlier kernels
            int s = 0; uint32_t ph = 0;
            TileWalk<PAIR, PAIR || EPI != EPI_GELU_TAB> tw;
            for (tw.start(p, rank); tw.valid(p); tw.next()) {
                const int tt = tw.tt, ct = tw.ct;
                bool ok = true;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(&empty_bar[s], ph ^ 1u, ctl, p.status, 1)) { ok = false; break; }
                    uint8_t* st = ring + s * p.stage_bytes;
                    if (PAIR) {
                        // both CTAs' bytes are counted on the even CTA's barrier (a copy of the odd CTA that lands
                        // before the expectation is set only makes the pending count negative for a while)
                        const uint32_t full0 = map_to_cta(smem_u32(&full_bar[s]), 0);
                        if (rank == 0) mbar_expect_tx(&full_bar[s], 2u * (uint32_t)p.stage_bytes);
                        tma_load_2d_pair(st, &map_w, full0, kb * BK, ct * CT);
                        // the activation rows of a tile are split evenly between the two CTAs, also in a ragged tile
                        tma_load_2d_pair(st + W_BYTES, &map_x, full0, kb * BK, tt * p.TN + (int)rank * (tile_tokens(p, tt) >> 1));
                    } else {
                        mbar_expect_tx(&full_bar[s], (uint32_t)p.stage_bytes);
                        tma_load_2d(st, &map_w, &full_bar[s], kb * BK, ct * CT);
                        tma_load_2d(st + W_BYTES, &map_x, &full_bar[s], kb * BK, tt * p.TN);
                    }
                    if (++s == stages) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if ((!PAIR || rank == 0) && elect_one()) {
            const uint32_t idesc_full = umma_idesc_i8(PAIR ? 2 * CT : CT, p.TN, true, true, false, false);
            // K-major, 128-byte swizzle: 8-row groups are 1024 bytes apart.  The address field of a descriptor counts
            // 16-byte units from the start of shared memory (all of it fits the field), so the descriptor of stage s,
            // k-step k is the ring's descriptor plus (s * stage_bytes + 32 k) / 16: the loop below adds, it does not
            // rebuild
            const uint64_t desc_ring = umma_smem_desc(smem_u32(ring), 16, 1024, 128);
            const uint32_t stage16 = (uint32_t)p.stage_bytes >> 4;
            int s = 0; uint32_t ph = 0, soff = 0;
            TileWalk<PAIR, PAIR || EPI != EPI_GELU_TAB> tw;
            tw.start(p, rank);
            for (int it = 0; tw.valid(p); ++it, tw.next()) {
                const int tt = tw.tt;
                const int ab = it & 1;
                // the epilogue warps have pulled this accumulator's previous contents into registers
                if (!mbar_wait(&acc_empty[ab], ((uint32_t)(it >> 1) & 1u) ^ 1u, ctl, p.status, 2)) break;
                tc_fence_after_sync();
                const uint32_t tacc = tmem_base + (uint32_t)(ab * ACC_COLS);
                const int nt = tile_tokens(p, tt);
                const uint32_t idesc = nt == p.TN ? idesc_full
                                                  : umma_idesc_i8(PAIR ? 2 * CT : CT, nt, true, true, false, false);
                bool ok = true;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(&full_bar[s], ph, ctl, p.status, 3)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint64_t da0 = desc_ring + soff, db0 = da0 + (W_BYTES >> 4);
#pragma unroll
                    for (int k = 0; k < BK / 32; ++k) {
                        const uint64_t da = da0 + 2 * k, db = db0 + 2 * k;      // a k-step is 32 bytes
                        if (PAIR) umma_i8_pair(tacc, da, db, idesc, (kb | k) != 0 ? 1u : 0u);
                        else umma_i8(tacc, da, db, idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    // frees the stage (in both CTAs of a pair) once these MMAs have read it
                    if (PAIR) umma_commit_pair(&empty_bar[s], 3); else umma_commit(&empty_bar[s]);
                    soff += stage16;
                    if (++s == stages) { s = 0; soff = 0; ph ^= 1u; }
                }
                if (!ok) break;
                if (PAIR) umma_commit_pair(&acc_full[ab], 3); else umma_commit(&acc_full[ab]);   // accumulator complete
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        // Warp (quad, part) owns TMEM lanes 32*quad.. (the only ones it may touch) = 32 output channels, and the
        // token columns part * TN/4 .. of every tile; lane = channel.  Nothing here synchronises across warps.
        const int ew = warp - 2;
        const int quad = warp & 3;
        const int part = ew >> 2;
        const int tpp = p.TN >> 2;                             // tokens per part: 16, 32, 48 or 64
        const int nchunks = tpp >> 4;                          // 16-token chunks: 1..4
        // Staging blocks of this warp, [tpp tokens][32 channels] int8 each: one for the outputs and one for the
        // residual, or two of each used by alternate tiles.  With two, a tile neither waits for the copy engine to
        // have read the previous tile's outputs nor for a residual block that could only be requested once the
        // previous one had been consumed; it pays where the K loop is too short to cover those latencies.
        const int two = p.epi_bufs - 1;                        // 0 or 1
        const uint32_t buf_bytes = (uint32_t)(EPI_WARPS * tpp * 32);
        uint8_t* out_blk0 = smem + ew * (tpp * 32);
        // where this lane's words go after the transpose: token (lane % 4) of a group of four, channels 4 (lane / 4) ..
        const uint32_t out_word0 = smem_u32(out_blk0) + (uint32_t)((lane & 3) * 32 + (lane >> 2) * 4);
        const unsigned sel1 = (lane & 1) ? 0x3715u : 0x6240u, sel2 = (lane & 2) ? 0x3276u : 0x5410u;
        uint8_t* res_blk0 = smem + p.off_res + ew * (tpp * 32);
        const uint32_t res_lane0 = smem_u32(res_blk0) + (uint32_t)lane;
        uint32_t res_ph = 0;                                   // bit b: phase of staging buffer b's barrier
        // the byte pack of the store saturates to int8: narrower ranges (activations below 8 bits) are clamped first
        const bool sat8 = EPI == EPI_GELU ? (p.gelu.out.qmin == -128 && p.gelu.out.qmax == 127) : (p.qmin == -128 && p.qmax == 127);
        const uint32_t tab_mid = smem_u32(smem + p.off_tab) + 32768u;      // address of table[0 + 32768]
        if (EPI == EPI_GELU_TAB) {
            // the GELU table is static data: copy it while the previous kernel may still be running
            const int4* src = reinterpret_cast<const int4*>(p.gelu_tab);
            int4* dst = reinterpret_cast<int4*>(smem + p.off_tab);
            for (int i = ew * 32 + lane; i < IPTQ_GELU_TABLE_SIZE / 16; i += EPI_WARPS * 32) dst[i] = __ldg(src + i);
            named_barrier(1, EPI_WARPS * 32);
        }
        // The residual term R_res((res - zp) << 16) depends on the residual byte alone: its 256 values are tabulated
        // once per CTA, with the arithmetic the epilogue would otherwise run per output, and an output then costs a
        // second shared-memory read instead of a high multiply and a shift.
        const uint32_t rlut_mid = smem_u32(smem + p.off_tab) + 512u;        // address of the entry of residual byte 0
        if (EPI == EPI_RESIDUAL) {
            int* rl = reinterpret_cast<int*>(smem + p.off_tab);
            const int i = ew * 32 + lane;
            if (i < 256) rl[i] = requant_core((i - 128) * 65536 - p.res_off, p.res_mult, p.res_rnd, p.res_shift);
            named_barrier(1, EPI_WARPS * 32);
        }
        grid_dep_wait();                                       // residual reads and output writes come after this
        // Nothing in a tile's epilogue waits for something that was started in the same tile: the channel constants
        // and the residual block of tile i + 1 are requested during tile i.
        auto load_consts = [&](int ct_, int& cm_, int& cs_, int& cb_) {
            const int c = ct_ * CT + quad * 32 + lane;
            cm_ = 1 << 30; cs_ = 1; cb_ = 0;
            if (c < p.N) {
                cm_ = __ldg(p.mult + c);
                cs_ = (int)__ldg(p.shift + c);
                cb_ = p.bias ? __ldg(p.bias + c) : 0;
            }
        };
        auto request_residual = [&](int tt_, int ct_, int b_) {
            const int c0_ = ct_ * CT + quad * 32, tok0_ = tt_ * p.TN + part * tpp;
            if (c0_ < p.N && tok0_ < p.M && lane == 0) {
                mbar_expect_tx(&res_bar[2 * ew + b_], (uint32_t)(tpp * 32));
                tma_load_2d(res_blk0 + (uint32_t)b_ * buf_bytes, &map_res, &res_bar[2 * ew + b_], c0_, tok0_);
            }
        };
        const uint32_t acc_empty0 = PAIR ? map_to_cta(smem_u32(&acc_empty[0]), 0) : 0u;   // the even CTA's pair of barriers
        TileWalk<PAIR, PAIR || EPI != EPI_GELU_TAB> tw;
        tw.start(p, rank);
        int tt = tw.tt, ct = tw.ct;
        bool have = tw.valid(p);
        int cm, cs, cb;
        if (have) {
            load_consts(ct, cm, cs, cb);
            if (EPI == EPI_RESIDUAL) request_residual(tt, ct, 0);
        }
        for (int it = 0; have; ++it) {
            int ncm, ncs, ncb;
            tw.next();
            const int ntt = tw.tt, nct = tw.ct;
            const bool nhave = tw.valid(p);
            if (nhave) load_consts(nct, ncm, ncs, ncb);        // in flight during this tile
            const int sb = it & two;                           // staging buffer of this tile
            // the other buffer's residual bytes were consumed a tile ago (every lane has passed that tile's end)
            if (EPI == EPI_RESIDUAL && two && nhave) request_residual(ntt, nct, sb ^ 1);
            const uint32_t out_word = out_word0 + (uint32_t)sb * buf_bytes, res_lane = res_lane0 + (uint32_t)sb * buf_bytes;
            const int ab = it & 1;
            const uint32_t abph = (uint32_t)(it >> 1) & 1u;
            const int c0 = ct * CT + quad * 32;               // first channel of this warp
            const int tok0 = tt * p.TN + part * tpp;          // first token of this warp
            const bool active = c0 < p.N && tok0 < p.M;       // warp-uniform
            // The output zero point, which is added after the shift, goes into the rounding constant, shifted left,
            // where every channel of the warp has a shift small enough for that (the sum stays below 2^31).
            const bool fold = EPI == EPI_REQUANT && __all_sync(0xffffffffu, cs <= 20);
            const int crnd = (1 << (cs - 1)) + (fold ? p.out_zp << cs : 0);
            // the residual epilogue, whose other half already is an add and a high multiply per output, is faster with
            // bias and rounding constant in the 64-bit addend of one wide multiply-add (measured: 5 % at K = 96)
            const long long c64 = (long long)cb * (long long)cm + ((long long)(1 << (cs - 1)) << 32);
            if (!mbar_wait(&acc_full[ab], abph, ctl, p.status, 4)) break;
            tc_fence_after_sync();
            // the store that last used this tile's output block has read it (one or two K loops ago)
            if (lane == 0) { if (two) bulk_wait_read_but_one(); else bulk_wait_read_all(); }
            __syncwarp();
            if (EPI == EPI_RESIDUAL && active) {
                if (!mbar_wait(&res_bar[2 * ew + sb], (res_ph >> sb) & 1u, ctl, p.status, 5)) break;
                res_ph ^= 1u << sb;
            }
            const uint32_t tacc = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(ab * ACC_COLS + part * tpp);
            uint32_t acc[2][16];
            tmem_ld16(tacc, acc[0]);
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                if (ch < nchunks) {                            // warp-uniform
                    tmem_wait_ld();                            // chunk ch is in registers
                    if (ch + 1 < nchunks) {
                        tmem_ld16(tacc + (uint32_t)((ch + 1) * 16), acc[(ch + 1) & 1]);   // in flight during the arithmetic
                    } else {
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) {                       // the MMA warp may refill this accumulator
                            if (PAIR) mbar_arrive_cluster(acc_empty0 + (uint32_t)(ab * 8)); else mbar_arrive(&acc_empty[ab]);
                        }
                    }
                    if (active) {
                        // Three passes over the chunk, so that the shared-memory reads (volatile, hence kept in
                        // program order with the stores) are issued back to back instead of one per stored byte.
                        int v[16], r[16];
                        if (EPI == EPI_RESIDUAL) {
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                asm volatile("ld.shared.s8 %0, [%1];" : "=r"(r[j]) : "r"(res_lane + (uint32_t)((ch * 16 + j) * 32)));
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(r[j]) : "r"(rlut_mid + (uint32_t)(r[j] * 4)));
                        }
                        // R of the header: hi32((acc + bias) * mult) + rounding constant, shifted.  The bias add is
                        // written as add-then-max against INT_MIN: a plain add is moved to the multiplier's pipe by the
                        // assembler, which is the pipe this loop is short of.
                        if (fold) {
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                v[j] = mad_hi(__viaddmax_s32((int)acc[ch & 1][j], cb, p.acc_floor), cm, crnd) >> cs;
                                if (!sat8) v[j] = max(p.qmin, min(p.qmax, v[j]));
                            }
                        } else
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            if (EPI == EPI_RESIDUAL) v[j] = mad_wide_hi((int)acc[ch & 1][j], cm, c64) >> cs;
                            else v[j] = mad_hi(__viaddmax_s32((int)acc[ch & 1][j], cb, p.acc_floor), cm, crnd) >> cs;
                            if (EPI == EPI_GELU_TAB) {
                                v[j] = max(-32768, min(32767, v[j])) + (int)tab_mid;
                            } else if (EPI == EPI_GELU) {
                                v[j] = requant_nosat(gelu_core<GELU_VARIANT>(v[j], p.gelu), p.gelu.out);
                                if (!sat8) v[j] = max(p.gelu.out.qmin, min(p.gelu.out.qmax, v[j]));
                            } else if (EPI == EPI_RESIDUAL) {
                                v[j] += r[j] + p.out_zp;
                                if (!sat8) v[j] = max(p.qmin, min(p.qmax, v[j]));
                            } else {
                                v[j] += p.out_zp;
                                if (!sat8) v[j] = max(p.qmin, min(p.qmax, v[j]));
                            }
                        }
                        if (EPI == EPI_GELU_TAB) {
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                asm volatile("ld.shared.s8 %0, [%1];" : "=r"(v[j]) : "r"((uint32_t)v[j]));
                        }
                        // Four tokens of this lane's channel are packed into a word (saturating to int8), then a 4 x 4
                        // byte transpose over the four lanes of a group (two shuffle + byte-permute rounds) leaves
                        // lane m of the group with token m of the four for the group's four channels: one 32-bit
                        // store per four outputs, every lane of the warp on its own bank (byte stores of four lanes
                        // into one word took 2.7 shared-memory passes each).
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            unsigned w = pack4_sat_s8(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
                            w = __byte_perm(w, __shfl_xor_sync(0xffffffffu, w, 1), sel1);
                            w = __byte_perm(w, __shfl_xor_sync(0xffffffffu, w, 2), sel2);
                            asm volatile("st.shared.b32 [%0], %1;" ::"r"(out_word + (uint32_t)((ch * 16 + 4 * g) * 32)), "r"(w) : "memory");
                        }
                    }
                }
            }
            if (active) {
                fence_proxy_async_smem();                     // this lane's shared-memory stores -> visible to the TMA engine
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(&map_y, out_blk0 + (uint32_t)sb * buf_bytes, c0, tok0);  // clipped at N and M
                    bulk_commit();
                }
            }
            __syncwarp();                                      // every lane has read its residual bytes of this tile
            if (EPI == EPI_RESIDUAL && !two && nhave) request_residual(ntt, nct, 0);
            have = nhave; tt = ntt; ct = nct; cm = ncm; cs = ncs; cb = ncb;
        }
        if (lane == 0) bulk_wait_all();                       // stores complete before shared memory goes away
    }

    // ------------------------------------------------------------ teardown (also reached after an abort)
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    if (ctl->abort) {
        // give copies that are still in flight time to land before shared memory is released
        for (int i = 0; i < 64; ++i) __nanosleep(2000);
        __syncthreads();
    }
    if (PAIR) cluster_sync();                                  // neither CTA leaves while the other may still reach into it
    if (warp == 1) {
        tc_fence_after_sync();
        if (PAIR) tmem_dealloc_pair(tmem_base, TMEM_COLS); else tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ---------------------------------------------------------------- W4: unpack nibbles to int8
__global__ void unpack_int4_kernel(const uint8_t* __restrict__ packed, int8_t* __restrict__ out, int64_t nbytes)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    grid_dep_launch();
    grid_dep_wait();                                // the scratch may still be read by the previous kernel
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nbytes; i += stride) {
        const unsigned b = packed[i];
        const int lo = (int)(b & 15u), hi = (int)(b >> 4);
        char2 v;
        v.x = (char)(lo >= 8 ? lo - 16 : lo);                 // element 2i   (low nibble)
        v.y = (char)(hi >= 8 ? hi - 16 : hi);                 // element 2i+1 (high nibble)
        reinterpret_cast<char2*>(out)[i] = v;
    }
}

static int unpack_int4_bytes_launch(const void* packed, int8_t* out, int64_t n_elems, cudaStream_t st)
{
    const int64_t nbytes = n_elems / 2;
    const int grid = (int)std::min<int64_t>((nbytes + 255) / 256, (int64_t)sm_count() * 8);
    launch_kernel(unpack_int4_kernel, grid, 256, 0, st, static_cast<const uint8_t*>(packed), out, nbytes);
    note_launch();
    return last_launch_status();
}

// Up to four weight matrices in one launch (the head of a W4 encoder block): 16 packed bytes -> 32 int8 per step.
// The low nibbles L and high nibbles H of a word are sign-extended byte-wise ((v ^ 8) - 8, with bit 7 set during the
// subtraction so that no borrow crosses a byte) and interleaved back into element order.
struct UnpackSegs {
    const uint4* src[4];
    uint4* dst[4];
    int64_t nvec[4];           // 16-byte input vectors per segment
};

__device__ __forceinline__ unsigned sext_nibbles(unsigned v)
{
    return (((v ^ 0x08080808u) | 0x80808080u) - 0x08080808u) ^ 0x80808080u;
}

__global__ void __launch_bounds__(256) unpack_int4_multi_kernel(const UnpackSegs s)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    grid_dep_launch();
    grid_dep_wait();                                // the scratch may still be read by the previous kernel
#pragma unroll 1
    for (int seg = 0; seg < 4; ++seg) {
        for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < s.nvec[seg]; i += stride) {
            const uint4 pk = __ldg(s.src[seg] + i);
            const unsigned w[4] = {pk.x, pk.y, pk.z, pk.w};
            unsigned o[8];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const unsigned lo = sext_nibbles(w[k] & 0x0f0f0f0fu), hi = sext_nibbles((w[k] >> 4) & 0x0f0f0f0fu);
                o[2 * k] = __byte_perm(lo, hi, 0x5140);        // elements 0..3 of the word: l0 h0 l1 h1
                o[2 * k + 1] = __byte_perm(lo, hi, 0x7362);    // elements 4..7: l2 h2 l3 h3
            }
            s.dst[seg][2 * i] = make_uint4(o[0], o[1], o[2], o[3]);
            s.dst[seg][2 * i + 1] = make_uint4(o[4], o[5], o[6], o[7]);
        }
    }
}

// count <= 4 matrices; falls back to one launch per matrix when a pointer or a size does not allow 16-byte vectors
int unpack_int4_multi_launch(const void* const* packed, int8_t* const* out, const int64_t* n_elems, int count,
                             cudaStream_t st)
{
    bool vec = count >= 1 && count <= 4;
    for (int i = 0; vec && i < count; ++i)
        vec = aligned16(packed[i]) && aligned16(out[i]) && n_elems[i] % 32 == 0;
    if (!vec) {
        for (int i = 0; i < count; ++i) {
            int rc = unpack_int4_bytes_launch(packed[i], out[i], n_elems[i], st);
            if (rc != IPTQ_OK) return rc;
        }
        return IPTQ_OK;
    }
    UnpackSegs s{};
    int64_t total = 0;
    for (int i = 0; i < count; ++i) {
        s.src[i] = static_cast<const uint4*>(packed[i]);
        s.dst[i] = reinterpret_cast<uint4*>(out[i]);
        s.nvec[i] = n_elems[i] / 32;
        total = std::max(total, s.nvec[i]);
    }
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((total + 255) / 256, (int64_t)sm_count() * 8));
    launch_kernel(unpack_int4_multi_kernel, grid, 256, 0, st, s);
    note_launch();
    return last_launch_status();
}

// one matrix: the vector kernel when pointers and size allow it, the byte-wise one otherwise
int unpack_int4_launch(const void* packed, int8_t* out, int64_t n_elems, cudaStream_t st)
{
    return unpack_int4_multi_launch(&packed, &out, &n_elems, 1, st);
}

// ---------------------------------------------------------------- launcher
template <int EPI, int GV, bool PAIR>
static int launch_gemm_as(const CUtensorMap& mw, const CUtensorMap& mx, const CUtensorMap& my, const CUtensorMap& mr,
                          const GemmParams& p, int grid, int smem_bytes, cudaStream_t st)
{
    auto kern = gemm_i8_kernel<EPI, GV, PAIR>;
    static bool configured[64];               // one attribute call per instantiation and device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return IPTQ_ERR_CUDA;
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT) != cudaSuccess)
            return IPTQ_ERR_CUDA;
        configured[dev] = true;
    }
    if (PAIR) launch_kernel_cluster(kern, grid, GEMM_THREADS, smem_bytes, st, 2u, mw, mx, my, mr, p);
    else launch_kernel(kern, grid, GEMM_THREADS, smem_bytes, st, mw, mx, my, mr, p);
    note_launch();
    return last_launch_status();
}

template <int EPI, int GV>
static int launch_gemm(const CUtensorMap& mw, const CUtensorMap& mx, const CUtensorMap& my, const CUtensorMap& mr,
                       const GemmParams& p, bool pair, int grid, int smem_bytes, cudaStream_t st)
{
    return pair ? launch_gemm_as<EPI, GV, true>(mw, mx, my, mr, p, grid, smem_bytes, st)
                : launch_gemm_as<EPI, GV, false>(mw, mx, my, mr, p, grid, smem_bytes, st);
}

int linear_check(const LinearArgs& a)
{
    if (!a.x || !a.w || !a.mult || !a.shift || !a.y) return IPTQ_ERR_NULL;
    if (a.M < 0 || a.M > (int64_t)1 << 30 || a.N < 16 || a.K < 16 || a.K > 4096 || (a.N & 15) || (a.K & 15))
        return IPTQ_ERR_SHAPE;
    if (!aligned16(a.x) || !aligned16(a.w) || !aligned16(a.y) || (a.residual && !aligned16(a.residual)) ||
        (a.bias && (reinterpret_cast<uintptr_t>(a.bias) & 3u)) || (reinterpret_cast<uintptr_t>(a.mult) & 3u))
        return IPTQ_ERR_ALIGN;
    if (a.residual) { int rc = check_requant(a.residual_rq); if (rc != IPTQ_OK) return rc; }
    if (a.gelu) {
        if (a.gelu->in_bits < 8 || a.gelu->in_bits > 16) return IPTQ_ERR_BITS;
        if (a.gelu->variant < 0 || a.gelu->variant > 2) return IPTQ_ERR_VARIANT;
        int rc = check_requant(&a.gelu->out); if (rc != IPTQ_OK) return rc;
        if (a.gelu->table && !aligned16(a.gelu->table)) return IPTQ_ERR_ALIGN;
    }
    if (a.out_bits < 4 || a.out_bits > 8) return IPTQ_ERR_BITS;
    if (!a.status) return IPTQ_ERR_WORKSPACE;
    return IPTQ_OK;
}

// Shared-memory layout for a tile width: output blocks, residual blocks, GELU table, barriers, then as many ring
// stages as fit.  Returns the number of stages (0: does not fit).
static int gemm_layout(GemmParams& p, int TN, bool pair, bool residual, bool table, int kblocks, int epi_bufs,
                       int* smem_bytes)
{
    const int blocks = epi_bufs * EPI_WARPS * (TN / 4) * 32;  // = 128 TN bytes per buffer
    p.TN = TN;
    p.epi_bufs = epi_bufs;
    p.off_res = blocks;
    p.off_tab = p.off_res + (residual ? blocks : 0);
    p.off_bar = p.off_tab + (table ? IPTQ_GELU_TABLE_SIZE : residual ? 1024 : 0);   // GELU table, or residual terms
    p.off_ring = (p.off_bar + (2 * MAX_STAGES + 4 + 2 * EPI_WARPS) * 8 + 16 + 1023) & ~1023;
    p.stage_bytes = W_BYTES + (pair ? TN / 2 : TN) * BK;      // a CTA of a pair stages half of the activation tile
    const int room = SMEM_LIMIT - 1024 - p.off_ring;          // 1024: slack for the alignment of the dynamic base
    if (room < 0) return 0;
    int stages = std::min(MAX_STAGES, room / p.stage_bytes);
    // a ring much longer than one tile's K loop buys nothing, and a smaller footprint lets the next kernel's CTAs
    // become resident earlier
    stages = std::min(stages, std::max(2, kblocks + 1));
    p.stages = stages;
    *smem_bytes = p.off_ring + stages * p.stage_bytes + 1024;
    return stages;
}

// CTA pairs pay where the mainloop waits for operands: a reduction of six blocks of K or more (measured on ViT-Base:
// QKV 40.3 -> 37.6 us, FC1 + GELU 66.5 -> 58.5 us, FC2 62.6 -> 49.7 us; at three blocks, DeiT-Small, pairs lose),
// 256 tokens per tile, at least two channel tiles, and three rounds of pair tiles or more.
static bool use_pairs(const LinearArgs& a, int n_ct, int kblocks, int sms)
{
    return kblocks >= 6 && a.M > 192 && n_ct >= 2 && sms >= 2 &&
           (int64_t)((n_ct + 1) / 2) * ((a.M + 255) / 256) >= 3 * (int64_t)(sms / 2);   // three rounds of pair tiles
}

// Tile width, ring depth, single CTAs or pairs, grid: fills p.TN, p.n_tt and the shared-memory layout.  Single CTAs
// take the widest tile that fits beside a ring of at least three stages and is not mostly padding: a wide tile
// amortises the weight tile (the operand bytes per MMA clock fall from 128 B at 128 tokens to 96 B at 256) and beat
// every narrower one that was measured, even where it leaves the last round of tiles half empty.
static int gemm_plan(GemmParams& p, int64_t M, bool residual, bool table, int sms, bool* pair_out, int* smem_bytes,
                     int* grid)
{
    const int kblocks = (p.K + BK - 1) / BK;
    LinearArgs shape{};
    shape.M = M;
    const bool pair = use_pairs(shape, p.n_ct, kblocks, sms);
    int best_tn = 0;
    // A long reduction over few tiles (at most two rounds of 256-token tiles) is paced by the K loop of the last
    // round: half-width tiles on twice the CTAs finish sooner (DeiT-Small FC2: 15.2 us at 256, 12.3 us at 128).
    const int64_t tiles256 = (int64_t)p.n_ct * ((M + 255) / 256), tiles128 = (int64_t)p.n_ct * ((M + 127) / 128);
    const bool narrow = !pair && kblocks >= 8 && M > 128 && tiles256 <= 2 * (int64_t)sms && tiles256 > sms / 2 &&
                        tiles128 <= 3 * (int64_t)sms;
    // Less than one round of 256-token tiles (small batches): the kernel's time is one tile's K loop followed by its
    // epilogue on a few SMs, so the narrowest tile that still fits one round wins, else two rounds of 128-token
    // tiles, whose second epilogue runs under nothing but is half as long (1576 tokens: 768 x 3072 16.5 -> 9.4 us,
    // 384 x 1536 11.3 -> 5.3 us, 2304 x 768 7.2 -> 6.7 us; 197 tokens: 5.6-8.3 -> 3.6-4.4 us).
    const bool small = !pair && !narrow && M > 64 && tiles256 <= sms;
    if (small) {
        const int64_t tiles64 = (int64_t)p.n_ct * ((M + 63) / 64);
        best_tn = tiles64 <= sms ? 64 : 128;
    } else if (pair) best_tn = 256;
    else for (int TN : {256, 192, 128, 64}) {
        if (narrow && TN > 128) continue;
        GemmParams q = p;
        int sb;
        if (TN > 64 && M <= TN - 64) continue;                // a narrower tile covers all tokens
        if (gemm_layout(q, TN, false, residual, table, kblocks, 1, &sb) < std::min(3, kblocks + 1)) continue;
        best_tn = TN;
        break;
    }
    if (best_tn == 0) return IPTQ_ERR_SHAPE;
    // Two staging buffers per epilogue warp where they cost no ring stage (short reductions, whose K loop does not
    // cover the latency of the output store and of the residual load).
    int epi_bufs = 1;
    {
        GemmParams q1 = p, q2 = p;
        int sb1, sb2;
        if (gemm_layout(q2, best_tn, pair, residual, table, kblocks, 2, &sb2) >=
            gemm_layout(q1, best_tn, pair, residual, table, kblocks, 1, &sb1)) epi_bufs = 2;
    }
    if (gemm_layout(p, best_tn, pair, residual, table, kblocks, epi_bufs, smem_bytes) < 2) return IPTQ_ERR_SHAPE;
    const int64_t n_tt = (M + p.TN - 1) / p.TN;
    if ((int64_t)p.n_ct * n_tt > (int64_t)1 << 30) return IPTQ_ERR_SHAPE;
    p.n_tt = (int)n_tt;
    *grid = pair ? 2 * (int)std::min<int64_t>((int64_t)((p.n_ct + 1) / 2) * n_tt, sms / 2)
                 : (int)std::min<int64_t>((int64_t)p.n_ct * n_tt, sms);
    *pair_out = pair;
    return IPTQ_OK;
}

int linear_launch(const LinearArgs& a, cudaStream_t st)
{
    const int rc0 = linear_check(a);
    if (rc0 != IPTQ_OK) return rc0;
    if (a.M == 0) return IPTQ_OK;

    GemmParams p;
    p.M = (int)a.M; p.N = a.N; p.K = a.K;
    p.n_ct = (a.N + CT - 1) / CT;
    p.bias = a.bias; p.mult = a.mult; p.shift = a.shift; p.out_zp = a.out_zp;
    p.acc_floor = INT_MIN;
    p.qmin = -(1 << (a.out_bits - 1)); p.qmax = (1 << (a.out_bits - 1)) - 1;
    p.res_mult = p.res_rnd = p.res_shift = p.res_off = 0;
    if (a.residual) {
        p.res_mult = a.residual_rq->mult; p.res_shift = a.residual_rq->shift;
        p.res_rnd = 1 << (a.residual_rq->shift - 1); p.res_off = a.residual_rq->zp * 65536;
    }
    p.status = a.status;
    if (a.gelu) p.gelu = to_dev(*a.gelu);
    else { iptq_gelu_consts z{}; z.in_bits = 8; z.out.shift = 1; p.gelu = to_dev(z); }
    const bool table = a.gelu && a.gelu->table;
    p.gelu_tab = table ? a.gelu->table : nullptr;

    const int kblocks = (a.K + BK - 1) / BK;
    bool pair = false;
    int smem_bytes = 0, grid = 0;
    const int rcp = gemm_plan(p, a.M, a.residual != nullptr, table, sm_count(), &pair, &smem_bytes, &grid);
    if (rcp != IPTQ_OK) return rcp;
    (void)kblocks;

    CUtensorMap mw, mx, my, mr;
    int rc;
    {
        const uint64_t dims[2] = {(uint64_t)a.K, (uint64_t)a.N};
        const uint64_t str[1] = {(uint64_t)a.K};
        const uint32_t box[2] = {BK, CT};
        if ((rc = make_tensor_map_u8(&mw, a.w, 2, dims, str, box, 128)) != IPTQ_OK) return rc;
    }
    {
        const uint64_t dims[2] = {(uint64_t)a.K, (uint64_t)a.M};
        const uint64_t str[1] = {(uint64_t)a.K};
        const uint32_t box[2] = {BK, (uint32_t)(pair ? p.TN / 2 : p.TN)};
        if ((rc = make_tensor_map_u8(&mx, a.x, 2, dims, str, box, 128)) != IPTQ_OK) return rc;
    }
    {
        // output and residual: one [TN / 4 tokens][32 channels] block per epilogue warp, clipped at M and N by the copy engine
        const uint64_t dims[2] = {(uint64_t)a.N, (uint64_t)a.M};
        const uint64_t str[1] = {(uint64_t)a.N};
        const uint32_t box[2] = {32, (uint32_t)(p.TN / 4)};
        if ((rc = make_tensor_map_u8(&my, a.y, 2, dims, str, box, 0)) != IPTQ_OK) return rc;
        if ((rc = make_tensor_map_u8(&mr, a.residual ? a.residual : a.y, 2, dims, str, box, 0)) != IPTQ_OK) return rc;
    }
    if (table) return launch_gemm<EPI_GELU_TAB, 0>(mw, mx, my, mr, p, pair, grid, smem_bytes, st);   // the variant is in the table
    if (a.gelu) {
        switch (a.gelu->variant) {
            case IPTQ_GELU_POLY4: return launch_gemm<EPI_GELU, IPTQ_GELU_POLY4>(mw, mx, my, mr, p, pair, grid, smem_bytes, st);
            case IPTQ_GELU_POLY2: return launch_gemm<EPI_GELU, IPTQ_GELU_POLY2>(mw, mx, my, mr, p, pair, grid, smem_bytes, st);
            default: return launch_gemm<EPI_GELU, IPTQ_GELU_SHIFT>(mw, mx, my, mr, p, pair, grid, smem_bytes, st);
        }
    }
    if (a.residual) return launch_gemm<EPI_RESIDUAL, 0>(mw, mx, my, mr, p, pair, grid, smem_bytes, st);
    return launch_gemm<EPI_REQUANT, 0>(mw, mx, my, mr, p, pair, grid, smem_bytes, st);
}

static size_t align256(size_t v) { return (v + 255) & ~size_t(255); }

// ---------------------------------------------------------------- library-owned scratch (no-allocation entry point)
// [status block | unpacked int8 weights].  Every GPU that loads the library holds this array until the
// process exits.  In host code the name below is only a stand-in for the symbol: the device address comes from
// cudaGetSymbolAddress(), asked once per device with that device current.
static __device__ __align__(256) uint8_t g_static_scratch[kStatusBytes + IPTQ_STATIC_SCRATCH_BYTES];

static int static_scratch_ptr(uint8_t** out)
{
    static std::mutex mu;
    static uint8_t* per_device[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return IPTQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!per_device[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return IPTQ_ERR_CUDA;
        per_device[dev] = static_cast<uint8_t*>(ptr);
    }
    *out = per_device[dev];
    return IPTQ_OK;
}

}  // namespace iptq

using namespace iptq;

extern "C" {

size_t iptq_linear_workspace_bytes(int64_t M, int N, int K, int w_bits)
{
    (void)M;
    size_t b = kStatusBytes;
    if (w_bits == 4 && N > 0 && K > 0) b += align256((size_t)N * (size_t)K);
    return b;
}

int iptq_linear_plan(int64_t M, int N, int K, int has_residual, int has_gelu_table, int sm_count_in,
                     iptq_linear_plan_info* out)
{
    if (!out) return IPTQ_ERR_NULL;
    if (M < 1 || M > (int64_t)1 << 30 || N < 16 || K < 16 || K > 4096 || (N & 15) || (K & 15)) return IPTQ_ERR_SHAPE;
    const int sms = sm_count_in > 0 ? sm_count_in : sm_count();
    if (sms < 1) return IPTQ_ERR_CUDA;
    GemmParams p{};
    p.M = (int)M; p.N = N; p.K = K;
    p.n_ct = (N + CT - 1) / CT;
    bool pair = false;
    int smem_bytes = 0, grid = 0;
    const int rc = gemm_plan(p, M, has_residual != 0, has_gelu_table != 0, sms, &pair, &smem_bytes, &grid);
    if (rc != IPTQ_OK) return rc;
    out->tile_tokens = p.TN; out->stages = p.stages; out->cta_pairs = pair ? 1 : 0;
    out->smem_bytes = smem_bytes; out->grid = grid;
    out->channel_tiles = p.n_ct; out->token_tiles = p.n_tt; out->staging_buffers = p.epi_bufs;
    return IPTQ_OK;
}

int iptq_linear(const int8_t* x, const void* w, int w_bits, const int32_t* bias, const int32_t* mult,
                const int8_t* shift, int32_t out_zp, const int8_t* residual, const iptq_requant* residual_rq,
                int8_t* y, int64_t M, int N, int K, void* ws, size_t ws_bytes, iptq_stream_t stream)
{
    return iptq_linear_bits(x, w, w_bits, bias, mult, shift, out_zp, residual, residual_rq, y, M, N, K, 8, ws, ws_bytes,
                            stream);
}

int iptq_linear_bits(const int8_t* x, const void* w, int w_bits, const int32_t* bias, const int32_t* mult,
                     const int8_t* shift, int32_t out_zp, const int8_t* residual, const iptq_requant* residual_rq,
                     int8_t* y, int64_t M, int N, int K, int out_bits, void* ws, size_t ws_bytes,
                     iptq_stream_t stream)
{
    if (w_bits != 8 && w_bits != 4) return IPTQ_ERR_BITS;
    if (out_bits < 4 || out_bits > 8) return IPTQ_ERR_BITS;
    if (!ws) return IPTQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return IPTQ_ERR_ALIGN;
    if (N < 1 || K < 1) return IPTQ_ERR_SHAPE;
    if (ws_bytes < iptq_linear_workspace_bytes(M, N, K, w_bits)) return IPTQ_ERR_WORKSPACE;
    if (!w) return IPTQ_ERR_NULL;
    // every argument is checked before the first launch (the unpack kernel included)
    const int8_t* w8 = w_bits == 4 ? static_cast<const int8_t*>(ws) + kStatusBytes : static_cast<const int8_t*>(w);
    LinearArgs a{x, w8, bias, mult, shift, out_zp, residual, residual_rq, nullptr, y, M, N, K,
                 static_cast<StatusBlock*>(ws), out_bits};
    int rc = linear_check(a);
    if (rc != IPTQ_OK) return rc;
    if (w_bits == 4) {
        if (M > 0 && (rc = unpack_int4_launch(w, const_cast<int8_t*>(w8), (int64_t)N * K, stream)) != IPTQ_OK) return rc;
    }
    return linear_launch(a, stream);
}

int iptq_linear_w4_static(const int8_t* x, const void* w_packed, const int32_t* bias, const int32_t* mult,
                          const int8_t* shift, int32_t out_zp, const int8_t* residual,
                          const iptq_requant* residual_rq, int8_t* y, int64_t M, int N, int K, void* status,
                          iptq_stream_t stream)
{
    if (!w_packed) return IPTQ_ERR_NULL;
    if (N < 1 || K < 1 || (K & 1)) return IPTQ_ERR_SHAPE;
    if ((size_t)N * (size_t)K > (size_t)IPTQ_STATIC_SCRATCH_BYTES) return IPTQ_ERR_WORKSPACE;
    if (status && (reinterpret_cast<uintptr_t>(status) & 255u)) return IPTQ_ERR_ALIGN;
    uint8_t* base = nullptr;
    int rc = static_scratch_ptr(&base);            // first call on this device: looks the array's address up
    if (rc != IPTQ_OK) return rc;
    StatusBlock* st = status ? static_cast<StatusBlock*>(status) : reinterpret_cast<StatusBlock*>(base);
    int8_t* w8 = reinterpret_cast<int8_t*>(base + kStatusBytes);
    LinearArgs a{x, w8, bias, mult, shift, out_zp, residual, residual_rq, nullptr, y, M, N, K, st};
    if ((rc = linear_check(a)) != IPTQ_OK) return rc;          // nothing is enqueued for a call that is rejected
    if (M == 0) return IPTQ_OK;
    // the built-in status block keeps the previous call's contents: it must start at zero
    if (!status && cudaMemsetAsync(st, 0, kStatusBytes, stream) != cudaSuccess) return IPTQ_ERR_CUDA;
    if ((rc = unpack_int4_launch(w_packed, w8, (int64_t)N * K, stream)) != IPTQ_OK) return rc;
    return linear_launch(a, stream);
}

size_t iptq_mlp_workspace_bytes(int64_t M, int D, int Dh, int w_bits)
{
    size_t b = kStatusBytes;
    if (M > 0 && Dh > 0) b += align256((size_t)M * (size_t)Dh);               // hidden activations
    if (w_bits == 4 && D > 0 && Dh > 0) b += 2 * align256((size_t)D * (size_t)Dh);
    return b;
}

int iptq_mlp_block(const int8_t* x, const void* w1, const int32_t* b1, const int32_t* m1, const int8_t* s1,
                   const iptq_gelu_consts* gelu, const void* w2, const int32_t* b2, const int32_t* m2,
                   const int8_t* s2, int32_t out_zp, const int8_t* residual, const iptq_requant* residual_rq,
                   int8_t* y, int64_t M, int D, int Dh, int w_bits, void* ws, size_t ws_bytes,
                   iptq_stream_t stream)
{
    if (w_bits != 8 && w_bits != 4) return IPTQ_ERR_BITS;
    if (!gelu || !w1) return IPTQ_ERR_NULL;
    if (!ws) return IPTQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return IPTQ_ERR_ALIGN;
    if (M < 0 || D < 1 || Dh < 1) return IPTQ_ERR_SHAPE;
    if (ws_bytes < iptq_mlp_workspace_bytes(M, D, Dh, w_bits)) return IPTQ_ERR_WORKSPACE;
    uint8_t* base = static_cast<uint8_t*>(ws);
    StatusBlock* status = reinterpret_cast<StatusBlock*>(base);
    int8_t* hidden = reinterpret_cast<int8_t*>(base + kStatusBytes);
    size_t off = kStatusBytes + align256((size_t)M * (size_t)Dh);
    const int8_t* w1_8 = static_cast<const int8_t*>(w1);
    const int8_t* w2_8 = static_cast<const int8_t*>(w2);
    int8_t* dsts[2] = {reinterpret_cast<int8_t*>(base + off),
                       reinterpret_cast<int8_t*>(base + off + align256((size_t)D * (size_t)Dh))};
    if (w_bits == 4) {
        w1_8 = dsts[0];
        if (w2) w2_8 = dsts[1];
    }
    // FC1 with the GELU epilogue; without FC2 the activations go straight to y
    LinearArgs fc1{x, w1_8, b1, m1, s1, 0, nullptr, nullptr, gelu, w2 ? hidden : y, M, Dh, D, status};
    LinearArgs fc2{hidden, w2_8, b2, m2, s2, out_zp, residual, residual_rq, nullptr, y, M, D, Dh, status};
    // every argument of both layers is checked before the first launch (the unpack kernel included)
    int rc = linear_check(fc1);
    if (rc == IPTQ_OK && w2) rc = linear_check(fc2);
    if (rc != IPTQ_OK) return rc;
    if (w_bits == 4) {
        const void* srcs[2] = {w1, w2};
        const int64_t ns[2] = {(int64_t)D * Dh, (int64_t)D * Dh};
        if (M > 0 && (rc = unpack_int4_multi_launch(srcs, dsts, ns, w2 ? 2 : 1, stream)) != IPTQ_OK) return rc;   // both matrices in one launch
    }
    rc = linear_launch(fc1, stream);
    if (rc != IPTQ_OK || !w2) return rc;
    return linear_launch(fc2, stream);
}

int iptq_unpack_int4(const void* packed, int8_t* out, int64_t n_elems, iptq_stream_t stream)
{
    if (n_elems < 0 || (n_elems & 1)) return IPTQ_ERR_SHAPE;
    if (n_elems == 0) return IPTQ_OK;
    if (!packed || !out) return IPTQ_ERR_NULL;
    if (!aligned16(packed) || !aligned16(out)) return IPTQ_ERR_ALIGN;
    return unpack_int4_launch(packed, out, n_elems, stream);
}

}  // extern "C"
