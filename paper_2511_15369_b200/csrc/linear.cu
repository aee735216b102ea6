// INT8 x INT8 -> INT32 GEMM on the 5th-generation tensor cores (tcgen05.mma.kind::i8, TMEM accumulators,
// TMA-fed shared-memory pipeline) with the integer epilogues of the path applied straight out of TMEM:
//   - per-channel dyadic requantisation (QKV, proj, FC2), optionally with the int8 residual branch;
//   - FC1: requantise to the GELU input scale, integer GELU (Sec. 3.3, Eqs. (3), (5)), requantise to int8.
// No int32 intermediate is written to HBM.
//
// One persistent CTA per SM, 14 warps: warp 0 = TMA producer, warp 1 = MMA issuer (owns TMEM),
// warps 2..13 = epilogue (three warps per TMEM lane quadrant, each taking a third of the tile's columns).
// The accumulator is double-buffered in TMEM so that the epilogue of tile i overlaps the mainloop of tile i+1.
// Per-column requantisation constants live in TMEM beside the accumulators (shared-memory reads of them would
// cost one load per output and saturate the load/store pipe); the bias is written into each accumulator before
// the MMAs start, which then always accumulate.
#include <algorithm>
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
enum { EPI_REQUANT = 0, EPI_RESIDUAL = 1, EPI_GELU = 2 };

constexpr int BM = 128;          // rows per tile = TMEM lanes
constexpr int BK = 128;          // bytes of K per stage = one 128-byte swizzle row = 4 MMA k-steps
constexpr int COLS = 32;         // columns per epilogue warp: bytes per output row, one 32-byte swizzle row
constexpr uint32_t TMEM_COLS = 512;

// Tile width BN is 96 or 128.  TMEM holds two accumulators plus per-column constant rows (one row = BN words,
// replicated over the 128 lanes so that a thread reads them with the same instruction as its accumulators):
//   BN =  96: mult, rounding constant, shift           (5 x 96 = 480 columns)
//   BN = 128: mult, shift - 1; the rounding constant 2^(shift-1) is rebuilt with one shift  (4 x 128 = 512 columns)
// GTAB: the FC1 epilogue reads the integer GELU from a 64 KB table in shared memory, which leaves room for a shorter ring.
// The ring takes what shared memory is left: deeper rings changed nothing at K = 384 and gave 3 % at K = 768 / 3072.
template <int BN, bool GTAB = false>
struct GemmCfg {
    static constexpr int STAGES = GTAB ? (BN == 96 ? 4 : 3) : (BN == 96 ? 7 : 5);
    static constexpr int EPI_PARTS = BN / COLS;          // epilogue warps per TMEM lane quadrant
    static constexpr int EPI_WARPS = 4 * EPI_PARTS;
    static constexpr int THREADS = 32 * (2 + EPI_WARPS);
    static constexpr uint32_t TM_MULT = 2 * BN, TM_RND = 3 * BN, TM_SHIFT = BN == 96 ? 4 * BN : 3 * BN;
    static constexpr bool HAS_RND = BN == 96;
};

struct GemmParams {
    int M, N, K;
    int num_m_tiles, num_n_tiles;
    int stages;                                       // ring stages in use
    const int32_t* bias; const int32_t* mult; const int8_t* shift;
    int out_zp;
    int qmin, qmax;                                   // output range of the plain / residual epilogues when it is not int8
    int res_mult, res_rnd, res_shift, res_off;        // residual branch: ((res << 16) - res_off) through R
    GeluDev gelu;
    const int8_t* gelu_tab;                           // device table of the integer GELU, or null
    StatusBlock* status;
};

template <int BN, bool GTAB = false>
struct GemmSmem {
    static constexpr int STAGES = GemmCfg<BN, GTAB>::STAGES;
    static constexpr int EPI_WARPS = GemmCfg<BN, GTAB>::EPI_WARPS;
    static constexpr int A_BYTES = BM * BK;
    static constexpr int B_BYTES = BN * BK;
    static constexpr int WARP_TILE = 32 * COLS;                                   // bytes of one warp's output block
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;                        // one ring stage: A tile, then B tile
    static constexpr int OFF_OUT = 0;                                             // [EPI_WARPS][32 rows][COLS] int8
    static constexpr int OFF_RES = OFF_OUT + EPI_WARPS * WARP_TILE;              // same shape, residual tiles
    static constexpr int OFF_BIAS = OFF_RES + EPI_WARPS * WARP_TILE;             // [EPI_WARPS][COLS] int32
    static constexpr int OFF_TAB = OFF_BIAS + EPI_WARPS * COLS * 4;              // GELU table (GTAB only)
    static constexpr int OFF_BAR = OFF_TAB + (GTAB ? IPTQ_GELU_TABLE_SIZE : 0);
    static constexpr int NUM_BARS = 2 * STAGES + 4 + EPI_WARPS;
    static constexpr int OFF_RING = (OFF_BAR + NUM_BARS * 8 + 16 + 1023) & ~1023; // the ring comes last: its length is a launch parameter
    static constexpr int total(int stages) { return OFF_RING + stages * STAGE_BYTES + 1024; }   // slack for 1024-byte alignment
    static constexpr int TOTAL = total(STAGES);
};

// Byte offset of 16-byte chunk `chunk` (0/1) of row `row` inside a [32][32]-byte block written/read by TMA with
// the 32-byte swizzle (chunk bit XOR bit 7 of the address); also keeps a warp's per-row 16-byte accesses
// conflict-free.
__device__ __forceinline__ uint32_t swz32(int row, int chunk) { return (uint32_t)(row * 32 + ((chunk ^ ((row >> 2) & 1)) << 4)); }

// One CTA works on ONE column tile (blockIdx.x % num_n_tiles) and walks down its row tiles, so the per-column
// constants are set up once per CTA: mult / rounding / shift in TMEM, the bias in shared memory, from where the
// epilogue writes it back into each accumulator it has just drained (the MMAs then always accumulate).
template <int BN, int EPI, int GELU_VARIANT, bool SAT8, bool GTAB>
__global__ void __launch_bounds__(GemmCfg<BN>::THREADS, 1)
gemm_i8_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_y, const __grid_constant__ CUtensorMap map_res,
               const GemmParams p)
{
    using L = GemmSmem<BN, GTAB>;
    using G = GemmCfg<BN, GTAB>;
    constexpr int STAGES = G::STAGES, EPI_WARPS = G::EPI_WARPS;
    constexpr uint32_t TM_MULT = G::TM_MULT, TM_RND = G::TM_RND, TM_SHIFT = G::TM_SHIFT;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sA = smem + L::OFF_RING;
    uint8_t* sB = sA + L::A_BYTES;
    const int stages = p.stages;                     // ring stages in use (<= STAGES)
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* acc_full = empty_bar + STAGES;      // [2]
    uint64_t* acc_empty = acc_full + 2;           // [2]
    uint64_t* res_bar = acc_empty + 2;            // [EPI_WARPS]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(res_bar + EPI_WARPS);
    CtaControl* ctl = reinterpret_cast<CtaControl*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int kblocks = (p.K + BK - 1) / BK;
    const int n0 = (int)(blockIdx.x % (unsigned)p.num_n_tiles) * BN;
    const int mt0 = (int)(blockIdx.x / (unsigned)p.num_n_tiles);
    const int mt_step = (int)(gridDim.x / (unsigned)p.num_n_tiles);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], EPI_WARPS); }
        for (int w = 0; w < EPI_WARPS; ++w) mbar_init(&res_bar[w], 1);
        ctl->abort = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
        prefetch_tensormap(&map_y);
        if (EPI == EPI_RESIDUAL) prefetch_tensormap(&map_res);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    grid_dep_launch();

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (elect_one()) {
            grid_dep_wait();                                   // the activations come from the previous kernel
            int s = 0; uint32_t ph = 0;
            for (int mt = mt0; mt < p.num_m_tiles; mt += mt_step) {
                bool ok = true;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(&empty_bar[s], ph ^ 1u, ctl, p.status, 1)) { ok = false; break; }
                    mbar_expect_tx(&full_bar[s], L::A_BYTES + L::B_BYTES);
                    tma_load_2d(sA + s * L::STAGE_BYTES, &map_a, &full_bar[s], kb * BK, mt * BM);
                    tma_load_2d(sB + s * L::STAGE_BYTES, &map_b, &full_bar[s], kb * BK, n0);
                    if (++s == stages) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            constexpr uint32_t idesc = umma_idesc_i8(BM, BN, true, true, false, false);
            int s = 0; uint32_t ph = 0;
            int it = 0;
            for (int mt = mt0; mt < p.num_m_tiles; mt += mt_step, ++it) {
                const int ab = it & 1;
                // the accumulator holds the bias, written by the epilogue warps (first at start-up, then after each drain)
                if (!mbar_wait(&acc_empty[ab], (uint32_t)(it >> 1) & 1u, ctl, p.status, 2)) break;
                tc_fence_after_sync();
                const uint32_t tacc = tmem_base + (uint32_t)(ab * BN);
                bool ok = true;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(&full_bar[s], ph, ctl, p.status, 3)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t a_addr = smem_u32(sA + s * L::STAGE_BYTES);
                    const uint32_t b_addr = smem_u32(sB + s * L::STAGE_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / 32; ++k) {
                        // K-major, 128-byte swizzle: 8-row groups are 1024 bytes apart; a k-step is 32 bytes
                        const uint64_t da = umma_smem_desc(a_addr + k * 32, 16, 1024, 128);
                        const uint64_t db = umma_smem_desc(b_addr + k * 32, 16, 1024, 128);
                        umma_i8(tacc, da, db, idesc, 1u);
                    }
                    umma_commit(&empty_bar[s]);               // frees the stage once these MMAs have read it
                    if (++s == stages) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
                umma_commit(&acc_full[ab]);                   // accumulator complete
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        // Warp (quad, part) owns TMEM lanes 32*quad.. (the only ones it may touch) and columns part*COLS.. of
        // every tile: it turns them into a [32 rows][COLS] int8 block in shared memory and stores that block
        // with one TMA copy; nothing in the epilogue synchronises across warps.
        const int ew = warp - 2;
        const int quad = warp & 3;
        const int part = ew >> 2;
        int* sbias = reinterpret_cast<int*>(smem + L::OFF_BIAS) + ew * COLS;
        const uint32_t bias_addr = smem_u32(sbias);
        const uint32_t out_blk = smem_u32(smem + L::OFF_OUT + ew * L::WARP_TILE);
        uint8_t* res_ptr = smem + L::OFF_RES + ew * L::WARP_TILE;
        const uint32_t res_blk = smem_u32(res_ptr);
        const int col0 = n0 + part * COLS;
        const uint32_t tlane = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(part * COLS);
        uint32_t res_ph = 0;
        {
            // ---- once per CTA: this warp's per-column constants (lane = column)
            const int n = col0 + lane;
            int cb = 0, cm = 1 << 30, cr = 1, cs = 1;
            if (n < p.N) {
                cs = (int)__ldg(p.shift + n);
                cb = p.bias ? __ldg(p.bias + n) : 0;
                cm = __ldg(p.mult + n);
                cr = 1 << (cs - 1);
            }
            if (!G::HAS_RND) cs -= 1;                         // the shift row holds shift - 1
            sbias[lane] = cb;
            __syncwarp();
            uint32_t v[16];
#pragma unroll
            for (int ch = 0; ch < COLS / 16; ++ch) {
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = (uint32_t)__shfl_sync(0xffffffffu, cm, ch * 16 + j);
                tmem_st16(tlane + TM_MULT + ch * 16, v);
                if (G::HAS_RND) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = (uint32_t)__shfl_sync(0xffffffffu, cr, ch * 16 + j);
                    tmem_st16(tlane + TM_RND + ch * 16, v);
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = (uint32_t)__shfl_sync(0xffffffffu, cs, ch * 16 + j);
                tmem_st16(tlane + TM_SHIFT + ch * 16, v);
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = (uint32_t)__shfl_sync(0xffffffffu, cb, ch * 16 + j);
                tmem_st16(tlane + ch * 16, v);                // both accumulators start from the bias
                tmem_st16(tlane + BN + ch * 16, v);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) { mbar_arrive(&acc_empty[0]); mbar_arrive(&acc_empty[1]); }
        }
        const uint32_t tab_mid = smem_u32(smem + L::OFF_TAB) + 32768u;      // address of table[0 + 32768]
        if (GTAB) {
            // the GELU table is static data: copy it while the previous kernel may still be running
            const int4* src = reinterpret_cast<const int4*>(p.gelu_tab);
            int4* dst = reinterpret_cast<int4*>(smem + L::OFF_TAB);
            for (int i = ew * 32 + lane; i < IPTQ_GELU_TABLE_SIZE / 16; i += EPI_WARPS * 32) dst[i] = __ldg(src + i);
            named_barrier(1, EPI_WARPS * 32);
        }
        grid_dep_wait();                                       // residual reads and output writes come after this
        int it = 0;
        for (int mt = mt0; mt < p.num_m_tiles; mt += mt_step, ++it) {
            const int ab = it & 1;
            const uint32_t abph = (uint32_t)(it >> 1) & 1u;
            const int row0 = mt * BM + quad * 32;
            const bool active = row0 < p.M && col0 < p.N;     // warp-uniform
            // the previous tile's store must have read the staging block before it is rewritten
            if (lane == 0) bulk_wait_read_all();
            __syncwarp();
            if (EPI == EPI_RESIDUAL && active && lane == 0) {
                mbar_expect_tx(&res_bar[ew], L::WARP_TILE);
                tma_load_2d(res_ptr, &map_res, &res_bar[ew], col0, row0);
            }
            if (!mbar_wait(&acc_full[ab], abph, ctl, p.status, 4)) break;
            tc_fence_after_sync();
            if (EPI == EPI_RESIDUAL && active) {
                if (!mbar_wait(&res_bar[ew], res_ph, ctl, p.status, 5)) break;
                res_ph ^= 1u;
            }
            const uint32_t tacc = tlane + (uint32_t)(ab * BN);
#pragma unroll
            for (int ch = 0; ch < COLS / 16; ++ch) {
                uint32_t acc[16], cm[16], cr[G::HAS_RND ? 16 : 1], cs[16];
                tmem_ld16(tacc + ch * 16, acc);
                tmem_ld16(tlane + TM_MULT + ch * 16, cm);
                if constexpr (G::HAS_RND) tmem_ld16(tlane + TM_RND + ch * 16, cr);
                tmem_ld16(tlane + TM_SHIFT + ch * 16, cs);
                uint32_t bv[16];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint4 t = ld_shared_v4(bias_addr + ch * 64 + q * 16);
                    bv[4 * q] = t.x; bv[4 * q + 1] = t.y; bv[4 * q + 2] = t.z; bv[4 * q + 3] = t.w;
                }
                tmem_wait_ld();
                tmem_st16(tacc + ch * 16, bv);                // re-arm this accumulator with the bias
                if (!active) continue;
                uint4 resv = make_uint4(0, 0, 0, 0);
                if (EPI == EPI_RESIDUAL) resv = ld_shared_v4(res_blk + swz32(lane, ch));
                const uint32_t resw[4] = {resv.x, resv.y, resv.z, resv.w};
                int o[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    int v;
                    if constexpr (G::HAS_RND) v = requant_core((int)acc[j], (int)cm[j], (int)cr[j], (int)cs[j]);
                    else v = (mad_hi((int)acc[j], (int)cm[j], 1 << cs[j]) >> cs[j]) >> 1;   // cs = shift - 1
                    if (EPI == EPI_GELU && GTAB) {
                        v = max(-32768, min(32767, v));
                        asm volatile("ld.shared.s8 %0, [%1];" : "=r"(v) : "r"(tab_mid + (uint32_t)v));
                    } else if (EPI == EPI_GELU) {
                        v = gelu_core<GELU_VARIANT>(v, p.gelu);
                        v = requant_nosat(v, p.gelu.out);
                        if (!SAT8) v = max(p.gelu.out.qmin, min(p.gelu.out.qmax, v));
                    } else if (EPI == EPI_RESIDUAL) {
                        // byte j of the residual word, sign-extended, widened by 2^16 and requantised
                        const int rb = (j & 3) == 0 ? sext_byte<0>(resw[j >> 2]) : (j & 3) == 1 ? sext_byte<1>(resw[j >> 2])
                                     : (j & 3) == 2 ? sext_byte<2>(resw[j >> 2]) : sext_byte<3>(resw[j >> 2]);
                        v += requant_core(rb * 65536 - p.res_off, p.res_mult, p.res_rnd, p.res_shift) + p.out_zp;
                    } else {
                        v += p.out_zp;
                    }
                    if (EPI != EPI_GELU && !SAT8) v = max(p.qmin, min(p.qmax, v));   // activations narrower than 8 bits
                    o[j] = v;
                }
                st_shared_v4(out_blk + swz32(lane, ch), pack4_sat_s8(o[0], o[1], o[2], o[3]),
                             pack4_sat_s8(o[4], o[5], o[6], o[7]), pack4_sat_s8(o[8], o[9], o[10], o[11]),
                             pack4_sat_s8(o[12], o[13], o[14], o[15]));
            }
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[ab]);       // the MMA warp may refill this accumulator
            if (active) {
                fence_proxy_async_smem();                     // this lane's st.shared -> visible to the TMA engine
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(&map_y, smem + L::OFF_OUT + ew * L::WARP_TILE, col0, row0);   // clipped at M and N
                    bulk_commit();
                }
            }
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
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, TMEM_COLS);
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
template <int BN, int EPI, int GV, bool SAT8, bool GTAB = false>
static int launch_gemm(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& my, const CUtensorMap& mr,
                       const GemmParams& p, cudaStream_t st)
{
    using L = GemmSmem<BN, GTAB>;
    auto kern = gemm_i8_kernel<BN, EPI, GV, SAT8, GTAB>;
    static bool configured[64];               // one attribute call per instantiation and device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return IPTQ_ERR_CUDA;
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::TOTAL) != cudaSuccess)
            return IPTQ_ERR_CUDA;
        configured[dev] = true;
    }
    // every CTA serves one column tile; the SMs are split evenly among the column tiles
    const int per_n = std::max(1, std::min(sm_count() / p.num_n_tiles, p.num_m_tiles));
    const int grid = p.num_n_tiles * per_n;
    // a ring much longer than one tile's K loop buys nothing, and a smaller footprint lets the next kernel's CTAs
    // become resident earlier
    GemmParams q = p;
    const int kblocks = (p.K + BK - 1) / BK;
    q.stages = std::max(2, std::min(L::STAGES, kblocks + 1));
    launch_kernel(kern, grid, GemmCfg<BN>::THREADS, L::total(q.stages), st, ma, mb, my, mr, q);
    note_launch();
    return last_launch_status();
}

template <int BN>
static int linear_launch_bn(const LinearArgs& a, cudaStream_t st);

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

int linear_launch(const LinearArgs& a, cudaStream_t st)
{
    const int rc0 = linear_check(a);
    if (rc0 != IPTQ_OK) return rc0;
    if (a.M == 0) return IPTQ_OK;
    // 128-wide tiles use the tensor core fully and re-read the activations less often, but rebuild the rounding
    // constant per output (two more instructions); measured, they win for the plain epilogue and for the tabulated
    // GELU epilogue at small K (ViT-Base FC1: 24 column tiles on 144 CTAs instead of 32 on 128), not for the
    // polynomial GELU or the residual epilogue
    const bool wide = a.N % 128 == 0 && (a.N % 96 != 0 || ((!a.gelu || a.gelu->table) && !a.residual && a.K <= 768));
    return wide ? linear_launch_bn<128>(a, st) : linear_launch_bn<96>(a, st);
}

template <int BN>
static int linear_launch_bn(const LinearArgs& a, cudaStream_t st)
{
    GemmParams p;
    p.M = (int)a.M; p.N = a.N; p.K = a.K;
    p.num_m_tiles = (int)((a.M + BM - 1) / BM);
    p.num_n_tiles = (a.N + BN - 1) / BN;
    p.bias = a.bias; p.mult = a.mult; p.shift = a.shift; p.out_zp = a.out_zp;
    p.qmin = -(1 << (a.out_bits - 1)); p.qmax = (1 << (a.out_bits - 1)) - 1;
    p.res_mult = p.res_rnd = p.res_shift = p.res_off = 0;
    if (a.residual) {
        p.res_mult = a.residual_rq->mult; p.res_shift = a.residual_rq->shift;
        p.res_rnd = 1 << (a.residual_rq->shift - 1); p.res_off = a.residual_rq->zp * 65536;
    }
    p.status = a.status;
    if (a.gelu) p.gelu = to_dev(*a.gelu);
    else { iptq_gelu_consts z{}; z.in_bits = 8; z.out.shift = 1; p.gelu = to_dev(z); }

    CUtensorMap ma, mb, my, mr;
    int rc;
    {
        const uint64_t dims[2] = {(uint64_t)a.K, (uint64_t)a.M};
        const uint64_t str[1] = {(uint64_t)a.K};
        const uint32_t box[2] = {BK, BM};
        if ((rc = make_tensor_map_u8(&ma, a.x, 2, dims, str, box, 128)) != IPTQ_OK) return rc;
    }
    {
        const uint64_t dims[2] = {(uint64_t)a.K, (uint64_t)a.N};
        const uint64_t str[1] = {(uint64_t)a.K};
        const uint32_t box[2] = {BK, BN};
        if ((rc = make_tensor_map_u8(&mb, a.w, 2, dims, str, box, 128)) != IPTQ_OK) return rc;
    }
    {
        // output and residual: one [32 rows][COLS] block per epilogue warp, clipped at M and N by the copy engine
        const uint64_t dims[2] = {(uint64_t)a.N, (uint64_t)a.M};
        const uint64_t str[1] = {(uint64_t)a.N};
        const uint32_t box[2] = {COLS, 32};
        if ((rc = make_tensor_map_u8(&my, a.y, 2, dims, str, box, 32)) != IPTQ_OK) return rc;
        if ((rc = make_tensor_map_u8(&mr, a.residual ? a.residual : a.y, 2, dims, str, box, 32)) != IPTQ_OK) return rc;
    }
    p.gelu_tab = a.gelu ? a.gelu->table : nullptr;
    if (a.gelu && a.gelu->table) {
        if (!aligned16(a.gelu->table)) return IPTQ_ERR_ALIGN;
        return launch_gemm<BN, EPI_GELU, 0, true, true>(ma, mb, my, mr, p, st);    // the variant is in the table
    }
    if (a.gelu) {
        const bool sat8 = a.gelu->out.qmin == -128 && a.gelu->out.qmax == 127;
#define IPTQ_GEMM_GELU(V) (sat8 ? launch_gemm<BN, EPI_GELU, V, true>(ma, mb, my, mr, p, st) \
                                : launch_gemm<BN, EPI_GELU, V, false>(ma, mb, my, mr, p, st))
        switch (a.gelu->variant) {
            case IPTQ_GELU_POLY4: return IPTQ_GEMM_GELU(IPTQ_GELU_POLY4);
            case IPTQ_GELU_POLY2: return IPTQ_GEMM_GELU(IPTQ_GELU_POLY2);
            default: return IPTQ_GEMM_GELU(IPTQ_GELU_SHIFT);
        }
#undef IPTQ_GEMM_GELU
    }
    if (a.out_bits != 8) {
        if (a.residual) return launch_gemm<BN, EPI_RESIDUAL, 0, false>(ma, mb, my, mr, p, st);
        return launch_gemm<BN, EPI_REQUANT, 0, false>(ma, mb, my, mr, p, st);
    }
    if (a.residual) return launch_gemm<BN, EPI_RESIDUAL, 0, true>(ma, mb, my, mr, p, st);
    return launch_gemm<BN, EPI_REQUANT, 0, true>(ma, mb, my, mr, p, st);
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
