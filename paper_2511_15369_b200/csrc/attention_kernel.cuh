#pragma once
// Kernel and per-variant launcher of the fused integer attention (included by attention.cu and by the
// attention_variant*.cu files, which instantiate one Softmax variant each so that they compile in parallel).
// Problems of N <= 64 tokens take the kernel of attention_window.cuh instead.
//
// Fused integer attention: S = Q K^T (tcgen05 INT8 -> int32 in TMEM) -> (+bias, mask) -> integer Softmax of
// Sec. 3.4 (Eqs. (6)-(15)) -> uint8 P written to shared memory in the tensor-core operand layout ->
// O = P V (u8 x s8 -> int32 in TMEM) -> dyadic requant -> int8, heads re-interleaved.
// Neither S nor P ever reaches HBM.
//
// The integer Softmax cannot be computed "online" (flash style): the floor in Eq. (9) depends on the final row
// maximum and P depends on floor(2^M / sum) before it multiplies V, so the whole score row is needed at once.
// A query row (<= 256 scores) is shared by four threads; each pulls its quarter (<= 64 scores) out of TMEM with one
// batch of loads and keeps it in registers through the three steps (max; exponentials + sum; probabilities), the
// four exchanging their partial max / sum through shared memory.  S leaves TMEM right after the load, so the MMA
// warp computes the next item's scores while the Softmax of the current one runs.
//
// Work item = (batch, head, 128-row query tile), handed out dynamically (full tiles first) through a counter in
// the workspace status block.  One CTA per SM, 20 warps: warps 0..15 = Softmax + output (warp w may only
// touch TMEM lanes 32*(w%4)..), warp 16 = TMA producer (3-stage ring of Q/K/V tiles), warp 17 = MMA issuer, warps
// 18 and 19 idle (they complete the group of four whose registers go to the Softmax warps).
// The output of item k is requantised after the Softmax of item k+1, when its P V product is certainly done.
#include <algorithm>

#include "tc_common.cuh"

namespace iptq {

constexpr int ATT_SOFTMAX_THREADS = 512;                 // warps 0..15
constexpr int ATT_SVC_WARP = ATT_SOFTMAX_THREADS / 32;   // the service group: TMA producer, MMA issuer, two idle warps
constexpr int ATT_THREADS = ATT_SOFTMAX_THREADS + 128;
// Registers per thread once the roles have split (setmaxnreg).  The CTA's pool is what it was launched with, 640
// threads x 96 registers; the service group keeps 32 per thread and the Softmax warps, which hold a quarter of a
// score row each, take 112 (16 x 112 + 4 x 32 = 20 x 96: all of the pool and no more).  At 96 the Softmax code
// spills 16-22 registers into its loops; at 112, one or two (ViT-Base attention 84.5 -> 76.5 us).
constexpr int ATT_LAUNCH_REGS = 96, ATT_SOFTMAX_REGS = 112, ATT_SVC_REGS = 32;
static_assert((ATT_SOFTMAX_THREADS / 32) * ATT_SOFTMAX_REGS + 4 * ATT_SVC_REGS <= (ATT_THREADS / 32) * ATT_LAUNCH_REGS,
              "the register counts after the split exceed the CTA's pool: reg_alloc would wait for ever");
constexpr int ATT_STAGES = 3;              // upper bound of the Q/K/V ring depth

struct AttnParams {
    int B, H, N, dh;
    int mtiles;            // ceil(N / 128)
    int items, full_items; // all work items; those of them that are full 128-row tiles (handed out first)
    int npad_s;            // N rounded up to 16: UMMA N of QK^T, TMEM columns of S
    int kpad;              // N rounded up to 32: UMMA K extent of P V
    int o_col;             // first TMEM column of O
    int q_bytes, k_bytes, v_bytes, stage_bytes;
    int p_off, p_bytes, xch_off, bar_off;
    int p_plane;           // bytes of one P operand; the logarithm candidate keeps two per buffer (p_bytes = 2 p_plane)
    int stages;            // Q/K/V ring depth (3, or 2 when the exponential table needs the room)
    int lut_off, lut_n;    // exponential table: e(d) for d < lut_n, 0 beyond (lut_n = 0: no table)
    const uint16_t* lut_src;   // the same table in device memory (copied), or null (built by each CTA)
    uint32_t tmem_cols;
    const int32_t* bias;   // [H, N, N] or null
    const int4* bias_q;    // window kernel: the same bias as [H][ceil(N/4) column quads][64 rows] of 4 columns each, or null
    const uint8_t* mask_id;// [B, N] or null
    int8_t* out;           // [B, N, H*dh]
    ExpDev ex; int M, f_shl, p_shr;
    RequantDev orq;
    StatusBlock* status;
};

// item index -> (batch*head, row tile): full tiles first, then the ragged last tiles
__device__ __forceinline__ void decode_item(const AttnParams& p, int it, int& bh, int& mt)
{
    const int full_per = p.N >> 7;                        // full 128-row tiles per (batch, head)
    if (it < p.full_items) { bh = it / full_per; mt = it - bh * full_per; }
    else                   { bh = it - p.full_items; mt = full_per; }
}

// USE_LUT: the integer exponential of Eqs. (7)-(14) depends only on d = max - s, is below 2^16 and vanishes for
// d >= lut_n (a few times x0); each CTA tabulates it once in shared memory with the same arithmetic and the
// Softmax step then costs one table read per score instead of some sixteen dependent integer instructions.
template <int DH, int VARIANT, bool HAS_BIAS, bool HAS_MASK, bool PSHR, bool USE_LUT>
__global__ void __launch_bounds__(ATT_THREADS, 1)
attention_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const AttnParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sP = smem + p.p_off;                                         // two P buffers
    int* xch_max = reinterpret_cast<int*>(smem + p.xch_off);              // [4 parts][128 rows]
    unsigned* xch_sum = reinterpret_cast<unsigned*>(xch_max + 512);       // [4 parts][128 rows]
    uint64_t* kv_full = reinterpret_cast<uint64_t*>(smem + p.bar_off);   // [ATT_STAGES]
    uint64_t* kv_empty = kv_full + ATT_STAGES;                            // [ATT_STAGES]
    uint64_t* s_full = kv_empty + ATT_STAGES;
    uint64_t* s_empty = s_full + 1;
    uint64_t* p_ready = s_empty + 1;                                      // [2]
    uint64_t* o_full = p_ready + 2;
    uint64_t* o_empty = o_full + 1;
    volatile int* item_of = reinterpret_cast<volatile int*>(o_empty + 1); // [ATT_STAGES] item held by a stage, -1 = stop
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(const_cast<int*>(item_of) + ATT_STAGES + 1);
    CtaControl* ctl = reinterpret_cast<CtaControl*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], 1); }
        mbar_init(s_full, 1);
        mbar_init(s_empty, ATT_SOFTMAX_THREADS / 32);       // one arrival per Softmax warp (512 arrivals on one
        mbar_init(&p_ready[0], ATT_SOFTMAX_THREADS / 32);  // barrier word serialise and cost more than the Softmax itself)
        mbar_init(&p_ready[1], ATT_SOFTMAX_THREADS / 32);
        mbar_init(o_full, 1);
        mbar_init(o_empty, ATT_SOFTMAX_THREADS / 32);
        ctl->abort = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_q);
        prefetch_tensormap(&map_k);
        prefetch_tensormap(&map_v);
    }
    if (warp == ATT_SVC_WARP + 1) {
        tmem_alloc(tmem_slot, p.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    grid_dep_launch();

    if (warp >= ATT_SVC_WARP) {
        // the service group: its four warps give registers back at one place, then two of them take a role
        reg_dealloc<ATT_SVC_REGS>();
        if (warp == ATT_SVC_WARP) {
            // ------------------------------------------------------------ TMA producer + work distribution
            if (elect_one()) {
                grid_dep_wait();                                   // q/k/v come from the previous kernel
                int s = 0; uint32_t ph = 0;
                for (;;) {
                    if (!mbar_wait_nocall(&kv_empty[s], ph ^ 1u, ctl, p.status, 11)) break;
                    const int it = atomicAdd(&p.status->work_next, 1);
                    if (it >= p.items) {
                        item_of[s] = -1;
                        mbar_arrive(&kv_full[s]);                  // release: the consumers see the stop mark
                        break;
                    }
                    int bh, mt;
                    decode_item(p, it, bh, mt);
                    const int h = bh % p.H, b = bh / p.H;
                    item_of[s] = it;
                    uint8_t* st = smem + s * p.stage_bytes;
                    mbar_expect_tx(&kv_full[s], (uint32_t)((128 + p.npad_s + p.kpad) * DH));   // bytes of the three full boxes
                    tma_load_4d(st, &map_q, &kv_full[s], 0, mt * 128, h, b);
                    tma_load_4d(st + p.q_bytes, &map_k, &kv_full[s], 0, 0, h, b);
                    tma_load_4d(st + p.q_bytes + p.k_bytes, &map_v, &kv_full[s], 0, 0, h, b);
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                }
                // the last CTA to finish re-arms the counters for the next launch that uses this workspace
                __threadfence();
                if (atomicAdd(&p.status->work_done, 1) == (int)gridDim.x - 1) {
                    p.status->work_next = 0;
                    p.status->work_done = 0;
                    __threadfence();
                }
            }
        } else if (warp == ATT_SVC_WARP + 1) {
            // ------------------------------------------------------------ MMA issuer: S(k), then P V of item k-1
            if (elect_one()) {
                const uint32_t idesc_s = umma_idesc_i8(128, p.npad_s, true, true, false, false);
                const uint32_t idesc_o = umma_idesc_i8(128, DH, false, true, false, true);     // u8 P (K-major) x s8 V (MN-major)
                const uint32_t tmem_o = tmem_base + (uint32_t)p.o_col;
                int s = 0; uint32_t ph = 0;
                int s_prev = 0;
                auto issue_pv = [&](int k) -> bool {                // k = item count index of the item whose P is ready
                    if (!mbar_wait_nocall(&p_ready[k & 1], (uint32_t)(k >> 1) & 1u, ctl, p.status, 14)) return false;
                    if (!mbar_wait_nocall(o_empty, ((uint32_t)k & 1u) ^ 1u, ctl, p.status, 12)) return false;   // previous O has been read
                    tc_fence_after_sync();
                    const uint32_t p_addr = smem_u32(sP + (k & 1) * p.p_bytes);
                    const uint32_t v_addr = smem_u32(smem + s_prev * p.stage_bytes) + p.q_bytes + p.k_bytes;
                    for (int ks = 0; ks < p.kpad / 32; ++ks) {
                        // A = P: K-major, 128-byte swizzle, column blocks of 128 keys are 16 KB apart
                        const uint64_t da = umma_smem_desc(p_addr + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024, 128);
                        // B = V [keys, DH]: MN-major (DH contiguous), DH-byte swizzle, 8-key groups 8*DH apart
                        const uint64_t db = umma_smem_desc(v_addr + ks * 32 * DH, 8 * DH, 8 * DH, DH);
                        umma_i8(tmem_o, da, db, idesc_o, ks != 0 ? 1u : 0u);
                        if constexpr (VARIANT == IPTQ_SM_LOG2) {
                            // low-order plane (probabilities 2^-8 .. 2^-15) into its own accumulator behind the first
                            const uint64_t da2 = umma_smem_desc(p_addr + p.p_plane + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024, 128);
                            umma_i8(tmem_o + (uint32_t)DH, da2, db, idesc_o, ks != 0 ? 1u : 0u);
                        }
                    }
                    umma_commit(&kv_empty[s_prev]);                // the stage may be refilled
                    umma_commit(o_full);
                    return true;
                };
                int k = 0;
                for (;; ++k) {
                    if (!mbar_wait_nocall(&kv_full[s], ph, ctl, p.status, 13)) break;
                    const bool stop = item_of[s] < 0;
                    if (!stop) {
                        if (!mbar_wait_nocall(s_empty, ((uint32_t)k & 1u) ^ 1u, ctl, p.status, 18)) break;   // S(k-1) is in registers
                        tc_fence_after_sync();
                        const uint32_t q_addr = smem_u32(smem + s * p.stage_bytes);
                        const uint32_t k_addr = q_addr + p.q_bytes;
                        // S = Q K^T: both operands K-major with DH-byte rows (DH-byte swizzle, 8-row groups 8*DH apart)
    #pragma unroll
                        for (int kk = 0; kk < DH / 32; ++kk) {
                            const uint64_t da = umma_smem_desc(q_addr + kk * 32, 16, 8 * DH, DH);
                            const uint64_t db = umma_smem_desc(k_addr + kk * 32, 16, 8 * DH, DH);
                            umma_i8(tmem_base, da, db, idesc_s, kk != 0 ? 1u : 0u);
                        }
                        umma_commit(s_full);
                    }
                    if (k > 0 && !issue_pv(k - 1)) break;
                    if (stop) break;
                    s_prev = s;
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else {
        // ------------------------------------------------------------ softmax + output warps
        reg_alloc<ATT_SOFTMAX_REGS>();
        const int quad = warp & 3;                             // TMEM lane quadrant this warp may touch
        const int part = warp >> 2;                            // which quarter of the columns
        const int rloc = quad * 32 + lane;                     // row inside the 128-row tile
        const uint32_t trow = tmem_base + ((uint32_t)(quad * 32) << 16);
        const uint32_t p_row0 = smem_u32(sP) + (uint32_t)((rloc >> 3) * 1024 + (rloc & 7) * 128);
        const int HD = p.H * DH;
        const int chunks = p.npad_s >> 4;                      // 16-column chunks of a row (<= 16)
        const int cbase = chunks >> 2, crem = chunks & 3;
        const int nch = cbase + (part < crem ? 1 : 0);         // this thread's chunks (<= 4) ...
        const int c_begin = part * cbase + min(part, crem);    // ... starting here
        const bool sat8 = p.orq.qmin == -128 && p.orq.qmax == 127;
        int s = 0; uint32_t ph = 0;
        uint16_t* lut = reinterpret_cast<uint16_t*>(smem + p.lut_off);
        const uint32_t lut_addr = smem_u32(lut);
        if (USE_LUT) {
            if (p.lut_src) {
                // written and fenced by iptq_softmax_table(): safe to read ahead of the dependency wait
                const int4* src = reinterpret_cast<const int4*>(p.lut_src);
                int4* dst = reinterpret_cast<int4*>(lut);
                for (int i = (int)threadIdx.x; i < (p.lut_n + 8) / 8; i += ATT_SOFTMAX_THREADS) dst[i] = __ldg(src + i);
            } else {
                for (int d = (int)threadIdx.x; d <= p.lut_n; d += ATT_SOFTMAX_THREADS)
                    lut[d] = d < p.lut_n ? (uint16_t)exp_core_nd<VARIANT>(-d, p.ex) : (uint16_t)0;
            }
            named_barrier(5, ATT_SOFTMAX_THREADS);              // the table is complete before anyone reads it
        }
        grid_dep_wait();                                       // output rows are written only after this

        // requantises and stores this thread's share of the output tile of item (b, h, mt), count index k
        auto epilogue = [&](int k, int b, int h, int mt) -> bool {
            if (!mbar_wait_nocall(o_full, (uint32_t)k & 1u, ctl, p.status, 16)) return false;
            tc_fence_after_sync();
            const int row = mt * 128 + rloc;
            constexpr int OPARTS = DH / 16;                    // threads of a row that hold 16 output columns each
            if (mt * 128 + quad * 32 < p.N && part < OPARTS) {
                uint32_t r[16];
                tmem_ld16(trow + (uint32_t)(p.o_col + part * 16), r);
                if constexpr (VARIANT == IPTQ_SM_LOG2) {
                    // O = 2^8 * (high plane product) + (low plane product), at scale 2^-15
                    uint32_t r2[16];
                    tmem_ld16(trow + (uint32_t)(p.o_col + DH + part * 16), r2);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j) r[j] = (uint32_t)(((int)r[j] << 8) + (int)r2[j]);
                }
                tmem_wait_ld();
                int o[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    o[j] = requant_nosat((int)r[j], p.orq);
                    if (!sat8) o[j] = max(p.orq.qmin, min(p.orq.qmax, o[j]));
                }
                if (row < p.N) {
                    int4 pk;
                    pk.x = (int)pack4_sat_s8(o[0], o[1], o[2], o[3]);
                    pk.y = (int)pack4_sat_s8(o[4], o[5], o[6], o[7]);
                    pk.z = (int)pack4_sat_s8(o[8], o[9], o[10], o[11]);
                    pk.w = (int)pack4_sat_s8(o[12], o[13], o[14], o[15]);
                    *reinterpret_cast<int4*>(p.out + ((size_t)b * p.N + row) * HD + h * DH + part * 16) = pk;
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(o_empty);
            return true;
        };

        int k = 0;
        int pb = 0, phd = 0, pmt = 0;                          // item whose output is still to be written
        bool ok = true;
        for (;; ++k) {
            // the four warps of a quadrant meet at two named barriers per item: a warp that gives up before them
            // arrives without waiting, so that a bounded wait running out can never strand the others
            if (!mbar_wait_nocall(&kv_full[s], ph, ctl, p.status, 17)) {   // acquire: the item number is visible
                named_barrier_arrive(1 + quad, 128); named_barrier_arrive(1 + quad, 128);
                ok = false;
                break;
            }
            const int it = item_of[s];
            if (it < 0) break;
            if (++s == p.stages) { s = 0; ph ^= 1u; }
            int bh, mt;
            decode_item(p, it, bh, mt);
            const int h = bh % p.H, b = bh / p.H;
            const int row = mt * 128 + rloc;
            const bool valid = row < p.N;
            const bool warp_rows = mt * 128 + quad * 32 < p.N;            // warp-uniform: any valid row in this warp
            const int32_t* brow = HAS_BIAS ? p.bias + ((size_t)h * p.N + (valid ? row : 0)) * p.N : nullptr;
            const uint8_t* mrow = HAS_MASK ? p.mask_id + (size_t)b * p.N : nullptr;
            const unsigned my_id = HAS_MASK ? mrow[valid ? row : 0] : 0u;
            const uint32_t p_row = p_row0 + (uint32_t)((k & 1) * p.p_bytes);

            if (!mbar_wait_nocall(s_full, (uint32_t)k & 1u, ctl, p.status, 15)) {
                named_barrier_arrive(1 + quad, 128); named_barrier_arrive(1 + quad, 128);
                ok = false;
                break;
            }
            tc_fence_after_sync();
            // ---- this thread's quarter of the score row, TMEM -> registers, in one batch
            uint32_t v[4][16];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (warp_rows && i < nch) tmem_ld16(trow + (uint32_t)((c_begin + i) * 16), v[i]);
            tmem_wait_ld();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(s_empty);               // the MMA warp may overwrite S with the next item's scores
            if (warp_rows) {
                // ---- row maximum over the real, unmasked columns (Eq. (6)); padding and masked pairs become
                //      kNoScore, a bias is added in place, so that the next step needs no case analysis
                int mx = INT_MIN, mx1 = INT_MIN, mx2 = INT_MIN, mx3 = INT_MIN;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (i < nch) {
                        const int c0 = (c_begin + i) * 16;
                        if (HAS_BIAS || HAS_MASK || c0 + 16 > p.N) {          // warp-uniform
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const int col = c0 + j;
                                int sc = (int)v[i][j];
                                bool use = col < p.N;
                                if (HAS_BIAS && use) sc += __ldg(brow + col);
                                if (HAS_MASK && use) use = (mrow[col] == my_id);
                                v[i][j] = (uint32_t)(use ? sc : kNoScore);
                            }
                        }
                        // four running maxima: one chain of 64 dependent min/max instructions would leave the
                        // thread waiting on itself
#pragma unroll
                        for (int j = 0; j < 16; j += 4) {
                            mx = max(mx, (int)v[i][j]);     mx1 = max(mx1, (int)v[i][j + 1]);
                            mx2 = max(mx2, (int)v[i][j + 2]); mx3 = max(mx3, (int)v[i][j + 3]);
                        }
                    }
                }
                mx = max(max(mx, mx1), max(mx2, mx3));
                xch_max[part * 128 + rloc] = mx;
                named_barrier(1 + quad, 128);
                mx = max(max(xch_max[rloc], xch_max[128 + rloc]), max(xch_max[256 + rloc], xch_max[384 + rloc]));
                // ---- integer exponentials (Eqs. (7)-(14)), in place, and their sum
                unsigned sum = 0, sum1 = 0, sum2 = 0, sum3 = 0;         // four partial sums, as for the maximum
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (i < nch) {
                        if (USE_LUT) {
                            // table addresses first, then the 16 reads back to back, then the sums
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                v[i][j] = lut_addr + 2u * min((unsigned)mx - v[i][j], (unsigned)p.lut_n);
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v[i][j]) : "r"(v[i][j]));
                        } else {
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                v[i][j] = exp_core_nd<VARIANT>(exp_distance(mx, (int)v[i][j]), p.ex);
                        }
#pragma unroll
                        for (int j = 0; j < 16; j += 4) {
                            sum += v[i][j]; sum1 += v[i][j + 1]; sum2 += v[i][j + 2]; sum3 += v[i][j + 3];
                        }
                    }
                }
                sum = (sum + sum1) + (sum2 + sum3);
                xch_sum[part * 128 + rloc] = sum;
                named_barrier(1 + quad, 128);
                sum = (xch_sum[rloc] + xch_sum[128 + rloc]) + (xch_sum[256 + rloc] + xch_sum[384 + rloc]);
                if constexpr (VARIANT == IPTQ_SM_LOG2) {
                    // ---- logarithm candidate: p = 2^-code as the 16-bit value 2^(15 - code), split into a high and
                    //      a low byte plane (exactly one of the two bytes is non-zero), both in the A-operand layout
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (i < nch) {
                            uint32_t wh[4], wl[4];
#pragma unroll
                            for (int q4 = 0; q4 < 4; ++q4) {
                                int hi[4], lo[4];
#pragma unroll
                                for (int t = 0; t < 4; ++t) {
                                    const unsigned code = log2_code(sum, v[i][q4 * 4 + t]);
                                    const unsigned w16 = code <= 15u ? (0x8000u >> code) : 0u;
                                    hi[t] = (int)(w16 >> 8);
                                    lo[t] = (int)(w16 & 0xffu);
                                }
                                wh[q4] = pack4_sat_u8(hi[0], hi[1], hi[2], hi[3]);
                                wl[q4] = pack4_sat_u8(lo[0], lo[1], lo[2], lo[3]);
                            }
                            const int c0 = (c_begin + i) * 16;
                            const int chunk = (c0 & 127) >> 4;
                            const uint32_t at = p_row + (uint32_t)((c0 >> 7) * 16384 + ((chunk ^ (rloc & 7)) << 4));
                            st_shared_v4(at, wh[0], wh[1], wh[2], wh[3]);
                            st_shared_v4(at + (uint32_t)p.p_plane, wl[0], wl[1], wl[2], wl[3]);
                        }
                    }
                } else {
                // ---- IntDiv (Eq. (15)) -> uint8 probabilities in the UMMA A-operand layout
                const unsigned f = intdiv_factor(sum, p.M) << p.f_shl;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (i < nch) {
                        uint32_t w[4];
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            int pv[4];
#pragma unroll
                            for (int t = 0; t < 4; ++t) {
                                unsigned x = __umulhi(f, v[i][q4 * 4 + t]);
                                if (PSHR) x >>= p.p_shr;
                                pv[t] = (int)x;
                            }
                            w[q4] = pack4_sat_u8(pv[0], pv[1], pv[2], pv[3]);      // values are <= 2^(b-1): nothing saturates
                        }
                        const int c0 = (c_begin + i) * 16;
                        const int chunk = (c0 & 127) >> 4;
                        st_shared_v4(p_row + (uint32_t)((c0 >> 7) * 16384 + ((chunk ^ (rloc & 7)) << 4)), w[0], w[1], w[2], w[3]);
                    }
                }
                }
            } else {
                named_barrier_arrive(1 + quad, 128); named_barrier_arrive(1 + quad, 128);   // keeps the barrier generations aligned
            }
            // key columns between npad_s and kpad (at most one 16-column chunk) meet zero rows of V, but the bytes
            // the tensor core reads there must be defined
            if (part == 3 && p.kpad > p.npad_s) {
                const int c0 = p.npad_s;
                const int chunk = (c0 & 127) >> 4;
                st_shared_v4(p_row + (uint32_t)((c0 >> 7) * 16384 + ((chunk ^ (rloc & 7)) << 4)), 0u, 0u, 0u, 0u);
                if constexpr (VARIANT == IPTQ_SM_LOG2)
                    st_shared_v4(p_row + (uint32_t)(p.p_plane + (c0 >> 7) * 16384 + ((chunk ^ (rloc & 7)) << 4)), 0u, 0u, 0u, 0u);
            }
            fence_proxy_async_smem();            // generic-proxy stores -> visible to the tensor core's reads
            __syncwarp();
            if (lane == 0) mbar_arrive(&p_ready[k & 1]);
            // ---- output of the previous item: its P V product was issued right after that item's Softmax
            if (k > 0 && !epilogue(k - 1, pb, phd, pmt)) { ok = false; break; }
            pb = b; phd = h; pmt = mt;
        }
        if (ok && k > 0) epilogue(k - 1, pb, phd, pmt);
    }

    // ------------------------------------------------------------ teardown (also reached after an abort)
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    if (ctl->abort) {
        for (int i = 0; i < 64; ++i) __nanosleep(2000);
        __syncthreads();
    }
    if (warp == ATT_SVC_WARP + 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

template <int DH, int VARIANT>
int launch_attn(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const AttnParams& p,
                       int smem_bytes, cudaStream_t st)
{
    const int grid = std::min(p.items, sm_count());
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return IPTQ_ERR_CUDA;
#define IPTQ_ATT_LAUNCH3(HB, HM, PS, LT)                                                                          \
    do {                                                                                                          \
        auto kern = attention_kernel<DH, VARIANT, HB, HM, PS, LT>;                                                \
        static int configured[64];          /* largest dynamic shared memory size set so far, per device */     \
        if (configured[dev] < smem_bytes) {                                                                       \
            /* the register counts the roles take after the split are sized for a launch with ATT_LAUNCH_REGS: a   \
               build that starts this kernel with fewer would leave its Softmax warps waiting for registers */     \
            cudaFuncAttributes fa;                                                                                \
            if (cudaFuncGetAttributes(&fa, kern) != cudaSuccess || ((fa.numRegs + 7) & ~7) != ATT_LAUNCH_REGS)   \
                return IPTQ_ERR_CUDA;                                                                             \
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) != cudaSuccess) \
                return IPTQ_ERR_CUDA;                                                                             \
            configured[dev] = smem_bytes;                                                                         \
        }                                                                                                         \
        launch_kernel(kern, grid, ATT_THREADS, smem_bytes, st, mq, mk, mv, p);                                    \
    } while (0)
#define IPTQ_ATT_LAUNCH2(HB, HM, PS)                                                                              \
    do {                                                                                                          \
        if (p.lut_n) IPTQ_ATT_LAUNCH3(HB, HM, PS, true); else IPTQ_ATT_LAUNCH3(HB, HM, PS, false);                \
    } while (0)
#define IPTQ_ATT_LAUNCH(HB, HM)                                                                                   \
    do {                                                                                                          \
        if (p.p_shr) IPTQ_ATT_LAUNCH2(HB, HM, true); else IPTQ_ATT_LAUNCH2(HB, HM, false);                        \
    } while (0)
    if (p.bias && p.mask_id) IPTQ_ATT_LAUNCH(true, true);
    else if (p.bias) IPTQ_ATT_LAUNCH(true, false);
    else if (p.mask_id) IPTQ_ATT_LAUNCH(false, true);
    else IPTQ_ATT_LAUNCH(false, false);
#undef IPTQ_ATT_LAUNCH
#undef IPTQ_ATT_LAUNCH2
#undef IPTQ_ATT_LAUNCH3
    note_launch();
    return last_launch_status();
}


}  // namespace iptq
