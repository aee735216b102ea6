#pragma once
// Fused integer attention for small problems (N <= 64 tokens: Swin windows).  Same arithmetic as attention_kernel,
// different decomposition, because here an item is dominated by serial latency (operand wait, TMEM round trips,
// one divide per row, output epilogue), not by the per-score work:
//   * an item is two (batch, head) problems, one per 64-row half of the 128-row tile; S = Q K^T is 128 x 128 and
//     each half looks at its own 64 columns only, P is block diagonal (the off-diagonal quarters are zeroed once);
//   * a row has at most 64 scores, so ONE thread keeps the whole row in registers: no exchange of partial
//     max / sum, no barrier inside an item;
//   * the Softmax warps form G independent groups of four (one warp per TMEM lane quadrant); group g owns its own
//     S / O columns in TMEM and its own P buffer and takes items g, g + G, ...: G items are in flight per SM and
//     cover each other's latencies.  G = 3 for head dimension 32, 2 for 64 and for the logarithm candidate
//     (512 TMEM columns hold G x (128 + output columns)).
// Warp 0 = TMA producer (ring of G + 2 operand stages) and work distribution, warp 1 = MMA issuer: Q K^T of item k,
// then P V of item k - (G - 1).
#include "attention_kernel.cuh"

namespace iptq {

constexpr int WIN_MAX_GROUPS = 3;
constexpr int WIN_MAX_STAGES = WIN_MAX_GROUPS + 2;

template <int DH, int VARIANT> struct WinCfg {
    static constexpr int OW = DH * (VARIANT == IPTQ_SM_LOG2 ? 2 : 1);       // TMEM columns of O (two planes for log2)
    static constexpr int G = (DH == 32 && VARIANT != IPTQ_SM_LOG2) ? 3 : 2;
    static constexpr int GCOLS = 128 + OW;                                  // S and O of one group
    static constexpr int THREADS = 64 + 128 * G;
    static constexpr int STAGES = G + 2;
    static constexpr int STAGE_BYTES = 3 * 128 * DH;                        // Q, K, V tiles of a pair
    static constexpr int P_BYTES = 16384 * (VARIANT == IPTQ_SM_LOG2 ? 2 : 1);
    static_assert(G * GCOLS <= 512, "TMEM");
};

// FULL: 48 < N <= 64, i.e. every row has its four 16-column chunks (the Swin window of 49 tokens): the chunk loops
// then carry no run-time conditions.
template <int DH, int VARIANT, bool HAS_BIAS, bool HAS_MASK, bool PSHR, bool USE_LUT, bool FULL>
__global__ void __launch_bounds__(WinCfg<DH, VARIANT>::THREADS, 1)
window_attention_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                        const __grid_constant__ CUtensorMap map_v, const AttnParams p)
{
    using W = WinCfg<DH, VARIANT>;
    constexpr int G = W::G, ST = W::STAGES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sP = smem + ST * W::STAGE_BYTES;                              // G P buffers
    uint16_t* lut = reinterpret_cast<uint16_t*>(smem + p.lut_off);
    uint64_t* kv_full = reinterpret_cast<uint64_t*>(smem + p.bar_off);    // [ST]
    uint64_t* kv_empty = kv_full + ST;                                     // [ST]
    uint64_t* s_full = kv_empty + ST;                                      // [G] each
    uint64_t* s_empty = s_full + G;
    uint64_t* p_ready = s_empty + G;
    uint64_t* o_full = p_ready + G;
    uint64_t* o_empty = o_full + G;
    volatile int* item_of = reinterpret_cast<volatile int*>(o_empty + G); // [ST] item held by a stage, -1 = stop
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(const_cast<int*>(item_of) + ST + 1);
    CtaControl* ctl = reinterpret_cast<CtaControl*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int problems = p.B * p.H;

    if (threadIdx.x == 0) {
        for (int s = 0; s < ST; ++s) { mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], 1); }
        for (int g = 0; g < G; ++g) {
            mbar_init(&s_full[g], 1);
            mbar_init(&s_empty[g], 4);                     // one arrival per warp of the group
            mbar_init(&p_ready[g], 4);
            mbar_init(&o_full[g], 1);
            mbar_init(&o_empty[g], 4);
        }
        ctl->abort = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_q);
        prefetch_tensormap(&map_k);
        prefetch_tensormap(&map_v);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, p.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    grid_dep_launch();

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer + work distribution
        if (elect_one()) {
            grid_dep_wait();                                   // q/k/v come from the previous kernel
            int s = 0; uint32_t ph = 0;
            int stops = 0;                                     // stop marks written so far (every group needs one)
            for (;;) {
                if (!mbar_wait(&kv_empty[s], ph ^ 1u, ctl, p.status, 21)) break;
                const int it = stops ? p.items : atomicAdd(&p.status->work_next, 1);
                if (it >= p.items) {
                    item_of[s] = -1;
                    mbar_arrive(&kv_full[s]);                  // release: the consumers see the stop mark
                    if (++stops == G) break;
                } else {
                    item_of[s] = it;
                    uint8_t* st = smem + s * W::STAGE_BYTES;
                    const int n_here = 2 * it + 1 < problems ? 2 : 1;
                    mbar_expect_tx(&kv_full[s], (uint32_t)(n_here * 3 * 64 * DH));
                    for (int w = 0; w < n_here; ++w) {
                        const int bh = 2 * it + w;
                        const int h = bh % p.H, b = bh / p.H;
                        uint8_t* half = st + w * 64 * DH;
                        tma_load_4d(half, &map_q, &kv_full[s], 0, 0, h, b);
                        tma_load_4d(half + 128 * DH, &map_k, &kv_full[s], 0, 0, h, b);
                        tma_load_4d(half + 256 * DH, &map_v, &kv_full[s], 0, 0, h, b);
                    }
                }
                if (++s == ST) { s = 0; ph ^= 1u; }
            }
            // the last CTA to finish re-arms the counters for the next launch that uses this workspace
            __threadfence();
            if (atomicAdd(&p.status->work_done, 1) == (int)gridDim.x - 1) {
                p.status->work_next = 0;
                p.status->work_done = 0;
                __threadfence();
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            const uint32_t idesc_s = umma_idesc_i8(128, 128, true, true, false, false);
            const uint32_t idesc_o = umma_idesc_i8(128, DH, false, true, false, true);     // u8 P (K-major) x s8 V (MN-major)
            auto issue_pv = [&](int j) -> bool {                // item count index j: its P is (about to be) ready
                const int g = j % G, n = j / G, sj = j % ST;
                if (!mbar_wait(&p_ready[g], (uint32_t)n & 1u, ctl, p.status, 24)) return false;
                if (!mbar_wait(&o_empty[g], ((uint32_t)n & 1u) ^ 1u, ctl, p.status, 22)) return false;   // previous O of the group has been read
                tc_fence_after_sync();
                const uint32_t tmem_o = tmem_base + (uint32_t)(g * W::GCOLS + 128);
                const uint32_t p_addr = smem_u32(sP + g * W::P_BYTES);
                const uint32_t v_addr = smem_u32(smem + sj * W::STAGE_BYTES) + 256 * DH;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {                // 128 keys in steps of 32
                    const uint64_t da = umma_smem_desc(p_addr + ks * 32, 16, 1024, 128);
                    const uint64_t db = umma_smem_desc(v_addr + ks * 32 * DH, 8 * DH, 8 * DH, DH);
                    umma_i8(tmem_o, da, db, idesc_o, ks != 0 ? 1u : 0u);
                    if constexpr (VARIANT == IPTQ_SM_LOG2) {
                        const uint64_t da2 = umma_smem_desc(p_addr + 16384 + ks * 32, 16, 1024, 128);
                        umma_i8(tmem_o + (uint32_t)DH, da2, db, idesc_o, ks != 0 ? 1u : 0u);
                    }
                }
                umma_commit(&kv_empty[sj]);                    // the stage may be refilled
                umma_commit(&o_full[g]);
                return true;
            };
            int k_stop = INT_MAX;
            for (int k = 0;; ++k) {
                if (k < k_stop) {
                    const int sk = k % ST;
                    if (!mbar_wait(&kv_full[sk], (uint32_t)(k / ST) & 1u, ctl, p.status, 23)) break;
                    if (item_of[sk] < 0) {
                        k_stop = k;
                    } else {
                        const int g = k % G, n = k / G;
                        if (!mbar_wait(&s_empty[g], ((uint32_t)n & 1u) ^ 1u, ctl, p.status, 28)) break;   // the group holds its previous S in registers
                        tc_fence_after_sync();
                        const uint32_t q_addr = smem_u32(smem + sk * W::STAGE_BYTES);
                        const uint32_t k_addr = q_addr + 128 * DH;
#pragma unroll
                        for (int kk = 0; kk < DH / 32; ++kk) {
                            const uint64_t da = umma_smem_desc(q_addr + kk * 32, 16, 8 * DH, DH);
                            const uint64_t db = umma_smem_desc(k_addr + kk * 32, 16, 8 * DH, DH);
                            umma_i8(tmem_base + (uint32_t)(g * W::GCOLS), da, db, idesc_s, kk != 0 ? 1u : 0u);
                        }
                        umma_commit(&s_full[g]);
                    }
                }
                const int j = k - (G - 1);
                if (j >= k_stop) break;
                if (j >= 0 && !issue_pv(j)) break;
            }
        }
    } else {
        // ------------------------------------------------------------ Softmax + output: one thread per tile row
        const int g = (warp - 2) >> 2;                         // group: owns S/O columns g * GCOLS.. and P buffer g
        const int quad = warp & 3;                             // TMEM lane quadrant this warp may touch
        const int rloc = quad * 32 + lane;                     // row inside the 128-row tile
        const int win = quad >> 1;                             // which problem of the pair
        const int row = rloc & 63;                             // row inside the problem
        const uint32_t tS = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(g * W::GCOLS + 64 * win);
        const uint32_t tO = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(g * W::GCOLS + 128);
        const uint32_t p_row = smem_u32(sP + g * W::P_BYTES) + (uint32_t)((rloc >> 3) * 1024 + (rloc & 7) * 128);
        const int HD = p.H * DH;
        const int nch = FULL ? 4 : ((p.N + 15) & ~15) >> 4;    // 16-column chunks of a row (1..4)
        const bool sat8 = p.orq.qmin == -128 && p.orq.qmax == 127;
        const uint32_t lut_addr = smem_u32(lut);
        const int tid = (int)threadIdx.x - 64;                 // 0 .. 128 G - 1
        {
            // P is block diagonal and key columns past the padded row length are never written: zero everything once
            int4* z = reinterpret_cast<int4*>(sP);
            for (int i = tid; i < G * W::P_BYTES / 16; i += 128 * G) z[i] = make_int4(0, 0, 0, 0);
            if (USE_LUT) {
                if (p.lut_src) {
                    // written and fenced by iptq_softmax_table(): safe to read ahead of the dependency wait
                    const int4* src = reinterpret_cast<const int4*>(p.lut_src);
                    int4* dst = reinterpret_cast<int4*>(lut);
                    for (int i = tid; i < (p.lut_n + 8) / 8; i += 128 * G) dst[i] = __ldg(src + i);
                } else {
                    for (int d = tid; d <= p.lut_n; d += 128 * G)
                        lut[d] = d < p.lut_n ? (uint16_t)exp_core_nd<VARIANT>(-d, p.ex) : (uint16_t)0;
                }
            }
            fence_proxy_async_smem();
            named_barrier(5, 128 * G);
        }
        grid_dep_wait();                                       // output rows are written only after this

        for (int k = g, n = 0;; k += G, ++n) {
            const int sk = k % ST;
            if (!mbar_wait(&kv_full[sk], (uint32_t)(k / ST) & 1u, ctl, p.status, 27)) break;   // acquire: the item number is visible
            const int it = item_of[sk];
            if (it < 0) break;
            int bh = 2 * it + win;
            const bool exists = bh < problems;
            if (!exists) bh = 0;
            const int h = bh % p.H, b = bh / p.H;
            const bool valid = exists && row < p.N;
            const bool warp_rows = exists && (quad & 1) * 32 < p.N;     // warp-uniform: any valid row in this warp
            // one thread per row: with the row-major bias the 32 lanes of a load hit 32 different sectors and a row
            // takes N loads; the re-laid-out copy gives a thread 4 columns per 16-byte load and a warp 512 contiguous bytes
            const int C4 = (p.N + 3) >> 2;
            const int32_t* brow = HAS_BIAS ? p.bias + ((size_t)h * p.N + (valid ? row : 0)) * p.N : nullptr;
            const int4* bq = HAS_BIAS && p.bias_q ? p.bias_q + (size_t)h * C4 * 64 + (valid ? row : 0) : nullptr;
            // the first chunk's quads are requested before the wait for the scores, the others one chunk ahead
            int4 bb[2][4];
            if (HAS_BIAS && bq && warp_rows) {
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) bb[0][q4] = q4 < C4 ? __ldg(bq + q4 * 64) : make_int4(0, 0, 0, 0);
            }
            // attention labels of the problem's tokens: lane l keeps those of columns l and l + 32, a column's label
            // then comes from a shuffle (all rows of a warp belong to the same problem)
            const uint8_t* mrow = HAS_MASK ? p.mask_id + (size_t)b * p.N : nullptr;
            const unsigned my_id = HAS_MASK ? mrow[valid ? row : 0] : 0u;
            const unsigned id_lo = HAS_MASK && lane < p.N ? mrow[lane] : 0x100u;
            const unsigned id_hi = HAS_MASK && lane + 32 < p.N ? mrow[lane + 32] : 0x100u;

            if (!mbar_wait(&s_full[g], (uint32_t)n & 1u, ctl, p.status, 25)) break;
            tc_fence_after_sync();
            uint32_t v[4][16];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (warp_rows && i < nch) tmem_ld16(tS + (uint32_t)(i * 16), v[i]);
            tmem_wait_ld();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_empty[g]);           // the MMA warp may overwrite S with the group's next item
            int mx = INT_MIN;
            // most windows of a shifted layout lie inside one region: all labels equal, nothing to mask (the labels
            // were requested before the wait for the scores and are first looked at here)
            const unsigned id_0 = __shfl_sync(0xffffffffu, id_lo, 0);
            const bool mixed = HAS_MASK && !__all_sync(0xffffffffu, (lane >= p.N || id_lo == id_0) && (lane + 32 >= p.N || id_hi == id_0));
            if (warp_rows) {
                // ---- row maximum over the real, unmasked columns (Eq. (6)); padding and masked pairs become kNoScore
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (i < nch) {
                        const int c0 = i * 16;
                        if (HAS_BIAS && bq) {
                            if (i + 1 < nch) {                                // next chunk's quads in flight meanwhile
#pragma unroll
                                for (int q4 = 0; q4 < 4; ++q4)
                                    bb[(i + 1) & 1][q4] = 4 * (i + 1) + q4 < C4 ? __ldg(bq + (4 * (i + 1) + q4) * 64) : make_int4(0, 0, 0, 0);
                            }
                            // the copy holds zeros past column N, so the bias is added without looking at the column
#pragma unroll
                            for (int q4 = 0; q4 < 4; ++q4) {
                                const int4 q = bb[i & 1][q4];
                                v[i][4 * q4] += (uint32_t)q.x; v[i][4 * q4 + 1] += (uint32_t)q.y;
                                v[i][4 * q4 + 2] += (uint32_t)q.z; v[i][4 * q4 + 3] += (uint32_t)q.w;
                            }
                        }
                        // each case is straight-line code: the conditions are warp-uniform and tested once per chunk
                        if (HAS_BIAS && !bq) {
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                if (c0 + j < p.N) v[i][j] += (uint32_t)__ldg(brow + c0 + j);
                        }
                        if (HAS_MASK && mixed) {
                            // labels past column N are 0x100 and match no row, so this also pads the row end
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const int col = c0 + j;                   // compile-time after unrolling: i and j are
                                const unsigned id = __shfl_sync(0xffffffffu, col < 32 ? id_lo : id_hi, col & 31);
                                v[i][j] = id == my_id ? v[i][j] : (uint32_t)kNoScore;
                            }
                        } else if (c0 + 16 > p.N) {
#pragma unroll
                            for (int j = 0; j < 16; ++j) v[i][j] = c0 + j < p.N ? v[i][j] : (uint32_t)kNoScore;
                        }
#pragma unroll
                        for (int j = 0; j < 16; ++j) mx = max(mx, (int)v[i][j]);
                    }
                }
                // ---- integer exponentials (Eqs. (7)-(14)), in place, and their sum
                unsigned sum = 0;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (i < nch) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            unsigned e;
                            if (USE_LUT) {
                                const unsigned d = min((unsigned)mx - v[i][j], (unsigned)p.lut_n);
                                asm volatile("ld.shared.u16 %0, [%1];" : "=r"(e) : "r"(lut_addr + 2u * d));
                            } else {
                                e = exp_core_nd<VARIANT>(exp_distance(mx, (int)v[i][j]), p.ex);
                            }
                            sum += e;
                            v[i][j] = e;
                        }
                    }
                }
                // ---- probabilities -> the UMMA A-operand layout (row rloc, key columns 64 win + 16 i ..)
                const unsigned f = VARIANT == IPTQ_SM_LOG2 ? 0u : intdiv_factor(sum, p.M) << p.f_shl;     // Eq. (15)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (i < nch) {
                        uint32_t wh[4], wl[4];
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            int hi[4], lo[4];
#pragma unroll
                            for (int t = 0; t < 4; ++t) {
                                if constexpr (VARIANT == IPTQ_SM_LOG2) {
                                    // p = 2^-code as the 16-bit value 2^(15 - code): exactly one byte is non-zero
                                    const unsigned code = log2_code(sum, v[i][q4 * 4 + t]);
                                    const unsigned w16 = code <= 15u ? (0x8000u >> code) : 0u;
                                    hi[t] = (int)(w16 >> 8);
                                    lo[t] = (int)(w16 & 0xffu);
                                } else {
                                    unsigned x = __umulhi(f, v[i][q4 * 4 + t]);
                                    if (PSHR) x >>= p.p_shr;
                                    hi[t] = (int)x;
                                    lo[t] = 0;
                                }
                            }
                            wh[q4] = pack4_sat_u8(hi[0], hi[1], hi[2], hi[3]);      // values are <= 2^(b-1): nothing saturates
                            wl[q4] = pack4_sat_u8(lo[0], lo[1], lo[2], lo[3]);
                        }
                        const int chunk = 4 * win + i;         // 16-key chunk inside the 128-key row of P
                        const uint32_t at = p_row + (uint32_t)((chunk ^ (rloc & 7)) << 4);
                        st_shared_v4(at, wh[0], wh[1], wh[2], wh[3]);
                        if constexpr (VARIANT == IPTQ_SM_LOG2) st_shared_v4(at + 16384u, wl[0], wl[1], wl[2], wl[3]);
                    }
                }
            }
            fence_proxy_async_smem();            // generic-proxy stores -> visible to the tensor core's reads
            __syncwarp();
            if (lane == 0) mbar_arrive(&p_ready[g]);
            // ---- output of this item: the other groups' items fill the time the P V product takes
            if (!mbar_wait(&o_full[g], (uint32_t)n & 1u, ctl, p.status, 26)) break;
            tc_fence_after_sync();
            if (warp_rows) {
                int8_t* orow = p.out + ((size_t)b * p.N + row) * HD + h * DH;
#pragma unroll
                for (int c = 0; c < DH / 16; ++c) {
                    uint32_t r[16];
                    tmem_ld16(tO + (uint32_t)(c * 16), r);
                    if constexpr (VARIANT == IPTQ_SM_LOG2) {
                        // O = 2^8 * (high plane product) + (low plane product), at scale 2^-15
                        uint32_t r2[16];
                        tmem_ld16(tO + (uint32_t)(DH + c * 16), r2);
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
                    if (valid) {
                        int4 pk;
                        pk.x = (int)pack4_sat_s8(o[0], o[1], o[2], o[3]);
                        pk.y = (int)pack4_sat_s8(o[4], o[5], o[6], o[7]);
                        pk.z = (int)pack4_sat_s8(o[8], o[9], o[10], o[11]);
                        pk.w = (int)pack4_sat_s8(o[12], o[13], o[14], o[15]);
                        *reinterpret_cast<int4*>(orow + c * 16) = pk;
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&o_empty[g]);
        }
    }

    // ------------------------------------------------------------ teardown (also reached after an abort)
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    if (ctl->abort) {
        for (int i = 0; i < 64; ++i) __nanosleep(2000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

// Geometry of the window kernel for (dh, variant): shared by the host code that sizes the launch.
struct WinGeom { int groups, stages, stage_bytes, p_bytes, gcols, threads; };
inline WinGeom window_geometry(int dh, int variant)
{
    WinGeom w;
    const bool log2 = variant == IPTQ_SM_LOG2;
    w.groups = (dh == 32 && !log2) ? 3 : 2;
    w.stages = w.groups + 2;
    w.stage_bytes = 3 * 128 * dh;
    w.p_bytes = 16384 * (log2 ? 2 : 1);
    w.gcols = 128 + dh * (log2 ? 2 : 1);
    w.threads = 64 + 128 * w.groups;
    return w;
}

template <int DH, int VARIANT>
int launch_window_attn(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const AttnParams& p,
                       int smem_bytes, cudaStream_t st)
{
    using W = WinCfg<DH, VARIANT>;
    const int grid = std::min(p.items, sm_count());
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return IPTQ_ERR_CUDA;
#define IPTQ_WIN_LAUNCH4(HB, HM, PS, LT, FL)                                                                      \
    do {                                                                                                          \
        auto kern = window_attention_kernel<DH, VARIANT, HB, HM, PS, LT, FL>;                                     \
        static int configured[64];          /* largest dynamic shared memory size set so far, per device */     \
        if (configured[dev] < smem_bytes) {                                                                       \
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) != cudaSuccess) \
                return IPTQ_ERR_CUDA;                                                                             \
            configured[dev] = smem_bytes;                                                                         \
        }                                                                                                         \
        launch_kernel(kern, grid, W::THREADS, smem_bytes, st, mq, mk, mv, p);                                     \
    } while (0)
#define IPTQ_WIN_LAUNCH3(HB, HM, PS, LT)                                                                          \
    do {                                                                                                          \
        if (p.N > 48) IPTQ_WIN_LAUNCH4(HB, HM, PS, LT, true); else IPTQ_WIN_LAUNCH4(HB, HM, PS, LT, false);       \
    } while (0)
#define IPTQ_WIN_LAUNCH2(HB, HM, PS)                                                                              \
    do {                                                                                                          \
        if (p.lut_n) IPTQ_WIN_LAUNCH3(HB, HM, PS, true); else IPTQ_WIN_LAUNCH3(HB, HM, PS, false);                \
    } while (0)
#define IPTQ_WIN_LAUNCH(HB, HM)                                                                                   \
    do {                                                                                                          \
        if (p.p_shr) IPTQ_WIN_LAUNCH2(HB, HM, true); else IPTQ_WIN_LAUNCH2(HB, HM, false);                        \
    } while (0)
    if (p.bias && p.mask_id) IPTQ_WIN_LAUNCH(true, true);
    else if (p.bias) IPTQ_WIN_LAUNCH(true, false);
    else if (p.mask_id) IPTQ_WIN_LAUNCH(false, true);
    else IPTQ_WIN_LAUNCH(false, false);
#undef IPTQ_WIN_LAUNCH
#undef IPTQ_WIN_LAUNCH2
#undef IPTQ_WIN_LAUNCH3
#undef IPTQ_WIN_LAUNCH4
    note_launch();
    return last_launch_status();
}

}  // namespace iptq
