// Chunk-prefill attention tiles on the 5th-generation tensor cores (tcgen05 + TMEM), included by sw_kernels.cu.
//
// One work item = one KV head x 256 query rows (two 128-row tiles).  A tile's rows are (token, query head of the
// group) pairs, token-major: row r <-> chunk token tok0 + r / g, head kvh*g + r % g, so all g query heads that
// share the KV head ride on the same K/V tiles.  Per 128-key KV tile j:
//     S_t = Q_t K_j^T          tcgen05.mma, A and B from shared memory (K-major, 128-byte swizzle), D in TMEM
//     P_t = exp2(S_t - m)      4 warps per tile, one thread per row (TMEM lane), P written back to TMEM as bf16
//     O_t += P_t V_j           tcgen05.mma, A from TMEM, B = V from shared memory (MN-major), D in TMEM
// Roles: warp 0 lane 0 issues TMA (Q once per item, K/V pages into a 2-stage ring), warp 1 lane 0 issues every
// MMA, warp 2 zeroes V rows past the end of the prompt (unwritten page slots), warps 4-7 / 8-11 run the online
// softmax of tile 0 / 1.  All hand-offs are mbarriers; every wait is bounded.
#pragma once

namespace sw {

template <int D>
struct PfGeo {
    static constexpr int kHalves = D / 64;
    static constexpr int kHalfBytes = 128 * 128;                 // [128 rows][64 elements], 128-byte swizzle
    static constexpr int kTileBytes = kHalves * kHalfBytes;      // one Q, K or V tile
    static constexpr int kQOffset = 0;                           // Q tile t at t * kTileBytes
    static constexpr int kKVOffset = 2 * kTileBytes;             // stage s: K at s * 2 * kTileBytes, then V
    static constexpr int kBytes = kKVOffset + 2 * 2 * kTileBytes;
    static constexpr int kPageBytes = kPageSize * 128;           // one page's rows inside a half
};

enum PfBar {
    kBarQFull = 0, kBarKFull = 1, kBarVLanded = 3, kBarVFull = 5, kBarKEmpty = 7, kBarVEmpty = 9,
    kBarSFull = 11, kBarPFull = 13, kBarODone = 15, kPfBars = 17
};

// register budgets per warpgroup during the prefill phase: 128 * 72 + 256 * 216 <= 384 * 168
constexpr int kPfRegsLaunch = 168, kPfRegsLight = 72, kPfRegsHeavy = 216;

struct PfShared {
    uint32_t smem;    // 1024-aligned shared address of the tile region
    uint32_t bars;    // shared address of the kPfBars mbarriers
    uint32_t tmem;    // TMEM base (lane 0, column 0 of the 512-column allocation)
    volatile int* abort_flag;
};

__device__ __forceinline__ void pf_init_barriers(uint32_t bars) {
    for (int i = 0; i < kPfBars; ++i) mbar_init(bars + i * 8, (i == kBarPFull || i == kBarPFull + 1) ? 4 : 1);
}

// Bounded wait that also gives up when another role of this CTA has given up.
__device__ __forceinline__ bool pf_wait(const PfShared& sh, int bar, uint32_t parity, int32_t* ctrl, int where) {
    const uint32_t addr = sh.bars + bar * 8;
    if (mbar_try_wait(addr, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t i = 0;; ++i) {
        if (mbar_try_wait(addr, parity)) return true;
        if ((i & 63) == 63) {
            if (*sh.abort_flag) return false;
            if (clock64() - t0 > kWaitBudgetCycles) break;
        }
    }
    *sh.abort_flag = 1;
    report(ctrl, SW_ERR_DEVICE_TIMEOUT, kSiteWait, (where << 8) | bar);
    return false;
}

// ---- work decomposition -------------------------------------------------------------------------------------------
// Items are ordered longest first: rank 0 is the last 256-row group of the chunk.  A "step" is one 128-key KV tile of
// one item.  All steps of all items form one line of length W that is cut into equal ranges, one per CTA, so every
// SM gets the same amount of tensor work whatever the chunk and prefix lengths are; an item cut by a range boundary
// is finished by several CTAs, each writing a partial (m, l, O) for its piece, and the last one to arrive merges.
struct PfPlan {
    int n_tp;           // 256-row groups of the chunk
    int total_steps;    // W
    int spc;            // steps per CTA (ceil(W / gridDim))
    const int* prefix;  // shared memory [n_tp + 1]: steps of one kv head's items before rank r
};

struct PfItem {
    int item;        // rank * Hkv + kvh
    int kvh;
    int tok0[2];     // first chunk token of each tile
    int nkv[2];      // KV tiles each tile attends in total (0 = tile has no rows)
    int start;       // index of the item's step 0 on the line of all steps
    int j0, j1;      // this CTA's piece of the item: KV tiles [j0, j1)
};

__device__ __forceinline__ int pf_tiles_of(const MixedParams& p, int tok0) {
    const int tt = 128 / p.group;  // tokens per tile
    if (tok0 >= p.C) return 0;
    return (p.P + min(tok0 + tt, p.C) - 1) / 128 + 1;
}
__device__ __forceinline__ int pf_num_groups(const MixedParams& p) {
    const int tok_per_item = 256 / p.group;
    return (p.C + tok_per_item - 1) / tok_per_item;
}
// steps of one item of rank r (the later tile, when it has rows, attends the most keys)
__device__ __forceinline__ int pf_steps_of_rank(const MixedParams& p, int n_tp, int r) {
    const int tt = 128 / p.group;
    const int tp = n_tp - 1 - r;
    return max(pf_tiles_of(p, (tp * 2) * tt), pf_tiles_of(p, (tp * 2 + 1) * tt));
}

// Built by all threads of the CTA; `prefix` needs n_tp + 1 ints, `scratch` kWarps + 1 ints.
__device__ __forceinline__ PfPlan pf_make_plan(const MixedParams& p, int* prefix, int* scratch) {
    PfPlan plan;
    plan.n_tp = pf_num_groups(p);
    const int per_thread = (plan.n_tp + kThreads - 1) / kThreads;
    const int beg = min(plan.n_tp, (int)threadIdx.x * per_thread);
    const int end = min(plan.n_tp, beg + per_thread);
    int local = 0;
    for (int r = beg; r < end; ++r) local += pf_steps_of_rank(p, plan.n_tp, r);
    int total = 0;
    int run = block_exclusive_scan(local, scratch, &total);
    for (int r = beg; r < end; ++r) {
        prefix[r] = run;
        run += pf_steps_of_rank(p, plan.n_tp, r);
    }
    if (threadIdx.x == 0) prefix[plan.n_tp] = total;
    __syncthreads();
    plan.total_steps = total * p.Hkv;
    plan.spc = (plan.total_steps + (int)gridDim.x - 1) / (int)gridDim.x;
    plan.prefix = prefix;
    return plan;
}

// The piece of the step line [x, range_end) that belongs to the item containing step x.
__device__ __forceinline__ PfItem pf_locate(const MixedParams& p, const PfPlan& plan, int x, int range_end) {
    int lo = 0, hi = plan.n_tp;  // largest rank with prefix[rank] * Hkv <= x
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (plan.prefix[mid] * p.Hkv <= x) lo = mid; else hi = mid;
    }
    const int rank = lo;
    const int nk = plan.prefix[rank + 1] - plan.prefix[rank];
    const int base = plan.prefix[rank] * p.Hkv;
    PfItem it;
    it.kvh = (x - base) / nk;
    it.item = rank * p.Hkv + it.kvh;
    it.start = base + it.kvh * nk;
    const int tt = 128 / p.group;
    const int tp = plan.n_tp - 1 - rank;
    for (int t = 0; t < 2; ++t) {
        it.tok0[t] = (tp * 2 + t) * tt;
        it.nkv[t] = pf_tiles_of(p, it.tok0[t]);
    }
    it.j0 = x - it.start;
    it.j1 = min(nk, range_end - it.start);
    return it;
}

// ---- role: TMA producer (one thread) ---------------------------------------------------------------------------
template <int D>
__device__ __forceinline__ bool pf_produce(const CUtensorMap* kv_map, const CUtensorMap* q_map, const MixedParams& p,
                                           const PfShared& sh, const PfItem& it, uint32_t& kv_it) {
    using G = PfGeo<D>;
    const int tt = 128 / p.group;
    // Q tiles (rows past the chunk are zero-filled by the tensor map's bounds)
    int active = (it.nkv[0] > it.j0) + (it.nkv[1] > it.j0);
    mbar_arrive_expect_tx(sh.bars + kBarQFull * 8, active * G::kTileBytes);
    for (int t = 0; t < 2; ++t)
        if (it.nkv[t] > it.j0)
            for (int h = 0; h < G::kHalves; ++h)
                tma_load_3d(sh.smem + G::kQOffset + t * G::kTileBytes + h * G::kHalfBytes, q_map, sh.bars + kBarQFull * 8,
                            h * 64, it.kvh * p.group, it.tok0[t]);
    (void)tt;
    const int npages = (p.P + p.C + kPageSize - 1) / kPageSize;
    for (int j = it.j0; j < it.j1; ++j, ++kv_it) {
        const uint32_t s = kv_it & 1, n = kv_it >> 1;
        const int pg0 = j * 8;
        const int nvp = min(8, npages - pg0);
        int ids[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) ids[i] = i < nvp ? p.prefill_pages[pg0 + i] : 0;
        const uint32_t kdst = sh.smem + G::kKVOffset + s * 2 * G::kTileBytes;
        const uint32_t vdst = kdst + G::kTileBytes;
        if (!pf_wait(sh, kBarKEmpty + s, (n & 1) ^ 1, p.ctrl, 1)) return false;
        mbar_arrive_expect_tx(sh.bars + (kBarKFull + s) * 8, nvp * G::kHalves * G::kPageBytes);
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (i < nvp)
                for (int h = 0; h < G::kHalves; ++h)
                    tma_load_4d(kdst + h * G::kHalfBytes + i * G::kPageBytes, kv_map, sh.bars + (kBarKFull + s) * 8, h * 64, 0,
                                it.kvh, ids[i]);
        if (!pf_wait(sh, kBarVEmpty + s, (n & 1) ^ 1, p.ctrl, 2)) return false;
        mbar_arrive_expect_tx(sh.bars + (kBarVLanded + s) * 8, nvp * G::kHalves * G::kPageBytes);
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (i < nvp)
                for (int h = 0; h < G::kHalves; ++h)
                    tma_load_4d(vdst + h * G::kHalfBytes + i * G::kPageBytes, kv_map, sh.bars + (kBarVLanded + s) * 8, h * 64,
                                0, p.Hkv + it.kvh, ids[i]);
    }
    return true;
}

// ---- role: V sanitizer (one warp) -------------------------------------------------------------------------------
// Keys at or past P + C are never attended, but their V rows still enter the P V product with weight zero; zero them
// so that whatever an unwritten page slot (or a stale buffer) holds cannot turn 0 * x into NaN.
template <int D>
__device__ __forceinline__ bool pf_sanitize(const MixedParams& p, const PfShared& sh, const PfItem& it, uint32_t& kv_it) {
    using G = PfGeo<D>;
    const int lane = threadIdx.x & 31;
    const int kv_total = p.P + p.C;
    for (int j = it.j0; j < it.j1; ++j, ++kv_it) {
        const uint32_t s = kv_it & 1, n = kv_it >> 1;
        if (!pf_wait(sh, kBarVLanded + s, n & 1, p.ctrl, 3)) return false;
        const int first_dead = max(0, kv_total - j * 128);
        if (first_dead < 128) {
            const uint32_t vdst = sh.smem + G::kKVOffset + s * 2 * G::kTileBytes + G::kTileBytes;
            const int chunks = (128 - first_dead) * 8;  // 16-byte pieces per half
            for (int h = 0; h < G::kHalves; ++h)
                for (int c = lane; c < chunks; c += 32) {
                    const uint32_t addr = vdst + h * G::kHalfBytes + (first_dead + c / 8) * 128 + (c % 8) * 16;
                    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0u) : "memory");
                }
            fence_proxy_async_smem();
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(sh.bars + (kBarVFull + s) * 8);
    }
    return true;
}

// ---- role: MMA issuer (one thread) ------------------------------------------------------------------------------
struct PfMmaState {
    uint32_t kv_it = 0, q_it = 0;
    uint32_t p_cnt[2] = {0, 0};
};

template <int D>
__device__ __forceinline__ void pf_issue_qk(const PfShared& sh, int t, uint32_t s) {
    using G = PfGeo<D>;
    constexpr uint32_t idesc = umma_idesc_bf16(128, 128, 0, 0);
    const uint32_t q = sh.smem + G::kQOffset + t * G::kTileBytes;
    const uint32_t k = sh.smem + G::kKVOffset + s * 2 * G::kTileBytes;
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
        const uint32_t off = (ks >> 2) * G::kHalfBytes + (ks & 3) * 32;
        tc_mma_ss(sh.tmem + t * 128, umma_desc_sw128(q + off, 16, 1024), umma_desc_sw128(k + off, 16, 1024), idesc, ks > 0);
    }
    tc_commit(sh.bars + (kBarSFull + t) * 8);
}

template <int D>
__device__ __forceinline__ void pf_issue_pv(const PfShared& sh, int t, uint32_t s, bool first) {
    using G = PfGeo<D>;
    constexpr uint32_t idesc = umma_idesc_bf16(128, D, 0, 1);  // B = V is MN-major: [key][d] with d contiguous
    const uint32_t v = sh.smem + G::kKVOffset + s * 2 * G::kTileBytes + G::kTileBytes;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks)  // 16 keys per instruction
        tc_mma_ts(sh.tmem + 256 + t * D, sh.tmem + t * 128 + ks * 8, umma_desc_sw128(v + ks * 2 * 1024, G::kHalfBytes, 1024),
                  idesc, !(first && ks == 0));
    tc_commit(sh.bars + (kBarODone + t) * 8);
}

template <int D>
__device__ __forceinline__ bool pf_mma(const MixedParams& p, const PfShared& sh, const PfItem& it, PfMmaState& st) {
    auto act = [&](int t, int j) { return j < it.j1 && j < it.nkv[t]; };
    auto last_active = [&](int j) { return act(1, j) ? 1 : 0; };
    if (!pf_wait(sh, kBarQFull, st.q_it & 1, p.ctrl, 4)) return false;
    {
        const uint32_t s = st.kv_it & 1, n = st.kv_it >> 1;
        if (!pf_wait(sh, kBarKFull + s, n & 1, p.ctrl, 5)) return false;
        tc_fence_after_sync();
        for (int t = 0; t < 2; ++t)
            if (act(t, it.j0)) pf_issue_qk<D>(sh, t, s);
        tc_commit(sh.bars + (kBarKEmpty + s) * 8);
    }
    for (int j = it.j0; j < it.j1; ++j) {
        const uint32_t cur = st.kv_it + (j - it.j0);
        const uint32_t s = cur & 1, n = cur >> 1;
        if (!pf_wait(sh, kBarVFull + s, n & 1, p.ctrl, 6)) return false;
        const bool more = j + 1 < it.j1;
        if (more && !pf_wait(sh, kBarKFull + (s ^ 1), ((cur + 1) >> 1) & 1, p.ctrl, 7)) return false;
        for (int t = 0; t < 2; ++t) {
            if (act(t, j)) {
                if (!pf_wait(sh, kBarPFull + t, st.p_cnt[t] & 1, p.ctrl, 8)) return false;
                st.p_cnt[t] += 1;
                tc_fence_after_sync();
                pf_issue_pv<D>(sh, t, s, j == it.j0);
            }
            if (t == last_active(j)) tc_commit(sh.bars + (kBarVEmpty + s) * 8);
            if (act(t, j + 1)) pf_issue_qk<D>(sh, t, s ^ 1);
            if (more && t == last_active(j + 1)) tc_commit(sh.bars + (kBarKEmpty + (s ^ 1)) * 8);
        }
    }
    st.kv_it += it.j1 - it.j0;
    st.q_it += 1;
    return true;
}

// ---- role: online softmax + epilogue (4 warps per tile, one thread per row) ---------------------------------------
// exp2 either on the special-function unit or, for a fixed share of the elements, as a cubic on the FMA pipe
// (round to nearest integer with the 1.5 * 2^23 trick, minimax cubic of 2^f on [-0.5, 0.5], relative error 7.5e-5 —
// far below the bf16 rounding of P — exponent added as integer bits).  The two pipes then share the row's 128 exps.
#ifndef SW_PF_POLY_EVERY
#define SW_PF_POLY_EVERY 0
#endif
#ifndef SW_PF_SPLIT_MAX
#define SW_PF_SPLIT_MAX 0
#endif
constexpr int kPolyEvery = SW_PF_POLY_EVERY;  // every kPolyEvery-th pair computes its first element with the polynomial; 0 = never
template <bool kPoly>
__device__ __forceinline__ float pf_exp2(float x) {
    if constexpr (!kPoly) {
        return fast_exp2(x);
    } else {
        x = fmaxf(x, -126.f);
        const float t = x + 12582912.f;
        const float f = x - (t - 12582912.f);
        float r = fmaf(f, 0.0551716648f, 0.2426111251f);
        r = fmaf(r, f, 0.6932609677f);
        r = fmaf(r, f, 0.9999280572f);
        return __int_as_float(__float_as_int(r) + (__float_as_int(t) << 23));
    }
}

struct PfSoftmaxState {
    uint32_t s_cnt = 0, o_cnt = 0;  // completions of this tile's S-ready / O-updated barriers consumed so far
};

// Scratch for items finished by several CTAs.  Slot = 2 * CTA + (0: the CTA's range starts inside the item,
// 1: the item starts inside the CTA's range); per slot and tile: m[128], l[128] and O[128][D], all fp32.
struct PfScratch {
    float* ml;         // [slots][2 tiles][2][128]
    float* o;          // [slots][2 tiles][128][D]
    int32_t* tickets;  // [items][2 tiles]
    volatile int* flags;  // shared memory, one int per tile: ticket value seen by the warpgroup's thread 0
};

template <int D>
__device__ __forceinline__ bool pf_softmax(const MixedParams& p, const PfShared& sh, const PfPlan& plan,
                                           const PfScratch& scr, const PfItem& it, int t, PfSoftmaxState& st) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j_end = min(it.j1, it.nkv[t]);
    if (j_end <= it.j0) return true;  // this tile has no step in this piece
    const int row = (warp & 3) * 32 + lane;
    const int tok = it.tok0[t] + row / p.group;
    const int head = it.kvh * p.group + row % p.group;
    const int pos = p.P + tok;
    const uint32_t lane_addr = sh.tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t s_addr = lane_addr + t * 128;  // P (bf16) aliases the first 64 columns of S
    const uint32_t o_addr = lane_addr + 256 + t * D;
    const float sl2 = p.sm_scale_log2;
    float m_ref = -INFINITY, l_sum = 0.f;
    uint32_t v[32];

    for (int j = it.j0; j < j_end; ++j) {
        if (!pf_wait(sh, kBarSFull + t, st.s_cnt & 1, p.ctrl, 9)) return false;
        st.s_cnt += 1;
        tc_fence_after_sync();
        // the whole row of S (128 fp32) in registers: one TMEM read per element
        uint32_t s[128];
        const int limit = pos - j * 128 + 1;  // columns [0, limit) are attended
        float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld_32x32b_x32(s_addr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
        tc_wait_ld();
        if (limit < 128) {
#pragma unroll
            for (int i = 0; i < 128; ++i) s[i] = i < limit ? s[i] : 0xff800000u;  // -inf: exp2 gives exactly 0
        }
#pragma unroll
        for (int i = 0; i < 128; i += 8) {
            mx0 = max3(mx0, __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
            mx1 = max3(mx1, __uint_as_float(s[i + 2]), __uint_as_float(s[i + 3]));
            mx2 = max3(mx2, __uint_as_float(s[i + 4]), __uint_as_float(s[i + 5]));
            mx3 = max3(mx3, __uint_as_float(s[i + 6]), __uint_as_float(s[i + 7]));
        }
        const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
        const float m_new = fmaxf(m_ref, mx * sl2);
        if (j == it.j0) {
            m_ref = m_new;
        } else {
            // lazy rescale: keep the old reference unless some row's maximum grew by more than 2^8
            // (a row whose keys were all masked so far has m_ref = -inf and no weight yet: it just adopts m_new)
            const bool need = m_new - m_ref > 8.0f;
            if (__any_sync(0xffffffffu, need)) {
                if (!pf_wait(sh, kBarODone + t, (st.o_cnt + (j - it.j0) - 1) & 1, p.ctrl, 10)) return false;
                tc_fence_after_sync();
                const float f = need ? fast_exp2(m_ref - m_new) : 1.f;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    tmem_ld_32x32b_x32(o_addr + c * 32, v);
                    tc_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * f);
                    tmem_st_32x32b_x32(o_addr + c * 32, v);
                }
                tc_wait_st();
                if (need) {
                    l_sum *= f;
                    m_ref = m_new;
                }
            }
        }
        // P = exp2(S * scale - m_ref), packed to bf16 over the columns of S (all of S is already in registers)
        const float neg_m = m_ref == -INFINITY ? 0.f : -m_ref;
        const uint64_t scale2 = pack_f32x2(sl2, sl2), negm2 = pack_f32x2(neg_m, neg_m);
        uint64_t sum_a = pack_f32x2(0.f, 0.f), sum_b = sum_a;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                // two columns per instruction: x = s * scale - m, P = 2^x, row sum, bf16 pack
                const uint64_t x2 = fma_f32x2(pack_f32x2(__uint_as_float(s[c * 32 + 2 * i]), __uint_as_float(s[c * 32 + 2 * i + 1])),
                                              scale2, negm2);
                float x0, x1;
                unpack_f32x2(x2, x0, x1);
                // the choice folds to a constant once the loop is unrolled
                const float p0 = (kPolyEvery != 0 && i % (kPolyEvery ? kPolyEvery : 1) == 0) ? pf_exp2<true>(x0)
                                                                                             : pf_exp2<false>(x0);
                const float p1 = fast_exp2(x1);
                if (i & 1) sum_b = add_f32x2(sum_b, pack_f32x2(p0, p1)); else sum_a = add_f32x2(sum_a, pack_f32x2(p0, p1));
                pk[i] = pack_bf16x2(p0, p1);
            }
            tmem_st_32x32b_x16(s_addr + c * 16, pk);
        }
        {
            float a0, a1, b0, b1;
            unpack_f32x2(sum_a, a0, a1);
            unpack_f32x2(sum_b, b0, b1);
            l_sum += (a0 + a1) + (b0 + b1);
        }
        tc_wait_st();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(sh.bars + (kBarPFull + t) * 8);
    }

    // the piece's O is complete once its last P V has been committed
    if (!pf_wait(sh, kBarODone + t, (st.o_cnt + (j_end - it.j0) - 1) & 1, p.ctrl, 11)) return false;
    st.o_cnt += j_end - it.j0;
    tc_fence_after_sync();
    const bool row_ok = tok < p.C;
    __nv_bfloat16* dst = p.out + ((int64_t)tok * p.Hq + head) * D;
    const bool whole = it.j0 == 0 && j_end == it.nkv[t];
    if (whole) {
        // epilogue of an item this CTA did alone: O / l -> bf16 -> out
        const float inv = 1.f / l_sum;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
            tmem_ld_32x32b_x32(o_addr + c * 32, v);
            tc_wait_ld();
            if (row_ok) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 w;
                    w.x = pack_bf16x2(__uint_as_float(v[8 * i + 0]) * inv, __uint_as_float(v[8 * i + 1]) * inv);
                    w.y = pack_bf16x2(__uint_as_float(v[8 * i + 2]) * inv, __uint_as_float(v[8 * i + 3]) * inv);
                    w.z = pack_bf16x2(__uint_as_float(v[8 * i + 4]) * inv, __uint_as_float(v[8 * i + 5]) * inv);
                    w.w = pack_bf16x2(__uint_as_float(v[8 * i + 6]) * inv, __uint_as_float(v[8 * i + 7]) * inv);
                    *reinterpret_cast<uint4*>(dst + c * 32 + i * 8) = w;
                }
            }
        }
        if (row_ok && p.lse) p.lse[(int64_t)tok * p.Hq + head] = (m_ref + __log2f(l_sum)) * 0.6931471805599453f;
        tc_fence_before_sync();
        return true;
    }

    // ---- the item is shared with other CTAs: publish this piece, the last piece to arrive merges all of them ----
    const int cta = blockIdx.x;
    const int first_cta = it.start / plan.spc;
    const int last_cta = (it.start + it.nkv[t] - 1) / plan.spc;
    const int my_slot = 2 * cta + (cta * plan.spc >= it.start ? 0 : 1);
    {
        float* ml = scr.ml + ((int64_t)my_slot * 2 + t) * 256;
        float* po = scr.o + (((int64_t)my_slot * 2 + t) * 128 + row) * D;
        ml[row] = m_ref;
        ml[128 + row] = l_sum;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
            tmem_ld_32x32b_x32(o_addr + c * 32, v);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 8; ++i)
                *reinterpret_cast<uint4*>(po + c * 32 + i * 4) = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
        }
    }
    tc_fence_before_sync();
    __threadfence();
    named_barrier_sync(2 + t, 128);
    if ((warp & 3) == 0 && lane == 0) scr.flags[t] = atomicAdd(&scr.tickets[it.item * 2 + t], 1);
    named_barrier_sync(2 + t, 128);
    const bool merger = scr.flags[t] == last_cta - first_cta;
    named_barrier_sync(2 + t, 128);  // everyone has read the flag before a later piece may overwrite it
    if (!merger) return true;
    __threadfence();
    if ((warp & 3) == 0 && lane == 0) scr.tickets[it.item * 2 + t] = 0;  // re-armed for the next launch
    float m_all = -INFINITY;
    for (int b = first_cta; b <= last_cta; ++b) {
        const int slot = 2 * b + (b * plan.spc >= it.start ? 0 : 1);
        m_all = fmaxf(m_all, __ldcg(scr.ml + ((int64_t)slot * 2 + t) * 256 + row));
    }
    float acc[D];
#pragma unroll
    for (int i = 0; i < D; ++i) acc[i] = 0.f;
    float l_all = 0.f;
    for (int b = first_cta; b <= last_cta; ++b) {
        const int slot = 2 * b + (b * plan.spc >= it.start ? 0 : 1);
        const float* ml = scr.ml + ((int64_t)slot * 2 + t) * 256;
        const float ms = __ldcg(ml + row);
        const float w = ms == -INFINITY ? 0.f : fast_exp2(ms - m_all);
        l_all += w * __ldcg(ml + 128 + row);
        const float4* po = reinterpret_cast<const float4*>(scr.o + (((int64_t)slot * 2 + t) * 128 + row) * D);
#pragma unroll
        for (int i = 0; i < D / 4; ++i) {
            const float4 x = __ldcg(po + i);
            acc[4 * i + 0] = fmaf(w, x.x, acc[4 * i + 0]);
            acc[4 * i + 1] = fmaf(w, x.y, acc[4 * i + 1]);
            acc[4 * i + 2] = fmaf(w, x.z, acc[4 * i + 2]);
            acc[4 * i + 3] = fmaf(w, x.w, acc[4 * i + 3]);
        }
    }
    if (row_ok) {
        const float inv = 1.f / l_all;
#pragma unroll
        for (int i = 0; i < D / 8; ++i) {
            uint4 w;
            w.x = pack_bf16x2(acc[8 * i + 0] * inv, acc[8 * i + 1] * inv);
            w.y = pack_bf16x2(acc[8 * i + 2] * inv, acc[8 * i + 3] * inv);
            w.z = pack_bf16x2(acc[8 * i + 4] * inv, acc[8 * i + 5] * inv);
            w.w = pack_bf16x2(acc[8 * i + 6] * inv, acc[8 * i + 7] * inv);
            *reinterpret_cast<uint4*>(dst + i * 8) = w;
        }
        if (p.lse) p.lse[(int64_t)tok * p.Hq + head] = (m_all + __log2f(l_all)) * 0.6931471805599453f;
    }
    return true;
}

// ---- the prefill phase of one CTA ----------------------------------------------------------------------------------
template <int D>
__device__ __forceinline__ void prefill_phase(const CUtensorMap* kv_map, const CUtensorMap* q_map, const MixedParams& p,
                                              const PfShared& sh, const PfPlan& plan, const PfScratch& scr) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int range_begin = min(plan.total_steps, (int)blockIdx.x * plan.spc);
    const int range_end = min(plan.total_steps, range_begin + plan.spc);
    uint32_t prod_kv_it = 0, san_kv_it = 0;
    PfMmaState mma_state;
    PfSoftmaxState sm_state;
    // The softmax warpgroups hold a whole row of S in registers; the TMA / MMA / sanitizer warps need few.  The two
    // kinds of warps run separate loops (so that each gets its own register budget) and meet at a named barrier at
    // the end of every piece.  (The caller guarantees a non-empty range: two register re-budgetings of a
    // warpgroup must be separated by a synchronisation of its warps.)
    auto piece_sync = [&]() {
        __syncwarp();
        tc_fence_before_sync();
        named_barrier_sync(1, kThreads);
        tc_fence_after_sync();
        return *sh.abort_flag == 0;
    };
    if (warp < 4) {
        setmaxnreg_dec<kPfRegsLight>();
        for (int x = range_begin; x < range_end;) {
            const PfItem it = pf_locate(p, plan, x, range_end);
            if (warp == 0) {
                if (lane == 0) pf_produce<D>(kv_map, q_map, p, sh, it, prod_kv_it);
            } else if (warp == 1) {
                if (lane == 0) pf_mma<D>(p, sh, it, mma_state);
            } else if (warp == 2) {
                pf_sanitize<D>(p, sh, it, san_kv_it);
            }
            x = it.start + it.j1;
            if (!piece_sync()) break;
        }
        setmaxnreg_inc<kPfRegsLaunch>();
    } else {
        setmaxnreg_inc<kPfRegsHeavy>();
        for (int x = range_begin; x < range_end;) {
            const PfItem it = pf_locate(p, plan, x, range_end);
            pf_softmax<D>(p, sh, plan, scr, it, (warp - 4) >> 2, sm_state);
            x = it.start + it.j1;
            if (!piece_sync()) break;
        }
        setmaxnreg_dec<kPfRegsLaunch>();
    }
}

}  // namespace sw
