// Chunk-prefill attention tiles on the 5th-generation tensor cores (tcgen05 + TMEM), included by sw_kernels.cu.
//
// One work item = one KV head x 256 query rows (two 128-row tiles).  A tile's rows are (token, query head of the
// group) pairs, token-major: row r <-> chunk token tok0 + r / g, head kvh*g + r % g, so all g query heads that
// share the KV head ride on the same K/V tiles.  Per 128-key KV tile j:
//     S_t = Q_t K_j^T          tcgen05.mma, A and B from shared memory (K-major, 128-byte swizzle), D in TMEM
//     P_t = exp2(S_t - m)      4 warps per tile, one thread per row (TMEM lane), P written back to TMEM as bf16
//     O_t += P_t V_j           tcgen05.mma, A from TMEM, B = V from shared memory (MN-major), D in TMEM
// Roles: warp 0 issues TMA (Q once per item, K/V pages into a 2-stage ring; lane i owns page i of a tile), warp 1
// issues every MMA (one elected lane), warp 2 zeroes V rows past the end of the prompt (unwritten page slots), warp 3
// fetches the next work item, warps 4-7 / 8-11 run the online softmax of tile 0 / 1.  All hand-offs are mbarriers;
// every wait is bounded.
//
// Operand tiles of K and V hold their 128 keys as sixteen 8-key groups, each group as head_dim/64 swizzled blocks of
// [8 slots][128 bytes] side by side: [group 0..15][block][8][128 B].  The 8-key groups of one 64-element block are thus a
// uniform stride apart (what the matrix descriptors need), and a page (two groups) is one contiguous stretch that ONE
// copy of 4 KB fills (head_dim 128): the tensor map views a page's rows of one head as {64 elements, 8 slots, block,
// slot group}.  The copy engine's cost is per copy; with one copy per 2 KB block the producer warp was busy for a whole
// step and K tiles arrived late.
#pragma once

namespace sw {

template <int D>
struct PfGeo {
    static constexpr int kHalves = D / 64;
    static constexpr int kHalfBytes = 128 * 128;                 // Q: [128 rows][64 elements], 128-byte swizzle
    static constexpr int kTileBytes = kHalves * kHalfBytes;      // one Q, K or V tile
    static constexpr int kQOffset = 0;                           // Q tile t at t * kTileBytes
    static constexpr int kKVOffset = 2 * kTileBytes;             // stage s: K at s * 2 * kTileBytes, then V
    static constexpr int kBytes = kKVOffset + 2 * 2 * kTileBytes;
    static constexpr int kAtomBytes = 8 * 128;                   // K, V: one [8 slots][64 elements] swizzled block
    static constexpr int kGroupStride = kHalves * kAtomBytes;    // K, V: 8 keys, [head_dim/64 blocks][8][128 B]
    static constexpr int kPageStride = 2 * kGroupStride;         // K, V: one page = two 8-key groups
};

// P of a tile is handed to the MMA warp in two halves (keys 0-63, then 64-127) so that the first four P V
// instructions run while the second half is still being exponentiated.
enum PfBar {
    kBarQFull = 0, kBarKFull = 1, kBarVLanded = 3, kBarVFull = 5, kBarKEmpty = 7, kBarVEmpty = 9,
    kBarSFull = 11, kBarPHalf = 13 /* [tile][half] */, kBarODone = 17, kPfBars = 19
};

// register budgets per warpgroup during the prefill phase: 128 * 72 + 256 * 216 <= 384 * 168
constexpr int kPfRegsLaunch = 168, kPfRegsLight = 72, kPfRegsHeavy = 216;

constexpr int kChunkTable = 88;  // ints into the CTA's scratch: P[8], C[8], first row[8], page-list offset[8], pieces[8] of the chunks
constexpr int kChunkTotals = 7 * 8;  // ints into the table: the plan's totals, after seven fields of eight chunks

struct PfShared {
    uint32_t smem;    // 1024-aligned shared address of the tile region
    uint32_t bars;    // shared address of the kPfBars mbarriers
    uint32_t tmem;    // TMEM base (lane 0, column 0 of the 512-column allocation)
    volatile int* abort_flag;
};

// Field `field` (0 prefix length, 1 tokens, 2 first row, 3 page-list offset, 4 pieces per tail item) of chunk `chunk` from the table in shared
// memory; its address follows from the tile region's, so no role keeps a pointer to it.
// A kernel that serves a single chunk (kMulti = false) reads the kernel parameters instead, which costs no register
// and no instruction in any role.
template <int D, bool kMulti>
__device__ __forceinline__ int pf_chunk(const MixedParams& p, const PfShared& sh, int field, int chunk) {
    if constexpr (!kMulti) {
        return field == 0 ? p.cP[0] : (field == 1 ? p.cC[0] : 0);
    } else {
        return lds_s32(sh.smem + Geo<D>::kMiscOffset + (kChunkTable + field * kMaxChunks + chunk) * 4);
    }
}

__device__ __forceinline__ void pf_init_barriers(uint32_t bars) {
    for (int i = 0; i < kPfBars; ++i) mbar_init(bars + i * 8, (i >= kBarPHalf && i < kBarPHalf + 4) ? 4 : 1);
}

// Bounded wait that also gives up when another role of this CTA has given up.
__device__ __forceinline__ bool pf_wait(const PfShared& sh, int bar, uint32_t parity, int32_t* ctrl, int where) {
    const uint32_t addr = sh.bars + bar * 8;
    if (mbar_try_wait(addr, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t i = 0;; ++i) {
        // (the long prefill launches run at the power cap: letting the hardware park a waiting warp for up to a
        // microsecond instead of polling measured 1-3 % faster)
        if (mbar_try_wait_suspend(addr, parity, 1000)) return true;
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
// Items (one KV head x 256 query rows) are ordered longest first: rank 0 is the last 256-row group of the chunk.
// A "step" is one 128-key KV tile of one item.  The G CTAs that take entries (PfPlan::ctas) pull them from a global
// counter.  The first n_whole entries are whole items; the remaining r = n_items mod G items (all of them when there
// are fewer items than CTAs) would leave most SMs idle in the last wave, so each of them is cut along the KV axis into k
// pieces that run side by side; every piece publishes a partial (m, l, O) and the last piece of an item to arrive
// merges them.  CTAs working at the same time thus stay at similar KV positions (their K/V tiles meet in L2).
constexpr int kPfMinPieceSteps = 4;   // never pieces shorter than this many KV steps
constexpr int kPfPieceCost = 1;       // steps' worth of work that cutting an item into one more piece costs
// Whole rounds of items beside decode requests: the decode pages need the memory system, not the SMs, and about
// kDecodeCtasAtFullRate CTAs' rings of page copies already draw the full rate.  So a few CTAs take no chunk-prefill work
// at all and stream decode pages from the start, as many as it takes for the two kinds of work to end together (G is
// the grid less those CTAs); the leftover items of the others' last round are cut into pieces that may run in several
// rounds.  Whoever runs out of its own kind of work takes the other.
constexpr int kDecodeCtasAtFullRate = 64;
constexpr float kDecodeCtasMinGain = 0.20f;   // share of the launch's CTA time the rule must save to be applied
constexpr float kDecodeCtasMinSteps = 48.f;   // and the shortest decode phase (at the full rate, in steps of an entry)
constexpr float kEntryCostSteps = 3.f;        // fill and drain of an entry, in steps
constexpr float kEntrySafety = 1.25f;
constexpr int kPfMinRoundPieceSteps = 24;  // pieces that run in several rounds: at least this many KV steps each
constexpr int kPfMaxRoundPieces = 12;

struct PfPlan {
    int longest, shortest;             // steps of the longest and of the shortest item (items are numbered chunk by chunk)
    int n_items;        // sum over chunks of (256-row groups) * Hkv
    int n_whole;        // entries [0, n_whole) are whole items
    int pieces;         // k: pieces per tail item (1 = tail items are whole too); several chunks: of the first chunk's
    int n_entries;      // n_whole + (n_items - n_whole) * k; several chunks: every chunk's tail items times its own k
    int ctas;           // CTAs that take entries (the first ones by index); the others start with decode units
    uint32_t table;     // several chunks: shared address of the chunk table (k of chunk j is field 4)
};

struct PfItem {
    int item;        // number of the item among all chunks' items; within its chunk: rank * Hkv + kvh
    int kvh;
    int chunk;       // which chunk of the iteration the item belongs to (its descriptors are in the shared table)
    int tok0[2];     // first chunk token of each tile
    int nkv[2];      // KV tiles each tile attends in total (0 = tile has no rows)
    int nk;          // steps of the item = max(nkv)
    int j0, j1;      // this entry's piece of the item: KV tiles [j0, j1)
    int piece;       // index of the piece (0 when the item is whole)
    int slot0;       // scratch slot of the item's piece 0 (tail items only)
    int pieces;      // pieces the item is cut into (several chunks: each chunk has its own count)
};

__device__ __forceinline__ int pf_tiles_of(int group, int P, int C, int tok0) {
    const int tt = 128 / group;  // tokens per tile
    if (tok0 >= C) return 0;
    return (P + min(tok0 + tt, C) - 1) / 128 + 1;
}
__device__ __forceinline__ int pf_num_groups(int group, int C) {
    const int tok_per_item = 256 / group;
    return (C + tok_per_item - 1) / tok_per_item;
}
// steps of one item of rank r of a chunk with n_tp groups (the later tile, when it has rows, attends the most keys)
__device__ __forceinline__ int pf_steps_of_rank(int group, int P, int C, int n_tp, int r) {
    const int tt = 128 / group;
    const int tp = n_tp - 1 - r;
    return max(pf_tiles_of(group, P, C, (tp * 2) * tt), pf_tiles_of(group, P, C, (tp * 2 + 1) * tt));
}
// first KV tile of piece i when nk steps are cut into k pieces
__device__ __forceinline__ int pf_piece_begin(int nk, int k, int i) { return (int)(((long long)nk * i) / k); }

// k ~ sqrt(steps / cost): a piece costs its steps plus a merge that grows with k (about one step's worth per piece
// merged, with partial results laid out so that publishing and merging are coalesced); never pieces shorter than the
// minimum.
__device__ __forceinline__ int pf_pieces_for(int steps) {
    int k = 1;
    while ((k + 1) * (k + 1) * kPfPieceCost <= steps) ++k;
    return max(1, min(k, steps / kPfMinPieceSteps));
}

// CTAs that take chunk-prefill entries when n_items items of wp steps in all run beside the decode requests (the
// others start with decode units); G when the plain order is kept.
__device__ __forceinline__ int pf_entry_ctas(const MixedParams& p, int G, int n_items, float wp, float decode_steps) {
    if (p.n <= 0 || n_items < G) return G;  // no decode requests, or not even one whole round of items
    // work in CTA-steps: the decode pages at the rate of one CTA, and with every CTA drawing 1 / G of the full rate
    const float wd = decode_steps * (float)kDecodeCtasAtFullRate, wd_all = decode_steps * (float)G;
    // CTA time the launch saves when few CTAs stream.  Entries run slower while pages are streamed beside them, so
    // below a fifth of the launch the plain order (every CTA turns to the decode units after its entries) is kept;
    // it is also kept beside a decode phase so short that latency, not the streaming rate, bounds it.
    if (decode_steps < kDecodeCtasMinSteps || wd_all - wd < kDecodeCtasMinGain * (wp + wd_all)) return G;
    // d CTAs streaming for the whole launch finish with the others when d / G is the decode share of the work
    const int d = (int)(wd * (float)G / (wp + wd) + 0.5f);
    if (d < kDecodeCtasAtFullRate) return G - min(d, G / 2);
    // The decode pages are the longer part: kDecodeCtasAtFullRate streaming CTAs or more draw the full rate, so the launch
    // cannot end before decode_steps, and the entries only have to be done by then.  They get as many CTAs as that takes
    // (every entry counted with its fill and drain, and with a margin: entries run slower beside streaming CTAs), at
    // least an eighth of the grid and at most what the full rate leaves.
    const int need = (int)ceilf(kEntrySafety * (wp + kEntryCostSteps * (float)n_items) / decode_steps);
    return min(max(need, max(1, G / 8)), G - min(kDecodeCtasAtFullRate, G / 2));
}
__device__ __forceinline__ float pf_decode_steps(const MixedParams& p) {  // the decode phase at the full rate, in steps
    return p.n > 0 ? (float)__ldg(p.decode_page_indptr + p.n) * (float)p.Hkv * p.steps_per_stage : 0.f;
}

// Several chunks in one iteration: the tail items (the last n_items mod G ones, G the CTAs that take entries) belong to chunks of very
// different lengths, e.g. the end of a long prompt next to the start of a new one.  Each chunk gets its own piece
// count, sized by its shortest item; while the tail entries outnumber the CTAs, the chunk with the shortest pieces
// gives one up.  Run by one whole warp in the kernel prologue, lane j owning chunk j; fills the chunk table:
// fields 0-3 the descriptors, 4 pieces per tail item, 5 items before the chunk, 6 tail entries before the chunk's
// tail items (fields 5 and 6 hold INT_MAX where nothing may match), then the plan's totals.
__device__ __forceinline__ void pf_fill_chunk_table(const MixedParams& p, int* tbl) {
    const int lane = threadIdx.x & 31;
    int P = 0, C = 0, row0 = 0, page0 = 0;
#pragma unroll
    for (int j = 0; j < kMaxChunks; ++j)
        if (lane == j) {
            P = p.cP[j];
            C = p.cC[j];
            row0 = p.cRow0[j];
            page0 = p.cPage0[j];
        }
    const bool live = lane < p.nchunks;
    const int n_tp = live ? pf_num_groups(p.group, C) : 0;
    const int cnt = n_tp * p.Hkv;
    auto scan = [&](int v) {  // inclusive, over the first kMaxChunks lanes
        for (int d = 1; d < kMaxChunks; d <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, v, d);
            if (lane >= d) v += u;
        }
        return v;
    };
    const int incl = scan(cnt);
    const int before = incl - cnt;
    const int n_items = __shfl_sync(0xffffffffu, incl, kMaxChunks - 1);
    int longest = 0, shortest = 0x7fffffff;
    if (n_tp > 0) {
        longest = pf_steps_of_rank(p.group, P, C, n_tp, 0);
        shortest = pf_steps_of_rank(p.group, P, C, n_tp, n_tp - 1);
    }
    // beside enough decode pages a few CTAs take no entry (the rule of the single-chunk plan; pieces in one round here)
    const int steps2 = __reduce_add_sync(0xffffffffu, n_tp > 0 ? (longest + shortest) * cnt : 0);
    const int G = pf_entry_ctas(p, (int)gridDim.x, n_items, 0.5f * (float)steps2, pf_decode_steps(p));
    const int n_whole = n_items - n_items % G;
    const int tail = max(0, before + cnt - max(before, n_whole));
    int k = tail > 0 ? pf_pieces_for(shortest) : 1;
    int total = __reduce_add_sync(0xffffffffu, tail * k);
    while (total > G) {  // warp-uniform
        const int key = (tail > 0 && k > 1) ? (((shortest / k) << 5) | lane) : 0x7fffffff;
        const int best = __reduce_min_sync(0xffffffffu, key);
        if (best == 0x7fffffff) break;  // every k is 1: the tail holds fewer items than there are CTAs
        if (key == best) k -= 1;
        total -= __shfl_sync(0xffffffffu, tail, best & 31);
    }
    const int acc = scan(tail * k) - tail * k;
    longest = __reduce_max_sync(0xffffffffu, longest);
    shortest = __reduce_min_sync(0xffffffffu, shortest);
    const int k0 = __shfl_sync(0xffffffffu, k, 0);
    if (lane < kMaxChunks) {
        tbl[lane] = P;
        tbl[kMaxChunks + lane] = C;
        tbl[2 * kMaxChunks + lane] = row0;
        tbl[3 * kMaxChunks + lane] = page0;
        tbl[4 * kMaxChunks + lane] = k;
        tbl[5 * kMaxChunks + lane] = live ? before : 0x7fffffff;
        tbl[6 * kMaxChunks + lane] = tail > 0 ? acc : 0x7fffffff;
    }
    if (lane == 0) {
        int* tot = tbl + kChunkTotals;
        tot[0] = n_items;
        tot[1] = n_whole;
        tot[2] = n_whole + total;
        tot[3] = longest;
        tot[4] = shortest;
        tot[5] = n_whole == 0 ? k0 : 1;
        tot[6] = G;
    }
}

template <bool kMulti>
__device__ __forceinline__ PfPlan pf_make_plan(const MixedParams& p, uint32_t table) {
    PfPlan plan;
    plan.table = table;
    if constexpr (kMulti) {  // worked out once per CTA by pf_fill_chunk_table
        const uint32_t tot = table + kChunkTotals * 4;
        plan.n_items = lds_s32(tot);
        plan.n_whole = lds_s32(tot + 4);
        plan.n_entries = lds_s32(tot + 8);
        plan.longest = lds_s32(tot + 12);
        plan.shortest = lds_s32(tot + 16);
        plan.pieces = lds_s32(tot + 20);
        plan.ctas = lds_s32(tot + 24);
        return plan;
    }
    int G = (int)gridDim.x;
    const int n_tp = pf_num_groups(p.group, p.cC[0]);
    plan.n_items = n_tp * p.Hkv;
    plan.longest = 0;
    plan.shortest = 0x7fffffff;
    if (n_tp > 0) {
        plan.longest = pf_steps_of_rank(p.group, p.cP[0], p.cC[0], n_tp, 0);
        plan.shortest = pf_steps_of_rank(p.group, p.cP[0], p.cC[0], n_tp, n_tp - 1);
    }
    const float decode_steps = pf_decode_steps(p);
    const int entry_ctas = pf_entry_ctas(p, G, plan.n_items, 0.5f * (float)(plan.longest + plan.shortest) * (float)plan.n_items,
                                         decode_steps);
    const bool rounds = entry_ctas < G;  // whole rounds of items (their lengths fall linearly with the rank) beside decode CTAs
    G = entry_ctas;
    plan.ctas = G;
    const int r = plan.n_items % G;
    plan.n_whole = plan.n_items - r;
    plan.pieces = 1;
    if (rounds && r > 0) {
        // The leftover items may run in several rounds of pieces: the k that ends the last round soonest (a piece costs
        // its steps plus its share of the merge), among those whose partial results fit the scratch.
        const int kmax = min(min(kPfMaxRoundPieces, p.pf_slots / r), max(1, plan.shortest / kPfMinRoundPieceSteps));
        int best = 0x7fffffff;
        for (int k = 1; k <= kmax; ++k) {
            const int t = ((r * k + G - 1) / G) * ((plan.shortest + k - 1) / k + (k > 1 ? 2 + k / 2 : 0));
            if (t < best) {
                best = t;
                plan.pieces = k;
            }
        }
    } else if (r > 0) {
        // the tail items are short ones; size the pieces by the shortest item, never more pieces than fit side by side
        plan.pieces = min(G / r, pf_pieces_for(plan.shortest));
    }
    if (!rounds && plan.pieces > 1 && p.n > 0) {
        // Beside a long decode phase the leftover items need not finish early, and every CTA they occupy is a CTA
        // that does not stream decode pages meanwhile: pieces about as long as the decode phase (all decode pages at
        // the streaming rate, counted in steps of an entry under decode traffic) are short enough.
        const int kmax = plan.pieces;
        plan.pieces = min(kmax, max(1, (int)ceilf((float)plan.shortest / decode_steps)));
        if (plan.n_whole == 0 && decode_steps >= kDecodeCtasMinSteps) {
            // Fewer items than CTAs beside a decode phase bound by the streaming rate: the CTAs without an entry stream
            // at (their number / kDecodeCtasAtFullRate) of the full rate while the pieces run, everybody streams what is
            // left afterwards; the k that ends the launch soonest.
            float best = 3.0e38f;
            for (int k = 1; k <= kmax; ++k) {
                const float t = (float)((plan.shortest + k - 1) / k + (k > 1 ? 2 + k / 2 : 0));
                const float rate = fminf(1.f, (float)(G - r * k) / (float)kDecodeCtasAtFullRate);
                const float end = t + fmaxf(0.f, decode_steps - t * rate);
                if (end < best) {
                    best = end;
                    plan.pieces = k;
                }
            }
        }
    }
    if (plan.pieces == 1) plan.n_whole = plan.n_items;
    plan.n_entries = plan.n_whole + (plan.n_items - plan.n_whole) * plan.pieces;
    return plan;
}

template <bool kMulti>
__device__ __forceinline__ PfItem pf_entry(const MixedParams& p, const PfPlan& plan, int entry) {
    PfItem it;
    it.pieces = plan.pieces;
    it.slot0 = 0;
    it.chunk = 0;
    int before = 0, cP = p.cP[0], cC = p.cC[0];
    if constexpr (!kMulti) {
        if (entry < plan.n_whole) {
            it.item = entry;
            it.piece = 0;
        } else {
            it.item = plan.n_whole + (entry - plan.n_whole) / plan.pieces;
            it.piece = (entry - plan.n_whole) % plan.pieces;
            it.slot0 = (it.item - plan.n_whole) * plan.pieces;
        }
    } else {
        // The entry's chunk is the last one whose threshold it reaches: for a whole item the items before the chunk,
        // for a tail entry the tail entries before the chunk's (tail entries are numbered chunk by chunk: a chunk's
        // tail items times the chunk's own piece count; the first chunk that has tail items has threshold 0).
        const bool whole = entry < plan.n_whole;
        const int key = whole ? entry : entry - plan.n_whole;
        const uint32_t thr = plan.table + (whole ? 5 : 6) * kMaxChunks * 4;
#pragma unroll
        for (int j = 1; j < kMaxChunks; ++j)
            if (key >= lds_s32(thr + j * 4)) it.chunk = j;
        const uint32_t col = plan.table + it.chunk * 4;
        cP = lds_s32(col);
        cC = lds_s32(col + kMaxChunks * 4);
        before = lds_s32(col + 5 * kMaxChunks * 4);
        if (whole) {
            it.item = entry;
            it.piece = 0;
        } else {
            it.pieces = lds_s32(col + 4 * kMaxChunks * 4);
            const int rel = key - lds_s32(col + 6 * kMaxChunks * 4);
            const int idx = rel / it.pieces;
            it.item = max(before, plan.n_whole) + idx;
            it.piece = rel - idx * it.pieces;
            it.slot0 = key - it.piece;
        }
    }
    const int local = it.item - before;
    const int rank = local / p.Hkv;
    it.kvh = local % p.Hkv;
    const int tt = 128 / p.group;
    const int tp = pf_num_groups(p.group, cC) - 1 - rank;
    for (int t = 0; t < 2; ++t) {
        it.tok0[t] = (tp * 2 + t) * tt;
        it.nkv[t] = pf_tiles_of(p.group, cP, cC, it.tok0[t]);
    }
    it.nk = max(it.nkv[0], it.nkv[1]);
    if (entry < plan.n_whole) {
        it.j0 = 0;
        it.j1 = it.nk;
    } else {
        it.j0 = pf_piece_begin(it.nk, it.pieces, it.piece);
        it.j1 = pf_piece_begin(it.nk, it.pieces, it.piece + 1);
    }
    return it;
}

// ---- role: TMA producer (one warp) ----------------------------------------------------------------------------
template <int D, bool kMulti>
__device__ __forceinline__ bool pf_produce(const CUtensorMap* kv_map, const CUtensorMap* q_map, const MixedParams& p,
                                           const PfShared& sh, const PfItem& it, uint32_t& kv_it) {
    using G = PfGeo<D>;
    // The whole warp runs the role: lane i owns page i of every 128-key tile (its page id, its TMA boxes), so the
    // eight pages of a tile are issued by one instruction instead of a loop of one thread.
    const int lane = threadIdx.x & 31;
    // Q tiles (rows past the chunk are zero-filled by the tensor map's bounds)
    if (lane == 0) {
        const int active = (it.nkv[0] > it.j0) + (it.nkv[1] > it.j0);
        mbar_arrive_expect_tx(sh.bars + kBarQFull * 8, active * G::kTileBytes);
        for (int t = 0; t < 2; ++t)
            if (it.nkv[t] > it.j0)
                for (int h = 0; h < G::kHalves; ++h)
                    tma_load_3d(sh.smem + G::kQOffset + t * G::kTileBytes + h * G::kHalfBytes, q_map, sh.bars + kBarQFull * 8,
                                h * 64, it.kvh * p.group, pf_chunk<D, kMulti>(p, sh, 2, it.chunk) + it.tok0[t]);
    }
    // fused launch: tiles that reach into the chunk's own keys wait until every CTA has written its share of them
    if (p.pool != nullptr && it.j1 * 128 > pf_chunk<D, kMulti>(p, sh, 0, it.chunk) && !wait_append(p)) {
        if (lane == 0) {
            *sh.abort_flag = 1;
            report(p.ctrl, SW_ERR_DEVICE_TIMEOUT, kSiteWait, it.item);
        }
        return false;
    }
    const int npages = (pf_chunk<D, kMulti>(p, sh, 0, it.chunk) + pf_chunk<D, kMulti>(p, sh, 1, it.chunk) + kPageSize - 1) / kPageSize;
    auto page_of = [&](int j) {
        int id = (lane < 8 && j * 8 + lane < npages) ? p.prefill_pages[pf_chunk<D, kMulti>(p, sh, 3, it.chunk) + j * 8 + lane] : 0;
        if (id < 0 || (int64_t)id >= p.num_pages) {
            // reported, and page 0 fetched in its place: a bad id never reaches the copy engine
            report(p.ctrl, SW_ERR_OUT_OF_RANGE, kSiteAttnPage, it.item);
            id = 0;
        }
        return id;
    };
    int id_next = page_of(it.j0);
    for (int j = it.j0; j < it.j1; ++j, ++kv_it) {
        const uint32_t s = kv_it & 1, n = kv_it >> 1;
        const int id = id_next;
        if (j + 1 < it.j1) id_next = page_of(j + 1);  // in flight while this tile is issued
        const int nvp = min(8, npages - j * 8);
        const uint32_t kdst = sh.smem + G::kKVOffset + s * 2 * G::kTileBytes;
        const uint32_t vdst = kdst + G::kTileBytes;
        if (!pf_wait(sh, kBarKEmpty + s, (n & 1) ^ 1, p.ctrl, 1)) return false;
        if (lane == 0) mbar_arrive_expect_tx(sh.bars + (kBarKFull + s) * 8, nvp * G::kPageStride);
        __syncwarp();
        if (lane < nvp)
            tma_load_5d(kdst + lane * G::kPageStride, kv_map, sh.bars + (kBarKFull + s) * 8, 0, 0, 0, 0, (2 * id) * p.Hkv + it.kvh);
        if (!pf_wait(sh, kBarVEmpty + s, (n & 1) ^ 1, p.ctrl, 2)) return false;
        if (lane == 0) mbar_arrive_expect_tx(sh.bars + (kBarVLanded + s) * 8, nvp * G::kPageStride);
        __syncwarp();
        if (lane < nvp)
            tma_load_5d(vdst + lane * G::kPageStride, kv_map, sh.bars + (kBarVLanded + s) * 8, 0, 0, 0, 0,
                        (2 * id + 1) * p.Hkv + it.kvh);
    }
    return true;
}

// ---- role: V sanitizer (one warp) -------------------------------------------------------------------------------
// Keys at or past P + C are never attended, but their V rows still enter the P V product with weight zero; zero them
// so that whatever an unwritten page slot (or a stale buffer) holds cannot turn 0 * x into NaN.
template <int D, bool kMulti>
__device__ __forceinline__ bool pf_sanitize(const MixedParams& p, const PfShared& sh, const PfItem& it, uint32_t& kv_it) {
    using G = PfGeo<D>;
    const int lane = threadIdx.x & 31;
    const int kv_total = pf_chunk<D, kMulti>(p, sh, 0, it.chunk) + pf_chunk<D, kMulti>(p, sh, 1, it.chunk);
    for (int j = it.j0; j < it.j1; ++j, ++kv_it) {
        const uint32_t s = kv_it & 1, n = kv_it >> 1;
        if (!pf_wait(sh, kBarVLanded + s, n & 1, p.ctrl, 3)) return false;
        const int first_dead = max(0, kv_total - j * 128);
        if (first_dead < 128) {
            const uint32_t vdst = sh.smem + G::kKVOffset + s * 2 * G::kTileBytes + G::kTileBytes;
            const int chunks = (128 - first_dead) * 8;  // 16-byte pieces per 64-element block
            for (int h = 0; h < G::kHalves; ++h)
                for (int c = lane; c < chunks; c += 32) {
                    const int key = first_dead + c / 8;
                    const uint32_t addr = vdst + (key >> 3) * G::kGroupStride + h * G::kAtomBytes + (key & 7) * 128 + (c % 8) * 16;
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

// The whole MMA warp runs this role in lockstep (waits included) so that addresses and descriptors stay in uniform
// registers; only the tcgen05.mma / tcgen05.commit instructions themselves are issued by the one elected lane.
template <int D>
__device__ __forceinline__ void pf_issue_qk(const PfShared& sh, int t, uint32_t s, bool leader) {
    using G = PfGeo<D>;
    constexpr uint32_t idesc = umma_idesc_bf16(128, 128, 0, 0);
    const uint64_t qd = umma_desc_sw128(sh.smem + G::kQOffset + t * G::kTileBytes, 16, 1024);
    const uint64_t kd = umma_desc_sw128(sh.smem + G::kKVOffset + s * 2 * G::kTileBytes, 16, G::kGroupStride);
    const uint32_t d_tmem = sh.tmem + t * 128;
    if (leader) {
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            // descriptor address units (16 bytes): 64-element block ks / 4, 16 elements = 32 bytes per slice
            const uint64_t qoff = (uint64_t)(((ks >> 2) * G::kHalfBytes + (ks & 3) * 32) >> 4);
            const uint64_t koff = (uint64_t)(((ks >> 2) * G::kAtomBytes + (ks & 3) * 32) >> 4);
            tc_mma_ss(d_tmem, qd + qoff, kd + koff, idesc, ks > 0);
        }
        tc_commit(sh.bars + (kBarSFull + t) * 8);
    }
}

// one half of O_t += P_t V: keys [64 * half, 64 * half + 64), 16 keys = one page per instruction (its two 8-key groups
// are one group stride apart, the 64-element blocks of a row one block apart)
template <int D>
__device__ __forceinline__ void pf_issue_pv_half(const PfShared& sh, int t, uint32_t s, int half, bool first, bool leader) {
    using G = PfGeo<D>;
    constexpr uint32_t idesc = umma_idesc_bf16(128, D, 0, 1);  // B = V is MN-major: [key][d] with d contiguous
    const uint64_t vd = umma_desc_sw128(sh.smem + G::kKVOffset + s * 2 * G::kTileBytes + G::kTileBytes + half * 4 * G::kPageStride,
                                        G::kAtomBytes, G::kGroupStride);
    const uint32_t d_tmem = sh.tmem + 256 + t * D;
    const uint32_t p_tmem = sh.tmem + t * 128 + half * 32;
    const uint32_t acc_first = first && half == 0 ? 0u : 1u;
    if (leader) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            tc_mma_ts(d_tmem, p_tmem + i * 8, vd + (uint64_t)(i * (G::kPageStride >> 4)), idesc, i == 0 ? acc_first : 1u);
        if (half == 1) tc_commit(sh.bars + (kBarODone + t) * 8);
    }
}

template <int D>
__device__ __forceinline__ bool pf_mma(const MixedParams& p, const PfShared& sh, const PfItem& it, PfMmaState& st) {
    const bool leader = elect_one();
    auto act = [&](int t, int j) { return j < it.j1 && j < it.nkv[t]; };
    auto last_active = [&](int j) { return act(1, j) ? 1 : 0; };
    auto commit = [&](int bar) {
        if (leader) tc_commit(sh.bars + bar * 8);
    };
    if (!pf_wait(sh, kBarQFull, st.q_it & 1, p.ctrl, 4)) return false;
    {
        const uint32_t s = st.kv_it & 1, n = st.kv_it >> 1;
        if (!pf_wait(sh, kBarKFull + s, n & 1, p.ctrl, 5)) return false;
        tc_fence_after_sync();
        for (int t = 0; t < 2; ++t)
            if (act(t, it.j0)) pf_issue_qk<D>(sh, t, s, leader);
        commit(kBarKEmpty + s);
    }
    for (int j = it.j0; j < it.j1; ++j) {
        const uint32_t cur = st.kv_it + (j - it.j0);
        const uint32_t s = cur & 1, n = cur >> 1;
        if (!pf_wait(sh, kBarVFull + s, n & 1, p.ctrl, 6)) return false;
        const bool more = j + 1 < it.j1;
        bool k_ready = false;  // K of tile j+1 is awaited as late as possible: right before its first use
        for (int t = 0; t < 2; ++t) {
            if (act(t, j)) {
                for (int half = 0; half < 2; ++half) {
                    if (!pf_wait(sh, kBarPHalf + 2 * t + half, st.p_cnt[t] & 1, p.ctrl, 8)) return false;
                    tc_fence_after_sync();
                    pf_issue_pv_half<D>(sh, t, s, half, j == it.j0, leader);
                }
                st.p_cnt[t] += 1;
            }
            if (t == last_active(j)) commit(kBarVEmpty + s);
            if (act(t, j + 1)) {
                if (!k_ready) {
                    if (!pf_wait(sh, kBarKFull + (s ^ 1), ((cur + 1) >> 1) & 1, p.ctrl, 7)) return false;
                    k_ready = true;
                }
                pf_issue_qk<D>(sh, t, s ^ 1, leader);
            }
            if (more && t == last_active(j + 1)) commit(kBarKEmpty + (s ^ 1));
        }
    }
    st.kv_it += it.j1 - it.j0;
    st.q_it += 1;
    return true;
}

// ---- role: online softmax + epilogue (4 warps per tile, one thread per row) ---------------------------------------
// The row's 128 exponentials are the longest stretch of a tile's softmax: the special-function unit delivers one warp
// instruction every 8 cycles, 1024 cycles per row, as long as the tensor core needs for a whole tile.  A fixed share of
// the column pairs is therefore exponentiated on the FMA pipe instead, two columns per instruction: x = n + f with n the
// nearest integer (1.5 * 2^23 trick), a minimax cubic of 2^f on [-0.5, 0.5] (relative error 7.5e-5, far below the bf16
// rounding of P), and n added to the exponent as integer bits.  Of every 8 pairs the first kPfFmaPairsOf8 take this path.
constexpr int kPfMaxChains = 4;      // independent chains of the row maximum
constexpr int kPfFmaPairsOf8 = 2;    // measured: 2 of 8 gains 2-4 %, 3 of 8 nothing, 4 of 8 loses (the FMA pipe fills up)
__device__ __forceinline__ void pf_exp2_pair_fma(uint64_t x2, float& p0, float& p1) {
    float x0, x1;
    unpack_f32x2(x2, x0, x1);
    const uint64_t xc = pack_f32x2(fmaxf(x0, -126.f), fmaxf(x1, -126.f));   // 2^-126 stands for zero (and for -inf)
    const uint64_t t = add_f32x2(xc, pack_f32x2(12582912.f, 12582912.f));  // low mantissa bits = n
    const uint64_t r = add_f32x2(t, pack_f32x2(-12582912.f, -12582912.f)); // n as a float
    const uint64_t f = fma_f32x2(r, pack_f32x2(-1.f, -1.f), xc);
    uint64_t q = fma_f32x2(f, pack_f32x2(0.0551716648f, 0.0551716648f), pack_f32x2(0.2426111251f, 0.2426111251f));
    q = fma_f32x2(q, f, pack_f32x2(0.6932609677f, 0.6932609677f));
    q = fma_f32x2(q, f, pack_f32x2(0.9999280572f, 0.9999280572f));
    float q0, q1, t0, t1;
    unpack_f32x2(q, q0, q1);
    unpack_f32x2(t, t0, t1);
    p0 = __int_as_float(__float_as_int(q0) + (__float_as_int(t0) << 23));
    p1 = __int_as_float(__float_as_int(q1) + (__float_as_int(t1) << 23));
}

struct PfSoftmaxState {
    uint32_t s_cnt = 0, o_cnt = 0;  // completions of this tile's S-ready / O-updated barriers consumed so far
};

// Scratch for the tail items cut into pieces.  Slot = (tail item index) * k + piece (at most gridDim slots);
// per slot and tile: m[128], l[128] and O[128][D], all fp32.
struct PfScratch {
    float* ml;         // [slots][2 tiles][2][128]
    float* o;          // [slots][2 tiles][D / 4 column chunks][128 rows][4]
    int32_t* tickets;  // [items][2 tiles]
    volatile int* flags;  // shared memory, one int per tile: ticket value seen by the warpgroup's thread 0
};

template <int D, bool kMulti>
__device__ __forceinline__ bool pf_softmax(const CUtensorMap* out_map, const MixedParams& p, const PfShared& sh,
                                           const PfPlan& plan, const PfScratch& scr, const PfItem& it, int t,
                                           PfSoftmaxState& st) {
    using G = PfGeo<D>;
    if (it.j1 <= it.j0) return true;  // an empty piece (more pieces than steps)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j_end = min(it.j1, it.nkv[t]);
    if (j_end <= it.j0) return true;  // this tile has no step in this piece
    const int row = (warp & 3) * 32 + lane;
    const int tok = it.tok0[t] + row / p.group;
    const int head = it.kvh * p.group + row % p.group;
    const int pos = pf_chunk<D, kMulti>(p, sh, 0, it.chunk) + tok;
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
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld_32x32b_x32(s_addr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
        tc_wait_ld();
        if (limit < 128) {
#pragma unroll
            for (int i = 0; i < 128; ++i) s[i] = i < limit ? s[i] : 0xff800000u;  // -inf: exp2 gives exactly 0
        }
        // row maximum: independent chains of 3-input max, then a short tree
        float mxv[kPfMaxChains];
#pragma unroll
        for (int c = 0; c < kPfMaxChains; ++c) mxv[c] = -INFINITY;
#pragma unroll
        for (int i = 0; i < 128; i += 2 * kPfMaxChains)
#pragma unroll
            for (int c = 0; c < kPfMaxChains; ++c)
                mxv[c] = max3(mxv[c], __uint_as_float(s[i + 2 * c]), __uint_as_float(s[i + 2 * c + 1]));
#pragma unroll
        for (int w = kPfMaxChains / 2; w > 0; w >>= 1)
#pragma unroll
            for (int c = 0; c < w; ++c) mxv[c] = fmaxf(mxv[c], mxv[c + w]);
        const float mx = mxv[0];
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
                float p0, p1;
                if ((i & 7) < kPfFmaPairsOf8) {   // folds to a constant once the loop is unrolled
                    pf_exp2_pair_fma(x2, p0, p1);
                } else {
                    float x0, x1;
                    unpack_f32x2(x2, x0, x1);
                    p0 = fast_exp2(x0);
                    p1 = fast_exp2(x1);
                }
                if (i & 1) sum_b = add_f32x2(sum_b, pack_f32x2(p0, p1)); else sum_a = add_f32x2(sum_a, pack_f32x2(p0, p1));
                pk[i] = pack_bf16x2(p0, p1);
            }
            tmem_st_32x32b_x16(s_addr + c * 16, pk);
            if (c == 1) {  // the first 64 keys of P are in place: the first half of P V may start
                tc_wait_st();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(sh.bars + (kBarPHalf + 2 * t) * 8);
            }
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
        if (lane == 0) mbar_arrive(sh.bars + (kBarPHalf + 2 * t + 1) * 8);
    }

    // the piece's O is complete once its last P V has been committed
    if (!pf_wait(sh, kBarODone + t, (st.o_cnt + (j_end - it.j0) - 1) & 1, p.ctrl, 11)) return false;
    st.o_cnt += j_end - it.j0;
    tc_fence_after_sync();
    const bool row_ok = tok < pf_chunk<D, kMulti>(p, sh, 1, it.chunk);
    const int64_t out_row = (int64_t)pf_chunk<D, kMulti>(p, sh, 2, it.chunk) + tok;
    __nv_bfloat16* dst = p.out + (out_row * p.Hq + head) * D;
    const bool whole = it.j0 == 0 && j_end == it.nkv[t];  // this piece holds every step of the tile
    if (whole) {
        // epilogue of an item this CTA did alone: O / l -> bf16 -> out
        const float inv = 1.f / l_sum;
        const int chunk_rows = pf_chunk<D, kMulti>(p, sh, 1, it.chunk);
        if (it.tok0[t] + 128 / p.group <= chunk_rows) {
            // Every row of the tile is a row of the chunk: the tile goes to the slot its Q tile came from (the last
            // Q K^T of the tile has long completed), in the same swizzled layout, and one thread hands it to the copy
            // engine, which writes whole 128-byte lines instead of 128 threads storing 16 bytes each.
            const uint32_t stage = sh.smem + G::kQOffset + t * G::kTileBytes + row * 128;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                tmem_ld_32x32b_x32(o_addr + c * 32, v);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int q = c * 4 + i;  // 16-byte piece of the row: half q / 8, position q % 8 (swizzled by the row)
                    sts_v4(stage + (q >> 3) * G::kHalfBytes + (((q & 7) ^ (row & 7)) << 4),
                           pack_bf16x2(__uint_as_float(v[8 * i + 0]) * inv, __uint_as_float(v[8 * i + 1]) * inv),
                           pack_bf16x2(__uint_as_float(v[8 * i + 2]) * inv, __uint_as_float(v[8 * i + 3]) * inv),
                           pack_bf16x2(__uint_as_float(v[8 * i + 4]) * inv, __uint_as_float(v[8 * i + 5]) * inv),
                           pack_bf16x2(__uint_as_float(v[8 * i + 6]) * inv, __uint_as_float(v[8 * i + 7]) * inv));
                }
            }
            if (p.lse) p.lse[out_row * p.Hq + head] = (m_ref + __log2f(l_sum)) * 0.6931471805599453f;
            tc_fence_before_sync();
            fence_proxy_async_smem();
            named_barrier_sync(2 + t, 128);
            if ((warp & 3) == 0 && lane == 0) {
                const int row0 = pf_chunk<D, kMulti>(p, sh, 2, it.chunk) + it.tok0[t];
#pragma unroll
                for (int h = 0; h < G::kHalves; ++h)
                    tma_store_3d(out_map, sh.smem + G::kQOffset + t * G::kTileBytes + h * G::kHalfBytes, h * 64,
                                 it.kvh * p.group, row0);
                tma_store_commit();
                // the slot is read before this thread reaches the barrier that lets the producer refill it
                tma_store_wait_read();
            }
            return true;
        }
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
        if (row_ok && p.lse) p.lse[out_row * p.Hq + head] = (m_ref + __log2f(l_sum)) * 0.6931471805599453f;
        tc_fence_before_sync();
        return true;
    }

    // ---- the item is shared with other CTAs: publish this piece, the last piece to arrive merges all of them ----
    // pieces of this item that hold steps of tile t: 0 .. last_piece (pieces are never empty: k <= nk / 4)
    int last_piece = 0;
    for (int i = 1; i < it.pieces; ++i)
        if (pf_piece_begin(it.nk, it.pieces, i) < it.nkv[t]) last_piece = i;
    const int n_mine = last_piece + 1;
    const int my_slot = it.slot0 + it.piece;
    {
        float* ml = scr.ml + ((int64_t)my_slot * 2 + t) * 256;
        // O of a (slot, tile) is stored by 16-byte column chunks: chunk q of all 128 rows, then chunk q + 1, so that
        // the 32 rows of a warp write (and the merging warp reads) 512 contiguous bytes per instruction
        float* po = scr.o + ((int64_t)my_slot * 2 + t) * 128 * D + row * 4;
        ml[row] = m_ref;
        ml[128 + row] = l_sum;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
            tmem_ld_32x32b_x32(o_addr + c * 32, v);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 8; ++i)
                *reinterpret_cast<uint4*>(po + (c * 8 + i) * 512) = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
        }
    }
    tc_fence_before_sync();
    __threadfence();
    named_barrier_sync(2 + t, 128);
    if ((warp & 3) == 0 && lane == 0) scr.flags[t] = atomicAdd(&scr.tickets[it.item * 2 + t], 1);
    named_barrier_sync(2 + t, 128);
    const bool merger = scr.flags[t] == n_mine - 1;
    named_barrier_sync(2 + t, 128);  // everyone has read the flag before a later piece may overwrite it
    if (!merger) return true;
    __threadfence();
    if ((warp & 3) == 0 && lane == 0) scr.tickets[it.item * 2 + t] = 0;  // re-armed for the next launch
    const float* ml0 = scr.ml + ((int64_t)it.slot0 * 2 + t) * 256 + row;  // piece i: + i * 512 floats
    float m_all = -INFINITY;
#pragma unroll 4
    for (int i = 0; i <= last_piece; ++i) m_all = fmaxf(m_all, __ldcg(ml0 + (int64_t)i * 512));
    // weights of the pieces: w_i = 2^(m_i - m_all); l = sum_i w_i l_i
    float l_all = 0.f;
#pragma unroll 4
    for (int i = 0; i <= last_piece; ++i) {
        const float ms = __ldcg(ml0 + (int64_t)i * 512);
        l_all += (ms == -INFINITY ? 0.f : fast_exp2(ms - m_all)) * __ldcg(ml0 + (int64_t)i * 512 + 128);
    }
    const float inv = 1.f / l_all;
    // 64 output columns at a time keeps the accumulators small, so that the loads of two pieces are in flight
    const float* o0 = scr.o + ((int64_t)it.slot0 * 2 + t) * 128 * D + row * 4;  // piece i: + i * 2 * 128 * D floats
#pragma unroll 1
    for (int c = 0; c < D / 64; ++c) {
        float acc[64];
#pragma unroll
        for (int i = 0; i < 64; ++i) acc[i] = 0.f;
#pragma unroll 2
        for (int i = 0; i <= last_piece; ++i) {
            const float ms = __ldcg(ml0 + (int64_t)i * 512);
            const float w = ms == -INFINITY ? 0.f : fast_exp2(ms - m_all);
            const float* po = o0 + (int64_t)i * 2 * 128 * D + c * 16 * 512;
            float4 x[16];
#pragma unroll
            for (int q = 0; q < 16; ++q) x[q] = __ldcg(reinterpret_cast<const float4*>(po + q * 512));
#pragma unroll
            for (int q = 0; q < 16; ++q) {
                acc[4 * q + 0] = fmaf(w, x[q].x, acc[4 * q + 0]);
                acc[4 * q + 1] = fmaf(w, x[q].y, acc[4 * q + 1]);
                acc[4 * q + 2] = fmaf(w, x[q].z, acc[4 * q + 2]);
                acc[4 * q + 3] = fmaf(w, x[q].w, acc[4 * q + 3]);
            }
        }
        if (row_ok) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                uint4 w;
                w.x = pack_bf16x2(acc[8 * i + 0] * inv, acc[8 * i + 1] * inv);
                w.y = pack_bf16x2(acc[8 * i + 2] * inv, acc[8 * i + 3] * inv);
                w.z = pack_bf16x2(acc[8 * i + 4] * inv, acc[8 * i + 5] * inv);
                w.w = pack_bf16x2(acc[8 * i + 6] * inv, acc[8 * i + 7] * inv);
                *reinterpret_cast<uint4*>(dst + c * 64 + i * 8) = w;
            }
        }
    }
    if (row_ok && p.lse) p.lse[out_row * p.Hq + head] = (m_all + __log2f(l_all)) * 0.6931471805599453f;
    return true;
}

// ---- the prefill phase of one CTA ----------------------------------------------------------------------------------
// `next` points at two shared-memory ints: the idle warp fetches the following entry from the global counter while
// the current one is processed and leaves it in next[iteration parity]; everyone reads it after the piece barrier.
template <int D, bool kMulti>
__device__ __forceinline__ void prefill_phase(const CUtensorMap* kv_map, const CUtensorMap* q_map, const CUtensorMap* out_map,
                                              const MixedParams& p, const PfShared& sh, const PfPlan& plan,
                                              const PfScratch& scr, int first_entry, volatile int* next) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint32_t prod_kv_it = 0, san_kv_it = 0;
    PfMmaState mma_state;
    PfSoftmaxState sm_state;
    // The softmax warpgroups hold a whole row of S in registers; the TMA / MMA / sanitizer warps need few.  The two
    // kinds of warps run separate loops (so that each gets its own register budget) and meet at a named barrier at
    // the end of every piece.  (The caller guarantees at least one entry: two register re-budgetings of a
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
        int entry = first_entry;
        for (int iter = 0; entry < plan.n_entries; ++iter) {
            const PfItem it = pf_entry<kMulti>(p, plan, entry);
            if (warp == 0) {
                if (it.j1 > it.j0) pf_produce<D, kMulti>(kv_map, q_map, p, sh, it, prod_kv_it);
            } else if (warp == 1) {
                if (it.j1 > it.j0) pf_mma<D>(p, sh, it, mma_state);
            } else if (warp == 2) {
                if (it.j1 > it.j0) pf_sanitize<D, kMulti>(p, sh, it, san_kv_it);
            } else {
                // entries 0 .. plan.ctas-1 are the CTAs' first ones; the counter hands out the rest
                if (lane == 0) next[iter & 1] = plan.ctas + atomicAdd(&p.ctrl[kCtrPrefill], 1);
            }
            if (!piece_sync()) break;
            entry = next[iter & 1];
        }
        setmaxnreg_inc<kPfRegsLaunch>();
    } else {
        setmaxnreg_inc<kPfRegsHeavy>();
        int entry = first_entry;
        for (int iter = 0; entry < plan.n_entries; ++iter) {
            const PfItem it = pf_entry<kMulti>(p, plan, entry);
            pf_softmax<D, kMulti>(out_map, p, sh, plan, scr, it, (warp - 4) >> 2, sm_state);
            if (!piece_sync()) break;
            entry = next[iter & 1];
        }
        tma_store_wait_all();  // the tiles handed to the copy engine are in global memory before the CTA moves on
        setmaxnreg_dec<kPfRegsLaunch>();
    }
}

}  // namespace sw
