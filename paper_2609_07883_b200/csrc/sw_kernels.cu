// sm_100a kernels of the mixed prefill-chunk + decode attention iteration.
//
//   sw_kv_append_kernel     scatter of this iteration's new K/V rows into their pages (Table 1, KV manager)
//   sw_mixed_attn_kernel    ONE persistent launch per iteration (Sec. 4.1).  Optionally it first writes the new K/V
//                           rows itself (the fused form of the append).  CTAs with chunk-prefill entries run them on
//                           the tensor cores (sw_prefill.cuh).  Every CTA then plans the split-KV decode units from
//                           the context lengths; a warp's first unit is fixed by its index, further ones come from a
//                           shared counter; a unit streams its K/V pages with TMA into the warp's shared-memory ring
//                           and keeps an online softmax in registers; of the units of one (request, kv head) the one
//                           that drew the last ticket merges the partial results.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "sw_internal.h"
#include "sw_ptx.cuh"

namespace sw {
using namespace swptx;

// ---------------------------------------------------------------------------------------------------------------
// device status: first problem wins
// ---------------------------------------------------------------------------------------------------------------
__device__ __forceinline__ void report(int32_t* ctrl, int code, int site, int index) {
    if (atomicCAS(&ctrl[kCtrStatus], 0, code) == 0) ctrl[kCtrDetail] = (site << 24) | (index & 0xFFFFFF);
}

// ---------------------------------------------------------------------------------------------------------------
// KV append
// ---------------------------------------------------------------------------------------------------------------
// One thread per (row, 16-byte piece of the row's Hkv*D elements); it copies that piece of K and of V.  `first` and
// `stride` spread the pieces over the calling threads.
// (P is AppendParams or MixedParams: the fields have the same names; every index into the chunk arrays is a
// compile-time constant so that the kernel parameters stay in constant memory.)
template <bool kMulti, class P>
__device__ __forceinline__ void append_rows(const P& p, int head_dim, int64_t first, int64_t stride) {
    const int pieces_per_row = p.Hkv * head_dim / 8;
    const int64_t total = (int64_t)(p.C + p.n) * pieces_per_row;
    for (int64_t idx = first; idx < total; idx += stride) {
        const int row = (int)(idx / pieces_per_row);
        const int piece = (int)(idx % pieces_per_row);
        int64_t pos;
        const int32_t* pages;
        int npages;
        if (row < p.C) {
            // the chunk this row belongs to: the last one that starts at or before it
            int cP = p.cP[0], cRow0 = 0, page0 = 0, page1 = p.num_prefill_pages;
#pragma unroll
            for (int j = 0; j < kMaxChunks; ++j)
                if (kMulti && j < p.nchunks && row >= p.cRow0[j]) {
                    cP = p.cP[j];
                    cRow0 = p.cRow0[j];
                    page0 = p.cPage0[j];
                    page1 = p.cPage0[j + 1];
                }
            pos = (int64_t)cP + (row - cRow0);
            pages = p.prefill_pages + page0;
            npages = page1 - page0;
        } else {
            const int i = row - p.C;
            const int len = p.decode_kv_len[i];
            if (len < 1) {
                report(p.ctrl, SW_ERR_OUT_OF_RANGE, kSiteAppendLen, i);
                continue;
            }
            pos = (int64_t)len - 1;
            const int beg = p.decode_page_indptr[i];
            pages = p.decode_pages + beg;
            npages = p.decode_page_indptr[i + 1] - beg;
        }
        const int64_t pi = pos / kPageSize;
        const int slot = (int)(pos % kPageSize);
        if (pi >= npages) {
            report(p.ctrl, SW_ERR_OUT_OF_RANGE, kSiteAppendLen, row);
            continue;
        }
        const int64_t page = pages[pi];
        if (page < 0 || page >= p.num_pages) {
            report(p.ctrl, SW_ERR_OUT_OF_RANGE, kSiteAppendPage, row);
            continue;
        }
        const int e0 = piece * 8;          // element offset inside the row's [Hkv][D]
        const int kvh = e0 / head_dim;
        const int e = e0 % head_dim;
        const int64_t src = (int64_t)row * p.Hkv * head_dim + e0;
        const int64_t dst_k = ((((int64_t)page * 2 + 0) * p.Hkv + kvh) * kPageSize + slot) * head_dim + e;
        const int64_t dst_v = ((((int64_t)page * 2 + 1) * p.Hkv + kvh) * kPageSize + slot) * head_dim + e;
        *reinterpret_cast<uint4*>(p.pool + dst_k) = *reinterpret_cast<const uint4*>(p.k_new + src);
        *reinterpret_cast<uint4*>(p.pool + dst_v) = *reinterpret_cast<const uint4*>(p.v_new + src);
    }
}

__global__ void sw_kv_append_kernel(const AppendParams p) {
    // launched with programmatic stream serialization: it may start while the previous kernel (the attention of
    // the previous iteration, possibly still reading this pool) drains; nothing is touched before this wait
    grid_launch_dependents();
    grid_dependency_wait();
    append_rows<true>(p, p.D, (int64_t)blockIdx.x * blockDim.x + threadIdx.x, (int64_t)gridDim.x * blockDim.x);
}

cudaError_t launch_kv_append(const AppendParams& p, int num_sms, cudaStream_t stream) {
    const int64_t total = (int64_t)(p.C + p.n) * (p.Hkv * p.D / 8);
    if (total == 0) return cudaSuccess;
    const int threads = 256;
    int64_t blocks = (total + threads - 1) / threads;
    if (blocks > (int64_t)num_sms * 8) blocks = (int64_t)num_sms * 8;   // eight 256-thread blocks fill an SM
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, sw_kv_append_kernel, p);
}

// Fused launches (append and attention in one kernel): every CTA writes its share of the new K/V rows at the start of
// the kernel and then adds one to a counter.  A page that can hold one of those rows (the last page of a decode
// request; the chunk's own keys) is not fetched before the counter shows every CTA's share.  The grid is one CTA per
// SM, so all CTAs are resident and the wait is short; it is bounded all the same.  Whole-warp call; false when the
// wait ran out.
__device__ __forceinline__ bool wait_append(const MixedParams& p) {
    if (p.pool == nullptr) return true;
    int ok = 1;
    if ((threadIdx.x & 31) == 0) {
        const long long t0 = clock64();
        while (ld_acquire_gpu(&p.ctrl[kCtrAppend]) < (int)gridDim.x) {
            if (clock64() - t0 > kWaitBudgetCycles) {
                ok = 0;
                break;
            }
            __nanosleep(64);
        }
    }
    ok = __shfl_sync(0xffffffffu, ok, 0);
    fence_proxy_async_global();  // the rows were written with plain stores and are read through TMA
    return ok != 0;
}

// ---------------------------------------------------------------------------------------------------------------
// mixed attention: shared-memory plan
// ---------------------------------------------------------------------------------------------------------------
constexpr int kStages = 2;  // K/V page buffers in flight per warp

template <int D>
struct Geo {
    static constexpr int kHalves = D / 64;                    // 128-byte swizzled column blocks per row
    static constexpr int kBlockBytes = kPageSize * 128;       // one [16 tokens][64 elems] swizzled block
    static constexpr int kStageBytes = 2 * kHalves * kBlockBytes;  // K then V of one (page, kv head)
    static constexpr int kRingBytes = kWarps * kStages * kStageBytes;
    static constexpr int kBarOffset = kRingBytes;                              // kWarps*kStages mbarriers
    static constexpr int kPfBarOffset = kBarOffset + kWarps * kStages * 8;     // barriers of the prefill tiles
    static constexpr int kPlanOffset = kPfBarOffset + 32 * 8;                  // int32 unit_prefix[kMaxDecode+1]
    static constexpr int kLenOffset = kPlanOffset + (kMaxDecode + 1) * 4 + 12;  // int32 kv_len[kMaxDecode]
    static constexpr int kIndptrOffset = kLenOffset + kMaxDecode * 4;           // int32 page_indptr[kMaxDecode+1]
    static constexpr int kMiscOffset = kIndptrOffset + (kMaxDecode + 1) * 4 + 12; // scan scratch, TMEM base, abort flag
    static constexpr int kSmemBytes = kMiscOffset + 768;   // 64 ints scan scratch and flags, the plan's counters, the chunk table
};

constexpr int kWideMergeSplits = 24;  // from this many units of a request on, its last g units share the merge
constexpr int kOneRoundMaxPages = 48;  // longest unit (pages) for which one round of units is planned
constexpr int kPlanCounters = 8;       // shared counters of the plan's block sums, zeroed in the kernel prologue
// When the CTAs of a single wave of prefill entries turn to decode units: a fixed start-up plus the time of the longest
// entry's 128-key steps (MixedParams::step_us each, with the other CTAs streaming decode pages at the same time); the
// decode units stream one (page, kv head) stage per MixedParams::stage_us meanwhile.  Both figures come from the
// device's clocks (see sw_create).
constexpr float kLateBaseUs = 1.0f;
constexpr int kMinEarlyCtas = 64;  // CTAs whose rings of page copies keep the memory system busy on their own
constexpr int kMinLateCtas = 24;   // fewer late CTAs than this: their delay is not worth units of two sizes
struct Plan {
    const int* len;     // shared-memory copies of the context lengths and page-list offsets
    const int* indptr;
    bool two_sizes;     // large units handed out by index to the early CTAs, small ones pulled by the late CTAs only
    int decode_units;   // units of all requests
    int total_items;
};

// Block-wide exclusive scan of one value per thread (kThreads threads): a warp scan, one barrier, then every thread
// adds up the warps before its own.  scratch: kWarps ints nobody has touched since the last barrier; one use only.
__device__ __forceinline__ int block_exclusive_scan(int v, int* scratch, int* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) scratch[warp] = inc;
    __syncthreads();
    int before = 0, all = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        const int t = scratch[w];
        all += t;
        if (w < warp) before += t;
    }
    *total = all;
    return before + inc - v;
}

// Block-wide sum of one value per thread: a warp reduction, one shared-memory add per warp, one barrier.  ctr is a
// counter that was zero before the previous barrier; one use only.
__device__ __forceinline__ int block_sum(int v, int* ctr) {
    const int w = __reduce_add_sync(0xffffffffu, v);
    if ((threadIdx.x & 31) == 0 && w != 0) atomicAdd(ctr, w);
    __syncthreads();
    return *reinterpret_cast<volatile int*>(ctr);
}

// One-class unit size: pages per unit when `warps_per_head` warps share `total_pages`.  Small batches are
// latency-bound: one round of units, as many as there are warps, gets every warp streaming at once.  Large batches are
// bandwidth-bound: a few rounds of smaller units shorten the tail.  Every request adds at most one ragged unit per
// head, hence the "- n".
__device__ __forceinline__ int plan_split_pages(const MixedParams& p, int total_pages, int warps_per_head) {
    const int one_round = (total_pages + warps_per_head - 1) / warps_per_head;  // pages per unit if run in one round
    const int rounds = one_round <= kOneRoundMaxPages ? 1 : (one_round <= 160 ? 2 : 4);
    int units_target = max(1, rounds * warps_per_head - p.n);
    units_target = min(units_target, max(1, p.target_items / p.Hkv));
    return max((total_pages + units_target - 1) / units_target, kMinSplitTokens / kPageSize);
}

// CTAs that start with chunk-prefill work turn to decode units later than the others.
struct LateJoin {
    int ctas;   // how many CTAs (0 = none, gridDim.x = all: both plan like a decode-only launch)
    float us;   // estimated delay of their first decode unit relative to the other CTAs' first
};

// Every CTA derives the same plan from the context lengths: no host planning, no extra launch.
//
// When some CTAs join late the plan may have two unit sizes (plan.two_sizes).  The decode phase is bandwidth-bound, so
// by the time the late CTAs arrive the others have streamed about late.us * pages_per_us pages; what is left then is
// shared evenly among all warps.  The first requests are cut into large units (streamed share + even share), one for
// each warp of the early CTAs and handed out by index; the remaining requests are cut into small units (the even
// share), which only the warps of the late CTAs pull from the counter.  Both counts are made to fit the warps that
// run them, so that no warp starts a second unit.  If the early warps are nearly done by the time the late ones arrive,
// the plan is sized for the early warps alone; if the early CTAs are few, their head start is small or there are many
// requests per warp, it falls back to units of one size pulled by everybody.
__device__ __forceinline__ Plan make_plan(const MixedParams& p, int* unit_prefix, int* len_s, int* indptr_s, int* scratch,
                                          LateJoin late, float pages_per_us) {
    Plan plan;
    plan.len = len_s;
    plan.indptr = indptr_s;
    plan.two_sizes = false;
    const int per_thread = (p.n + kThreads - 1) / kThreads;
    const int beg = min(p.n, (int)threadIdx.x * per_thread);
    const int end = min(p.n, beg + per_thread);
    // total context in pages (fits an int: n <= 2048 requests of < 2^27 pages)
    int pages_local = 0;
    for (int i = beg; i < end; ++i) {
        const int len = p.decode_kv_len[i];
        pages_local += len > 0 ? (len + kPageSize - 1) / kPageSize : 0;
        len_s[i] = len;                              // the units read these from shared memory later
        indptr_s[i] = p.decode_page_indptr[i];
    }
    if (threadIdx.x == 0 && p.n > 0) indptr_s[p.n] = p.decode_page_indptr[p.n];
    int* ctr = scratch + 64;  // kPlanCounters counters zeroed in the kernel prologue, one per block sum
    const int total_pages = block_sum(pages_local, ctr++);

    const int G = (int)gridDim.x;
    constexpr int kMinPages = kMinSplitTokens / kPageSize;
    int split_a = 0, split_b = 0;  // pages per unit of the first requests / of the rest
    int a_pages = 0x7fffffff;      // requests whose pages start below this (per head) are cut with split_a
    if (late.ctas <= 0 || late.ctas >= G) {
        split_a = split_b = plan_split_pages(p, total_pages, max(1, G * kWarps / p.Hkv));
    } else {
        const float early = (float)((G - late.ctas) * kWarps), all = (float)(G * kWarps);
        const float pages = (float)total_pages * p.Hkv;
        const float streamed = fminf(pages, pages_per_us * late.us);
        const float even = (pages - streamed) / all;
        // units and pages (per head) of the early warps and of the late ones; a request adds about half a ragged unit
        const float a_units = early / p.Hkv, b_units = (all - early) / p.Hkv;
        const float a_share = fminf((float)total_pages, a_units * (streamed / early + even));
        const float b_share = (float)total_pages - a_share;
        const float a_ragged = 0.6f * p.n * a_share / fmaxf(1.f, (float)total_pages);
        const float b_ragged = 0.6f * p.n - a_ragged;
        if (G - late.ctas < kMinEarlyCtas || late.ctas < kMinLateCtas || streamed < 0.25f * pages) {
            // Too few early CTAs to keep the memory system busy on their own (the estimate of what they stream would
            // not hold), or a head start that is small next to the whole phase: one unit size, every warp pulls.
            split_a = split_b = plan_split_pages(p, total_pages, max(1, G * kWarps / p.Hkv));
        } else if (pages - streamed < (float)(late.ctas * kWarps * kMinPages)) {
            split_a = split_b = plan_split_pages(p, total_pages, max(1, (G - late.ctas) * kWarps / p.Hkv));
        } else if (a_ragged > 0.25f * a_units || b_ragged > 0.25f * b_units) {
            // too many requests per warp for one even unit each: units pulled by every warp balance better
            split_a = split_b = plan_split_pages(p, total_pages, max(1, G * kWarps / p.Hkv));
        } else {
            split_a = max(kMinPages, (int)ceilf(a_share / (a_units - a_ragged)));
            split_b = max(kMinPages, (int)ceilf(b_share / (b_units - b_ragged)));
            a_pages = (int)a_share;
            plan.two_sizes = true;
        }
    }
    int pages_before = 0;
    if (plan.two_sizes) {
        int unused;
        pages_before = block_exclusive_scan(pages_local, scratch + 16, &unused);
        // count the units of either size and grow the size until they fit their warps (the estimates are rarely off)
        const int a_units = (G - late.ctas) * kWarps / p.Hkv, b_units = late.ctas * kWarps / p.Hkv;
        for (int pass = 0; pass < (kPlanCounters - 1) / 2; ++pass) {
            int cnt_a = 0, cnt_b = 0, before = pages_before;
            for (int i = beg; i < end; ++i) {
                const int pg = len_s[i] > 0 ? (len_s[i] + kPageSize - 1) / kPageSize : 0;
                if (before < a_pages) cnt_a += (pg + split_a - 1) / split_a; else cnt_b += (pg + split_b - 1) / split_b;
                before += pg;
            }
            const int total_a = block_sum(cnt_a, ctr++);
            const int total_b = block_sum(cnt_b, ctr++);
            if (total_a <= a_units && total_b <= b_units) break;
            if (total_a > a_units) split_a = (int)(((int64_t)split_a * total_a + a_units - 1) / a_units) + 1;
            if (total_b > b_units) split_b = (int)(((int64_t)split_b * total_b + b_units - 1) / b_units) + 1;
        }
    }
    int units_local = 0;
    for (int i = beg; i < end; ++i) {
        const int len = len_s[i];
        const int pg = len > 0 ? (len + kPageSize - 1) / kPageSize : 0;
        const int split = pages_before < a_pages ? split_a : split_b;
        units_local += (pg + split - 1) / split;
        pages_before += pg;
    }
    pages_before -= pages_local;
    int total_units = 0;
    int run = block_exclusive_scan(units_local, scratch, &total_units);
    for (int i = beg; i < end; ++i) {
        unit_prefix[i] = run;
        const int len = len_s[i];
        const int pg = len > 0 ? (len + kPageSize - 1) / kPageSize : 0;
        const int split = pages_before < a_pages ? split_a : split_b;
        run += (pg + split - 1) / split;
        pages_before += pg;
    }
    if (threadIdx.x == 0) unit_prefix[p.n] = total_units;
    __syncthreads();
    plan.decode_units = total_units;
    plan.total_items = total_units * p.Hkv;
    return plan;
}

// ---------------------------------------------------------------------------------------------------------------
// one split-KV unit on one warp
// ---------------------------------------------------------------------------------------------------------------
struct Unit {
    int q_row;          // row of q / out
    int kvh;            // KV head
    int len;            // keys attended by this row in total
    int t_begin, t_end; // this unit's key range
    int nsplit;         // units of this (row, kv head); 1 = write the result directly
    int split;          // index among them
    int ticket;         // ticket slot (decode request * Hkv + kvh)
    int slot;           // partial-result slot
    const int32_t* pages;
};

template <int D>
struct WarpRing {
    uint32_t buf;   // shared address of this warp's first stage
    uint32_t bar;   // shared address of this warp's first mbarrier
    uint32_t it;    // pages consumed so far (stage = it % kStages, parity = (it / kStages) & 1)
};

// Lane 0 arms the stage's barrier and fetches the page with one copy: the head's K blocks, then its V blocks.
template <int D>
__device__ __forceinline__ void issue_page(const CUtensorMap* kvp_map, const WarpRing<D>& ring, uint32_t issue_it, int page,
                                           int kvh) {
    if ((threadIdx.x & 31) == 0) {
        const uint32_t stage = issue_it % kStages;
        const uint32_t bar = ring.bar + stage * 8;
        mbar_arrive_expect_tx(bar, Geo<D>::kStageBytes);
        // a decode page is read once: evict-first keeps it from pushing the chunk's K/V tiles out of L2
        tma_load_5d_hint(ring.buf + stage * Geo<D>::kStageBytes, kvp_map, bar, 0, 0, 0, 2 * page, kvh, l2_policy_evict_first());
    }
}

// Merge of the splits of one (request, kv head) by the last unit to arrive, all rows together so that the loads of
// one pass are in flight at once.  G >= group size is a compile-time bound: rows beyond the group read row 0 with
// weight zero, which keeps the loops free of branches.  Slots of the splits are Hkv apart.
// The warp merges rows [row0, row0 + nrows) of the group (all of them, or one row when several units share the merge);
// J = splits whose partial outputs are loaded together.
template <int D, int G, int J = (G >= 8 ? 2 : (G == 4 ? 4 : 8))>
__device__ __forceinline__ void merge_splits(const MixedParams& p, const Unit& u, int row0, int nrows) {
    constexpr int V = D / 32;                 // output columns per lane
    const int lane = threadIdx.x & 31;
    const int g = p.group;
    const int slot0 = u.slot - u.split * p.Hkv;
    const int ns = u.nsplit;
    const float* ml0 = p.part_ml + (int64_t)slot0 * (2 * kMaxGroup);  // split s: + s * ml_stride
    const int64_t ml_stride = (int64_t)p.Hkv * (2 * kMaxGroup);
    // pass 1: lanes take splits; per row the running maximum and the row sum rescaled to it, then one warp reduction
    float m_all[G], l_all[G], m_first[G];
#pragma unroll
    for (int r = 0; r < G; ++r) {
        m_all[r] = -INFINITY;
        l_all[r] = 0.f;
        m_first[r] = -INFINITY;
    }
    for (int s0 = 0; s0 < ns; s0 += 32) {
        const int sidx = min(s0 + lane, ns - 1);
        const bool live = s0 + lane < ns;
        float ms[G], ls[G];
#pragma unroll
        for (int r = 0; r < G; ++r) {
            const int rr = row0 + (r < nrows ? r : 0);
            ms[r] = __ldcg(ml0 + sidx * ml_stride + rr);
            ls[r] = __ldcg(ml0 + sidx * ml_stride + kMaxGroup + rr);
        }
#pragma unroll
        for (int r = 0; r < G; ++r) {
            if (!live) ms[r] = -INFINITY;
            if (s0 == 0) m_first[r] = ms[r];
            const float m_new = fmaxf(m_all[r], ms[r]);
            const float a = m_all[r] == -INFINITY ? 0.f : fast_exp2((m_all[r] - m_new) * p.sm_scale_log2);
            const float b = ms[r] == -INFINITY ? 0.f : fast_exp2((ms[r] - m_new) * p.sm_scale_log2);
            l_all[r] = l_all[r] * a + ls[r] * b;
            m_all[r] = m_new;
        }
    }
#pragma unroll
    for (int r = 0; r < G; ++r) {
        float mw = m_all[r];
#pragma unroll
        for (int o2 = 16; o2 > 0; o2 >>= 1) mw = fmaxf(mw, __shfl_xor_sync(0xffffffffu, mw, o2));
        float lw = m_all[r] == -INFINITY ? 0.f : l_all[r] * fast_exp2((m_all[r] - mw) * p.sm_scale_log2);
#pragma unroll
        for (int o2 = 16; o2 > 0; o2 >>= 1) lw += __shfl_xor_sync(0xffffffffu, lw, o2);
        m_all[r] = mw;
        l_all[r] = lw;
    }
    // pass 2: weighted sum of the partial outputs; lanes take V adjacent columns of every row, J splits per batch
    float acc[G][V];
#pragma unroll
    for (int r = 0; r < G; ++r)
#pragma unroll
        for (int v = 0; v < V; ++v) acc[r][v] = 0.f;
    const float* po0 = p.part_o + (int64_t)slot0 * g * D + lane * V;  // split s, row r: + s * po_stride + r * D
    const int64_t po_stride = (int64_t)p.Hkv * g * D;
    for (int s0 = 0; s0 < ns; s0 += 32) {
        float w[G];
#pragma unroll
        for (int r = 0; r < G; ++r) {
            float ms = m_first[r];
            if (s0 > 0) {
                ms = __ldcg(ml0 + min(s0 + lane, ns - 1) * ml_stride + row0 + (r < nrows ? r : 0));
                if (s0 + lane >= ns) ms = -INFINITY;
            }
            w[r] = (ms == -INFINITY || r >= nrows) ? 0.f : fast_exp2((ms - m_all[r]) * p.sm_scale_log2);
        }
        const int cnt = min(32, ns - s0);
        for (int j0 = 0; j0 < cnt; j0 += J) {
            float x[J][G][V];
#pragma unroll
            for (int j = 0; j < J; ++j) {
                const float* src = po0 + (s0 + min(j0 + j, cnt - 1)) * po_stride;
#pragma unroll
                for (int r = 0; r < G; ++r) {
                    const float* row = src + (row0 + (r < nrows ? r : 0)) * D;
                    if constexpr (V == 4) {
                        const float4 t = __ldcg(reinterpret_cast<const float4*>(row));
                        x[j][r][0] = t.x, x[j][r][1] = t.y, x[j][r][2] = t.z, x[j][r][3] = t.w;
                    } else {
                        const float2 t = __ldcg(reinterpret_cast<const float2*>(row));
                        x[j][r][0] = t.x, x[j][r][1] = t.y;
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < J; ++j) {
#pragma unroll
                for (int r = 0; r < G; ++r) {
                    float wj = __shfl_sync(0xffffffffu, w[r], (j0 + j) & 31);
                    if (j0 + j >= cnt) wj = 0.f;
#pragma unroll
                    for (int v = 0; v < V; ++v) acc[r][v] = fmaf(wj, x[j][r][v], acc[r][v]);
                }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < G; ++r) {
        if (r < nrows) {
            const float inv = 1.f / l_all[r];
            const int hd = u.kvh * g + row0 + r;
            __nv_bfloat16* dst = p.out + ((int64_t)u.q_row * p.Hq + hd) * D + lane * V;
            if constexpr (V == 4) {
                *reinterpret_cast<uint2*>(dst) = make_uint2(pack_bf16x2(acc[r][0] * inv, acc[r][1] * inv),
                                                            pack_bf16x2(acc[r][2] * inv, acc[r][3] * inv));
            } else {
                *reinterpret_cast<uint32_t*>(dst) = pack_bf16x2(acc[r][0] * inv, acc[r][1] * inv);
            }
            if (p.lse && lane == 0) p.lse[(int64_t)u.q_row * p.Hq + hd] = m_all[r] * p.sm_scale + __logf(l_all[r]);
        }
    }
}

// Which row of the group a unit of a request with many units merges (-1: none).  Not inlined: the rare case should
// not cost the common one registers or instructions.
__device__ __noinline__ int wide_merge_row(int nsplit, int split, int kvh, int g, int Hkv) {
    const int d = nsplit - 1 - split;
    if (nsplit >= 2 * g * Hkv) {
        const int q = d >> 1;
        return (!(d & 1) && q % Hkv == kvh && q / Hkv < g) ? q / Hkv : -1;
    }
    return d < g ? d : -1;
}

// Runs one unit; returns false if a bounded wait expired.
template <int D>
__device__ bool run_unit(const CUtensorMap* kvp_map, const MixedParams& p, const Unit& u, WarpRing<D>& ring, int fixed_items, bool pulls,
                         int& next_item) {
    constexpr int KS = D / 16;  // k-slices of QK^T; also pairs of 8-wide output column tiles of PV
    const int lane = threadIdx.x & 31;
    const int qrow_in_group = lane >> 2;  // accumulator row held in c0/c1
    const int g = p.group;

    // A fragments of Q: rows 0..g-1 are the query heads sharing this KV head, rows >= g are zero
    uint32_t qa[KS][2];
    {
        const __nv_bfloat16* qbase = p.q + ((int64_t)u.q_row * p.Hq + (int64_t)u.kvh * g) * D;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            uint32_t v0 = 0, v1 = 0;
            if (qrow_in_group < g) {
                const uint32_t* src = reinterpret_cast<const uint32_t*>(qbase + qrow_in_group * D + ks * 16 + (lane & 3) * 2);
                v0 = src[0];
                v1 = src[4];  // +8 elements
            }
            qa[ks][0] = v0;
            qa[ks][1] = v1;
        }
    }

    float o[2 * KS][2];
#pragma unroll
    for (int i = 0; i < 2 * KS; ++i) o[i][0] = o[i][1] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;

    const int pg0 = u.t_begin / kPageSize;
    const int pg1 = (u.t_end + kPageSize - 1) / kPageSize;
    const int npg = pg1 - pg0;

    // per-lane shared-memory offsets of the ldmatrix rows (128-byte swizzle: 16-byte chunk ^= row % 8)
    const int k_tok = ((lane >> 4) << 3) + (lane & 7);
    const int k_sel = (lane >> 3) & 1;
    const int v_tok = (((lane >> 3) & 1) << 3) + (lane & 7);
    const int v_sel = lane >> 4;
    const int swz = lane & 7;

    int ids = 0;
    int issued = 0;
    bool append_timeout = false;
    const uint32_t it0 = ring.it;  // ring position of this unit's first page
    auto issue_next = [&]() {
        if ((issued & 31) == 0) {
            const int pi = pg0 + issued + lane;
            ids = pi < pg1 ? u.pages[pi] : 0;
        }
        int page = __shfl_sync(0xffffffffu, ids, issued & 31);
        if (page < 0 || (int64_t)page >= p.num_pages) {
            // a bad id never reaches the copy engine: the problem is reported and page 0 is fetched in its place, so
            // the barrier still receives the bytes it expects
            if (lane == 0) report(p.ctrl, SW_ERR_OUT_OF_RANGE, kSiteAttnPage, u.q_row);
            page = 0;
        }
        // the request's last page holds the row this iteration appends
        if (p.pool != nullptr && (pg0 + issued + 1) * kPageSize >= u.len && !wait_append(p)) {
            if (lane == 0) report(p.ctrl, SW_ERR_DEVICE_TIMEOUT, kSiteWait, u.q_row);
            append_timeout = true;
        }
        issue_page<D>(kvp_map, ring, it0 + issued, page, u.kvh);
        ++issued;
    };
    for (int k = 0; k < kStages && k < npg; ++k) issue_next();
    // Once this unit's last page is on its way the following unit is claimed from the shared counter: the counter's
    // round trip hides behind the last pages, and no warp hoards a unit while others are still idle.
    // With the claim the unit draws its ticket among the units of its (request, kv head): the last ticket makes it
    // the one that merges.  Both answers are read at the end of the unit, when they have long arrived.
    // A request cut into many units (kWideMergeSplits or more) has g mergers per kv head, fixed in advance among its
    // last units, one query-head row each.  Such a unit will wait for the request's other units, so it must not hold
    // a claimed unit meanwhile (another merger could be waiting for that one): it claims its next unit after the merge.
    // With enough units the mergers of the different heads and rows are every other unit from the end (row j of head
    // h: unit nsplit - 1 - 2 (j Hkv + h)), which puts them on different SMs; otherwise the last g units of each head.
    const bool wide = g > 1 && u.nsplit >= kWideMergeSplits;
    const int merge_row = wide ? wide_merge_row(u.nsplit, u.split, u.kvh, g, p.Hkv) : -1;
    bool claimed = merge_row >= 0;
    int ticket = 0;  // lane 0
    auto claim_next = [&]() {
        if (!claimed && issued >= npg) {
            claimed = true;
            if (lane == 0) {
                next_item = pulls ? fixed_items + atomicAdd(&p.ctrl[kCtrWork], 1) : 0x7fffffff;
                if (u.nsplit > 1 && !wide) ticket = atomicAdd(&p.tickets[u.ticket], 1);
            }
        }
    };
    claim_next();

    for (int k = 0; k < npg; ++k) {
        if (append_timeout) return false;
        const uint32_t stage = ring.it % kStages;
        const uint32_t parity = (ring.it / kStages) & 1;
        const uint32_t sK = ring.buf + stage * Geo<D>::kStageBytes;
        const uint32_t sV = sK + Geo<D>::kHalves * Geo<D>::kBlockBytes;
        if (!mbar_wait(ring.bar + stage * 8, parity)) {
            report(p.ctrl, SW_ERR_DEVICE_TIMEOUT, kSiteWait, u.q_row);
            return false;
        }
        const int t0 = (pg0 + k) * kPageSize;

        // S = Q K^T for 16 keys
        float s[2][4];
#pragma unroll
        for (int i = 0; i < 2; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            const int chunk = 2 * ks + k_sel;
            const uint32_t addr = sK + (chunk >> 3) * Geo<D>::kBlockBytes + k_tok * 128 + (((chunk & 7) ^ swz) << 4);
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4(addr, b0, b1, b2, b3);
            mma_bf16_16816(s[0], qa[ks][0], 0u, qa[ks][1], 0u, b0, b1);
            mma_bf16_16816(s[1], qa[ks][0], 0u, qa[ks][1], 0u, b2, b3);
        }
        // mask keys outside [t_begin, t_end)
        const int valid_hi = u.t_end - t0;   // keys with index >= valid_hi are masked
        const int valid_lo = u.t_begin - t0; // keys with index <  valid_lo are masked (always <= 0 here)
        float mx = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int key = nt * 8 + (lane & 3) * 2 + j;
                const float v = (key < valid_hi && key >= valid_lo) ? s[nt][j] : -INFINITY;
                s[nt][j] = v;
                mx = fmaxf(mx, v);
            }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_run, mx);
        const float corr = fast_exp2((m_run - m_new) * p.sm_scale_log2);
        const float mb = m_new * p.sm_scale_log2;
        float pr[2][2];
        float psum = 0.f;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                pr[nt][j] = fast_exp2(fmaf(s[nt][j], p.sm_scale_log2, -mb));
                psum += pr[nt][j];
            }
        l_run = l_run * corr + psum;
        m_run = m_new;
#pragma unroll
        for (int i = 0; i < 2 * KS; ++i) {
            o[i][0] *= corr;
            o[i][1] *= corr;
        }
        const uint32_t pa0 = pack_bf16x2(pr[0][0], pr[0][1]);
        const uint32_t pa2 = pack_bf16x2(pr[1][0], pr[1][1]);

        // the unwritten slots of a partly filled last page hold whatever the pool held: zero those V rows so that
        // 0 * garbage cannot produce NaN
        if (valid_hi < kPageSize) {
            __syncwarp();
            const int dead_rows = kPageSize - valid_hi;
            for (int c = lane; c < dead_rows * (D / 8); c += 32) {
                const int row = valid_hi + c / (D / 8);
                const int chunk = c % (D / 8);
                const uint32_t addr = sV + (chunk >> 3) * Geo<D>::kBlockBytes + row * 128 + (((chunk & 7) ^ (row & 7)) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0u) : "memory");
            }
            __syncwarp();
        }

        // O += P V
#pragma unroll
        for (int dn = 0; dn < KS; ++dn) {
            const int chunk = 2 * dn + v_sel;
            const uint32_t addr = sV + (chunk >> 3) * Geo<D>::kBlockBytes + v_tok * 128 + (((chunk & 7) ^ swz) << 4);
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4_trans(addr, b0, b1, b2, b3);
            float acc0[4] = {o[2 * dn][0], o[2 * dn][1], 0.f, 0.f};
            float acc1[4] = {o[2 * dn + 1][0], o[2 * dn + 1][1], 0.f, 0.f};
            mma_bf16_16816(acc0, pa0, 0u, pa2, 0u, b0, b1);
            mma_bf16_16816(acc1, pa0, 0u, pa2, 0u, b2, b3);
            o[2 * dn][0] = acc0[0];
            o[2 * dn][1] = acc0[1];
            o[2 * dn + 1][0] = acc1[0];
            o[2 * dn + 1][1] = acc1[1];
        }
        ring.it += 1;
        __syncwarp();  // every lane is done reading this stage before it is refilled
        if (valid_hi < kPageSize) fence_proxy_async_smem();
        if (issued < npg) issue_next();
        claim_next();
    }

    // finish: row sums across the quad
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    const bool row_ok = qrow_in_group < g;
    const int head = u.kvh * g + qrow_in_group;
    if (u.nsplit == 1) {
        if (row_ok) {
            const float inv = 1.f / l_run;
            __nv_bfloat16* dst = p.out + ((int64_t)u.q_row * p.Hq + head) * D + (lane & 3) * 2;
#pragma unroll
            for (int i = 0; i < 2 * KS; ++i)
                *reinterpret_cast<uint32_t*>(dst + i * 8) = pack_bf16x2(o[i][0] * inv, o[i][1] * inv);
            if (p.lse && (lane & 3) == 0) p.lse[(int64_t)u.q_row * p.Hq + head] = m_run * p.sm_scale + __logf(l_run);
        }
        return true;
    }

    // Partial result -> scratch.  The units that did not draw the last ticket publish it (fence, then one more on the
    // `ready` counter, without waiting for anything); the one that did waits until the others have and merges.  It is
    // usually the last to finish, so its wait is short, and no fence or ticket round trip sits between its last page
    // and the merge.
    if (row_ok) {
        float* po = p.part_o + ((int64_t)u.slot * g + qrow_in_group) * D + (lane & 3) * 2;
#pragma unroll
        for (int i = 0; i < 2 * KS; ++i) *reinterpret_cast<float2*>(po + i * 8) = make_float2(o[i][0], o[i][1]);
        if ((lane & 3) == 0) {
            p.part_ml[(int64_t)u.slot * (2 * kMaxGroup) + qrow_in_group] = m_run;
            p.part_ml[(int64_t)u.slot * (2 * kMaxGroup) + kMaxGroup + qrow_in_group] = l_run;
        }
    }
    if (wide) {
        // Many splits (one long context cut for all the warps): a single warp would load their partial outputs a few
        // at a time.  Every unit publishes its partial result; g of the request's last units then merge one row of
        // the group each.  A waiting merger holds no claimed unit, and the units it waits for are run by warps that wait
        // for nothing or are claimed by such warps: a request has 24 units or more only if it holds 23 units' worth
        // of pages, so at most target_items / 23 (request, kv head) pairs have mergers, fewer than 1500 warps even
        // with groups of 8, and some warp is always free to claim.  The last merger to finish re-arms the counter.
        __threadfence();
        __syncwarp();
        if (lane == 0) atomicAdd(&p.ready[u.ticket], 1);
        if (merge_row < 0) return true;
        int ok = 1;
        if (lane == 0) {
            const long long t0 = clock64();
            while (ld_acquire_gpu(&p.ready[u.ticket]) < u.nsplit) {
                if (clock64() - t0 > kWaitBudgetCycles) {
                    ok = 0;
                    break;
                }
                __nanosleep(64);
            }
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) {
            if (lane == 0) report(p.ctrl, SW_ERR_DEVICE_TIMEOUT, kSiteWait, u.q_row);
            return false;
        }
        merge_splits<D, 1, 16>(p, u, merge_row, 1);
        if (lane == 0) {
            if (atomicAdd(&p.ready[u.ticket], 1) == u.nsplit + g - 1) p.ready[u.ticket] = 0;  // ready for the next launch
            next_item = pulls ? fixed_items + atomicAdd(&p.ctrl[kCtrWork], 1) : 0x7fffffff;
        }
        return true;
    }
    ticket = __shfl_sync(0xffffffffu, ticket, 0);
    const bool merger = ticket == u.nsplit - 1;
    if (!merger) {
        __threadfence();
        __syncwarp();
        if (lane == 0) atomicAdd(&p.ready[u.ticket], 1);
        return true;
    }
    // last ticket: merge all splits of this (request, kv head) once the others are published
    __syncwarp();  // this warp's own partial result, written above by all lanes, is ordered before the loads below
    int ok = 1;
    if (lane == 0) {
        const long long t0 = clock64();
        while (ld_acquire_gpu(&p.ready[u.ticket]) < u.nsplit - 1) {
            if (clock64() - t0 > kWaitBudgetCycles) {
                ok = 0;
                break;
            }
            __nanosleep(64);
        }
        p.tickets[u.ticket] = 0;  // ready for the next launch
        p.ready[u.ticket] = 0;
    }
    ok = __shfl_sync(0xffffffffu, ok, 0);
    if (!ok) {
        if (lane == 0) report(p.ctrl, SW_ERR_DEVICE_TIMEOUT, kSiteWait, u.q_row);
        return false;
    }
    switch (g) {
        case 1: merge_splits<D, 1>(p, u, 0, 1); break;
        case 2: merge_splits<D, 2>(p, u, 0, 2); break;
        case 4: merge_splits<D, 4>(p, u, 0, 4); break;
        default: merge_splits<D, kMaxGroup>(p, u, 0, g); break;
    }
    return true;
}

}  // namespace sw
#include "sw_prefill.cuh"
namespace sw {

// ---------------------------------------------------------------------------------------------------------------
// the persistent kernel
// ---------------------------------------------------------------------------------------------------------------
template <int D, bool kMulti>
__global__ void __launch_bounds__(kThreads, 1) sw_mixed_attn_kernel(const __grid_constant__ CUtensorMap kv_map,
                                                                       const __grid_constant__ CUtensorMap kvp_map,
                                                                    const __grid_constant__ CUtensorMap q_map,
                                                                    const __grid_constant__ CUtensorMap out_map,
                                                                    const MixedParams p) {
    static_assert(PfGeo<D>::kBytes <= Geo<D>::kRingBytes, "prefill tiles must fit the region shared with the decode ring");
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    int* unit_prefix = reinterpret_cast<int*>(smem + Geo<D>::kPlanOffset);
    int* scratch = reinterpret_cast<int*>(smem + Geo<D>::kMiscOffset);

    const bool tensor_prefill = p.C > 0;
    volatile int* misc = reinterpret_cast<volatile int*>(scratch + 32);  // [0] TMEM base, [1] abort flag, [2..3] ticket flags
    if (threadIdx.x >= 32 && threadIdx.x < 32 + kPlanCounters) scratch[64 + threadIdx.x - 32] = 0;  // block-sum counters
    // the chunks' descriptors go to shared memory: the roles of the chunk-prefill phase look them up by the item's chunk
    // number instead of carrying them in registers
    if (kMulti && warp == 2) pf_fill_chunk_table(p, scratch + kChunkTable);
    if (threadIdx.x == 0) {
        tma_prefetch_desc(&kv_map);
        tma_prefetch_desc(&kvp_map);
        for (int i = 0; i < kWarps * kStages; ++i) mbar_init(base + Geo<D>::kBarOffset + i * 8, 1);
        if (tensor_prefill) {
            tma_prefetch_desc(&q_map);
            tma_prefetch_desc(&out_map);
            pf_init_barriers(base + Geo<D>::kPfBarOffset);
        }
        misc[0] = 0;
        misc[1] = 0;
        fence_mbar_init();
    }
    // Everything above touched only shared memory and kernel parameters.  From here on the kernel reads what earlier
    // kernels of the stream wrote (the pool after the KV append, q, the page tables): wait for them to finish.
    grid_dependency_wait();
    grid_launch_dependents();
    if (p.pool != nullptr) {
        // fused launch: this CTA's share of the new K/V rows, then its mark on the counter the readers wait for
        append_rows<kMulti>(p, D, (int64_t)blockIdx.x * kThreads + threadIdx.x, (int64_t)gridDim.x * kThreads);
        fence_proxy_async_global();
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) atomicAdd(&p.ctrl[kCtrAppend], 1);
    }
    __syncthreads();

    // chunk-prefill tiles first (long, tensor-bound); the decode units below fill the tail
    // The first prefill entry of a CTA is its own index and the first decode unit of a warp is fixed as well: neither
    // waits for a counter.  CTAs that start with prefill work take all their decode units from the counter.
    int prefill_ctas = 0;
    LateJoin late{0, 0.f};
    if (tensor_prefill) {
        const PfPlan pplan = pf_make_plan<kMulti>(p, base + Geo<D>::kMiscOffset + kChunkTable * 4);
        prefill_ctas = min(pplan.n_entries, pplan.ctas);
        late.ctas = prefill_ctas;
        late.us = kLateBaseUs + p.step_us * ((pplan.longest + pplan.pieces - 1) / pplan.pieces);
        if (pplan.n_items >= pplan.ctas)  // whole rounds: the prefill CTAs share all items' steps
            late.us = kLateBaseUs + p.step_us * (0.5f * (float)(pplan.longest + pplan.shortest) * (float)pplan.n_items / (float)pplan.ctas);
        const int first_entry = blockIdx.x;
        if (first_entry < prefill_ctas) {  // CTA-uniform: this CTA has prefill work
            if (warp == 1) {
                tmem_alloc(smem_u32(const_cast<int*>(&misc[0])), 512);
                tmem_relinquish();
            }
            tc_fence_before_sync();
            __syncthreads();
            tc_fence_after_sync();
            PfShared sh;
            sh.smem = base;
            sh.bars = base + Geo<D>::kPfBarOffset;
            sh.tmem = (uint32_t)misc[0];
            sh.abort_flag = &misc[1];
            PfScratch scr;
            scr.ml = p.pf_ml;
            scr.o = p.pf_o;
            scr.tickets = p.pf_tickets;
            scr.flags = &misc[2];
            prefill_phase<D, kMulti>(&kv_map, &q_map, &out_map, p, sh, pplan, scr, first_entry, &misc[5]);
            tc_fence_before_sync();
            __syncthreads();
            if (warp == 1) tmem_dealloc(sh.tmem, 512);
        }
        __syncthreads();
    }

    const Plan plan = make_plan(p, unit_prefix, reinterpret_cast<int*>(smem + Geo<D>::kLenOffset),
                                reinterpret_cast<int*>(smem + Geo<D>::kIndptrOffset), scratch, late,
                                p.stages_per_us);
    if (plan.total_items > p.max_items) {
        if (threadIdx.x == 0) report(p.ctrl, SW_ERR_WORKSPACE, kSiteScratch, plan.total_items);
    } else {
        WarpRing<D> ring;
        ring.buf = base + warp * kStages * Geo<D>::kStageBytes;
        ring.bar = base + Geo<D>::kBarOffset + warp * kStages * 8;
        ring.it = 0;
        const int fixed_items = ((int)gridDim.x - prefill_ctas) * kWarps;  // units handed out without the counter
        // with two unit sizes the early CTAs run their one large unit each and leave the counter to the late CTAs
        const bool pulls = !plan.two_sizes || (int)blockIdx.x < prefill_ctas;
        int item = ((int)blockIdx.x - prefill_ctas) * kWarps + warp;
        if ((int)blockIdx.x < prefill_ctas) {
            if (lane == 0) item = fixed_items + atomicAdd(&p.ctrl[kCtrWork], 1);
            item = __shfl_sync(0xffffffffu, item, 0);
        }
        while (item < plan.total_items) {
            int next_item = 0;  // lane 0: claimed inside run_unit
            Unit u;
            bool ok = true;
            {
                const int di = item;
                const int unit = di / p.Hkv;
                u.kvh = di % p.Hkv;
                int lo = 0, hi = p.n;  // largest i with unit_prefix[i] <= unit
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (unit_prefix[mid] <= unit) lo = mid; else hi = mid;
                }
                const int i = lo;
                u.q_row = p.C + i;
                u.len = plan.len[i];
                u.split = unit - unit_prefix[i];
                u.nsplit = unit_prefix[i + 1] - unit_prefix[i];
                // the request's pages are shared out evenly among its units (no ragged last unit)
                const int req_pages = (u.len + kPageSize - 1) / kPageSize;
                const int unit_pages = (req_pages + u.nsplit - 1) / u.nsplit;
                u.t_begin = min(u.len, u.split * unit_pages * kPageSize);
                u.t_end = min(u.len, u.t_begin + unit_pages * kPageSize);
                u.ticket = i * p.Hkv + u.kvh;
                u.slot = di;
                const int beg = plan.indptr[i];
                u.pages = p.decode_pages + beg;
                ok = (u.len + kPageSize - 1) / kPageSize <= plan.indptr[i + 1] - beg;
            }
            if (!ok) {
                if (lane == 0) {
                    report(p.ctrl, SW_ERR_OUT_OF_RANGE, kSiteAttnLen, u.q_row);
                    next_item = pulls ? fixed_items + atomicAdd(&p.ctrl[kCtrWork], 1) : 0x7fffffff;
                }
            } else if (!run_unit<D>(&kvp_map, p, u, ring, fixed_items, pulls, next_item)) {
                break;
            }
            item = __shfl_sync(0xffffffffu, next_item, 0);
        }
    }

    // the last CTA to finish re-arms the work counter for the next launch
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const int done = atomicAdd(&p.ctrl[kCtrDone], 1);
        if (done == (int)gridDim.x - 1) {
            p.ctrl[kCtrWork] = 0;
            p.ctrl[kCtrPrefill] = 0;
            p.ctrl[kCtrAppend] = 0;
            p.ctrl[kCtrDone] = 0;
            __threadfence();
        }
    }
}

// Self-test of the bounded wait: one warp waits on a barrier that nothing will ever complete; the wait must give up
// after `budget_cycles`, record SW_ERR_DEVICE_TIMEOUT in the status word and let the kernel end normally.
__global__ void sw_selftest_wait_kernel(int32_t* ctrl, long long budget_cycles) {
    __shared__ __align__(8) unsigned long long bar;
    const uint32_t addr = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(addr, 1);
        fence_mbar_init();
    }
    __syncwarp();
    if (!mbar_wait(addr, 0, budget_cycles) && threadIdx.x == 0) report(ctrl, SW_ERR_DEVICE_TIMEOUT, kSiteWait, 0xABCD);
}

cudaError_t launch_selftest_wait(int32_t* ctrl, long long budget_cycles, cudaStream_t stream) {
    sw_selftest_wait_kernel<<<1, 32, 0, stream>>>(ctrl, budget_cycles);
    return cudaGetLastError();
}

size_t mixed_attn_smem_bytes(int head_dim) {
    return (head_dim == 64 ? Geo<64>::kSmemBytes : Geo<128>::kSmemBytes) + 1024;
}

// The kernel exists in two forms per head size: for iterations with at most one prefill chunk, whose descriptors are
// then plain kernel parameters, and for iterations with several (descriptors looked up per work item).
cudaError_t configure_kernels(int head_dim) {
    const int bytes = (int)mixed_attn_smem_bytes(head_dim);
    cudaError_t e;
    if (head_dim == 64) {
        e = cudaFuncSetAttribute(sw_mixed_attn_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e != cudaSuccess) return e;
        return cudaFuncSetAttribute(sw_mixed_attn_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    }
    e = cudaFuncSetAttribute(sw_mixed_attn_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(sw_mixed_attn_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

// CTAs of the persistent kernel that one SM can hold at a time (the smaller figure of the two forms).  The fused launch
// makes CTAs wait for one another's share of the KV append, which is only safe when the whole grid is resident.
cudaError_t mixed_attn_resident_ctas_per_sm(int head_dim, int* out) {
    const size_t bytes = mixed_attn_smem_bytes(head_dim);
    int a = 0, b = 0;
    cudaError_t e;
    if (head_dim == 64) {
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, sw_mixed_attn_kernel<64, false>, kThreads, bytes);
        if (e != cudaSuccess) return e;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, sw_mixed_attn_kernel<64, true>, kThreads, bytes);
    } else {
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, sw_mixed_attn_kernel<128, false>, kThreads, bytes);
        if (e != cudaSuccess) return e;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, sw_mixed_attn_kernel<128, true>, kThreads, bytes);
    }
    *out = a < b ? a : b;
    return e;
}

cudaError_t launch_mixed_attn(int head_dim, const KvMaps& kv_maps, const CUtensorMap& q_map, const CUtensorMap& out_map,
                              const MixedParams& p,
                              int num_sms, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)num_sms);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = mixed_attn_smem_bytes(head_dim);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // prologue overlaps the previous kernel's tail
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const bool multi = p.nchunks > 1;
    if (head_dim == 64)
        return multi ? cudaLaunchKernelEx(&cfg, sw_mixed_attn_kernel<64, true>, kv_maps.half, kv_maps.page, q_map, out_map, p)
                     : cudaLaunchKernelEx(&cfg, sw_mixed_attn_kernel<64, false>, kv_maps.half, kv_maps.page, q_map, out_map, p);
    return multi ? cudaLaunchKernelEx(&cfg, sw_mixed_attn_kernel<128, true>, kv_maps.half, kv_maps.page, q_map, out_map, p)
                 : cudaLaunchKernelEx(&cfg, sw_mixed_attn_kernel<128, false>, kv_maps.half, kv_maps.page, q_map, out_map, p);
}

}  // namespace sw
