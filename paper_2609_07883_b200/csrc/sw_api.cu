// C-ABI entry points of the device path: context, KV append, the mixed attention launch, the host-buffer
// iteration and the cost probe.  Host code only validates, marshals and launches.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "sw.h"
#include "sw_error.h"
#include "sw_internal.h"

namespace {

using sw::EncodeTiledFn;

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Offsets of the regions inside the caller's workspace.
struct WsLayout {
    size_t ctrl, tickets, part_ml, part_o, pf_tickets, pf_ml, pf_o, st_q, st_k, st_v, st_out, st_lse, st_pages, total;
    int pf_slots;
    int max_items;
};

bool layout_supported(const sw_layout& l) {
    if (l.num_q_heads <= 0 || l.num_kv_heads <= 0 || l.num_pages <= 0) return false;
    if (l.head_dim != 64 && l.head_dim != 128) return false;
    if (l.page_size != sw::kPageSize) return false;
    if (l.num_q_heads % l.num_kv_heads != 0) return false;
    const int g = l.num_q_heads / l.num_kv_heads;
    if (!(g == 1 || g == 2 || g == 4 || g == 8)) return false;
    if (l.num_pages > (int64_t)1 << 30) return false;
    if (2 * l.num_pages * l.num_kv_heads >= (int64_t)1 << 31) return false;  // (page, K|V, head) blocks are int32 coordinates
    return true;
}

WsLayout ws_layout(const sw_layout& l, int max_chunk, int max_decode, int64_t max_pages) {
    WsLayout w{};
    const int g = l.num_q_heads / l.num_kv_heads;
    const size_t rows = (size_t)max_chunk + max_decode;
    w.max_items = sw::kTargetItems + max_decode * l.num_kv_heads;
    size_t off = 0;
    w.ctrl = off;     off = align_up(off + sw::kCtrWords * 4, 256);
    w.tickets = off;  off = align_up(off + (size_t)std::max(1, max_decode) * l.num_kv_heads * 4 * 2, 256);  // tickets, ready
    w.part_ml = off;  off = align_up(off + (size_t)w.max_items * 2 * sw::kMaxGroup * 4, 256);
    w.part_o = off;   off = align_up(off + (size_t)w.max_items * g * l.head_dim * 4, 256);
    // 256-row groups of the chunks of one iteration: every chunk may end in a ragged group
    const size_t groups = ((size_t)max_chunk + (256 / g) - 1) / (256 / g) + sw::kMaxChunks;
    w.pf_tickets = off; off = align_up(off + std::max<size_t>(1, groups) * l.num_kv_heads * 2 * 4, 256);
    // pieces of items publish partial results: one slot per CTA, more where a single chunk can hold a whole round of
    // items (its leftover items may then be cut into pieces that run in several rounds; the plan never uses more slots
    // than it is given)
    const size_t single_chunk_items = ((size_t)max_chunk + (256 / g) - 1) / (256 / g) * l.num_kv_heads;
    w.pf_slots = single_chunk_items >= 96 ? sw::kPfRoundSlots : sw::kMaxCtas;
    w.pf_ml = off;    off = align_up(off + (size_t)w.pf_slots * 2 * 256 * 4, 256);
    w.pf_o = off;     off = align_up(off + (max_chunk > 0 ? (size_t)w.pf_slots * 2 * 128 * l.head_dim * 4 : 0), 256);
    w.st_q = off;     off = align_up(off + rows * l.num_q_heads * l.head_dim * 2, 256);
    w.st_k = off;     off = align_up(off + rows * l.num_kv_heads * l.head_dim * 2, 256);
    w.st_v = off;     off = align_up(off + rows * l.num_kv_heads * l.head_dim * 2, 256);
    w.st_out = off;   off = align_up(off + rows * l.num_q_heads * l.head_dim * 2, 256);
    w.st_lse = off;   off = align_up(off + rows * l.num_q_heads * 4, 256);
    w.st_pages = off; off = align_up(off + ((size_t)max_pages + 2 * (size_t)max_decode + 8) * 4, 256);
    w.total = off;
    return w;
}

}  // namespace

struct sw_ctx {
    sw_layout layout;
    int device = 0;
    int num_sms = 0;
    float stage_us = 0.f, step_us = 0.f;  // planning estimates from the device's clocks (sw::device_timing)
    bool grid_resident = false;  // the persistent grid fits the device at once (needed by the fused append + attention launch)
    int max_chunk = 0, max_decode = 0;
    int64_t max_pages = 0;
    uint8_t* ws = nullptr;
    WsLayout w{};
    EncodeTiledFn encode = nullptr;
    struct MapEntry {
        const void* pool;
        sw::KvMaps maps;
    };
    std::vector<MapEntry> kv_maps;  // small cache: one entry per pool of a layer stack
    cudaEvent_t ev0 = nullptr, ev1 = nullptr;
};

namespace {

#define SW_CUDA(call)                                                                                        \
    do {                                                                                                     \
        cudaError_t e_ = (call);                                                                             \
        if (e_ != cudaSuccess) return sw_fail(SW_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_));  \
    } while (0)

// Launching calls run on the caller's current device: a context serves the device it was created on and refuses any other
// (its workspace, tensor maps and kernel attributes belong to that device).
sw_status check_current_device(const sw_ctx* ctx, const char* who) {
    int current = -1;
    SW_CUDA(cudaGetDevice(&current));
    if (current != ctx->device)
        return sw_fail(SW_ERR_INVALID_ARG, "%s: the context belongs to device %d but device %d is current", who, ctx->device,
                       current);
    return SW_OK;
}

sw_status kv_map_for(sw_ctx* ctx, const void* pool, const sw::KvMaps** out) {
    for (auto& e : ctx->kv_maps)
        if (e.pool == pool) {
            *out = &e.maps;
            return SW_OK;
        }
    const sw_layout& l = ctx->layout;
    if ((reinterpret_cast<uintptr_t>(pool) & 15) != 0) return sw_fail(SW_ERR_INVALID_ARG, "kv_pool must be 16-byte aligned");
    sw_ctx::MapEntry e;
    e.pool = pool;
    CUresult r = sw::encode_kv_maps(ctx->encode, l, pool, &e.maps);
    if (r != CUDA_SUCCESS) return sw_fail(SW_ERR_CUDA, "cuTensorMapEncodeTiled(kv pool) failed with CUresult %d", (int)r);
    if (ctx->kv_maps.size() >= 128) ctx->kv_maps.erase(ctx->kv_maps.begin());
    ctx->kv_maps.push_back(e);
    *out = &ctx->kv_maps.back().maps;
    return SW_OK;
}

// The prefill chunks of a batch in the form the kernels take (single-chunk batches become one chunk).
struct Chunks {
    int n = 0;
    int rows = 0;  // chunk rows of the iteration = sum of the chunk lengths
    int P[sw::kMaxChunks] = {}, C[sw::kMaxChunks] = {}, row0[sw::kMaxChunks] = {}, page0[sw::kMaxChunks + 1] = {};
};
static_assert(SW_MAX_CHUNKS == sw::kMaxChunks, "the header states the limit");

sw_status chunks_of(const sw_batch* b, const char* who, Chunks* out) {
    Chunks c;
    if (b->num_chunks < 0 || b->num_chunks > sw::kMaxChunks)
        return sw_fail(SW_ERR_INVALID_ARG, "%s: num_chunks %d outside 0..%d", who, b->num_chunks, sw::kMaxChunks);
    if (b->num_chunks == 0) {
        if (b->chunk_len > 0) {
            c.n = 1;
            c.P[0] = b->prefix_len;
            c.C[0] = b->chunk_len;
            c.rows = b->chunk_len;
            c.page0[1] = b->num_prefill_pages;
        }
    } else {
        if (!b->chunk_prefix_lens || !b->chunk_lens || !b->chunk_page_indptr)
            return sw_fail(SW_ERR_INVALID_ARG, "%s: chunk arrays missing", who);
        int64_t rows = 0;
        for (int j = 0; j < b->num_chunks; ++j) {
            if (b->chunk_prefix_lens[j] < 0 || b->chunk_lens[j] < 1)
                return sw_fail(SW_ERR_INVALID_ARG, "%s: chunk %d has prefix %d and length %d", who, j, b->chunk_prefix_lens[j],
                               b->chunk_lens[j]);
            if (b->chunk_page_indptr[j + 1] < b->chunk_page_indptr[j] || b->chunk_page_indptr[0] != 0)
                return sw_fail(SW_ERR_INVALID_ARG, "%s: chunk_page_indptr must start at 0 and not decrease", who);
            c.P[j] = b->chunk_prefix_lens[j];
            c.C[j] = b->chunk_lens[j];
            c.row0[j] = (int)rows;
            c.page0[j] = b->chunk_page_indptr[j];
            rows += b->chunk_lens[j];
            if (rows > sw::kMaxChunk) return sw_fail(SW_ERR_UNSUPPORTED, "%s: more than %d chunk rows", who, sw::kMaxChunk);
        }
        c.n = b->num_chunks;
        c.rows = (int)rows;
        c.page0[c.n] = b->chunk_page_indptr[c.n];
        if (c.page0[c.n] != b->num_prefill_pages)
            return sw_fail(SW_ERR_INVALID_ARG, "%s: chunk_page_indptr ends at %d, num_prefill_pages is %d", who, c.page0[c.n],
                           b->num_prefill_pages);
    }
    for (int j = c.n; j <= sw::kMaxChunks; ++j) c.page0[j] = c.page0[c.n];
    *out = c;
    return SW_OK;
}

sw_status check_batch(const sw_ctx* ctx, const sw_batch* b, const char* who, Chunks* chunks) {
    if (!ctx || !b) return sw_fail(SW_ERR_INVALID_ARG, "%s: null context or batch", who);
    if (b->prefix_len < 0 || b->chunk_len < 0 || b->num_decode < 0 || b->num_prefill_pages < 0)
        return sw_fail(SW_ERR_INVALID_ARG, "%s: negative size in batch", who);
    sw_status cs = chunks_of(b, who, chunks);
    if (cs != SW_OK) return cs;
    if (chunks->rows > ctx->max_chunk || b->num_decode > ctx->max_decode)
        return sw_fail(SW_ERR_WORKSPACE, "%s: %d chunk rows / num_decode %d exceed the context's limits %d / %d", who,
                       chunks->rows, b->num_decode, ctx->max_chunk, ctx->max_decode);
    if (b->num_decode > sw::kMaxDecode)
        return sw_fail(SW_ERR_UNSUPPORTED, "%s: at most %d decode requests per iteration", who, sw::kMaxDecode);
    for (int j = 0; j < chunks->n; ++j) {
        const int64_t need = ((int64_t)chunks->P[j] + chunks->C[j] + sw::kPageSize - 1) / sw::kPageSize;
        const int have = chunks->page0[j + 1] - chunks->page0[j];
        if (!b->prefill_pages || have < need)
            return sw_fail(SW_ERR_OUT_OF_RANGE, "%s: prefill page list has %d entries, P+C needs %lld", who, have,
                           (long long)need);
    }
    if (b->num_decode > 0 && (!b->decode_kv_len || !b->decode_page_indptr || !b->decode_pages))
        return sw_fail(SW_ERR_INVALID_ARG, "%s: decode arrays missing", who);
    return SW_OK;
}

}  // namespace

extern "C" {

size_t sw_workspace_bytes(const sw_layout* layout, int32_t max_chunk, int32_t max_decode, int64_t max_pages) {
    if (!layout || !layout_supported(*layout) || max_chunk < 0 || max_decode < 0 || max_pages < 0 ||
        max_decode > sw::kMaxDecode || max_chunk > sw::kMaxChunk)
        return 0;
    return ws_layout(*layout, max_chunk, max_decode, max_pages).total;
}

sw_status sw_create(const sw_layout* layout, int device, void* workspace, size_t workspace_bytes, int32_t max_chunk,
                    int32_t max_decode, int64_t max_pages, sw_ctx** out) {
    if (!layout || !out) return sw_fail(SW_ERR_INVALID_ARG, "sw_create: null argument");
    if (!layout_supported(*layout))
        return sw_fail(SW_ERR_UNSUPPORTED,
                       "sw_create: supported shapes are head_dim 64|128, page_size 16, q/kv head ratio 1|2|4|8");
    if (max_chunk < 0 || max_decode < 0 || max_pages < 0 || max_decode > sw::kMaxDecode || max_chunk > sw::kMaxChunk)
        return sw_fail(SW_ERR_INVALID_ARG, "sw_create: limits out of range (max_decode <= %d, max_chunk <= %d)", sw::kMaxDecode,
                       sw::kMaxChunk);
    const WsLayout w = ws_layout(*layout, max_chunk, max_decode, max_pages);
    if (!workspace || workspace_bytes < w.total || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0)
        return sw_fail(SW_ERR_WORKSPACE, "sw_create: workspace must be 256-byte aligned and hold %zu bytes", w.total);
    cudaDeviceProp prop;
    SW_CUDA(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10)
        return sw_fail(SW_ERR_UNSUPPORTED, "sw_create: device %d is compute capability %d.%d; this library is sm_100a only",
                       device, prop.major, prop.minor);
    // the set-up below runs with `device` current; the caller's current device is put back before returning
    int caller_device = device;
    SW_CUDA(cudaGetDevice(&caller_device));
    struct Restore {
        int dev, want;
        ~Restore() {
            if (dev != want) cudaSetDevice(dev);
        }
    } restore{caller_device, device};
    if (caller_device != device) SW_CUDA(cudaSetDevice(device));
    int mem_khz = 0, bus_bits = 0, sm_khz = 0;
    SW_CUDA(cudaDeviceGetAttribute(&mem_khz, cudaDevAttrMemoryClockRate, device));
    SW_CUDA(cudaDeviceGetAttribute(&bus_bits, cudaDevAttrGlobalMemoryBusWidth, device));
    SW_CUDA(cudaDeviceGetAttribute(&sm_khz, cudaDevAttrClockRate, device));
    sw_ctx* ctx = new (std::nothrow) sw_ctx();
    if (!ctx) return sw_fail(SW_ERR_INVALID_ARG, "sw_create: out of host memory");
    ctx->layout = *layout;
    if (ctx->layout.sm_scale <= 0.f) ctx->layout.sm_scale = 1.0f / std::sqrt((float)layout->head_dim);
    ctx->device = device;
    ctx->num_sms = std::min(prop.multiProcessorCount, sw::kMaxCtas);
    sw::device_timing(mem_khz, bus_bits, sm_khz, layout->head_dim, &ctx->stage_us, &ctx->step_us);
    ctx->max_chunk = max_chunk;
    ctx->max_decode = max_decode;
    ctx->max_pages = max_pages;
    ctx->ws = static_cast<uint8_t*>(workspace);
    ctx->w = w;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
        delete ctx;
        return sw_fail(SW_ERR_CUDA, "sw_create: cuTensorMapEncodeTiled is not available from the driver");
    }
    ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
    e = cudaMemset(ctx->ws, 0, w.pf_ml);  // control words, tickets and split-KV scratch start at zero
    if (e == cudaSuccess) e = sw::configure_kernels(layout->head_dim);
    int per_sm = 0;
    if (e == cudaSuccess) e = sw::mixed_attn_resident_ctas_per_sm(layout->head_dim, &per_sm);
    // The fused launch lets CTAs wait for one another's share of the KV append, so the whole grid has to be resident.
    // Where it would not be (fewer SMs than the properties promise cannot be seen here, but a smaller shared-memory
    // or register budget can) sw_mixed_iteration_run issues the append as a launch of its own.
    ctx->grid_resident = (int64_t)per_sm * prop.multiProcessorCount >= ctx->num_sms;
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        delete ctx;
        return sw_fail(SW_ERR_CUDA, "sw_create: device set-up failed: %s", cudaGetErrorString(e));
    }
    *out = ctx;
    return SW_OK;
}

void sw_destroy(sw_ctx* ctx) {
    if (!ctx) return;
    if (ctx->ev0) cudaEventDestroy(ctx->ev0);
    if (ctx->ev1) cudaEventDestroy(ctx->ev1);
    delete ctx;
}

sw_status sw_kv_append(sw_ctx* ctx, void* kv_pool, const sw_batch* batch, const void* k_new, const void* v_new,
                       void* stream) {
    Chunks ch;
    sw_status st = check_batch(ctx, batch, "sw_kv_append", &ch);
    if (st != SW_OK) return st;
    if (ch.rows + batch->num_decode == 0) return SW_OK;
    if (!kv_pool || !k_new || !v_new) return sw_fail(SW_ERR_INVALID_ARG, "sw_kv_append: null tensor");
    st = check_current_device(ctx, "sw_kv_append");
    if (st != SW_OK) return st;
    if (((reinterpret_cast<uintptr_t>(kv_pool) | reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new)) & 15) != 0)
        return sw_fail(SW_ERR_INVALID_ARG, "sw_kv_append: tensors must be 16-byte aligned");
    sw::AppendParams p{};
    p.Hkv = ctx->layout.num_kv_heads;
    p.D = ctx->layout.head_dim;
    p.num_pages = ctx->layout.num_pages;
    p.C = ch.rows;
    p.n = batch->num_decode;
    p.nchunks = ch.n;
    std::memcpy(p.cP, ch.P, sizeof p.cP);
    std::memcpy(p.cC, ch.C, sizeof p.cC);
    std::memcpy(p.cRow0, ch.row0, sizeof p.cRow0);
    std::memcpy(p.cPage0, ch.page0, sizeof p.cPage0);
    p.prefill_pages = batch->prefill_pages;
    p.num_prefill_pages = batch->num_prefill_pages;
    p.decode_kv_len = batch->decode_kv_len;
    p.decode_page_indptr = batch->decode_page_indptr;
    p.decode_pages = batch->decode_pages;
    p.k_new = static_cast<const __nv_bfloat16*>(k_new);
    p.v_new = static_cast<const __nv_bfloat16*>(v_new);
    p.pool = static_cast<__nv_bfloat16*>(kv_pool);
    p.ctrl = reinterpret_cast<int32_t*>(ctx->ws + ctx->w.ctrl);
    SW_CUDA(sw::launch_kv_append(p, ctx->num_sms, static_cast<cudaStream_t>(stream)));
    return SW_OK;
}

namespace {
// The attention launch; with k_new / v_new non-null the same launch first writes those rows into the pool.
sw_status run_mixed(sw_ctx* ctx, void* kv_pool, const sw_batch* batch, const void* k_new, const void* v_new, const void* q,
                    void* out, float* lse, void* stream, const char* who) {
    Chunks ch;
    sw_status st = check_batch(ctx, batch, who, &ch);
    if (st != SW_OK) return st;
    if (ch.rows + batch->num_decode == 0) return SW_OK;
    if (!kv_pool || !q || !out) return sw_fail(SW_ERR_INVALID_ARG, "%s: null tensor", who);
    st = check_current_device(ctx, who);
    if (st != SW_OK) return st;
    if (((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(k_new) |
          reinterpret_cast<uintptr_t>(v_new)) & 15) != 0)
        return sw_fail(SW_ERR_INVALID_ARG, "%s: tensors must be 16-byte aligned", who);
    const sw::KvMaps* kv_maps = nullptr;
    st = kv_map_for(ctx, kv_pool, &kv_maps);
    if (st != SW_OK) return st;
    const sw_layout& l = ctx->layout;
    sw::MixedParams p{};
    p.Hq = l.num_q_heads;
    p.Hkv = l.num_kv_heads;
    p.group = l.num_q_heads / l.num_kv_heads;
    p.num_pages = l.num_pages;
    p.sm_scale = l.sm_scale;
    p.sm_scale_log2 = l.sm_scale * 1.4426950408889634f;
    p.stage_us = ctx->stage_us;
    p.step_us = ctx->step_us;
    p.stages_per_us = 1.f / ctx->stage_us;
    p.steps_per_stage = ctx->stage_us / ctx->step_us;
    p.C = ch.rows;
    p.n = batch->num_decode;
    p.nchunks = ch.n;
    std::memcpy(p.cP, ch.P, sizeof p.cP);
    std::memcpy(p.cC, ch.C, sizeof p.cC);
    std::memcpy(p.cRow0, ch.row0, sizeof p.cRow0);
    std::memcpy(p.cPage0, ch.page0, sizeof p.cPage0);
    p.prefill_pages = batch->prefill_pages;
    p.num_prefill_pages = batch->num_prefill_pages;
    p.decode_kv_len = batch->decode_kv_len;
    p.decode_page_indptr = batch->decode_page_indptr;
    p.decode_pages = batch->decode_pages;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.out = static_cast<__nv_bfloat16*>(out);
    p.lse = lse;
    if (k_new) {
        p.k_new = static_cast<const __nv_bfloat16*>(k_new);
        p.v_new = static_cast<const __nv_bfloat16*>(v_new);
        p.pool = static_cast<__nv_bfloat16*>(kv_pool);
    }
    p.ctrl = reinterpret_cast<int32_t*>(ctx->ws + ctx->w.ctrl);
    p.tickets = reinterpret_cast<int32_t*>(ctx->ws + ctx->w.tickets);
    p.ready = p.tickets + (size_t)std::max(1, ctx->max_decode) * l.num_kv_heads;
    p.part_ml = reinterpret_cast<float*>(ctx->ws + ctx->w.part_ml);
    p.part_o = reinterpret_cast<float*>(ctx->ws + ctx->w.part_o);
    p.max_items = ctx->w.max_items;
    p.target_items = sw::kTargetItems;
    p.pf_ml = reinterpret_cast<float*>(ctx->ws + ctx->w.pf_ml);
    p.pf_o = reinterpret_cast<float*>(ctx->ws + ctx->w.pf_o);
    p.pf_slots = ctx->w.pf_slots;
    p.pf_tickets = reinterpret_cast<int32_t*>(ctx->ws + ctx->w.pf_tickets);
    // q as [row][head][element] restricted to the chunk rows: one box = 128 tile rows (token-major, the g heads of a
    // KV head minor) x 64 elements; rows past the chunk read as zero
    CUtensorMap q_map = kv_maps->half, out_map = kv_maps->half;
    if (p.C > 0) {
        const cuuint64_t dims[3] = {(cuuint64_t)l.head_dim, (cuuint64_t)l.num_q_heads, (cuuint64_t)p.C};
        const cuuint64_t strides[2] = {(cuuint64_t)l.head_dim * 2, (cuuint64_t)l.num_q_heads * l.head_dim * 2};
        const cuuint32_t box[3] = {64, (cuuint32_t)p.group, (cuuint32_t)(128 / p.group)};
        const cuuint32_t elem_strides[3] = {1, 1, 1};
        CUresult r = ctx->encode(&q_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(q), dims, strides, box,
                                 elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return sw_fail(SW_ERR_CUDA, "cuTensorMapEncodeTiled(q) failed with CUresult %d", (int)r);
        // out has the same shape: tiles whose 128 rows all lie inside a chunk are stored through this map
        r = ctx->encode(&out_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, out, dims, strides, box, elem_strides,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return sw_fail(SW_ERR_CUDA, "cuTensorMapEncodeTiled(out) failed with CUresult %d", (int)r);
    }
    SW_CUDA(sw::launch_mixed_attn(l.head_dim, *kv_maps, q_map, out_map, p, ctx->num_sms, static_cast<cudaStream_t>(stream)));
    return SW_OK;
}

// Append + attention: one launch, or two where the persistent grid would not be resident at once.
sw_status run_iteration(sw_ctx* ctx, void* kv_pool, const sw_batch* batch, const void* k_new, const void* v_new, const void* q,
                        void* out, float* lse, void* stream, const char* who) {
    if (ctx && !ctx->grid_resident) {
        sw_status st = sw_kv_append(ctx, kv_pool, batch, k_new, v_new, stream);
        if (st != SW_OK) return st;
        return run_mixed(ctx, kv_pool, batch, nullptr, nullptr, q, out, lse, stream, who);
    }
    return run_mixed(ctx, kv_pool, batch, k_new, v_new, q, out, lse, stream, who);
}
}  // namespace

sw_status sw_mixed_attn_run(sw_ctx* ctx, const void* kv_pool, const sw_batch* batch, const void* q, void* out, float* lse,
                            void* stream) {
    return run_mixed(ctx, const_cast<void*>(kv_pool), batch, nullptr, nullptr, q, out, lse, stream, "sw_mixed_attn_run");
}

sw_status sw_mixed_iteration_run(sw_ctx* ctx, void* kv_pool, const sw_batch* batch, const void* k_new, const void* v_new,
                                 const void* q, void* out, float* lse, void* stream) {
    if (!k_new || !v_new) return sw_fail(SW_ERR_INVALID_ARG, "sw_mixed_iteration_run: null tensor");
    return run_iteration(ctx, kv_pool, batch, k_new, v_new, q, out, lse, stream, "sw_mixed_iteration_run");
}

sw_status sw_mixed_iteration_host(sw_ctx* ctx, void* kv_pool, const sw_batch* hb, const void* h_q, const void* h_k_new,
                                  const void* h_v_new, void* h_out, float* h_lse, void* stream) {
    sw_status st = SW_OK;
    if (!ctx || !hb) return sw_fail(SW_ERR_INVALID_ARG, "sw_mixed_iteration_host: null context or batch");
    Chunks hch;
    st = chunks_of(hb, "sw_mixed_iteration_host", &hch);
    if (st != SW_OK) return st;
    if (hb->chunk_len < 0 || hb->num_decode < 0 || hb->num_prefill_pages < 0 || hch.rows > ctx->max_chunk ||
        hb->num_decode > ctx->max_decode)
        return sw_fail(SW_ERR_WORKSPACE, "sw_mixed_iteration_host: batch exceeds the context's limits");
    const int rows = hch.rows + hb->num_decode;
    if (rows == 0) return SW_OK;
    if (!h_q || !h_k_new || !h_v_new || !h_out || !kv_pool)
        return sw_fail(SW_ERR_INVALID_ARG, "sw_mixed_iteration_host: null tensor");
    const int n = hb->num_decode;
    if (n > 0 && (!hb->decode_kv_len || !hb->decode_page_indptr || !hb->decode_pages))
        return sw_fail(SW_ERR_INVALID_ARG, "sw_mixed_iteration_host: decode arrays missing");
    const int64_t n_dec_pages = n > 0 ? hb->decode_page_indptr[n] : 0;
    if (n_dec_pages < 0 || n_dec_pages + hb->num_prefill_pages > ctx->max_pages)
        return sw_fail(SW_ERR_WORKSPACE, "sw_mixed_iteration_host: %lld page-table entries exceed max_pages %lld",
                       (long long)(n_dec_pages + hb->num_prefill_pages), (long long)ctx->max_pages);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const sw_layout& l = ctx->layout;
    const size_t q_bytes = (size_t)rows * l.num_q_heads * l.head_dim * 2;
    const size_t kv_bytes = (size_t)rows * l.num_kv_heads * l.head_dim * 2;
    uint8_t* ws = ctx->ws;
    int32_t* d_pages = reinterpret_cast<int32_t*>(ws + ctx->w.st_pages);
    int32_t* d_len = d_pages;                         // [n]
    int32_t* d_indptr = d_len + ctx->max_decode;      // [n+1]
    int32_t* d_dec_pages = d_indptr + ctx->max_decode + 2;
    int32_t* d_pf_pages = d_dec_pages + n_dec_pages;
    SW_CUDA(cudaMemcpyAsync(ws + ctx->w.st_q, h_q, q_bytes, cudaMemcpyHostToDevice, s));
    SW_CUDA(cudaMemcpyAsync(ws + ctx->w.st_k, h_k_new, kv_bytes, cudaMemcpyHostToDevice, s));
    SW_CUDA(cudaMemcpyAsync(ws + ctx->w.st_v, h_v_new, kv_bytes, cudaMemcpyHostToDevice, s));
    if (n > 0) {
        SW_CUDA(cudaMemcpyAsync(d_len, hb->decode_kv_len, (size_t)n * 4, cudaMemcpyHostToDevice, s));
        SW_CUDA(cudaMemcpyAsync(d_indptr, hb->decode_page_indptr, (size_t)(n + 1) * 4, cudaMemcpyHostToDevice, s));
        if (n_dec_pages > 0)
            SW_CUDA(cudaMemcpyAsync(d_dec_pages, hb->decode_pages, (size_t)n_dec_pages * 4, cudaMemcpyHostToDevice, s));
    }
    if (hb->num_prefill_pages > 0)
        SW_CUDA(cudaMemcpyAsync(d_pf_pages, hb->prefill_pages, (size_t)hb->num_prefill_pages * 4, cudaMemcpyHostToDevice, s));
    sw_batch db = *hb;
    db.prefill_pages = d_pf_pages;
    db.decode_kv_len = d_len;
    db.decode_page_indptr = d_indptr;
    db.decode_pages = d_dec_pages;
    float* d_lse = h_lse ? reinterpret_cast<float*>(ws + ctx->w.st_lse) : nullptr;
    st = sw_mixed_iteration_run(ctx, kv_pool, &db, ws + ctx->w.st_k, ws + ctx->w.st_v, ws + ctx->w.st_q, ws + ctx->w.st_out,
                                d_lse, stream);
    if (st != SW_OK) return st;
    SW_CUDA(cudaMemcpyAsync(h_out, ws + ctx->w.st_out, q_bytes, cudaMemcpyDeviceToHost, s));
    if (h_lse) SW_CUDA(cudaMemcpyAsync(h_lse, d_lse, (size_t)rows * l.num_q_heads * 4, cudaMemcpyDeviceToHost, s));
    SW_CUDA(cudaStreamSynchronize(s));
    return SW_OK;
}

namespace {
// Times iterations of `layers` launches each: attention alone, or (k_new / v_new given) append + attention in one launch.
sw_status probe(sw_ctx* ctx, void* const* kv_pools, int32_t layers, const sw_batch* batch, const void* k_new,
                const void* v_new, const void* q, void* out, int32_t warmup, int32_t reps, int64_t* p50_ns, int64_t* p99_ns,
                int64_t* samples_ns, void* stream, const char* who) {
    if (!ctx || !kv_pools || layers < 1 || reps < 1 || warmup < 0 || !p50_ns || !p99_ns)
        return sw_fail(SW_ERR_INVALID_ARG, "%s: invalid argument", who);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (!ctx->ev0) SW_CUDA(cudaEventCreate(&ctx->ev0));
    if (!ctx->ev1) SW_CUDA(cudaEventCreate(&ctx->ev1));
    std::vector<int64_t> t((size_t)reps);
    for (int r = -warmup; r < reps; ++r) {
        SW_CUDA(cudaEventRecord(ctx->ev0, s));
        for (int layer = 0; layer < layers; ++layer) {
            sw_status st = k_new ? run_iteration(ctx, kv_pools[layer], batch, k_new, v_new, q, out, nullptr, stream, who)
                                 : run_mixed(ctx, kv_pools[layer], batch, nullptr, nullptr, q, out, nullptr, stream, who);
            if (st != SW_OK) return st;
        }
        SW_CUDA(cudaEventRecord(ctx->ev1, s));
        SW_CUDA(cudaEventSynchronize(ctx->ev1));
        float ms = 0.f;
        SW_CUDA(cudaEventElapsedTime(&ms, ctx->ev0, ctx->ev1));
        if (r >= 0) t[(size_t)r] = (int64_t)std::llround((double)ms * 1e6);
    }
    if (samples_ns) std::memcpy(samples_ns, t.data(), sizeof(int64_t) * (size_t)reps);
    std::sort(t.begin(), t.end());
    // nearest-rank percentiles: the ceil(q * reps)-th smallest sample
    auto rank = [&](double qv) { return t[(size_t)std::max<int64_t>(1, (int64_t)std::ceil(qv * reps)) - 1]; };
    *p50_ns = rank(0.50);
    *p99_ns = rank(0.99);
    return SW_OK;
}
}  // namespace

sw_status sw_cost_probe(sw_ctx* ctx, void* const* kv_pools, int32_t layers, const sw_batch* batch, const void* q, void* out,
                        int32_t warmup, int32_t reps, int64_t* p50_ns, int64_t* p99_ns, int64_t* samples_ns, void* stream) {
    return probe(ctx, kv_pools, layers, batch, nullptr, nullptr, q, out, warmup, reps, p50_ns, p99_ns, samples_ns, stream,
                 "sw_cost_probe");
}

sw_status sw_cost_probe_iteration(sw_ctx* ctx, void* const* kv_pools, int32_t layers, const sw_batch* batch, const void* k_new,
                                  const void* v_new, const void* q, void* out, int32_t warmup, int32_t reps, int64_t* p50_ns,
                                  int64_t* p99_ns, int64_t* samples_ns, void* stream) {
    if (!k_new || !v_new) return sw_fail(SW_ERR_INVALID_ARG, "sw_cost_probe_iteration: null tensor");
    return probe(ctx, kv_pools, layers, batch, k_new, v_new, q, out, warmup, reps, p50_ns, p99_ns, samples_ns, stream,
                 "sw_cost_probe_iteration");
}

sw_status sw_check_status(sw_ctx* ctx, void* stream, int32_t* code, int32_t* detail) {
    if (!ctx) return sw_fail(SW_ERR_INVALID_ARG, "sw_check_status: null context");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int32_t words[2] = {0, 0};
    int32_t* d = reinterpret_cast<int32_t*>(ctx->ws + ctx->w.ctrl) + sw::kCtrStatus;
    SW_CUDA(cudaMemcpyAsync(words, d, sizeof words, cudaMemcpyDeviceToHost, s));
    SW_CUDA(cudaStreamSynchronize(s));
    if (words[0] != 0) {
        // A launch that reported a problem may have skipped units or left early, so the work counters and tickets
        // may not have been re-armed: clear them together with the status words (the stream is idle here).
        SW_CUDA(cudaMemsetAsync(ctx->ws + ctx->w.ctrl, 0, ctx->w.part_ml - ctx->w.ctrl, s));
        SW_CUDA(cudaMemsetAsync(ctx->ws + ctx->w.pf_tickets, 0, ctx->w.pf_ml - ctx->w.pf_tickets, s));
        SW_CUDA(cudaStreamSynchronize(s));
    }
    if (code) *code = words[0];
    if (detail) *detail = words[1];
    if (words[0] != 0)
        return sw_fail((sw_status)words[0], "device reported status %d at site %d index %d", words[0], (words[1] >> 24) & 0xFF,
                       words[1] & 0xFFFFFF);
    return SW_OK;
}

sw_status sw_selftest_wait_timeout(sw_ctx* ctx, int64_t budget_cycles, void* stream) {
    if (!ctx || budget_cycles < 0 || budget_cycles > 4000000000LL)
        return sw_fail(SW_ERR_INVALID_ARG, "sw_selftest_wait_timeout: invalid argument (budget of at most 4e9 cycles)");
    SW_CUDA(sw::launch_selftest_wait(reinterpret_cast<int32_t*>(ctx->ws + ctx->w.ctrl), (long long)budget_cycles,
                                     static_cast<cudaStream_t>(stream)));
    return SW_OK;
}

}  // extern "C"
