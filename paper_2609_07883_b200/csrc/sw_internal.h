// Internal definitions shared by the library's host code and kernels (not part of the ABI).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sw.h"

namespace sw {

constexpr int kPageSize = 16;           // tokens per page
constexpr int kMaxDecode = 2048;        // decode requests per iteration (prefix-sum array lives in shared memory)
constexpr int kThreads = 384;           // 12 warps per CTA, one CTA per SM
constexpr int kWarps = kThreads / 32;
constexpr int kTargetItems = 4096;      // split-KV units aimed at per launch (bounds the partial-result scratch)
constexpr int kMinSplitTokens = 128;    // never split a decode context finer than this
constexpr int kMaxGroup = 8;            // query heads per KV head
constexpr int kMaxCtas = 192;           // persistent CTAs (one per SM) the scratch is sized for
constexpr int kPfRoundSlots = 3 * kMaxCtas;  // partial results of chunk-prefill pieces that run in several rounds
constexpr int kMaxChunks = 8;           // prefill chunks (of different prompts) in one iteration
constexpr int kMaxChunk = 65536;        // chunk tokens per iteration (256-row groups are planned in shared memory)

// Control words at the start of the workspace.
// kCtrAppend counts the CTAs of a fused launch that have finished writing their share of the new K/V rows.
enum CtrlWord { kCtrWork = 0, kCtrDone = 1, kCtrStatus = 2, kCtrDetail = 3, kCtrPrefill = 4, kCtrAppend = 5, kCtrWords = 64 };

// Device-detected problem locators written to kCtrDetail (high byte = site, low 24 bits = index).
enum DetailSite { kSiteAppendPage = 1, kSiteAppendLen = 2, kSiteAttnLen = 3, kSiteAttnPage = 4, kSiteWait = 5,
                  kSiteScratch = 6, kSiteTmem = 7 };

struct MixedParams {
    // shape
    int Hq, Hkv, group;
    int64_t num_pages;
    float sm_scale;       // softmax scale
    float sm_scale_log2;  // sm_scale * log2(e)
    // planning estimates, from the device's clocks (device_timing): microseconds in which the whole device streams one
    // (page, kv head) stage of K and V, and microseconds of one 128-key step of a chunk-prefill entry
    float stage_us, step_us;
    float stages_per_us, steps_per_stage;   // 1 / stage_us and stage_us / step_us, worked out on the host
    // batch.  C is the number of chunk rows of the iteration: the rows of its prefill chunks, one chunk after the
    // other.  Chunk j has cC[j] tokens at prefix cP[j], starts at row cRow0[j] and its prompt's page list starts at
    // prefill_pages[cPage0[j]] (cPage0[nchunks] = num_prefill_pages).
    int C, n;
    int nchunks;
    int cP[kMaxChunks], cC[kMaxChunks], cRow0[kMaxChunks], cPage0[kMaxChunks + 1];
    const int32_t* prefill_pages;
    int num_prefill_pages;
    const int32_t* decode_kv_len;
    const int32_t* decode_page_indptr;
    const int32_t* decode_pages;
    const __nv_bfloat16* q;
    __nv_bfloat16* out;
    float* lse;
    // fused KV append (sw_mixed_iteration_run): the rows' new K/V and the pool to write them to; null when the append
    // ran as a launch of its own
    const __nv_bfloat16* k_new;
    const __nv_bfloat16* v_new;
    __nv_bfloat16* pool;
    // scratch
    int32_t* ctrl;
    int32_t* tickets;   // [max_decode * Hkv]: order in which the units of a (request, kv head) near their end
    int32_t* ready;     // [max_decode * Hkv]: how many of them have published their partial result
    float* part_ml;     // [max_items][2 * kMaxGroup]  (m then l per query head of the group)
    float* part_o;      // [max_items][group * D]
    int max_items;      // partial-result slots available
    int target_items;   // split-KV units aimed at (<= max_items - n*Hkv)
    // scratch of prefill items finished by several CTAs
    float* pf_ml;        // [pf_slots][2][2][128]
    float* pf_o;         // [pf_slots][2][D / 4][128][4]
    int pf_slots;        // kMaxCtas, or kPfRoundSlots where a chunk can hold a whole round of items
    int32_t* pf_tickets; // [items][2]
};

struct AppendParams {
    int Hkv, D;
    int64_t num_pages;
    int C, n;
    int nchunks;
    int cP[kMaxChunks], cC[kMaxChunks], cRow0[kMaxChunks], cPage0[kMaxChunks + 1];
    const int32_t* prefill_pages;
    int num_prefill_pages;
    const int32_t* decode_kv_len;
    const int32_t* decode_page_indptr;
    const int32_t* decode_pages;
    const __nv_bfloat16* k_new;
    const __nv_bfloat16* v_new;
    __nv_bfloat16* pool;
    int32_t* ctrl;
};

// Tensor maps of one KV pool [page][K|V][kv head][slot][element].  A (page, K|V, kv head) block of 16 slots x head_dim
// elements reads as head_dim/64 x 2 swizzle atoms of [8 slots][64 elements] (1 KB each in shared memory).
//   half: 5-D {element % 64, slot % 8, element / 64, slot / 8, block} with block = (2 * page + K|V) * Hkv + kv head; box = one
//         block, landing as [slot group][64-element block][8][128 B]: the chunk-prefill producer fetches the eight pages
//         of a 128-key operand tile with eight such copies (one per page, K and V separately).
//   page: 5-D {element % 64, slot, element / 64, 2 * page + K|V, kv head}; box = all of one head's K and V in a page, as
//         2 x head_dim/64 blocks of [16][128 B], K blocks first: a decode unit fetches a page with one copy.
struct KvMaps {
    CUtensorMap half;
    CUtensorMap page;
};
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
inline CUresult encode_kv_maps(EncodeTiledFn encode, const sw_layout& l, const void* pool, KvMaps* out) {
    const cuuint64_t row = (cuuint64_t)l.head_dim * 2;                 // bytes of one slot of one head
    const cuuint64_t head = (cuuint64_t)kPageSize * row;               // one head's K (or V) in a page
    const cuuint64_t side = (cuuint64_t)l.num_kv_heads * head;         // all K (or all V) of a page
    const cuuint32_t ones[5] = {1, 1, 1, 1, 1};
    {
        const cuuint64_t dims[5] = {64, 8, (cuuint64_t)l.head_dim / 64, 2, (cuuint64_t)2 * l.num_pages * l.num_kv_heads};
        const cuuint64_t strides[4] = {row, 128, 8 * row, head};
        const cuuint32_t box[5] = {64, 8, (cuuint32_t)l.head_dim / 64, 2, 1};
        CUresult r = encode(&out->half, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(pool), dims, strides, box, ones,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return r;
    }
    const cuuint64_t dims[5] = {64, (cuuint64_t)kPageSize, (cuuint64_t)l.head_dim / 64, (cuuint64_t)2 * l.num_pages,
                                (cuuint64_t)l.num_kv_heads};
    const cuuint64_t strides[4] = {row, 128, side, head};
    const cuuint32_t box[5] = {64, (cuuint32_t)kPageSize, (cuuint32_t)l.head_dim / 64, 2, 1};
    return encode(&out->page, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(pool), dims, strides, box, ones,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

// launchers (sw_kernels.cu)
cudaError_t launch_kv_append(const AppendParams& p, int num_sms, cudaStream_t stream);
// MixedParams::stage_us / step_us for a device: the memory system streams about 0.76 of clock x bus width x 2 (measured
// against a plain copy on B200: 6.2 of 8.2 TB/s), and a 128-key step of a chunk-prefill entry takes about 4300 SM
// cycles while other CTAs stream decode pages (measured; 2.2 us at 1965 MHz).
inline void device_timing(int mem_clock_khz, int bus_width_bits, int sm_clock_khz, int head_dim, float* stage_us, float* step_us) {
    // a driver that reports no clock leaves the plan with B200's nominal figures rather than with a division by zero
    if (mem_clock_khz <= 0) mem_clock_khz = 3996000;
    if (bus_width_bits <= 0) bus_width_bits = 8192;
    if (sm_clock_khz <= 0) sm_clock_khz = 1965000;
    const double bytes_per_us = 0.76 * 2.0 * (double)mem_clock_khz * 1e3 * ((double)bus_width_bits / 8.0) / 1e6;
    const double stage_bytes = 2.0 * kPageSize * head_dim * 2;   // K and V rows of one head in a page
    *stage_us = (float)(stage_bytes / bytes_per_us);
    *step_us = (float)(4300.0 / ((double)sm_clock_khz / 1e3));
}
cudaError_t launch_mixed_attn(int head_dim, const KvMaps& kv_maps, const CUtensorMap& q_map, const CUtensorMap& out_map,
                              const MixedParams& p,
                              int num_sms, cudaStream_t stream);
cudaError_t configure_kernels(int head_dim);
cudaError_t mixed_attn_resident_ctas_per_sm(int head_dim, int* out);
cudaError_t launch_selftest_wait(int32_t* ctrl, long long budget_cycles, cudaStream_t stream);
size_t mixed_attn_smem_bytes(int head_dim);

}  // namespace sw
