// sw_decode_attn_static: decode-only attention for callers that cannot allocate device memory.
//
// Everything the attention kernel needs beyond its inputs and outputs (work counters, per-request tickets and the
// split-KV partial results) lives in one file-scope device array of fixed size that every GPU loading this library
// holds until the process exits.  No context, no workspace, no allocation of any kind.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>

#include "sw.h"
#include "sw_error.h"
#include "sw_internal.h"

namespace {

// Limits of the static variant (see include/sw.h).
constexpr int kStaticMaxDecode = SW_STATIC_MAX_DECODE;   // requests per call
constexpr int kStaticTargetItems = 512;                  // split-KV units aimed at
constexpr int kStaticMaxKvHeads = 8;
constexpr int kStaticMaxItems = kStaticTargetItems + kStaticMaxDecode * kStaticMaxKvHeads;
constexpr size_t kPartOBytesPerItem = 4096;              // group * head_dim * 4 <= 8 * 128 * 4

constexpr size_t kOffCtrl = 0;
constexpr size_t kOffTickets = 256;
constexpr size_t kOffPartMl = kOffTickets + (size_t)kStaticMaxDecode * kStaticMaxKvHeads * 4 * 2;  // tickets, ready
constexpr size_t kOffPartO = kOffPartMl + (size_t)kStaticMaxItems * 2 * sw::kMaxGroup * 4;
constexpr size_t kScratchBytes = kOffPartO + (size_t)kStaticMaxItems * kPartOBytesPerItem;
static_assert(kOffPartMl % 256 == 0 && kOffPartO % 256 == 0, "regions stay 256-byte aligned");
static_assert(kScratchBytes <= SW_STATIC_SCRATCH_BYTES, "the header states the size of the static scratch");

// In host code this name is only a stand-in for the symbol; the device address comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[SW_STATIC_SCRATCH_BYTES];

using sw::EncodeTiledFn;

struct DeviceState {
    bool ready = false;
    unsigned char* scratch = nullptr;  // device address of g_static_scratch on this device
    int num_sms = 0;
    int mem_khz = 0, bus_bits = 0, sm_khz = 0;
    bool configured[2] = {false, false};  // head_dim 64, 128
    EncodeTiledFn encode = nullptr;
};
constexpr int kMaxDevices = 64;
DeviceState g_devices[kMaxDevices];

#define SW_CUDA(call)                                                                                        \
    do {                                                                                                     \
        cudaError_t e_ = (call);                                                                             \
        if (e_ != cudaSuccess) return sw_fail(SW_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_));  \
    } while (0)

// Every call: `device` must be the caller's current device (the launch, the clearing of the scratch and the address of
// the scratch all belong to the current device; nothing here changes it).  Once per device: the set-up below.
sw_status setup_device(int device, DeviceState** out) {
    if (device < 0 || device >= kMaxDevices) return sw_fail(SW_ERR_INVALID_ARG, "device index %d out of range", device);
    int current = -1;
    SW_CUDA(cudaGetDevice(&current));
    if (current != device)
        return sw_fail(SW_ERR_INVALID_ARG, "sw_decode_attn_static: device %d was named but device %d is current", device,
                       current);
    DeviceState& st = g_devices[device];
    if (!st.ready) {
        cudaDeviceProp prop;
        SW_CUDA(cudaGetDeviceProperties(&prop, device));
        if (prop.major != 10)
            return sw_fail(SW_ERR_UNSUPPORTED, "device %d is compute capability %d.%d; this library is sm_100a only", device,
                           prop.major, prop.minor);
        void* ptr = nullptr;
        SW_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn)
            return sw_fail(SW_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
        st.scratch = static_cast<unsigned char*>(ptr);
        st.num_sms = prop.multiProcessorCount < sw::kMaxCtas ? prop.multiProcessorCount : sw::kMaxCtas;
        SW_CUDA(cudaDeviceGetAttribute(&st.mem_khz, cudaDevAttrMemoryClockRate, device));
        SW_CUDA(cudaDeviceGetAttribute(&st.bus_bits, cudaDevAttrGlobalMemoryBusWidth, device));
        SW_CUDA(cudaDeviceGetAttribute(&st.sm_khz, cudaDevAttrClockRate, device));
        st.encode = reinterpret_cast<EncodeTiledFn>(fn);
        st.ready = true;
    }
    *out = &st;
    return SW_OK;
}

}  // namespace

extern "C" sw_status sw_decode_attn_static(const sw_layout* layout, int device, const void* kv_pool, const sw_batch* batch,
                                           const void* q, void* out, float* lse, void* stream) {
    if (!layout || !batch) return sw_fail(SW_ERR_INVALID_ARG, "sw_decode_attn_static: null layout or batch");
    const sw_layout& l = *layout;
    if ((l.head_dim != 64 && l.head_dim != 128) || l.page_size != sw::kPageSize || l.num_kv_heads <= 0 ||
        l.num_q_heads % l.num_kv_heads != 0 || l.num_pages <= 0 || l.num_pages > ((int64_t)1 << 30) ||
        2 * l.num_pages * l.num_kv_heads >= ((int64_t)1 << 31))
        return sw_fail(SW_ERR_UNSUPPORTED, "sw_decode_attn_static: unsupported shape");
    const int g = l.num_q_heads / l.num_kv_heads;
    if (!(g == 1 || g == 2 || g == 4 || g == 8)) return sw_fail(SW_ERR_UNSUPPORTED, "sw_decode_attn_static: unsupported head ratio");
    if (l.num_kv_heads > kStaticMaxKvHeads)
        return sw_fail(SW_ERR_WORKSPACE, "sw_decode_attn_static: at most %d KV heads fit the static scratch", kStaticMaxKvHeads);
    if (batch->chunk_len != 0 || batch->num_chunks != 0)
        return sw_fail(SW_ERR_UNSUPPORTED, "sw_decode_attn_static: decode-only (chunk_len must be 0)");
    if (batch->num_decode < 0 || batch->num_decode > kStaticMaxDecode)
        return sw_fail(SW_ERR_WORKSPACE, "sw_decode_attn_static: num_decode %d exceeds the static limit %d", batch->num_decode,
                       kStaticMaxDecode);
    if (batch->num_decode == 0) return SW_OK;
    if (!kv_pool || !q || !out || !batch->decode_kv_len || !batch->decode_page_indptr || !batch->decode_pages)
        return sw_fail(SW_ERR_INVALID_ARG, "sw_decode_attn_static: null tensor");
    if (((reinterpret_cast<uintptr_t>(kv_pool) | reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out)) & 15) != 0)
        return sw_fail(SW_ERR_INVALID_ARG, "sw_decode_attn_static: tensors must be 16-byte aligned");
    DeviceState* st = nullptr;
    sw_status rc = setup_device(device, &st);
    if (rc != SW_OK) return rc;
    const int hd = l.head_dim == 64 ? 0 : 1;
    if (!st->configured[hd]) {
        SW_CUDA(sw::configure_kernels(l.head_dim));
        st->configured[hd] = true;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    // tensor maps of the pool, encoded on the stack for this call
    sw::KvMaps kv_maps;
    CUresult r = sw::encode_kv_maps(st->encode, l, kv_pool, &kv_maps);
    if (r != CUDA_SUCCESS) return sw_fail(SW_ERR_CUDA, "cuTensorMapEncodeTiled(kv pool) failed with CUresult %d", (int)r);

    // the array keeps whatever the previous call left: counters and tickets must start at zero
    SW_CUDA(cudaMemsetAsync(st->scratch + kOffCtrl, 0, kOffPartMl - kOffCtrl, s));

    sw::MixedParams p{};
    p.Hq = l.num_q_heads;
    p.Hkv = l.num_kv_heads;
    p.group = g;
    p.num_pages = l.num_pages;
    p.sm_scale = l.sm_scale > 0.f ? l.sm_scale : 1.0f / std::sqrt((float)l.head_dim);
    p.sm_scale_log2 = p.sm_scale * 1.4426950408889634f;
    sw::device_timing(st->mem_khz, st->bus_bits, st->sm_khz, l.head_dim, &p.stage_us, &p.step_us);
    p.stages_per_us = 1.f / p.stage_us;
    p.steps_per_stage = p.stage_us / p.step_us;
    p.C = 0;
    p.n = batch->num_decode;
    p.decode_kv_len = batch->decode_kv_len;
    p.decode_page_indptr = batch->decode_page_indptr;
    p.decode_pages = batch->decode_pages;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.out = static_cast<__nv_bfloat16*>(out);
    p.lse = lse;
    p.ctrl = reinterpret_cast<int32_t*>(st->scratch + kOffCtrl);
    p.tickets = reinterpret_cast<int32_t*>(st->scratch + kOffTickets);
    p.ready = p.tickets + kStaticMaxDecode * kStaticMaxKvHeads;
    p.part_ml = reinterpret_cast<float*>(st->scratch + kOffPartMl);
    p.part_o = reinterpret_cast<float*>(st->scratch + kOffPartO);
    p.max_items = kStaticMaxItems;
    p.target_items = kStaticTargetItems;
    SW_CUDA(sw::launch_mixed_attn(l.head_dim, kv_maps, kv_maps.half, kv_maps.half, p, st->num_sms, s));
    return SW_OK;
}
