// ps_push_static: the cumulative push for callers that must not allocate.
//
// Some programs that embed this library cannot call cudaMalloc at the point
// where they need a push: a plug-in running inside a host application that has
// handed every free byte of the GPU to its own pool, a serving loop with a
// fixed memory budget (for instance under an MPS memory limit), or a
// latency-critical section in which the device-wide synchronisation that
// cudaMalloc and cudaFree imply is not acceptable.  Such a caller can neither
// allocate the workspace that ps_create wants nor ask this library to do it.
// For them the scratch memory of a (small) push lives in a file-scope device
// array that is part of the loaded library image: it exists on every GPU that
// loads the library, from load until the process exits.
#include <mutex>
#include <string.h>

#include "ps_internal.cuh"

namespace psb {

constexpr uint64_t kStaticMaxKeys = PS_PUSH_STATIC_MAX_KEYS;
constexpr uint32_t kStaticMaxRowLen = PS_PUSH_STATIC_MAX_ROW_LEN;

constexpr size_t pad256(size_t x) { return (x + 255) / 256 * 256; }
constexpr size_t kOffStatus = 0;
constexpr size_t kOffKeysA = kOffStatus + pad256(sizeof(DevStatus));
constexpr size_t kOffKeysB = kOffKeysA + pad256(kStaticMaxKeys * 4);
constexpr size_t kOffValsA = kOffKeysB + pad256(kStaticMaxKeys * 4);
constexpr size_t kOffValsB = kOffValsA + pad256(kStaticMaxKeys * 4);
constexpr size_t kOffHist = kOffValsB + pad256(kStaticMaxKeys * 4);
constexpr size_t kOffSortCtl =
    kOffHist + pad256((size_t)kMaxSortPasses * ((kStaticMaxKeys + kSortTile - 1) / kSortTile) * kRadix * 4);
constexpr size_t kStaticGroups = (kStaticMaxKeys + kGroupSpan - 1) / kGroupSpan;
constexpr size_t kOffCarry = kOffSortCtl + pad256(((size_t)kSortCtlWords + kStaticGroups) * 4);
constexpr size_t kOffStarters =
    kOffCarry + pad256(((kStaticMaxKeys + kReduceTile - 1) / kReduceTile) * 2 * (size_t)kStaticMaxRowLen * 8);
constexpr size_t kOffStarterCount = kOffStarters + pad256(((kStaticMaxKeys + kReduceTile - 1) / kReduceTile) * 16);
constexpr size_t kOffGroupSum = kOffStarterCount + 256;
constexpr size_t kStaticBytes = kOffGroupSum + pad256(kStaticGroups * (size_t)kStaticMaxRowLen * 8);

// About 2.3 MB per GPU.  In host code this name is only a handle for the
// runtime; the address a kernel can use comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_push_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
struct PerDevice {
    bool ready;
    unsigned char* scratch;     // device address of g_push_scratch on this GPU
    int sm_count;
};
static PerDevice g_dev[kMaxDevices];
static std::mutex g_mu;

// Once per device, with that device current: look up where the array lives on it.
static ps_status_t device_setup(int device, PerDevice* out) {
    std::lock_guard<std::mutex> lock(g_mu);
    PerDevice& d = g_dev[device];
    if (!d.ready) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_push_scratch) != cudaSuccess || ptr == nullptr) return PS_ERR_CUDA;
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms <= 0)
            return PS_ERR_CUDA;
        d.scratch = (unsigned char*)ptr;
        d.sm_count = sms;
        d.ready = true;
    }
    *out = d;
    return PS_OK;
}

}  // namespace psb

using namespace psb;

extern "C" ps_status_t ps_push_static(void* d_store, const void* d_table, uint64_t num_keys, uint32_t row_len,
                                      uint64_t slots_per_part, const uint64_t* d_keys, uint64_t n,
                                      const float* d_updates, void* stream) {
    if (!d_store || !d_table) return PS_ERR_INVALID_ARG;
    if (num_keys == 0 || num_keys >= 0xFFFFFFFFull || row_len == 0 || slots_per_part == 0) return PS_ERR_INVALID_ARG;
    if (row_len % 4 != 0 || row_len > kStaticMaxRowLen) return PS_ERR_UNSUPPORTED;
    if (n > kStaticMaxKeys) return PS_ERR_WORKSPACE;
    if (n == 0) return PS_OK;
    if (!d_keys || !d_updates || ((uintptr_t)d_updates & 15) || ((uintptr_t)d_store & 15)) return PS_ERR_INVALID_ARG;
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return PS_ERR_CUDA;
    PerDevice dev;
    const ps_status_t rc = device_setup(device, &dev);
    if (rc != PS_OK) return rc;

    // A throw-away handle whose scratch pointers all lie inside the static array.
    ps_store tmp;
    memset(&tmp, 0, sizeof tmp);
    tmp.cfg.num_keys = num_keys;
    tmp.cfg.row_len = row_len;
    tmp.cfg.num_workers = 1;
    tmp.cfg.slots_per_part = slots_per_part;
    tmp.cfg.device = device;
    tmp.max_keys = kStaticMaxKeys;
    int bits = 0;
    while (bits < 32 && (num_keys >> bits) != 0) ++bits;
    tmp.key_bits = bits < 1 ? 1 : bits;
    tmp.sort_blocks_cap = (uint32_t)((kStaticMaxKeys + kSortTile - 1) / kSortTile);
    tmp.store = (float*)d_store;
    tmp.table = (uint2*)const_cast<void*>(d_table);
    tmp.status = (DevStatus*)(dev.scratch + kOffStatus);
    tmp.keysA = (uint32_t*)(dev.scratch + kOffKeysA);
    tmp.keysB = (uint32_t*)(dev.scratch + kOffKeysB);
    tmp.valsA = (uint32_t*)(dev.scratch + kOffValsA);
    tmp.valsB = (uint32_t*)(dev.scratch + kOffValsB);
    tmp.tile_state = (uint32_t*)(dev.scratch + kOffHist);
    tmp.sort_ctl = (uint32_t*)(dev.scratch + kOffSortCtl);
    tmp.group_done = tmp.sort_ctl + kSortCtlWords;
    tmp.group_sum = (double*)(dev.scratch + kOffGroupSum);
    tmp.carry = (double*)(dev.scratch + kOffCarry);
    tmp.starters = (uint4*)(dev.scratch + kOffStarters);
    tmp.starter_count = (unsigned int*)(dev.scratch + kOffStarterCount);
    tmp.epoch = 1;
    tmp.sm_count = dev.sm_count;

    cudaStream_t s = (cudaStream_t)stream;
    // The array keeps whatever the previous call left: the status words must start at zero.
    if (cudaMemsetAsync(tmp.status, 0, sizeof(DevStatus), s) != cudaSuccess) return PS_ERR_CUDA;
    // ... and so must the two words of the sort's grid barrier, should an earlier call have given up inside it
    if (cudaMemsetAsync(tmp.sort_ctl, 0, 2 * sizeof(uint32_t), s) != cudaSuccess) return PS_ERR_CUDA;
    launch_prepare_keys(&tmp, d_keys, n, s);
    run_push_pipeline(&tmp, (uint32_t)n, d_updates, nullptr, 0, s);
    if (cudaGetLastError() != cudaSuccess) return PS_ERR_CUDA;
    unsigned int code = 0;
    if (cudaMemcpyAsync(&code, &tmp.status->sticky, sizeof code, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return PS_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return PS_ERR_CUDA;
    return (ps_status_t)code;
}
