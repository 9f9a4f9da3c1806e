// locmoe_capacity_noalloc: the capacity stage for callers that cannot hand over a workspace.
//
// Who needs this: a host program that embeds the router but owns no device allocator of its own --
// for example a plug-in running inside a serving process that has already reserved the whole HBM for
// its pools (a cudaMalloc there fails or fragments the pool), or a C caller that is only ever given the
// input and output buffers of an op and has no way to ask its framework for scratch.  Such a caller can
// still run the angular-deviation / capacity step: the per-expert minima that the ordinary entry point
// keeps in the caller's workspace live here in a fixed array inside the library's own device image.
//
// The price: the array has a fixed size (so the expert count is limited, see kNoAllocMaxExperts), every
// GPU that loads the library carries it until the process exits, and ALL calls on a device share it.
#include <mutex>

#include "common.cuh"

namespace locmoe {
namespace {

// Largest expert count the built-in scratch serves.  The capacity kernels need at most 8 rows of E
// 32-bit codes (one row per CTA of the cluster kernel), i.e. 8 * 8192 * 4 bytes = 256 KiB per GPU.
constexpr int kNoAllocMaxExperts = 8192;
constexpr size_t kNoAllocWords = (size_t)8 * kNoAllocMaxExperts;

// The scratch itself.  In HOST code this name is only a handle for the runtime, not a device address:
// it must never be passed to a kernel.  The device address is fetched with cudaGetSymbolAddress below.
static __device__ __align__(256) uint32_t g_noalloc_scratch[kNoAllocWords];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the scratch on the CURRENT device; looked up once per device and cached.  The cached
// address belongs to the device's primary context as it was at the first call: after cudaDeviceReset (or in
// a process that switches to another context on the same device) it is stale, and the entry point must not
// be used any more.
int scratch_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return LOCMOE_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return LOCMOE_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return LOCMOE_OK;
}

}  // namespace
}  // namespace locmoe

using namespace locmoe;

extern "C" int locmoe_capacity_noalloc(const locmoe_shape_t* shape, const int32_t* idx, const float* cos_sim,
                                       const locmoe_capacity_rule_t* rule, float* delta_e, float* theta_e,
                                       locmoe_capacity_t* cap_dev, void* stream) {
    if (!shape || !idx || !cos_sim || !rule || !delta_e || !theta_e || !cap_dev) return LOCMOE_ERR_NULL;
    if (shape->T < 1 || shape->H < 2 || shape->E < 1 || shape->n_nodes < 1 || shape->dev_per_node < 1)
        return LOCMOE_ERR_SHAPE;
    if (shape->H % shape->E != 0) return LOCMOE_ERR_SHAPE;
    const long long D = (long long)shape->n_nodes * shape->dev_per_node;
    if (D > shape->E || shape->E % D != 0) return LOCMOE_ERR_SHAPE;
    if (shape->E > kNoAllocMaxExperts) return LOCMOE_ERR_TOO_LARGE;  // beyond the built-in scratch
    if (rule->bound_form < LOCMOE_BOUND_BETA || rule->bound_form > LOCMOE_BOUND_EXP) return LOCMOE_ERR_DTYPE;
    if (rule->T_global < 0) return LOCMOE_ERR_SHAPE;
    if (!(rule->min_mult >= 0.0) || !(rule->capacity_factor >= 0.0) || rule->delta_override != rule->delta_override)
        return LOCMOE_ERR_SHAPE;
    if ((uintptr_t)cap_dev % 8) return LOCMOE_ERR_ALIGN;
    void* scratch = nullptr;
    int rc = scratch_address(&scratch);  // first call on this device: one-time look-up of the array's address
    if (rc) return rc;
    // Nothing in the scratch has to start at zero: the one-cluster kernel overwrites every row it later
    // reads, and the multi-kernel path re-initialises its E words with a memset node on the same stream.
    return launch_capacity(*shape, idx, cos_sim, *rule, delta_e, theta_e, cap_dev, scratch,
                           static_cast<cudaStream_t>(stream));
}
