// Library-level entry points and the cached device check shared by all segments.
#include "kop_common.cuh"

namespace kop {
namespace {

constexpr int kMaxDevices = 64;
// 0 = not probed, 1 = supported, -1 = unsupported. Benign race: every writer stores the same value.
int g_device_state[kMaxDevices];
int g_sm_count[kMaxDevices];

}  // namespace

kop_status_t check_device()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return KOP_ERR_CUDA;
    }
    if (dev < 0 || dev >= kMaxDevices) return KOP_ERR_UNSUPPORTED_DEVICE;
    if (g_device_state[dev] == 0) {
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            (void)cudaGetLastError();
            return KOP_ERR_CUDA;
        }
        g_sm_count[dev] = sms;
        g_device_state[dev] = (major == 10) ? 1 : -1;     // the binary holds sm_100a code only
    }
    return g_device_state[dev] == 1 ? KOP_OK : KOP_ERR_UNSUPPORTED_DEVICE;
}

int sm_count()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices || g_sm_count[dev] <= 0)
        return 148;
    return g_sm_count[dev];
}

}  // namespace kop

extern "C" int kop_version(void) { return 100; /* 0.1.0 */ }

extern "C" const char* kop_status_string(kop_status_t status)
{
    switch (status) {
    case KOP_OK: return "KOP_OK";
    case KOP_ERR_NULL_POINTER: return "KOP_ERR_NULL_POINTER";
    case KOP_ERR_BAD_SHAPE: return "KOP_ERR_BAD_SHAPE";
    case KOP_ERR_BAD_STRIDE: return "KOP_ERR_BAD_STRIDE";
    case KOP_ERR_UNSUPPORTED_DTYPE: return "KOP_ERR_UNSUPPORTED_DTYPE";
    case KOP_ERR_MISALIGNED: return "KOP_ERR_MISALIGNED";
    case KOP_ERR_BAD_ALIAS: return "KOP_ERR_BAD_ALIAS";
    case KOP_ERR_WORKSPACE_TOO_SMALL: return "KOP_ERR_WORKSPACE_TOO_SMALL";
    case KOP_ERR_UNSUPPORTED_DEVICE: return "KOP_ERR_UNSUPPORTED_DEVICE";
    case KOP_ERR_CUDA: return "KOP_ERR_CUDA";
    case KOP_ERR_CUBLAS: return "KOP_ERR_CUBLAS";
    }
    return "KOP_ERR_UNKNOWN";
}
