// so_grad_check_static: the global gradient check for callers that cannot
// allocate device memory.
//
// The regular check (so_grad_check) keeps its tile sums in a scratch arena the
// caller allocates and binds.  Some callers have no allocator to ask: code that
// runs inside another framework's memory pool with nothing left in it, a
// library initialiser or a signal-safe diagnostic path where cudaMalloc (a
// device-wide synchronising call) is not acceptable, a plug-in that is handed
// raw pointers only.  For them this file carries its own scratch: one fixed
// array in device global memory that is part of the loaded library image on
// every GPU that uses it, until the process exits.  Nothing here calls
// cudaMalloc, cudaFree, or any routine that allocates (host or device).
#include "superoffload.h"

#include <cmath>
#include <mutex>

#include "so_types.h"

using namespace so;

namespace {

constexpr int64_t kStaticMaxElems = SO_STATIC_CHECK_MAX_ELEMS;
constexpr int64_t kStaticMaxTiles = (kStaticMaxElems + kTileElems - 1) / kTileElems;
constexpr int kMaxDevices = 64;

// The scratch itself: one double per 1024-element tile (512 KB).  In host code
// this name is only a handle for the runtime, not a device address -- a kernel
// given `g_tile_sums` directly would read host memory or fault -- so the host
// side asks the runtime for the real address once per device (below).
static __device__ __align__(256) double g_tile_sums[kStaticMaxTiles];

struct DeviceSetup {
    bool ready = false;
    double *tile_sums = nullptr;      // device address of g_tile_sums on this device
    int num_sms = 0;
    int occ_check = 0, occ_check_f32 = 0;
};

DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

// Fold the tile sums of one flat gradient (strided per-thread sums, then a
// shared-memory tree: for up to 4096 tiles, i.e. 4 Mi elements, this is the order
// in which the regular reduction folds a one-segment bucket, so the bits agree;
// beyond that the regular check folds per 4096-tile segment first and the two
// results are equal to rounding), then
// derive norm and clip coefficient on the device (IEEE sqrt and division are
// correctly rounded, so the values equal a host computation from the same sum)
// and write the result record to the caller's device buffer.
__global__ void __launch_bounds__(kReduceThreads)
static_check_finish_kernel(const double *tile_sums, uint32_t n_tiles, double max_grad_norm,
                           so_grad_stats *out)
{
    __shared__ double s_sum[kReduceThreads];
    __shared__ int s_bad[kReduceThreads];
    double acc = 0.0;
    int bad = 0;
    for (uint32_t i = threadIdx.x; i < n_tiles; i += kReduceThreads) {
        const double x = tile_sums[i];
        const uint32_t hi = (uint32_t)__double2hiint(x);
        bad |= ((hi & 0x7FF00000u) == 0x7FF00000u);
        acc = __dadd_rn(acc, x);
    }
    s_sum[threadIdx.x] = acc;
    s_bad[threadIdx.x] = bad;
    __syncthreads();
    for (int s = kReduceThreads / 2; s > 0; s >>= 1) {
        if ((int)threadIdx.x < s) {
            s_sum[threadIdx.x] = __dadd_rn(s_sum[threadIdx.x], s_sum[threadIdx.x + s]);
            s_bad[threadIdx.x] |= s_bad[threadIdx.x + s];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const double sumsq = s_sum[0];
        const double norm = __dsqrt_rn(sumsq);
        double coef = 1.0;
        if (max_grad_norm > 0.0) {
            const double c = __ddiv_rn(max_grad_norm, __dadd_rn(norm, 1e-6));
            coef = c < 1.0 ? c : 1.0;
        }
        out->sumsq = sumsq;
        out->norm = norm;
        out->clip_coef = coef;
        out->nonfinite = s_bad[0];
        out->reserved = 0;
    }
}

// Once per device, with that device current: resolve the device address of the
// static array and cache the launch geometry.  Allocates nothing.
so_status setup_device(int device, DeviceSetup **out)
{
    if (device < 0 || device >= kMaxDevices) return SO_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    DeviceSetup &d = g_setup[device];
    if (!d.ready) {
        double *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_tile_sums);
        if (e != cudaSuccess || ptr == nullptr) return SO_ERR_CUDA;
        e = cudaDeviceGetAttribute(&d.num_sms, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess) return SO_ERR_CUDA;
        e = grad_check_occupancy(SO_GRAD_BF16, &d.occ_check);
        if (e != cudaSuccess) return SO_ERR_CUDA;
        e = grad_check_occupancy(SO_GRAD_FP32, &d.occ_check_f32);
        if (e != cudaSuccess) return SO_ERR_CUDA;
        d.tile_sums = ptr;
        d.ready = true;
    }
    *out = &d;
    return SO_OK;
}

}  // namespace

extern "C" so_status so_grad_check_static(const void *grad, int64_t n_elems, int32_t grad_dtype,
                                          double max_grad_norm, void *stream,
                                          so_grad_stats *out_device)
{
    if (!out_device || n_elems < 0 || (n_elems > 0 && !grad)) return SO_ERR_INVALID_ARG;
    if (grad_dtype != SO_GRAD_BF16 && grad_dtype != SO_GRAD_FP32) return SO_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(grad) & 15u) != 0) return SO_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(out_device) & 7u) != 0) return SO_ERR_INVALID_ARG;
    if (!std::isfinite(max_grad_norm)) return SO_ERR_INVALID_ARG;
    if (n_elems > kStaticMaxElems) return SO_ERR_TOO_LARGE;

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return SO_ERR_CUDA;
    DeviceSetup *d = nullptr;
    const so_status s = setup_device(device, &d);
    if (s != SO_OK) return s;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint32_t n_tiles = (uint32_t)((n_elems + kTileElems - 1) / kTileElems);
    if (n_tiles > 0) {
        // one "bucket" that is the whole buffer; every tile sum the finish
        // kernel reads is written by this launch, so nothing left over from an
        // earlier call is ever read and nothing needs clearing
        CheckArgs a;
        a.grad = grad;
        a.partials = d->tile_sums;
        a.unscale[0] = a.unscale[1] = a.unscale[2] = 1.0;
        a.verdict = nullptr;
        a.pick = 0;
        a.geo.stride = 0;
        a.geo.tiles_per_slot = n_tiles;
        a.geo.bucket_elems = (uint32_t)n_elems;
        a.geo.last_elems = (uint32_t)n_elems;
        a.geo.last_bucket = 0;
        a.n_entries = 1;
        for (int i = 0; i < kMaxBatch; ++i) a.bucket[i] = 0;
        int64_t blocks = ((int64_t)n_tiles + kWarpsPerBlock - 1) / kWarpsPerBlock;
        const int occ = grad_dtype == SO_GRAD_BF16 ? d->occ_check : d->occ_check_f32;
        const int64_t cap = (int64_t)d->num_sms * (occ > 0 ? occ : 1);
        if (blocks > cap) blocks = cap;
        if (launch_grad_check(a, grad_dtype, (unsigned)blocks, st) != cudaSuccess) return SO_ERR_CUDA;
        if (cudaGetLastError() != cudaSuccess) return SO_ERR_CUDA;
    }
    static_check_finish_kernel<<<1, kReduceThreads, 0, st>>>(d->tile_sums, n_tiles, max_grad_norm,
                                                            out_device);
    if (cudaGetLastError() != cudaSuccess) return SO_ERR_CUDA;
    return SO_OK;
}
