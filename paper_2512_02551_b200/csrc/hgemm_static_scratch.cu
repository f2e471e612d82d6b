// hgemm_run_splitk_static: the split-K GEMM with its scratch memory built into the library.
//
// Some callers may not allocate device memory at all once they are running: code that executes
// inside a memory-frozen serving process, inside another library's callback, or under a
// fixed-footprint policy where every byte of HBM was handed out at start-up.  hgemm_plan needs
// cudaMalloc for the split-K workspace, so those callers could never use split-K.  This entry point
// gives them the same kernel with the workspace, the arrival counters and the status word placed in
// one file-scope __device__ array: no context, no plan, and no call to cudaMalloc, cudaFree or any
// other allocating routine.  The array itself gets its memory when the CUDA runtime loads this
// file's module on a device -- with lazy module loading (CUDA's default) that is the first call of
// this entry point on that device, with CUDA_MODULE_LOADING=EAGER it is context creation.  A process
// whose memory is frozen later should therefore make one call per device (or load eagerly) before
// the freeze; every later call leaves the amount of free device memory unchanged.
//
// Cost and limits: every GPU that loads the library holds the array (kScratchBytes + one control
// page) until the process exits; a call whose partial sums need more than that is refused; all
// calls share the one array, so two calls that overlap on the GPU would corrupt each other.
// Every system header that hgemm_kernel.cuh and ptx_sm100.cuh include is included here first, at
// global scope: the kernel header is pulled in inside an anonymous namespace below, and a system
// header first seen there would declare its names (std:: among them) inside that namespace.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>
#include <cstring>
#include <mutex>
#include <type_traits>

#include "../../include/hgemm.h"
#include "hgemm_planner.h"

// This translation unit compiles its own, internal-linkage copy of the one kernel instantiation it
// launches (the library's other copy lives in hgemm_api.cu).  The kernel does not need it -- it
// receives the scratch address through its parameters like any workspace -- but it keeps this entry
// point self-contained: the array, the code that resolves its device address and the launch that
// uses it sit in one file, and nothing in the plan-based code path changed when it was added.  The
// price is a second compile of that instantiation and a duplicate of it in the binary.
namespace {
#include "hgemm_kernel.cuh"
} // namespace

namespace {

constexpr size_t kScratchBytes = size_t(8) << 20;   // fp32 partial sums: 8 MiB
constexpr size_t kControlBytes = 4096;              // arrival counters (2 x uint32 per tile) + status word
constexpr int kMaxDevices = 64;
constexpr size_t kStatusOffset = kControlBytes - 256;   // the status word sits at the end of the control page

// In host code this name is only a handle for cudaGetSymbolAddress; the device address it stands
// for is looked up once per device below.  Layout: [control page | partial sums].
static __device__ __align__(256) unsigned char g_static_scratch[kControlBytes + kScratchBytes];

typedef CUresult (*encode_tiled_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct DeviceState {
    bool ready = false;
    unsigned char *scratch = nullptr;   // device address of g_static_scratch on this device
    int num_sms = 0;
    encode_tiled_fn encode = nullptr;
};
DeviceState g_devices[kMaxDevices];     // fixed table: no heap allocation on any path
std::mutex g_setup_mutex;               // first calls from several threads fill the table one at a time

// Once per device, with that device current: resolve the array's device address, read the SM
// count, fetch the tensor-map encoder, raise the kernel's shared-memory limit.  None of these
// allocates device memory.
hgemm_status_t setup_device(int device, DeviceState **out)
{
    if (device < 0 || device >= kMaxDevices) return HGEMM_ERR_INVALID_ARG;
    DeviceState &d = g_devices[device];
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!d.ready) {
        int major = 0, minor = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
            cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, device) != cudaSuccess) {
            (void)cudaGetLastError();
            return HGEMM_ERR_CUDA;
        }
        if (major != 10 || minor != 0) return HGEMM_ERR_ARCH;
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || ptr == nullptr) {
            (void)cudaGetLastError();
            return HGEMM_ERR_CUDA;
        }
        if (cudaDeviceGetAttribute(&d.num_sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
            (void)cudaGetLastError();
            return HGEMM_ERR_CUDA;
        }
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || fn == nullptr) {
            (void)cudaGetLastError();
            return HGEMM_ERR_CUDA;
        }
        e = cudaFuncSetAttribute(hgemm_dev::hgemm_umma_kernel<1, false, 1, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 int(hgemm_host::kSmemOptInBytes));
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            return HGEMM_ERR_CUDA;
        }
        d.scratch = static_cast<unsigned char *>(ptr);
        d.encode = reinterpret_cast<encode_tiled_fn>(fn);
        d.ready = true;
    }
    *out = &d;
    return HGEMM_OK;
}

bool encode_2d(const DeviceState &d, CUtensorMap *map, const void *base, uint64_t inner, uint64_t outer, uint32_t box_inner,
               uint32_t box_outer, CUtensorMapSwizzle swizzle)
{
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {inner * 2};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    return d.encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

} // namespace

extern "C" hgemm_status_t hgemm_run_splitk_static(int64_t M, int64_t N, int64_t K, int32_t block_n, int32_t split_k,
                                                  const void *A, const void *B, void *C, void *stream)
{
    if (!A || !B || !C) return HGEMM_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B) | reinterpret_cast<uintptr_t>(C)) & 15u)
        return HGEMM_ERR_INVALID_ARG;

    // the fixed configuration of this variant: 1-CTA family, 64-wide K stages, workspace split-K
    hgemm_config_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cfg.family = HGEMM_FAMILY_UMMA_1CTA;
    cfg.block_m = 128;
    cfg.block_n = block_n;
    cfg.block_k = 64;
    cfg.split_k = split_k;
    cfg.split_mode = HGEMM_SPLIT_WORKSPACE;
    cfg.raster_group = 1;
    cfg.epilogue = HGEMM_EPILOGUE_DIRECT;
    cfg.stages = 1;
    if (block_n >= 32 && block_n <= 256 && block_n % 32 == 0)
        cfg.stages = std::max(1, std::min(6, hgemm_host::max_stages(cfg.family, block_n, cfg.block_k)));
    hgemm_status_t st = hgemm_host::validate_shape_aligned(M, N, K);   // no padded copies here: nothing may be allocated
    if (st != HGEMM_OK) return st;
    st = hgemm_host::validate(M, N, K, cfg);
    if (st != HGEMM_OK) return st;

    // the size check comes before anything touches the GPU
    const int64_t tiles = ((M + 127) / 128) * ((N + block_n - 1) / block_n);
    const int64_t partial_bytes = split_k > 1 ? hgemm_host::workspace_bytes(M, N, K, cfg) : 0;
    const int64_t counter_bytes = split_k > 1 ? hgemm_host::counter_bytes(M, N, cfg) : 0;
    if (partial_bytes > int64_t(kScratchBytes) || counter_bytes > int64_t(kStatusOffset)) return HGEMM_ERR_SCRATCH_LIMIT;

    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess) {
        (void)cudaGetLastError();
        return HGEMM_ERR_CUDA;
    }
    DeviceState *d = nullptr;
    st = setup_device(device, &d);
    if (st != HGEMM_OK) return st;
    if (split_k > 1 && split_k > d->num_sms) return HGEMM_ERR_UNSUPPORTED;   // the slices of a tile must be co-resident

    CUtensorMap tmap_a, tmap_b, tmap_c;
    if (!encode_2d(*d, &tmap_a, A, uint64_t(K), uint64_t(M), 64, 128, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !encode_2d(*d, &tmap_b, B, uint64_t(K), uint64_t(N), 64, uint32_t(block_n), CU_TENSOR_MAP_SWIZZLE_128B) ||
        !encode_2d(*d, &tmap_c, C, uint64_t(N), uint64_t(M), 32, 32, CU_TENSOR_MAP_SWIZZLE_64B))
        return HGEMM_ERR_CUDA;

    // The array keeps whatever the last call left.  The partial sums need no clearing (every slot
    // that is read is written first); the counters and the status word must start at zero.  Without
    // K slices the kernel touches neither, and the array is left alone.
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (split_k > 1 && cudaMemsetAsync(d->scratch, 0, kControlBytes, s) != cudaSuccess) {
        (void)cudaGetLastError();
        return HGEMM_ERR_CUDA;
    }

    hgemm_dev::KernelParams p;
    std::memset(&p, 0, sizeof(p));
    p.M = int32_t(M);
    p.N = int32_t(N);
    p.K = int32_t(K);
    p.tiles_m = int32_t((M + 127) / 128);
    p.tiles_n = int32_t((N + block_n - 1) / block_n);
    p.split_k = split_k;
    p.first_split_tile = split_k > 1 ? 0 : int32_t(tiles);
    p.total_work = int32_t(tiles) * split_k;
    p.block_k = 64;
    p.kblocks = int32_t((K + 63) / 64);
    p.block_n = block_n;
    p.stages = cfg.stages;
    p.raster_group = 1;
    p.fd_per_group = hgemm_dev::make_fast_div(uint32_t(p.tiles_n));
    p.fd_raster = hgemm_dev::make_fast_div(1u);
    p.fd_last_group = hgemm_dev::make_fast_div(1u);
    p.fd_split = hgemm_dev::make_fast_div(uint32_t(std::max(1, split_k)));
    p.fd_pieces = hgemm_dev::make_fast_div(1u);
    int32_t cols = 32;
    while (cols < 2 * block_n) cols <<= 1;
    p.tmem_cols = cols;
    p.epilogue_tma = 0;
    p.cluster_split = 0;
    p.idesc = (1u << 4) | (uint32_t(block_n >> 3) << 17) | (uint32_t(128 >> 4) << 24);   // fp32 accumulate, fp16 A/B, K-major
    p.idesc_tail = p.idesc;
    p.workspace = reinterpret_cast<float *>(d->scratch + kControlBytes);
    p.workspace_floats = static_cast<unsigned long long>(kScratchBytes / 4);
    p.counter_words = static_cast<unsigned long long>(kStatusOffset / 4);
    p.counters = reinterpret_cast<uint32_t *>(d->scratch);
    p.status = reinterpret_cast<uint32_t *>(d->scratch + kStatusOffset);
    p.C = static_cast<__half *>(C);
    p.wait_budget = 2000000000LL;
    p.trace = nullptr;
    p.debug_skip = 0;
    p.tail_pieces = 1;
    p.acc_f16 = 0;
    p.scaled = 0;
    p.alpha = 1.0f;
    p.beta = 0.0f;
    p.epoch = 1;          // the control page was cleared just above: every call is the counters' first launch

    cudaLaunchConfig_t lc;
    std::memset(&lc, 0, sizeof(lc));
    lc.gridDim = dim3(unsigned(std::min<int64_t>(p.total_work, d->num_sms)), 1, 1);
    lc.blockDim = dim3(hgemm_dev::kThreads, 1, 1);
    lc.dynamicSmemBytes = size_t(hgemm_host::kSmemOptInBytes);
    lc.stream = s;
    cudaError_t e = cudaLaunchKernelEx(&lc, hgemm_dev::hgemm_umma_kernel<1, false, 1, false, false>, tmap_a, tmap_b, tmap_c, tmap_b, p);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return HGEMM_ERR_CUDA;
    }
    return HGEMM_OK;
}
