// sd_op_linear_static: the tensor-core linear operator for callers that must not allocate.
//
// The stream-K GEMM leaves split accumulators in a workspace that sd_op_linear takes from its
// caller.  Some callers cannot provide one: a plugin that runs inside another program's
// inference loop, or code that runs while device memory is fully handed out to a pool, gets
// input and output buffers and nothing else, and a cudaMalloc there would either fail or stall
// the whole device.  For them the workspace lives in the library image itself, in a file-scope
// device array of fixed size that every GPU loading the library holds until the process exits.
//
// The array's name is only a host-side handle; kernels must be given the device address, which
// cudaGetSymbolAddress returns for the device that is current at the time.  The address is
// looked up once per device, on the first call made with that device current.
#include <stdio.h>
#include <string.h>

#include <mutex>

#include "gemm_tc.h"

namespace {

static __device__ __align__(256) unsigned char g_linear_scratch[SD_STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
std::mutex g_mu;
void* g_scratch_addr[MAX_DEVICES];      // device address of g_linear_scratch on each device, once known

// Device address of the scratch array on the current device (nullptr on failure).
void* scratch_on_current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return nullptr;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_linear_scratch) != cudaSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        g_scratch_addr[dev] = p;
    }
    return g_scratch_addr[dev];
}

}  // namespace

extern "C" sd_status sd_op_linear_static(const void* x, const void* w, float* y, int rows, int n_out, int n_in,
                                         void* cuda_stream) {
    using namespace sd;
    if (!x || !w || !y || rows < 1 || n_out < 1 || n_in < 1) return SD_ERR_INVALID_ARG;
    if (!gemm_tc_supported(rows, n_out, n_in)) return SD_ERR_UNSUPPORTED;
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n_sm < 1)
        return SD_ERR_CUDA;
    const GemmGeom g = gemm_geometry(rows, n_out, n_in, n_sm);
    if (g.grid < 1) return SD_ERR_UNSUPPORTED;
    if (gemm_partials_bytes(g) > (size_t)SD_STATIC_SCRATCH_BYTES) {
        fprintf(stderr, "[sd] sd_op_linear_static: %d x %d x %d needs %zu bytes of scratch, the built-in array holds %d\n",
                rows, n_out, n_in, gemm_partials_bytes(g), (int)SD_STATIC_SCRATCH_BYTES);
        return SD_ERR_CAPACITY;
    }
    char* scratch = (char*)scratch_on_current_device();
    if (!scratch) return SD_ERR_CUDA;
    TensorMap tw, tx;
    if (!make_tensor_map_bf16(&tw, w, n_out, n_in, 128) || !make_tensor_map_bf16(&tx, x, rows, n_in, g.m_pad)) return SD_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // Every accumulator word that is read is written by this call's own GEMM first, so the array needs no clearing.
    Epilogue e;
    memset(&e, 0, sizeof(e));
    e.mode = EPI_PLAIN; e.y = y; e.n_out_rows = rows; e.row_stride = 1; e.row_offset = 0;
    if (launch_gemm_streamk(tw, tx, g, (float*)scratch, nullptr, nullptr, 0, st) != cudaSuccess ||
        launch_fused_step(g, e, (const float*)scratch, nullptr, nullptr, 1, st) != cudaSuccess)
        return SD_ERR_CUDA;
    return SD_OK;
}
