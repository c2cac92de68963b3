// parle_softmax_ce_static: the softmax cross-entropy backward + per-replica mean
// loss of the inner step, for callers that cannot provide (or allocate) a
// scratch buffer.  The per-row losses live in a fixed array inside the library
// image instead of the caller's workspace.
#include <mutex>

#include <math.h>

#include "common.cuh"

using namespace parle;

namespace {

constexpr int kFlagBytes = 256;                         // status slots, cleared at every call
constexpr size_t kScratchBytes = kFlagBytes + (size_t)PARLE_STATIC_LOSS_MAX_ROWS * sizeof(float);

// One copy per GPU that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

// Row-wise softmax cross-entropy backward, one warp per row (same arithmetic as
// the inner step's kernel): dlogits = (softmax - onehot)/B, row loss into the
// static array, whose device address the host passes in as `scratch`.
__global__ void __launch_bounds__(256)
softmax_ce_static_kernel(const float *__restrict__ logits, const int32_t *__restrict__ labels,
                         float *__restrict__ dlogits, int rows, int B, int C, unsigned char *scratch) {
    const int row = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
    const int lane = threadIdx.x % 32;
    if (row >= rows) return;
    int *slots = reinterpret_cast<int *>(scratch);
    float *row_loss = reinterpret_cast<float *>(scratch + kFlagBytes);
    const float *lg = logits + (size_t)row * C;
    float mx = -INFINITY;
    for (int j = lane; j < C; j += 32) mx = fmaxf(mx, lg[j]);
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float s = 0.f;
    for (int j = lane; j < C; j += 32) s += __expf(lg[j] - mx);
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const int label = labels[row];
    const bool label_ok = (label >= 0 && label < C);
    const float inv_s = 1.f / s, inv_B = 1.f / (float)B;
    for (int j = lane; j < C; j += 32) {
        float d = __expf(lg[j] - mx) * inv_s;
        if (j == label) d -= 1.f;
        dlogits[(size_t)row * C + j] = d * inv_B;
    }
    if (lane == 0) {
        row_loss[row] = label_ok ? (mx + __logf(s) - lg[label]) : 0.f;
        if (!label_ok) slots[SLOT_BAD_LABEL] = 1;
    }
}

// loss[g] = mean of replica g's row losses; one block per replica, fixed-order tree.
__global__ void __launch_bounds__(256)
loss_mean_static_kernel(float *__restrict__ loss, int B, const unsigned char *scratch) {
    __shared__ float sh[256];
    const float *row_loss = reinterpret_cast<const float *>(scratch + kFlagBytes);
    const int g = blockIdx.x;
    float s = 0.f;
    for (int i = threadIdx.x; i < B; i += 256) s += row_loss[(size_t)g * B + i];
    sh[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) loss[g] = sh[0] / (float)B;
}

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void *g_scratch_addr[kMaxDevices] = {};                 // device address of g_static_scratch, per device

// In host code `g_static_scratch` is only a handle for the symbol; the address a
// kernel can use has to be asked for, once per device, with that device current.
int scratch_for_current_device(unsigned char **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PARLE_ECUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return PARLE_ECUDA;
        g_scratch_addr[dev] = p;
    }
    *out = static_cast<unsigned char *>(g_scratch_addr[dev]);
    return PARLE_OK;
}

}  // namespace

extern "C" int parle_softmax_ce_static(const float *logits, const int32_t *labels, int n, int B, int C,
                                       float *dlogits, float *loss, int32_t *flags, void *cuda_stream) {
    if (!logits || !labels || !dlogits || !loss || n < 1 || B < 1 || C < 1) return PARLE_EINVAL;
    const long long rows = (long long)n * B;
    if (rows > PARLE_STATIC_LOSS_MAX_ROWS) return PARLE_ETOOBIG;
    unsigned char *scratch = nullptr;
    int rc = scratch_for_current_device(&scratch);
    if (rc != PARLE_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int *slots = reinterpret_cast<int *>(scratch);
    // the flag slots must start at zero; the row losses in use are fully overwritten below
    if (cudaMemsetAsync(slots, 0, kFlagBytes, stream) != cudaSuccess) return PARLE_ECUDA;
    softmax_ce_static_kernel<<<((int)rows + 7) / 8, 256, 0, stream>>>(logits, labels, dlogits, (int)rows, B, C, scratch);
    if (cudaGetLastError() != cudaSuccess) return PARLE_ECUDA;
    loss_mean_static_kernel<<<n, 256, 0, stream>>>(loss, B, scratch);
    if (cudaGetLastError() != cudaSuccess) return PARLE_ECUDA;
    if (flags) {
        // SLOT_BAD_LABEL holds 0/1; report it as the PARLE_FLAG_BAD_LABEL bit would be (0 or non-zero)
        if (cudaMemcpyAsync(flags, slots + SLOT_BAD_LABEL, sizeof(int32_t), cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
            return PARLE_ECUDA;
    }
    return PARLE_OK;
}
