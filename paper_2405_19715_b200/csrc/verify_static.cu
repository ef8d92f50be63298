// specdec_verify_correct_static: verify/correct for callers that must not allocate.
//
// Some users of this library run where cudaMalloc is off limits: inside a serving loop that
// has handed all device memory to its own pool, in a plugin whose host forbids driver
// allocations after start-up, or in a latency-critical path where an allocation's implicit
// synchronisation is unacceptable.  Creating a specdec_ctx allocates, so this entry point
// takes no context.  Its scratch (accept flags, per-position draws, per-row arrival counters
// and a status word) lives in one fixed array in the library's device image instead.
#include <cstdarg>
#include <cstdio>
#include <mutex>

#include "verify_unit.cuh"

namespace {

using namespace sd;

constexpr int STATIC_MAX_UNITS = SPECDEC_STATIC_MAX_UNITS;     // B * (K + 1) of one call
constexpr size_t OFF_FLAGS = 0;
constexpr size_t OFF_DRAWS = OFF_FLAGS + sizeof(int32_t) * STATIC_MAX_UNITS;
constexpr size_t OFF_MASS = OFF_DRAWS + sizeof(int32_t) * STATIC_MAX_UNITS;
constexpr size_t OFF_ARRIVE = OFF_MASS + sizeof(float) * STATIC_MAX_UNITS;
constexpr size_t OFF_STATUS = OFF_ARRIVE + sizeof(int32_t) * STATIC_MAX_UNITS;
constexpr size_t SCRATCH_BYTES = OFF_STATUS + 256;

// Lives in every GPU that loads the library, from load until the process exits (about 256 KB).
// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
std::mutex g_mutex;
unsigned char* g_scratch_addr[MAX_DEVICES] = {};     // device address of the array, per device
uint32_t g_epoch[MAX_DEVICES] = {};

constexpr int STATIC_THREADS = 512;

// The unit body of the one-CTA-per-unit kernel, with the fixed array as its scratch.
template <typename T, bool VEC>
__global__ void __launch_bounds__(STATIC_THREADS, 2) verify_static_kernel(const VerifyParams P) {
    extern __shared__ float slab_sum[];
    __shared__ UnitShared sh;
    direct_unit<T, VEC, STATIC_THREADS>(P, slab_sum, sh);
}

int report(char* err, size_t err_len, int code, const char* fmt, ...) {
    if (err && err_len) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(err, err_len, fmt, ap);
        va_end(ap);
    }
    return code;
}

template <typename T>
cudaError_t launch_static(const VerifyParams& p, cudaStream_t s) {
    constexpr int N = Elem<T>::EPV;
    const int nslab = ((p.V + N - 1) / N + 31) / 32;
    const size_t smem = (size_t)nslab * sizeof(float);
    const bool vec = (p.V % N == 0) && (reinterpret_cast<uintptr_t>(p.target) % 16 == 0) &&
                     (reinterpret_cast<uintptr_t>(p.draft) % 16 == 0);
    auto kern = vec ? verify_static_kernel<T, true> : verify_static_kernel<T, false>;
    kern<<<p.B * (p.K + 1), STATIC_THREADS, smem, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

extern "C" int specdec_verify_correct_static(const void* target_logits, const void* draft_logits,
                                             specdec_dtype dtype, const int32_t* cand_tokens,
                                             const int32_t* cand_len, const float* uniforms, float temperature,
                                             int B, int K, int V, int32_t* n_accepted, int32_t* next_token,
                                             uint32_t* data_status, void* stream, char* err, size_t err_len) {
    if (!target_logits || !draft_logits || !cand_tokens || !uniforms || !n_accepted || !next_token)
        return report(err, err_len, SPECDEC_EINVAL, "verify_correct_static: null pointer argument");
    if (dtype != SPECDEC_F32 && dtype != SPECDEC_BF16)
        return report(err, err_len, SPECDEC_EINVAL, "verify_correct_static: unknown dtype %d", (int)dtype);
    if (reinterpret_cast<uintptr_t>(target_logits) % 4 != 0 || reinterpret_cast<uintptr_t>(draft_logits) % 4 != 0)
        return report(err, err_len, SPECDEC_EINVAL, "verify_correct_static: logit tensors must be 4-byte aligned");
    if (B < 1 || K < 1 || V < 1)
        return report(err, err_len, SPECDEC_EINVAL, "verify_correct_static: B, K, V must be >= 1");
    if (!(temperature > 0.f) || temperature > 3.0e38f)
        return report(err, err_len, SPECDEC_EINVAL, "verify_correct_static: temperature must be positive and finite");
    if ((long long)B * (K + 1) > STATIC_MAX_UNITS)
        return report(err, err_len, SPECDEC_EUNSUPPORTED,
                      "verify_correct_static: B*(K+1) = %lld exceeds the fixed scratch of %d (row, position) units; "
                      "use specdec_verify_correct with a context for larger batches",
                      (long long)B * (K + 1), STATIC_MAX_UNITS);
    if (V > SPECDEC_STATIC_MAX_V)
        return report(err, err_len, SPECDEC_EUNSUPPORTED, "verify_correct_static: V = %d exceeds %d", V,
                      SPECDEC_STATIC_MAX_V);
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= MAX_DEVICES)
        return report(err, err_len, SPECDEC_ECUDA, "verify_correct_static: no usable current device (%s)",
                      cudaGetErrorString(e));
    unsigned char* base;
    uint32_t epoch;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!g_scratch_addr[dev]) {
            // First call on this device: resolve the array's device address (no allocation).
            void* p = nullptr;
            e = cudaGetSymbolAddress(&p, g_static_scratch);
            if (e != cudaSuccess)
                return report(err, err_len, SPECDEC_ECUDA, "verify_correct_static: cudaGetSymbolAddress: %s",
                              cudaGetErrorString(e));
            g_scratch_addr[dev] = static_cast<unsigned char*>(p);
        }
        base = g_scratch_addr[dev];
        g_epoch[dev] = (g_epoch[dev] + 1) & 0x3fffffffu;
        if (g_epoch[dev] == 0) g_epoch[dev] = 1;
        epoch = g_epoch[dev];
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The array keeps the previous call's contents.  Arrival counters must start at zero; accept
    // flags carry the call's epoch, so stale ones read as "unknown" -- except after the 30-bit
    // epoch wraps, when they are cleared too.  Draws are written before they are read.
    e = cudaMemsetAsync(base + OFF_ARRIVE, 0, sizeof(int32_t) * (size_t)B, s);
    if (e == cudaSuccess && epoch == 1) e = cudaMemsetAsync(base + OFF_FLAGS, 0, sizeof(int32_t) * STATIC_MAX_UNITS, s);
    if (e != cudaSuccess)
        return report(err, err_len, SPECDEC_ECUDA, "verify_correct_static: cudaMemsetAsync: %s", cudaGetErrorString(e));
    VerifyParams p;
    p.target = target_logits;
    p.draft = draft_logits;
    p.tokens = cand_tokens;
    p.lens = cand_len;
    p.uniforms = uniforms;
    p.c = (float)(1.4426950408889634 / (double)temperature);
    p.B = B;
    p.K = K;
    p.V = V;
    p.n_acc = n_accepted;
    p.next = next_token;
    p.ratio = nullptr;
    p.stats = nullptr;
    p.rmass = nullptr;
    p.flags = reinterpret_cast<int32_t*>(base + OFF_FLAGS);
    p.draws = reinterpret_cast<int32_t*>(base + OFF_DRAWS);
    p.draw_mass = reinterpret_cast<float*>(base + OFF_MASS);
    p.arrive = reinterpret_cast<int32_t*>(base + OFF_ARRIVE);
    p.status = data_status ? data_status : reinterpret_cast<uint32_t*>(base + OFF_STATUS);
    p.norms = nullptr;
    p.tasks = nullptr;
    p.task_ctl = nullptr;
    p.task_ready = nullptr;
    p.epoch = epoch;
    e = dtype == SPECDEC_BF16 ? launch_static<__nv_bfloat16>(p, s) : launch_static<float>(p, s);
    if (e != cudaSuccess)
        return report(err, err_len, SPECDEC_ECUDA, "verify_correct_static: launch: %s", cudaGetErrorString(e));
    return SPECDEC_OK;
}
