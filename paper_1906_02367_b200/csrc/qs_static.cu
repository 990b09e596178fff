// Master update without any allocation: a context-free variant of the decode step.
//
// qs_unpack_accumulate keeps one word per coordinate ("which workers sent this index") in
// scratch that qs_init allocates.  Some callers cannot allocate at all: code that runs where
// cudaMalloc is forbidden or would stall everyone (inside a latency-critical serving loop, in a
// process whose device memory is handed out once at start-up by another component, or under a
// memory budget that is already spent when the library is first called).  For them this file
// keeps that scratch in a fixed array that is part of the library image, so every GPU that loads
// the library carries it (4 MiB) until the process exits, and the entry point only launches
// kernels and one memset.
//
// The array is shared by every call on a device and keeps what the last call left in it, so each
// call clears the part it uses first, and two calls that overlap on the same GPU (different
// streams or threads) would race on it: run them one after another.
#include <cmath>
#include <mutex>

#include "qs_common.cuh"

namespace {

constexpr long long STATIC_MAX_D = QS_STATIC_MAX_D;   // coordinates the fixed scratch can cover
constexpr int MAX_DEVICES = 64;

// one word per coordinate: bit r set = worker r sent this index in the call being decoded
static __device__ __align__(256) uint32_t g_senders[STATIC_MAX_D];

struct StaticArgs {
    int R, s, quantizer, bl, bi;
    uint32_t d, k, active;          // active: bit mask of the workers taking part
    float cscale;
    float* x;
    const uint32_t* wire;
    long long stride;
    uint32_t* senders;              // device address of g_senders
};

__device__ __forceinline__ uint32_t field(const uint32_t* w, uint64_t bitpos, uint32_t width) {
    const uint64_t q = bitpos >> 5;
    const uint32_t o = (uint32_t)(bitpos & 31u);
    uint32_t v = w[q] >> o;
    if (o + width > 32u) v |= w[q + 1] << (32u - o);
    return width >= 32u ? v : (v & ((1u << width) - 1u));
}

__device__ __forceinline__ uint32_t stream_words(uint32_t n, uint32_t width) {
    return (uint32_t)(((uint64_t)n * width + 31u) >> 5);
}

// entries a worker's record holds; a count above k is not a record of this operator: ignore it
__device__ __forceinline__ uint32_t record_entries(const StaticArgs& a, const uint32_t* row) {
    const uint32_t n = row[0];
    return n <= a.k ? n : 0u;
}

__device__ __forceinline__ float record_value(const StaticArgs& a, const uint32_t* row, uint32_t n, uint32_t j) {
    const uint32_t* w_sgn = row + 2 + stream_words(n, a.bi);
    const uint32_t* w_lvl = w_sgn + stream_words(n, 1);
    const bool neg = (w_sgn[j >> 5] >> (j & 31u)) & 1u;
    const float N = __uint_as_float(row[1]);
    float g;
    if (qs::qz_is_sign(a.quantizer)) {
        g = N / (float)a.k;
    } else {
        const int level = (int)field(w_lvl, (uint64_t)j * a.bl, a.bl) + 1;
        g = (N * (float)level) / (float)a.s;
        if (a.quantizer == QS_QSGD_SCALED) g = g * a.cscale;
    }
    return neg ? -g : g;
}

__global__ void __launch_bounds__(256) static_mark_kernel(const StaticArgs a) {
    const uint64_t total = (uint64_t)a.R * a.k;
    for (uint64_t id = (uint64_t)blockIdx.x * 256u + threadIdx.x; id < total; id += (uint64_t)gridDim.x * 256u) {
        const uint32_t r = (uint32_t)(id / a.k), j = (uint32_t)(id % a.k);
        if (!((a.active >> r) & 1u)) continue;
        const uint32_t* row = a.wire + (size_t)r * a.stride;
        if (j >= record_entries(a, row)) continue;
        const uint32_t i = field(row + 2, (uint64_t)j * a.bi, a.bi);
        if (i < a.d) atomicOr(&a.senders[i], 1u << r);
    }
}

// the lowest worker that sent an index adds the values of all its senders in increasing worker
// order, updates x and clears the word again
__global__ void __launch_bounds__(256) static_apply_kernel(const StaticArgs a) {
    const uint64_t total = (uint64_t)a.R * a.k;
    for (uint64_t id = (uint64_t)blockIdx.x * 256u + threadIdx.x; id < total; id += (uint64_t)gridDim.x * 256u) {
        const uint32_t r = (uint32_t)(id / a.k), j = (uint32_t)(id % a.k);
        if (!((a.active >> r) & 1u)) continue;
        const uint32_t* row = a.wire + (size_t)r * a.stride;
        const uint32_t n = record_entries(a, row);
        if (j >= n) continue;
        const uint32_t i = field(row + 2, (uint64_t)j * a.bi, a.bi);
        if (i >= a.d) continue;
        const uint32_t senders = a.senders[i];
        if (!senders || (uint32_t)(__ffs(senders) - 1) != r) continue;
        float acc = 0.0f;
        acc = acc + record_value(a, row, n, j);
        uint32_t rest = senders & (senders - 1u);
        while (rest) {
            const uint32_t r2 = (uint32_t)(__ffs(rest) - 1);
            rest &= rest - 1u;
            const uint32_t* row2 = a.wire + (size_t)r2 * a.stride;
            const uint32_t n2 = record_entries(a, row2);
            uint32_t lo = 0, hi = n2;             // first position whose index is not below i
            while (lo < hi) {
                const uint32_t mid = (lo + hi) >> 1;
                if (field(row2 + 2, (uint64_t)mid * a.bi, a.bi) < i) lo = mid + 1; else hi = mid;
            }
            if (lo < n2) acc = acc + record_value(a, row2, n2, lo);
        }
        a.x[i] = a.x[i] - acc / (float)a.R;
        a.senders[i] = 0u;
    }
}

int ceil_log2_host(unsigned long long v) {
    int b = 0;
    while ((1ull << b) < v) ++b;
    return b;
}

// device address of g_senders, looked up once per device
std::mutex g_lock;
uint32_t* g_addr[MAX_DEVICES] = {nullptr};

int scratch_address(uint32_t** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return QS_CUDA;
    std::lock_guard<std::mutex> hold(g_lock);
    if (!g_addr[dev]) {
        // In host code the name g_senders is only a handle for the runtime, not a device
        // pointer: the address a kernel can use has to be asked for, on the device it lives on.
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_senders) != cudaSuccess || !p) {
            cudaGetLastError();
            return QS_CUDA;
        }
        g_addr[dev] = static_cast<uint32_t*>(p);
    }
    *out = g_addr[dev];
    return QS_OK;
}

}  // namespace

extern "C" {

int qs_unpack_accumulate_static(int R, int64_t d, int64_t k, int s, int quantizer, float* x, const uint32_t* wire,
                                int64_t stride_words, const uint8_t* worker_mask, void* cuda_stream) {
    if (d > STATIC_MAX_D) return QS_TOO_LARGE;
    if (R < 1 || R > qs::MAX_R || d < 1 || k < 1 || k > d || s < 1 || s > 65535 || !x || !wire) return QS_INVALID_ARG;
    if (quantizer != QS_QSGD && quantizer != QS_QSGD_SCALED && quantizer != QS_SIGN_L1 && quantizer != QS_SIGN_L2) return QS_INVALID_ARG;
    StaticArgs a;
    a.R = R; a.s = s; a.quantizer = quantizer;
    a.d = (uint32_t)d; a.k = (uint32_t)k;
    a.bl = ceil_log2_host((unsigned long long)s) < 1 ? 1 : ceil_log2_host((unsigned long long)s);
    a.bi = ceil_log2_host((unsigned long long)d) < 1 ? 1 : ceil_log2_host((unsigned long long)d);
    const long long need = 2 + (long long)qs::words_for(a.k, a.bi) + qs::words_for(a.k, 1) +
                           (!qs::qz_is_sign(quantizer) ? (long long)qs::words_for(a.k, a.bl) : 0);
    if (stride_words < need) return QS_CAPACITY;
    const double b1 = (double)k / ((double)s * (double)s), b2 = std::sqrt((double)k) / (double)s;
    a.cscale = (float)(1.0 / (1.0 + (b1 < b2 ? b1 : b2)));
    a.active = 0;
    for (int r = 0; r < R; ++r)
        if (!worker_mask || worker_mask[r]) a.active |= 1u << r;
    a.x = x; a.wire = wire; a.stride = stride_words;
    const int rc = scratch_address(&a.senders);
    if (rc != QS_OK) return rc;
    if (!a.active) return QS_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // the array keeps whatever the previous call (or an interrupted one) left: start from zero
    if (cudaMemsetAsync(a.senders, 0, sizeof(uint32_t) * (size_t)d, st) != cudaSuccess) { cudaGetLastError(); return QS_CUDA; }
    const unsigned long long total = (unsigned long long)R * (unsigned long long)k;
    const int grid = (int)((total + 255) / 256 < 4096 ? (total + 255) / 256 : 4096);
    static_mark_kernel<<<grid, 256, 0, st>>>(a);
    static_apply_kernel<<<grid, 256, 0, st>>>(a);
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return QS_CUDA; }
    return QS_OK;
}

}  // extern "C"
