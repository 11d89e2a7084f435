// kvq_decode_static: the full-prefix read for callers that may not allocate device memory.
//
// kvq_decode creates two small device objects with cudaMalloc the first time a plan is used: the
// plan's status word and, for the tensor-core kernel, the [D, D] fp32 inverse-transform table.
// Some callers cannot afford that call at all: an inference server that handed every byte of HBM
// to its own pool at start-up (cudaMalloc then fails), a latency-critical decode loop (cudaMalloc
// synchronises the whole device), a plug-in that is only allowed to touch memory it was given.
// For them this file keeps the same two objects in one fixed block of device memory that is part
// of the library image, and runs the D = 128 fp16 tensor-core kernel on it (the dense 128 x 128 form; kvq_decode
// takes one radix-2 step out of it on plans without a rotation).
//
// The block is shared by every call on a device and keeps what the last call left in it:
//   - the table belongs to ONE plan at a time; a call with another plan rewrites it first, with a
//     small kernel on the caller's stream;
//   - a call made while its stream is being captured always records that rewrite in front of the
//     decode and leaves the host's note of "whose table is in the block" alone: what the block holds
//     when the graph is replayed is not known at capture time.  A replay rewrites the table without
//     the host seeing it, so once a call has been captured on a device every later call there,
//     captured or not, rewrites the table first (a 128-CTA kernel of a few microseconds);
//   - the status word is cleared on the caller's stream before every launch;
//   - two calls that overlap on the GPU (different streams, no ordering between them) race on the
//     block.  Serialise them, or use kvq_decode.
#include <mutex>

#include "kvq_internal.h"

namespace {

constexpr int kStaticMaxD = 128;                            // largest head dim the block has room for
constexpr int kTableFloats = kStaticMaxD * kStaticMaxD;     // 64 KiB of fp32 table
constexpr int kStatusFloats = 64;                           // 256 B: the status word and padding
constexpr int kScratchFloats = kTableFloats + kStatusFloats;

// 65,792 bytes in every GPU context that loads the library, held until the process exits.
// In host code this name is only a handle for cudaGetSymbolAddress, never an address to pass on.
static __device__ __align__(256) float kvq_static_scratch[kScratchFloats];

struct SignWords {
    uint32_t w[128];   // same packing as kvq_plan::sign_xor: bit 15 / bit 31 of word m = s_{2m} / s_{2m+1} negative
};

// table[n][c] = s_n M[c][n], M the real orthogonal DFT matrix of Eq. 1-2 (the same table kvq_decode
// builds on the host), evaluated in fp64 and rounded once to fp32.
__global__ void kvq_static_fill_kernel(float *table, int D, const __grid_constant__ SignWords signs)
{
    const int n = blockIdx.x, c = threadIdx.x, H = D / 2;
    if (n >= D || c >= D) return;
    const double rs = 1.0 / sqrt((double)D), r2 = sqrt(2.0 / (double)D);
    double m;
    if (c == 0) m = rs;
    else if (c == H) m = (n & 1) ? -rs : rs;
    else if (c < H) m = r2 * cospi(2.0 * (double)((c * n) % D) / (double)D);
    else m = -r2 * sinpi(2.0 * (double)(((c - H) * n) % D) / (double)D);
    const bool neg = (signs.w[n >> 1] >> ((n & 1) ? 31 : 15)) & 1u;
    table[n * D + c] = (float)(neg ? -m : m);
}

struct DeviceSlot {
    float *block = nullptr;   // device address of kvq_static_scratch on this device
    bool table_valid = false;
    bool replays_possible = false;   // a call was recorded into a graph: replays rewrite the table when the host is not looking
    int table_D = 0;
    uint64_t table_seed = 0;
};

DeviceSlot g_slots[kvq::kMaxDevices];
std::mutex g_mu;

bool misaligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

}  // namespace

extern "C" kvq_status_t kvq_decode_static(kvq_plan_t *plan, const uint8_t *packed, const void *scales, int64_t N,
                                          const float *lambda, int64_t n_lambda, int64_t rows_per_lambda, void *out,
                                          kvq_dtype_t dtype, uint32_t *status_word, void *cuda_stream)
{
    using namespace kvq;
    if (!plan || N < 0) return KVQ_ERR_INVALID_ARG;
    if (dtype != KVQ_F16 && dtype != KVQ_BF16) return KVQ_ERR_INVALID_ARG;
    if (plan->D > kStaticMaxD) return KVQ_ERR_SCRATCH_LIMIT;                 // the table would not fit the block
    if (plan->D != 128 || dtype != KVQ_F16 || plan->group != 32 || plan->bits != 4 || plan->rot)
        return KVQ_ERR_UNSUPPORTED_DIM;   // the kernel behind it: D = 128, fp16, groups of 32, 4-bit codes, no rotation
    if (N == 0) return KVQ_OK;
    if (N >= ((int64_t)1 << 31)) return KVQ_ERR_INVALID_ARG;   // the kernel addresses rows through 32-bit tensor-map coordinates
    if (!packed || !scales || !out || !lambda || n_lambda < 1) return KVQ_ERR_INVALID_ARG;
    if (n_lambda > 1) {
        if (rows_per_lambda < 1) return KVQ_ERR_INVALID_ARG;
        if ((N + rows_per_lambda - 1) / rows_per_lambda > n_lambda) return KVQ_ERR_INVALID_ARG;
    }
    if (misaligned16(packed) || misaligned16(scales) || misaligned16(out) || misaligned16(lambda)) return KVQ_ERR_ALIGNMENT;
    if (status_word && (reinterpret_cast<uintptr_t>(status_word) & 3u)) return KVQ_ERR_ALIGNMENT;

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return KVQ_ERR_CUDA;
    }
    if (dev < 0 || dev >= kvq::kMaxDevices) return KVQ_ERR_INVALID_ARG;

    std::lock_guard<std::mutex> lk(g_mu);
    DeviceSlot &slot = g_slots[dev];
    if (!slot.block) {
        // set-up, once per device, with that device current: ask the runtime where the block lives
        float *p = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void **>(&p), kvq_static_scratch) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return KVQ_ERR_CUDA;
        }
        slot.block = p;
    }
    float *table = slot.block;
    uint32_t *own_status = reinterpret_cast<uint32_t *>(slot.block + kTableFloats);
    uint32_t *status = status_word ? status_word : own_status;

    // A captured call runs later, possibly many times, after calls this host code never sees in that order: it carries
    // its own table fill, and the host's note of what the block holds is neither trusted nor updated.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) {
        (void)cudaGetLastError();
        return KVQ_ERR_CUDA;
    }
    const bool capturing = cap != cudaStreamCaptureStatusNone;
    if (capturing) slot.replays_possible = true;   // from now on no eager call on this device can know what the block holds
    if (capturing || slot.replays_possible || !slot.table_valid || slot.table_D != plan->D || slot.table_seed != plan->seed) {
        SignWords sw;
        for (int i = 0; i < 128; ++i) sw.w[i] = plan->sign_xor[i];
        if (!capturing) slot.table_valid = false;
        kvq_static_fill_kernel<<<plan->D, plan->D, 0, stream>>>(table, plan->D, sw);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return KVQ_ERR_CUDA;
        if (!capturing) {
            slot.table_valid = true;
            slot.table_D = plan->D;
            slot.table_seed = plan->seed;
        }
    }
    if (cudaMemsetAsync(status, 0, sizeof(uint32_t), stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return KVQ_ERR_CUDA;
    }

    GemmParams g;
    g.packed = packed;
    g.scales = scales;
    g.lambda = lambda;
    g.out = out;
    g.b0 = table;
    g.N = N;
    g.n_lambda = n_lambda;
    g.rows_per_lambda = rows_per_lambda < 1 ? 1 : rows_per_lambda;
    g.per_vector = 0;
    g.status = status;
    if (umma_decode(128, false, 4, N, g, plan->sign_xor, stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return KVQ_ERR_CUDA;
    }
    return KVQ_OK;
}
