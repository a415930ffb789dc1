// mxq_greedy_accept: the verification step of a speculative-decoding round (Sec. III-A:
// drafted tokens after the first mismatch are dropped; Sec. III-B: G accepted tokens plus
// one token of the target's own).
//
// The cost is reading the logits once (B*R*V elements): an HBM stream.  Each CTA takes one
// slice of one logits row and reduces it to a (value, index) pair; the last CTA of a
// sequence to finish (found with a ticket counter, so nobody waits) combines the slices in
// index order, which keeps the result independent of scheduling, and then walks the draft.
#include <limits.h>

#include "mxq_device.cuh"
#include "mxq_host.h"

namespace mxq {

constexpr int kAcceptThreads = 256;
constexpr int64_t kSliceQuantum = 2048;  // slice lengths are multiples of this many logits
constexpr int64_t kTargetCtas = 592;     // 4 per SM on a 148-SM part
constexpr int kTickets = 1024;           // ticket counters live in a fixed region: sequence b uses ticket b % kTickets

struct Best {
    float v;
    int idx;
};

// a beats b when it is larger, or equal with a lower index.  NaN never beats anything.
__device__ __forceinline__ Best better(Best a, Best b) {
    return (b.v > a.v || (b.v == a.v && b.idx < a.idx)) ? b : a;
}

__device__ __forceinline__ void consider(Best &best, float x, int idx) {
    if (x > best.v) {  // strictly greater: earlier index keeps a tie; NaN and -inf never enter
        best.v = x;
        best.idx = idx;
    }
}

struct Slicing {
    int slices;
    int64_t slice_len;
};

static Slicing slicing_for(int64_t B, int R, int64_t V) {
    const int64_t rows = B * R;
    int64_t want = (kTargetCtas + rows - 1) / rows;
    const int64_t most = (V + kSliceQuantum - 1) / kSliceQuantum;
    if (want > most) want = most;
    if (want < 1) want = 1;
    int64_t len = (V + want - 1) / want;
    len = (len + kSliceQuantum - 1) / kSliceQuantum * kSliceQuantum;
    Slicing s;
    s.slice_len = len;
    s.slices = (int)((V + len - 1) / len);
    return s;
}

static size_t ticket_bytes() { return (size_t)kTickets * sizeof(unsigned); }

template <typename T>
__device__ __forceinline__ float logit_value(T x);
template <>
__device__ __forceinline__ float logit_value<float>(float x) { return x; }
template <>
__device__ __forceinline__ float logit_value<uint16_t>(uint16_t x) { return bf16_bits_to_float(x); }

// T = float or uint16_t (BF16 bits).  grid.x = B * R * slices.
template <typename T>
__global__ void __launch_bounds__(kAcceptThreads)
greedy_accept_kernel(const T *__restrict__ logits, int64_t B, int R, int64_t V, int slices, int64_t slice_len, bool vec_ok,
                     const int32_t *__restrict__ draft, int Tn, int32_t *__restrict__ accept_len,
                     int32_t *__restrict__ next_token, Best *__restrict__ partial, unsigned *__restrict__ tickets) {
    constexpr int kVec = 16 / sizeof(T);
    const int64_t cta = blockIdx.x;
    const int slice = (int)(cta % slices);
    const int64_t row = cta / slices;  // b * R + r
    const int64_t b = row / R;
    const T *p = logits + row * V;
    const int64_t lo = (int64_t)slice * slice_len;
    const int64_t hi = min(V, lo + slice_len);

    Best best = {-INFINITY, INT_MAX};
    if (vec_ok) {
        const int64_t nvec = (hi - lo) / kVec;  // lo is a multiple of kSliceQuantum, rows are 16-byte aligned
        const uint4 *pv = reinterpret_cast<const uint4 *>(p + lo);
        // four 16-byte loads in flight per lane (ascending index order is kept, so ties still go to the lowest index)
        int64_t i = threadIdx.x;
        for (; i + 3 * kAcceptThreads < nvec; i += 4 * kAcceptThreads) {
            uint4 q4[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) q4[u] = ld_stream_u4(pv + i + u * kAcceptThreads);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint4 q = q4[u];
                const int base = (int)(lo + (i + u * kAcceptThreads) * kVec);
                if constexpr (sizeof(T) == 4) {
                    consider(best, __uint_as_float(q.x), base);
                    consider(best, __uint_as_float(q.y), base + 1);
                    consider(best, __uint_as_float(q.z), base + 2);
                    consider(best, __uint_as_float(q.w), base + 3);
                } else {
                    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        consider(best, __uint_as_float(w[j] << 16), base + 2 * j);
                        consider(best, __uint_as_float(w[j] & 0xFFFF0000u), base + 2 * j + 1);
                    }
                }
            }
        }
        for (; i < nvec; i += kAcceptThreads) {
            const uint4 q = ld_stream_u4(pv + i);
            const int base = (int)(lo + i * kVec);
            if constexpr (sizeof(T) == 4) {
                consider(best, __uint_as_float(q.x), base);
                consider(best, __uint_as_float(q.y), base + 1);
                consider(best, __uint_as_float(q.z), base + 2);
                consider(best, __uint_as_float(q.w), base + 3);
            } else {
                const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    consider(best, __uint_as_float(w[j] << 16), base + 2 * j);
                    consider(best, __uint_as_float(w[j] & 0xFFFF0000u), base + 2 * j + 1);
                }
            }
        }
        for (int64_t i = lo + nvec * kVec + threadIdx.x; i < hi; i += kAcceptThreads)
            consider(best, logit_value<T>(p[i]), (int)i);
    } else {
        for (int64_t i = lo + threadIdx.x; i < hi; i += kAcceptThreads) consider(best, logit_value<T>(p[i]), (int)i);
    }

#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Best other;
        other.v = __shfl_xor_sync(0xffffffffu, best.v, o);
        other.idx = __shfl_xor_sync(0xffffffffu, best.idx, o);
        best = better(best, other);
    }
    __shared__ Best warp_best[kAcceptThreads / 32];
    __shared__ int verifier[MXQ_MAX_T + 1];
    __shared__ bool is_last;
    if ((threadIdx.x & 31) == 0) warp_best[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kAcceptThreads / 32; ++w) best = better(best, warp_best[w]);
        partial[row * slices + slice] = best;
        __threadfence();
        // sequences b, b + kTickets, ... share a counter; whoever arrives last finishes all of them
        const int64_t group = b % kTickets;
        const int64_t members = (B - group + kTickets - 1) / kTickets;
        const unsigned arrived = atomicAdd(&tickets[group], 1u);
        is_last = arrived == (unsigned)(members * R * slices) - 1u;
    }
    __syncthreads();
    if (!is_last) return;

    // every slice of every row of this group of sequences has been published
    __threadfence();
    for (int64_t bb = b % kTickets; bb < B; bb += kTickets) {
        if (threadIdx.x < R) {
            const Best *pr = partial + (bb * R + threadIdx.x) * slices;
            Best r = {-INFINITY, INT_MAX};
            for (int s = 0; s < slices; ++s) {
                Best q;
                q.v = __ldcg(&pr[s].v);
                q.idx = __ldcg(&pr[s].idx);
                r = better(r, q);
            }
            verifier[threadIdx.x] = (r.idx == INT_MAX) ? 0 : r.idx;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int G = Tn;
            for (int i = 0; i < Tn; ++i) {
                if (i >= R || draft[bb * Tn + i] != verifier[i]) {
                    G = i;
                    break;
                }
            }
            accept_len[bb] = G;
            next_token[bb] = (G < R) ? verifier[G] : -1;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) tickets[b % kTickets] = 0;  // ready for the next call
}

__global__ void accept_tokens_kernel(const int32_t *__restrict__ draft, const int32_t *__restrict__ verifier, int64_t B,
                                     int Tn, int R, int32_t *__restrict__ accept_len, int32_t *__restrict__ next_token) {
    const int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    int G = Tn;
    for (int i = 0; i < Tn; ++i) {
        if (i >= R || draft[b * Tn + i] != verifier[b * R + i]) {
            G = i;
            break;
        }
    }
    accept_len[b] = G;
    next_token[b] = (G < R) ? verifier[b * R + G] : -1;
}

static bool accept_shape_ok(int64_t B, int R, int64_t V, int T) {
    return B >= 1 && V >= 1 && V <= INT_MAX - 1 && T >= 1 && T <= MXQ_MAX_T && (R == T || R == T + 1) &&
           B * (int64_t)R <= (int64_t)INT_MAX / 1024;
}

// ---------------------------------------------------------------------------------------------
// Built-in scratch for mxq_greedy_accept_static: lives in the library image, so every GPU that
// loads the library holds these bytes until the process exits.  Same layout as the caller-provided
// workspace of mxq_greedy_accept: ticket counters first, then the per-slice (value, index) pairs.
// ---------------------------------------------------------------------------------------------
constexpr size_t kStaticScratchBytes = (size_t)1 << 20;  // 1 MiB
static __device__ __align__(256) unsigned char g_accept_scratch[kStaticScratchBytes];

// Device address of g_accept_scratch on the current device.  In host code the array's name is only a
// handle for the runtime, never a device address, so the address is asked for once per device (with that
// device current) and remembered.  Returns nullptr if the runtime refuses.
static void *static_scratch_for_current_device() {
    static void *cached[64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (cached[dev] == nullptr) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_accept_scratch) != cudaSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        cached[dev] = ptr;
    }
    return cached[dev];
}

}  // namespace mxq

extern "C" {
#pragma GCC visibility push(default)

size_t mxq_accept_workspace_bytes(int64_t B, int R, int64_t V) {
    if (B < 1 || R < 1 || R > MXQ_MAX_T + 1 || V < 1) return 0;
    const mxq::Slicing s = mxq::slicing_for(B, R, V);
    return mxq::ticket_bytes() + (size_t)B * R * s.slices * sizeof(mxq::Best);
}

int mxq_greedy_accept(const void *logits, int logits_dtype, int64_t B, int R, int64_t V, const int32_t *draft,
                      int T, int32_t *accept_len, int32_t *next_token, void *workspace, size_t workspace_bytes,
                      void *stream) {
    if (!logits || !draft || !accept_len || !next_token) return MXQ_ERR_NULL;
    if (!mxq::accept_shape_ok(B, R, V, T)) return MXQ_ERR_SHAPE;
    if (logits_dtype != MXQ_F32 && logits_dtype != MXQ_BF16) return MXQ_ERR_DTYPE;
    if (!mxq::aligned16(logits) || !mxq::aligned16(workspace)) return MXQ_ERR_ALIGN;
    if (!workspace || workspace_bytes < mxq_accept_workspace_bytes(B, R, V)) return MXQ_ERR_WORKSPACE;
    const mxq::Slicing s = mxq::slicing_for(B, R, V);
    unsigned *tickets = (unsigned *)workspace;
    mxq::Best *partial = (mxq::Best *)((char *)workspace + mxq::ticket_bytes());
    const unsigned grid = (unsigned)(B * R * s.slices);
    cudaStream_t st = (cudaStream_t)stream;
    if (logits_dtype == MXQ_F32) {
        const bool vec_ok = (V % 4) == 0;
        mxq::greedy_accept_kernel<float><<<grid, mxq::kAcceptThreads, 0, st>>>(
            (const float *)logits, B, R, V, s.slices, s.slice_len, vec_ok, draft, T, accept_len, next_token, partial, tickets);
    } else {
        const bool vec_ok = (V % 8) == 0;
        mxq::greedy_accept_kernel<uint16_t><<<grid, mxq::kAcceptThreads, 0, st>>>(
            (const uint16_t *)logits, B, R, V, s.slices, s.slice_len, vec_ok, draft, T, accept_len, next_token, partial,
            tickets);
    }
    return mxq::launch_status();
}

int mxq_greedy_accept_tokens(const int32_t *draft, const int32_t *verifier, int64_t B, int T, int R,
                             int32_t *accept_len, int32_t *next_token, void *stream) {
    if (!draft || !verifier || !accept_len || !next_token) return MXQ_ERR_NULL;
    if (B < 1 || T < 1 || T > MXQ_MAX_T || !(R == T || R == T + 1)) return MXQ_ERR_SHAPE;
    const unsigned grid = (unsigned)((B + 127) / 128);
    mxq::accept_tokens_kernel<<<grid, 128, 0, (cudaStream_t)stream>>>(draft, verifier, B, T, R, accept_len, next_token);
    return mxq::launch_status();
}

int mxq_greedy_accept_static(const void *logits, int logits_dtype, int64_t B, int R, int64_t V, const int32_t *draft,
                             int T, int32_t *accept_len, int32_t *next_token, void *stream) {
    if (!logits || !draft || !accept_len || !next_token) return MXQ_ERR_NULL;
    if (!mxq::accept_shape_ok(B, R, V, T)) return MXQ_ERR_SHAPE;
    if (logits_dtype != MXQ_F32 && logits_dtype != MXQ_BF16) return MXQ_ERR_DTYPE;
    if (!mxq::aligned16(logits)) return MXQ_ERR_ALIGN;
    // the scratch this shape needs must fit the built-in array; nothing is ever allocated to make room
    if (mxq_accept_workspace_bytes(B, R, V) > mxq::kStaticScratchBytes) return MXQ_ERR_WORKSPACE;
    void *scratch = mxq::static_scratch_for_current_device();  // first call on a device: one runtime query
    if (!scratch) return MXQ_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps whatever the previous call left; the ticket counters must start at zero
    if (cudaMemsetAsync(scratch, 0, mxq::ticket_bytes(), st) != cudaSuccess) {
        (void)cudaGetLastError();
        return MXQ_ERR_CUDA;
    }
    const mxq::Slicing s = mxq::slicing_for(B, R, V);
    unsigned *tickets = (unsigned *)scratch;
    mxq::Best *partial = (mxq::Best *)((char *)scratch + mxq::ticket_bytes());
    const unsigned grid = (unsigned)(B * R * s.slices);
    if (logits_dtype == MXQ_F32) {
        mxq::greedy_accept_kernel<float><<<grid, mxq::kAcceptThreads, 0, st>>>(
            (const float *)logits, B, R, V, s.slices, s.slice_len, (V % 4) == 0, draft, T, accept_len, next_token, partial,
            tickets);
    } else {
        mxq::greedy_accept_kernel<uint16_t><<<grid, mxq::kAcceptThreads, 0, st>>>(
            (const uint16_t *)logits, B, R, V, s.slices, s.slice_len, (V % 8) == 0, draft, T, accept_len, next_token,
            partial, tickets);
    }
    return mxq::launch_status();
}

size_t mxq_greedy_accept_static_max_bytes(void) { return mxq::kStaticScratchBytes; }

#pragma GCC visibility pop
}  // extern "C"
