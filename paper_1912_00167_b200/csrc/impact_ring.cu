// Circular buffer C(N, K) of device-resident train batches (Algorithm 1; Section 3.2), and
// the byte-exact copy / gather kernels behind it.
//
// Slot bookkeeping is a few integers per slot and lives on the host, where the learner loop
// that calls push / sample runs; the payload never leaves HBM.  A sample is normally
// zero-copy (the loss kernel reads the slot in place); the fused copy kernel serves pushes
// from device memory and the optional gather into caller buffers.
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <new>
#include <vector>

#include "impact.h"
#include "impact_internal.h"

namespace impact {
namespace {

constexpr int kMaxFields = 16;
constexpr size_t kFieldAlign = 256;

struct CopySegments {
    const char* src[kMaxFields];
    char* dst[kMaxFields];
    unsigned long long bytes[kMaxFields];
    unsigned long long vec_end[kMaxFields];  // running count of 16-byte units up to and including segment f
    int n;
};

// Copies up to kMaxFields byte ranges in one launch.  Every range is walked in 16-byte
// units; the last unit of a range whose length is not a multiple of 16 is copied bytewise.
__global__ void __launch_bounds__(256) multi_copy_kernel(const CopySegments s) {
    grid_dependency_wait();
    const unsigned long long total = s.vec_end[s.n - 1];
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    unsigned long long v = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    constexpr int U = 4;
    while (v < total) {
        uint4 x[U];
        char* out[U];
        int tail[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const unsigned long long vu = v + u * stride;
            tail[u] = -1;
            out[u] = nullptr;
            if (vu < total) {
                int f = 0;
                while (vu >= s.vec_end[f]) ++f;
                const unsigned long long off = (vu - (f ? s.vec_end[f - 1] : 0ull)) * 16ull;
                out[u] = s.dst[f] + off;
                if (off + 16ull <= s.bytes[f]) {
                    x[u] = __ldcs(reinterpret_cast<const uint4*>(s.src[f] + off));
                } else {
                    tail[u] = (int)(s.bytes[f] - off);
                    for (int i = 0; i < tail[u]; ++i) out[u][i] = s.src[f][off + i];
                    out[u] = nullptr;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (out[u]) __stcs(reinterpret_cast<uint4*>(out[u]), x[u]);
        v += U * stride;
    }
}

// dst[i, :] = src[idx[i], :], rows of `units` elements of type V.
template <typename V>
__global__ void __launch_bounds__(256) gather_rows_kernel(const V* __restrict__ src,
                                                          const int32_t* __restrict__ idx,
                                                          long long n, long long n_src_rows,
                                                          long long units, V* __restrict__ dst) {
    grid_dependency_wait();
    const long long total = n * units;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < total; v += stride) {
        const long long i = v / units;
        const long long c = v - i * units;
        long long r = idx[i];
        r = r < 0 ? 0 : (r >= n_src_rows ? n_src_rows - 1 : r);
        dst[v] = src[r * units + c];
    }
}

// Reads `n_read` 16-byte units and writes `n_write` of them back out (n_write <= n_read): a loss launch's byte mix
// with no arithmetic in between.  What is read but not written is folded into one word per thread that is stored
// only if it has an impossible value, so that the loads cannot be dropped.
__global__ void __launch_bounds__(256) stream_copy_kernel(const uint4* __restrict__ src, unsigned long long n_read,
                                                          uint4* __restrict__ dst, unsigned long long n_write,
                                                          unsigned int* __restrict__ sink) {
    grid_dependency_wait();
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    unsigned int fold = 0;
    constexpr int U = 4;
    for (unsigned long long v = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; v < n_read; v += U * stride) {
        uint4 x[U];
#pragma unroll
        for (int u = 0; u < U; ++u)
            x[u] = (v + u * stride < n_read) ? __ldcs(src + v + u * stride) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (v + u * stride < n_write) dst[v + u * stride] = x[u];
            else fold |= x[u].x ^ x[u].y ^ x[u].z ^ x[u].w;
        }
    }
    if (fold == 0xFFFFFFFFu && n_read == 1) *sink = fold;  // (never: keeps the unwritten loads alive)
}

// ---- bookkeeping resident on the device ---------------------------------------------------------------------
// The same few integers per slot as on the host, in device memory, so that a learner iteration -- push a worker
// batch into a free slot, obtain a batch, loss and gradients -- can be enqueued (or captured into a CUDA graph)
// without the host ever seeing a slot number.  One warp does the bookkeeping; it is the protocol of
// impact_buffer_push / impact_buffer_sample statement by statement (docs/ring_protocol.md), so both modes give the
// same trace for the same seed.
struct RingDeviceHeader {
    int32_t write_cursor, read_cursor;
    uint32_t n_events, pad;
    uint64_t draws, pushes;
};
constexpr int kEventLog = 4096;  // the most recent push / sample outcomes, for the host to read back
constexpr int kMaxDeviceSlots = 1024;  // slots a buffer may have for its bookkeeping to go to the device

struct RingDeviceView {
    RingDeviceHeader* hd;
    int32_t* valid;
    int32_t* count;
    uint64_t* fresh;   // per slot: the extra pointer that came with the batch pushed into it
    int4* events;      // (op, status, slot, k_before); op 1 = push, 2 = sample
    CopySegments* plan;
    char* storage;
    unsigned long long slot_stride;
    unsigned long long field_offset[kMaxFields], field_bytes[kMaxFields];
    int32_t N, K, n_fields, mode;
    uint64_t seed;
};

__device__ __forceinline__ uint64_t splitmix64_at_dev(uint64_t seed, uint64_t n) {
    uint64_t z = seed + (n + 1) * 0x9E3779B97F4A7C15ull;
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ull;
    z ^= z >> 27; z *= 0x94D049BB133111EBull;
    z ^= z >> 31;
    return z;
}

// One learner-side step of the bookkeeping: (1) if `sources` is given, the next candidate batch goes into the
// first free slot at or after the write cursor (none free: nothing happens, the event says FULL), and the copy
// that the following kernel performs is written to `plan`; (2) a live slot is drawn and the inputs of the loss
// call are resolved into `inputs`.
__global__ void __launch_bounds__(32) ring_step_kernel(const RingDeviceView v, const impact_ring_field_map map,
                                                       const void* learner_logits, const float* values,
                                                       const float* bootstrap_values, const void* const* sources,
                                                       int32_t n_candidates, int32_t do_sample,
                                                       impact_loss_inputs* inputs) {
    grid_dependency_wait();
    // the slots' flags and counts are staged in shared memory by the whole warp (one trip to L2 instead of one per
    // slot); lane 0 then walks them exactly as the host code does and writes back what it changed
    __shared__ int32_t valid_s[kMaxDeviceSlots], count_s[kMaxDeviceSlots];
    __shared__ uint64_t fresh_s[kMaxDeviceSlots];
    for (int32_t i = threadIdx.x; i < v.N; i += 32) {
        valid_s[i] = v.valid[i];
        count_s[i] = v.count[i];
        fresh_s[i] = v.fresh[i];
    }
    RingDeviceHeader hd = *v.hd;
    // (the candidate's pointers too: lane f fetches the f-th, all at once)
    __shared__ const void* cand_s[kMaxFields + 1];
    if (sources && (int)threadIdx.x <= v.n_fields)
        cand_s[threadIdx.x] = sources[(size_t)(hd.pushes % (uint64_t)n_candidates) * (size_t)(v.n_fields + 1) + threadIdx.x];
    __syncwarp();
    if (threadIdx.x != 0) return;
    v.plan->n = 0;
    if (sources) {
        int32_t slot = -1;
        for (int32_t i = 0; i < v.N; ++i) {
            const int32_t s = (hd.write_cursor + i) % v.N;
            if (!valid_s[s]) { slot = s; break; }
        }
        if (slot >= 0) {
            const void* const* cand = cand_s;
            int n = 0;
            unsigned long long units = 0;
            for (int f = 0; f < v.n_fields; ++f) {
                if (!cand[f]) continue;
                v.plan->src[n] = static_cast<const char*>(cand[f]);
                v.plan->dst[n] = v.storage + (unsigned long long)slot * v.slot_stride + v.field_offset[f];
                v.plan->bytes[n] = v.field_bytes[f];
                units += (v.field_bytes[f] + 15ull) / 16ull;
                v.plan->vec_end[n] = units;
                ++n;
            }
            v.plan->n = n;
            v.fresh[slot] = reinterpret_cast<uint64_t>(cand[v.n_fields]);
            fresh_s[slot] = reinterpret_cast<uint64_t>(cand[v.n_fields]);
            valid_s[slot] = 1;
            count_s[slot] = 0;
            v.valid[slot] = 1;
            v.count[slot] = 0;
            hd.write_cursor = (slot + 1) % v.N;
            hd.pushes += 1;
        }
        v.events[hd.n_events++ % kEventLog] = make_int4(1, slot >= 0 ? IMPACT_OK : IMPACT_ERR_FULL, slot, 0);
    }
    if (do_sample) {
        int32_t live = 0;
        for (int32_t s = 0; s < v.N; ++s) live += valid_s[s] ? 1 : 0;
        int32_t pick = -1;
        if (live > 0) {
            if (v.mode == IMPACT_SAMPLE_UNIFORM) {
                const uint64_t u = splitmix64_at_dev(v.seed, hd.draws++);
                uint64_t j = __umul64hi(u, (uint64_t)live);  // floor(u * live / 2^64)
                for (int32_t s = 0; s < v.N; ++s) {
                    if (!valid_s[s]) continue;
                    if (j == 0) { pick = s; break; }
                    --j;
                }
            } else {
                for (int32_t i = 0; i < v.N; ++i) {
                    const int32_t s = (hd.read_cursor + i) % v.N;
                    if (valid_s[s]) { pick = s; break; }
                }
                hd.read_cursor = (pick + 1) % v.N;
            }
        }
        int32_t k_before = 0;
        if (pick >= 0) {
            k_before = count_s[pick];
            v.count[pick] = k_before + 1;
            if (k_before + 1 >= v.K) v.valid[pick] = 0;
            auto field = [&](int32_t f) -> const void* {
                return f >= 0 ? v.storage + (unsigned long long)pick * v.slot_stride + v.field_offset[f] : nullptr;
            };
            impact_loss_inputs in;
            in.learner_logits = learner_logits;
            in.values = values;
            in.bootstrap_values = bootstrap_values;
            in.actions = static_cast<const int32_t*>(field(map.actions));
            in.rewards = static_cast<const float*>(field(map.rewards));
            in.discounts = static_cast<const float*>(field(map.discounts));
            in.worker_logp = static_cast<const float*>(field(map.worker_logp));
            const void* in_slot = field(map.target_logits);
            const void* fresh = reinterpret_cast<const void*>(fresh_s[pick]);
            if (k_before == 0 && fresh && in_slot) {  // first traversal: the target network's output is appended now
                in.target_logits = fresh;
                in.target_logits_copy = const_cast<void*>(in_slot);
            } else {
                in.target_logits = in_slot;
                in.target_logits_copy = nullptr;
            }
            in.status = IMPACT_OK;
            in.slot = pick;
            in.k_before = k_before;
            in.pad = 0;
            *inputs = in;
        } else {
            inputs->status = IMPACT_ERR_EMPTY;  // the pointers of the previous draw stay in place
        }
        v.events[hd.n_events++ % kEventLog] = make_int4(2, pick >= 0 ? IMPACT_OK : IMPACT_ERR_EMPTY, pick, k_before);
    }
    *v.hd = hd;
}

// multi_copy_kernel with its segments read from device memory (an empty plan copies nothing).
__global__ void __launch_bounds__(256) multi_copy_planned_kernel(const CopySegments* plan) {
    grid_dependency_wait();
    // the plan is staged in shared memory by the block's first threads, eight bytes each: one trip to L2 instead of
    // one for the count, one for the segment ends and one for the addresses
    __shared__ CopySegments plan_s;
    constexpr int kWords = (int)(sizeof(CopySegments) / 8);
    static_assert(sizeof(CopySegments) % 8 == 0 && kWords <= 256, "staged by one pass of the block");
    if ((int)threadIdx.x < kWords)
        reinterpret_cast<unsigned long long*>(&plan_s)[threadIdx.x] =
            reinterpret_cast<const unsigned long long*>(plan)[threadIdx.x];  // (through L1: the blocks of an SM share the lines)
    __syncthreads();
    plan = &plan_s;
    const int n = plan->n;
    if (n == 0) return;
    const unsigned long long total = plan->vec_end[n - 1];
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    constexpr int U = 4;
    for (unsigned long long v0 = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; v0 < total; v0 += U * stride) {
        uint4 x[U];
        char* out[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const unsigned long long vu = v0 + u * stride;
            out[u] = nullptr;
            if (vu < total) {
                int f = 0;
                while (vu >= plan->vec_end[f]) ++f;
                const unsigned long long off = (vu - (f ? plan->vec_end[f - 1] : 0ull)) * 16ull;
                const char* src = plan->src[f] + off;
                char* dst = plan->dst[f] + off;
                if (off + 16ull <= plan->bytes[f]) {
                    x[u] = __ldcs(reinterpret_cast<const uint4*>(src));
                    out[u] = dst;
                } else {
                    const int tail = (int)(plan->bytes[f] - off);
                    for (int i = 0; i < tail; ++i) dst[i] = src[i];
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (out[u]) __stcs(reinterpret_cast<uint4*>(out[u]), x[u]);
    }
}

int blocks_for(unsigned long long work_items, int per_thread, const DeviceInfo* di) {
    unsigned long long blocks = (work_items + 256ull * per_thread - 1) / (256ull * per_thread);
    const unsigned long long cap = (unsigned long long)di->sm_count * 8ull;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

// n-th output of SplitMix64 (Steele, Lea, Flood 2014) for the stream that starts at `seed`:
// the additive state after n+1 steps, passed through the two multiply-xorshift rounds.
uint64_t splitmix64_at(uint64_t seed, uint64_t n) {
    uint64_t z = seed + (n + 1) * 0x9E3779B97F4A7C15ull;
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ull;
    z ^= z >> 27; z *= 0x94D049BB133111EBull;
    z ^= z >> 31;
    return z;
}

struct StateHeader {
    uint32_t magic, version;
    int32_t N, K, n_fields, mode;
    int32_t write_cursor, read_cursor;
    uint64_t seed, draws;
};
constexpr uint32_t kStateMagic = 0x494D5043u;  // "IMPC"

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace
}  // namespace impact

using namespace impact;

struct impact_buffer {
    int32_t N = 0, K = 0, n_fields = 0, mode = 0;
    uint64_t seed = 0, draws = 0;
    int32_t write_cursor = 0, read_cursor = 0;
    std::vector<int32_t> valid, count;
    size_t field_bytes[kMaxFields] = {};
    size_t field_offset[kMaxFields] = {};
    size_t slot_stride = 0;
    char* storage = nullptr;
    bool owns_storage = false;
    // bookkeeping on the device (impact_buffer_device_begin): one allocation, laid out as
    // [header | valid N | count N | fresh N | events | copy plan]
    char* device_state = nullptr;
    bool device_mode = false;
    size_t device_state_bytes() const {
        return align_up16(sizeof(RingDeviceHeader)) + align_up16(sizeof(int32_t) * (size_t)N) * 2 +
               align_up16(sizeof(uint64_t) * (size_t)N) + sizeof(int4) * (size_t)kEventLog + align_up16(sizeof(CopySegments));
    }
    static size_t align_up16(size_t x) { return (x + 15) / 16 * 16; }
    RingDeviceView view() const {
        RingDeviceView v;
        char* p = device_state;
        v.hd = reinterpret_cast<RingDeviceHeader*>(p); p += align_up16(sizeof(RingDeviceHeader));
        v.valid = reinterpret_cast<int32_t*>(p); p += align_up16(sizeof(int32_t) * (size_t)N);
        v.count = reinterpret_cast<int32_t*>(p); p += align_up16(sizeof(int32_t) * (size_t)N);
        v.fresh = reinterpret_cast<uint64_t*>(p); p += align_up16(sizeof(uint64_t) * (size_t)N);
        v.events = reinterpret_cast<int4*>(p); p += sizeof(int4) * (size_t)kEventLog;
        v.plan = reinterpret_cast<CopySegments*>(p);
        v.storage = storage;
        v.slot_stride = slot_stride;
        for (int f = 0; f < kMaxFields; ++f) { v.field_offset[f] = field_offset[f]; v.field_bytes[f] = field_bytes[f]; }
        v.N = N; v.K = K; v.n_fields = n_fields; v.mode = mode;
        v.seed = seed;
        return v;
    }

    char* field_ptr(int32_t slot, int32_t f) const {
        return storage + (size_t)slot * slot_stride + field_offset[f];
    }
};

static bool valid_fields(int32_t n_fields, const size_t* field_bytes) {
    if (n_fields < 1 || n_fields > kMaxFields || !field_bytes) return false;
    for (int f = 0; f < n_fields; ++f)
        if (field_bytes[f] == 0) return false;
    return true;
}

extern "C" size_t impact_buffer_storage_bytes(int32_t N, int32_t n_fields, const size_t* field_bytes) {
    if (N < 1 || !valid_fields(n_fields, field_bytes)) return 0;
    size_t stride = 0;
    for (int f = 0; f < n_fields; ++f) stride += align_up(field_bytes[f], kFieldAlign);
    return stride * (size_t)N;
}

extern "C" int32_t impact_buffer_create(int32_t N, int32_t K, int32_t n_fields, const size_t* field_bytes,
                                        uint64_t seed, int32_t sample_mode, void* storage,
                                        impact_buffer** out) {
    if (!out || N < 1 || K < 1 || !valid_fields(n_fields, field_bytes)) return IMPACT_ERR_INVALID_ARG;
    if (sample_mode != IMPACT_SAMPLE_UNIFORM && sample_mode != IMPACT_SAMPLE_ROUND_ROBIN)
        return IMPACT_ERR_INVALID_ARG;
    if (storage && (reinterpret_cast<uintptr_t>(storage) % kFieldAlign) != 0) return IMPACT_ERR_INVALID_ARG;
    impact_buffer* h = new (std::nothrow) impact_buffer();
    if (!h) return IMPACT_ERR_INVALID_ARG;
    h->N = N; h->K = K; h->n_fields = n_fields; h->mode = sample_mode; h->seed = seed;
    h->valid.assign((size_t)N, 0);
    h->count.assign((size_t)N, 0);
    size_t off = 0;
    for (int f = 0; f < n_fields; ++f) {
        h->field_bytes[f] = field_bytes[f];
        h->field_offset[f] = off;
        off += align_up(field_bytes[f], kFieldAlign);
    }
    h->slot_stride = off;
    if (storage) {
        h->storage = static_cast<char*>(storage);
    } else {
        void* mem = nullptr;
        cudaError_t e = cudaMalloc(&mem, off * (size_t)N);
        if (e != cudaSuccess) { delete h; return record_cuda_error(e); }
        h->storage = static_cast<char*>(mem);
        h->owns_storage = true;
    }
    *out = h;
    return IMPACT_OK;
}

extern "C" int32_t impact_buffer_destroy(impact_buffer* h) {
    if (!h) return IMPACT_ERR_INVALID_ARG;
    int32_t st = IMPACT_OK;
    if (h->owns_storage || h->device_state) {
        cudaError_t e = cudaDeviceSynchronize();
        if (e == cudaSuccess && h->owns_storage) e = cudaFree(h->storage);
        if (e == cudaSuccess && h->device_state) e = cudaFree(h->device_state);
        if (e != cudaSuccess) st = record_cuda_error(e);
    }
    delete h;
    return st;
}

// Enqueue one fused copy of the given segments.
static int32_t launch_copy(const CopySegments& segs, cudaStream_t stream) {
    if (segs.n == 0) return IMPACT_OK;
    const DeviceInfo* di = current_device_info();
    if (!di) return IMPACT_ERR_CUDA;
    const unsigned long long total = segs.vec_end[segs.n - 1];
    IMPACT_CUDA_TRY(launch_serialized(multi_copy_kernel, dim3(blocks_for(total, 4, di)), dim3(256), 0, stream, segs));
    return IMPACT_OK;
}

static void add_segment(CopySegments& s, const void* src, void* dst, size_t bytes) {
    const int f = s.n++;
    s.src[f] = static_cast<const char*>(src);
    s.dst[f] = static_cast<char*>(dst);
    s.bytes[f] = bytes;
    s.vec_end[f] = (f ? s.vec_end[f - 1] : 0ull) + (bytes + 15) / 16;
}

extern "C" int32_t impact_buffer_push(impact_buffer* h, const void* const* field_src, int32_t src_location,
                                      int32_t* slot_out, void* stream) {
    if (!h || !field_src || !slot_out || h->device_mode) return IMPACT_ERR_INVALID_ARG;
    if (src_location != IMPACT_SRC_DEVICE && src_location != IMPACT_SRC_HOST) return IMPACT_ERR_INVALID_ARG;
    if (src_location == IMPACT_SRC_DEVICE)
        for (int f = 0; f < h->n_fields; ++f)
            if (field_src[f] && !aligned16(field_src[f])) return IMPACT_ERR_INVALID_ARG;
    int32_t slot = -1;
    for (int32_t i = 0; i < h->N; ++i) {
        const int32_t s = (h->write_cursor + i) % h->N;
        if (!h->valid[s]) { slot = s; break; }
    }
    if (slot < 0) return IMPACT_ERR_FULL;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (src_location == IMPACT_SRC_DEVICE) {
        CopySegments segs;
        segs.n = 0;
        for (int f = 0; f < h->n_fields; ++f)
            if (field_src[f]) add_segment(segs, field_src[f], h->field_ptr(slot, f), h->field_bytes[f]);
        int32_t st = launch_copy(segs, cs);
        if (st != IMPACT_OK) return st;
    } else {
        for (int f = 0; f < h->n_fields; ++f)
            if (field_src[f])
                IMPACT_CUDA_TRY(cudaMemcpyAsync(h->field_ptr(slot, f), field_src[f], h->field_bytes[f],
                                                cudaMemcpyHostToDevice, cs));
    }
    h->valid[slot] = 1;
    h->count[slot] = 0;
    h->write_cursor = (slot + 1) % h->N;
    *slot_out = slot;
    return IMPACT_OK;
}

extern "C" int32_t impact_buffer_sample(impact_buffer* h, int32_t* slot_out, int32_t* k_before_out,
                                        void* const* gather_dst, void* stream) {
    if (!h || !slot_out || !k_before_out || h->device_mode) return IMPACT_ERR_INVALID_ARG;
    if (gather_dst)
        for (int f = 0; f < h->n_fields; ++f)
            if (gather_dst[f] && !aligned16(gather_dst[f])) return IMPACT_ERR_INVALID_ARG;
    int32_t live = 0;
    for (int32_t s = 0; s < h->N; ++s) live += h->valid[s] ? 1 : 0;
    if (live == 0) return IMPACT_ERR_EMPTY;
    int32_t pick = -1;
    uint64_t draws = h->draws;
    int32_t read_cursor = h->read_cursor;
    if (h->mode == IMPACT_SAMPLE_UNIFORM) {
        const uint64_t u = splitmix64_at(h->seed, draws++);
        // floor(u * live / 2^64): unbiased up to 2^-64, no modulo
        uint64_t j = (uint64_t)(((unsigned __int128)u * (uint64_t)live) >> 64);
        for (int32_t s = 0; s < h->N; ++s) {
            if (!h->valid[s]) continue;
            if (j == 0) { pick = s; break; }
            --j;
        }
    } else {
        for (int32_t i = 0; i < h->N; ++i) {
            const int32_t s = (read_cursor + i) % h->N;
            if (h->valid[s]) { pick = s; break; }
        }
        read_cursor = (pick + 1) % h->N;
    }
    if (gather_dst) {
        CopySegments segs;
        segs.n = 0;
        for (int f = 0; f < h->n_fields; ++f)
            if (gather_dst[f]) add_segment(segs, h->field_ptr(pick, f), gather_dst[f], h->field_bytes[f]);
        int32_t st = launch_copy(segs, static_cast<cudaStream_t>(stream));
        if (st != IMPACT_OK) return st;  // bookkeeping untouched on failure
    }
    h->draws = draws;
    h->read_cursor = read_cursor;
    *slot_out = pick;
    *k_before_out = h->count[pick];
    h->count[pick] += 1;
    if (h->count[pick] >= h->K) h->valid[pick] = 0;
    return IMPACT_OK;
}

extern "C" int32_t impact_buffer_append(impact_buffer* h, int32_t slot, int32_t field, const void* src,
                                        void* stream) {
    if (!h || !src || slot < 0 || slot >= h->N || field < 0 || field >= h->n_fields || !aligned16(src))
        return IMPACT_ERR_INVALID_ARG;
    CopySegments segs;
    segs.n = 0;
    add_segment(segs, src, h->field_ptr(slot, field), h->field_bytes[field]);
    return launch_copy(segs, static_cast<cudaStream_t>(stream));
}

extern "C" void* impact_buffer_slot_ptr(impact_buffer* h, int32_t slot, int32_t field) {
    if (!h || slot < 0 || slot >= h->N || field < 0 || field >= h->n_fields) return nullptr;
    return h->field_ptr(slot, field);
}

// Brings the host copy of the bookkeeping up to date with the device's (device mode only); synchronises `stream`.
static int32_t download_state(impact_buffer* h, cudaStream_t cs) {
    const RingDeviceView v = h->view();
    RingDeviceHeader hd;
    IMPACT_CUDA_TRY(cudaMemcpyAsync(&hd, v.hd, sizeof(hd), cudaMemcpyDeviceToHost, cs));
    IMPACT_CUDA_TRY(cudaMemcpyAsync(h->valid.data(), v.valid, sizeof(int32_t) * (size_t)h->N, cudaMemcpyDeviceToHost, cs));
    IMPACT_CUDA_TRY(cudaMemcpyAsync(h->count.data(), v.count, sizeof(int32_t) * (size_t)h->N, cudaMemcpyDeviceToHost, cs));
    IMPACT_CUDA_TRY(cudaStreamSynchronize(cs));
    h->write_cursor = hd.write_cursor;
    h->read_cursor = hd.read_cursor;
    h->draws = hd.draws;
    return IMPACT_OK;
}

extern "C" int32_t impact_buffer_device_begin(impact_buffer* h, void* stream) {
    if (!h || h->device_mode) return IMPACT_ERR_INVALID_ARG;
    if (h->N > kMaxDeviceSlots) return IMPACT_ERR_UNSUPPORTED;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (!h->device_state) {
        void* mem = nullptr;
        IMPACT_CUDA_TRY(cudaMalloc(&mem, h->device_state_bytes()));
        h->device_state = static_cast<char*>(mem);
    }
    IMPACT_CUDA_TRY(cudaMemsetAsync(h->device_state, 0, h->device_state_bytes(), cs));
    const RingDeviceView v = h->view();
    RingDeviceHeader hd = {};
    hd.write_cursor = h->write_cursor;
    hd.read_cursor = h->read_cursor;
    hd.draws = h->draws;
    // (pageable sources: the copies have read them when the calls return)
    IMPACT_CUDA_TRY(cudaMemcpyAsync(v.hd, &hd, sizeof(hd), cudaMemcpyHostToDevice, cs));
    IMPACT_CUDA_TRY(cudaMemcpyAsync(v.valid, h->valid.data(), sizeof(int32_t) * (size_t)h->N, cudaMemcpyHostToDevice, cs));
    IMPACT_CUDA_TRY(cudaMemcpyAsync(v.count, h->count.data(), sizeof(int32_t) * (size_t)h->N, cudaMemcpyHostToDevice, cs));
    h->device_mode = true;
    return IMPACT_OK;
}

extern "C" int32_t impact_buffer_device_end(impact_buffer* h, void* stream) {
    if (!h || !h->device_mode) return IMPACT_ERR_INVALID_ARG;
    const int32_t st = download_state(h, static_cast<cudaStream_t>(stream));
    if (st != IMPACT_OK) return st;
    h->device_mode = false;
    return IMPACT_OK;
}

extern "C" int32_t impact_buffer_device_step(impact_buffer* h, const impact_ring_field_map* map,
                                             const void* learner_logits, const float* values,
                                             const float* bootstrap_values, const void* const* push_sources,
                                             int32_t n_candidates, impact_loss_inputs* inputs_out, void* stream) {
    if (!h || !h->device_mode) return IMPACT_ERR_INVALID_ARG;
    if (push_sources && (n_candidates < 1 || (reinterpret_cast<uintptr_t>(push_sources) & 7u) != 0)) return IMPACT_ERR_INVALID_ARG;
    impact_ring_field_map m = {-1, -1, -1, -1, -1};
    if (inputs_out) {
        if (!map || !aligned16(inputs_out)) return IMPACT_ERR_INVALID_ARG;
        m = *map;
        const int32_t* fs = &m.actions;
        for (int i = 0; i < 5; ++i)
            if (fs[i] < -1 || fs[i] >= h->n_fields) return IMPACT_ERR_INVALID_ARG;
    } else if (!push_sources) {
        return IMPACT_ERR_INVALID_ARG;  // nothing to do
    }
    const DeviceInfo* di = current_device_info();
    if (!di) return IMPACT_ERR_CUDA;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const RingDeviceView v = h->view();
    IMPACT_CUDA_TRY(launch_serialized(ring_step_kernel, dim3(1), dim3(32), 0, cs, v, m, learner_logits, values,
                                      bootstrap_values, push_sources, n_candidates, inputs_out ? 1 : 0, inputs_out));
    if (push_sources) {
        unsigned long long units = 0;
        for (int f = 0; f < h->n_fields; ++f) units += (h->field_bytes[f] + 15) / 16;
        // (a grid of two blocks per SM: most steps find every slot live and copy nothing, and an empty launch should
        // cost as little as possible)
        int blocks = blocks_for(units, 4, di);
        if (blocks > 2 * di->sm_count) blocks = 2 * di->sm_count;
        IMPACT_CUDA_TRY(launch_serialized(multi_copy_planned_kernel, dim3(blocks), dim3(256), 0, cs,
                                          static_cast<const CopySegments*>(v.plan)));
    }
    return IMPACT_OK;
}

extern "C" int32_t impact_buffer_device_events(impact_buffer* h, int32_t* events_out, int32_t max_events,
                                               int32_t* n_out, void* stream) {
    if (!h || !h->device_mode || !events_out || !n_out || max_events < 1) return IMPACT_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const RingDeviceView v = h->view();
    RingDeviceHeader hd;
    std::vector<int4> log((size_t)kEventLog);
    IMPACT_CUDA_TRY(cudaMemcpyAsync(&hd, v.hd, sizeof(hd), cudaMemcpyDeviceToHost, cs));
    IMPACT_CUDA_TRY(cudaMemcpyAsync(log.data(), v.events, sizeof(int4) * (size_t)kEventLog, cudaMemcpyDeviceToHost, cs));
    IMPACT_CUDA_TRY(cudaStreamSynchronize(cs));
    uint32_t have = hd.n_events < (uint32_t)kEventLog ? hd.n_events : (uint32_t)kEventLog;
    if (have > (uint32_t)max_events) have = (uint32_t)max_events;
    for (uint32_t i = 0; i < have; ++i) {  // oldest first
        const int4 e = log[(hd.n_events - have + i) % kEventLog];
        events_out[4 * i + 0] = e.x; events_out[4 * i + 1] = e.y; events_out[4 * i + 2] = e.z; events_out[4 * i + 3] = e.w;
    }
    *n_out = (int32_t)have;
    return IMPACT_OK;
}

extern "C" int32_t impact_buffer_live(const impact_buffer* h) {
    if (!h) return IMPACT_ERR_INVALID_ARG;
    if (h->device_mode) {
        const int32_t st = download_state(const_cast<impact_buffer*>(h), nullptr);
        if (st != IMPACT_OK) return st;
    }
    int32_t live = 0;
    for (int32_t s = 0; s < h->N; ++s) live += h->valid[s] ? 1 : 0;
    return live;
}

extern "C" size_t impact_buffer_state_bytes(const impact_buffer* h) {
    if (!h) return 0;
    return sizeof(StateHeader) + 2 * sizeof(int32_t) * (size_t)h->N;
}

extern "C" int32_t impact_buffer_export_state(const impact_buffer* h, void* blob, size_t blob_bytes) {
    if (!h || !blob || blob_bytes < impact_buffer_state_bytes(h)) return IMPACT_ERR_INVALID_ARG;
    if (h->device_mode) {  // the device holds the truth: fetch it (default stream; synchronises)
        const int32_t st = download_state(const_cast<impact_buffer*>(h), nullptr);
        if (st != IMPACT_OK) return st;
    }
    StateHeader hd;
    memset(&hd, 0, sizeof(hd));
    hd.magic = kStateMagic; hd.version = 1;
    hd.N = h->N; hd.K = h->K; hd.n_fields = h->n_fields; hd.mode = h->mode;
    hd.write_cursor = h->write_cursor; hd.read_cursor = h->read_cursor;
    hd.seed = h->seed; hd.draws = h->draws;
    char* out = static_cast<char*>(blob);
    memcpy(out, &hd, sizeof(hd));
    memcpy(out + sizeof(hd), h->valid.data(), sizeof(int32_t) * (size_t)h->N);
    memcpy(out + sizeof(hd) + sizeof(int32_t) * (size_t)h->N, h->count.data(), sizeof(int32_t) * (size_t)h->N);
    return IMPACT_OK;
}

extern "C" int32_t impact_buffer_import_state(impact_buffer* h, const void* blob, size_t blob_bytes) {
    if (!h || !blob || blob_bytes < impact_buffer_state_bytes(h) || h->device_mode) return IMPACT_ERR_INVALID_ARG;
    StateHeader hd;
    const char* in = static_cast<const char*>(blob);
    memcpy(&hd, in, sizeof(hd));
    if (hd.magic != kStateMagic || hd.version != 1 || hd.N != h->N || hd.K != h->K ||
        hd.n_fields != h->n_fields || (hd.mode != IMPACT_SAMPLE_UNIFORM && hd.mode != IMPACT_SAMPLE_ROUND_ROBIN))
        return IMPACT_ERR_INVALID_ARG;
    if (hd.write_cursor < 0 || hd.write_cursor >= h->N || hd.read_cursor < 0 || hd.read_cursor >= h->N)
        return IMPACT_ERR_INVALID_ARG;
    const int32_t* v = reinterpret_cast<const int32_t*>(in + sizeof(hd));
    const int32_t* c = v + h->N;
    for (int32_t s = 0; s < h->N; ++s)
        if ((v[s] != 0 && v[s] != 1) || c[s] < 0 || c[s] > h->K) return IMPACT_ERR_INVALID_ARG;
    h->mode = hd.mode; h->seed = hd.seed; h->draws = hd.draws;
    h->write_cursor = hd.write_cursor; h->read_cursor = hd.read_cursor;
    h->valid.assign(v, v + h->N);
    h->count.assign(c, c + h->N);
    return IMPACT_OK;
}

extern "C" int32_t impact_gather_rows(const void* src, const int32_t* idx, int64_t n, int64_t n_src_rows,
                                      size_t row_bytes, void* dst, void* stream) {
    if (!src || !idx || !dst || n < 0 || n_src_rows < 1 || row_bytes == 0) return IMPACT_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(idx) & 3u) != 0) return IMPACT_ERR_INVALID_ARG;
    if (n == 0) return IMPACT_OK;
    const DeviceInfo* di = current_device_info();
    if (!di) return IMPACT_ERR_CUDA;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const uintptr_t both = reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst) | row_bytes;
    if ((both & 15u) == 0) {
        const long long units = (long long)(row_bytes / 16);
        IMPACT_CUDA_TRY(launch_serialized(gather_rows_kernel<uint4>, dim3(blocks_for((unsigned long long)n * units, 4, di)), dim3(256), 0, cs,
                                          static_cast<const uint4*>(src), idx, (long long)n, (long long)n_src_rows, units, static_cast<uint4*>(dst)));
    } else if ((both & 3u) == 0) {
        const long long units = (long long)(row_bytes / 4);
        IMPACT_CUDA_TRY(launch_serialized(gather_rows_kernel<uint32_t>, dim3(blocks_for((unsigned long long)n * units, 4, di)), dim3(256), 0, cs,
                                          static_cast<const uint32_t*>(src), idx, (long long)n, (long long)n_src_rows, units, static_cast<uint32_t*>(dst)));
    } else {
        const long long units = (long long)row_bytes;
        IMPACT_CUDA_TRY(launch_serialized(gather_rows_kernel<unsigned char>, dim3(blocks_for((unsigned long long)n * units, 4, di)), dim3(256), 0, cs,
                                          static_cast<const unsigned char*>(src), idx, (long long)n, (long long)n_src_rows, units, static_cast<unsigned char*>(dst)));
    }
    IMPACT_CUDA_TRY(cudaGetLastError());
    return IMPACT_OK;
}

extern "C" int32_t impact_stream_copy(const void* src, size_t read_bytes, void* dst, size_t write_bytes, void* stream) {
    if (!src || !dst || !aligned16(src) || !aligned16(dst) || read_bytes == 0 || write_bytes > read_bytes ||
        (read_bytes & 15u) != 0 || (write_bytes & 15u) != 0 || write_bytes < 16)
        return IMPACT_ERR_INVALID_ARG;
    const DeviceInfo* di = current_device_info();
    if (!di) return IMPACT_ERR_CUDA;
    const unsigned long long n_read = read_bytes / 16, n_write = write_bytes / 16;
    IMPACT_CUDA_TRY(launch_serialized(stream_copy_kernel, dim3(blocks_for(n_read, 4, di)), dim3(256), 0,
                                      static_cast<cudaStream_t>(stream), static_cast<const uint4*>(src), n_read,
                                      static_cast<uint4*>(dst), n_write, reinterpret_cast<unsigned int*>(dst)));
    return IMPACT_OK;
}
