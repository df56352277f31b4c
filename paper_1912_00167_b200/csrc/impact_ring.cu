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
    if (h->owns_storage) {
        cudaError_t e = cudaDeviceSynchronize();
        if (e == cudaSuccess) e = cudaFree(h->storage);
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
    if (!h || !field_src || !slot_out) return IMPACT_ERR_INVALID_ARG;
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
    if (!h || !slot_out || !k_before_out) return IMPACT_ERR_INVALID_ARG;
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

extern "C" int32_t impact_buffer_live(const impact_buffer* h) {
    if (!h) return IMPACT_ERR_INVALID_ARG;
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
    if (!h || !blob || blob_bytes < impact_buffer_state_bytes(h)) return IMPACT_ERR_INVALID_ARG;
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
