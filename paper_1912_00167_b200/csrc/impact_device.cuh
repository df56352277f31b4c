// Device building blocks of the fused IMPACT loss kernels (sm_100a).
//
// Work decomposition shared by all loss kernels:
//   * one thread per time step ("row"); a tile is up to NT consecutive rows of the row-major
//     [B*T, width] tensors, which is one contiguous slab of global memory;
//   * short trajectories (T <= NT) are packed, floor(NT/T) whole trajectories per tile; long
//     ones are cut into tiles that are linked by one scalar (swept from the END backwards inside
//     one block) or by published affine aggregates (tiles on different blocks) -- either way
//     every byte is read once;
//   * slabs reach shared memory by bulk asynchronous copies (one instruction per slab) and
//     keep their dense layout; gradients overwrite the staged rows in place and leave by bulk
//     stores;
//   * sums are reduced in a fixed order: per thread, per warp, per block, and across blocks
//     either by the last block to arrive (ticket) or, in the persistent kernels, by one
//     collecting group that reads every block's tagged row.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace impact {
namespace dev {

constexpr int kNumSums = 7;  // surrogate, value, entropy, kl, clipped, rho-truncated, ratio

// ---- 16-byte vectors of storage elements ---------------------------------------------
template <typename T> struct Pack;
template <> struct Pack<float> {
    static constexpr int kElems = 4;
    static __device__ __forceinline__ void unpack(const uint4& v, float (&f)[4]) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ uint4 pack(const float (&f)[4]) {
        return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]),
                          __float_as_uint(f[2]), __float_as_uint(f[3]));
    }
    static __device__ __forceinline__ float to_float(float x) { return x; }
    static __device__ __forceinline__ float from_float(float x) { return x; }
};
template <> struct Pack<__nv_bfloat16> {
    static constexpr int kElems = 8;
    static __device__ __forceinline__ void unpack(const uint4& v, float (&f)[8]) {
        // a bf16 is the upper half of an fp32: widening is a shift, exact
        f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
        f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
        f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xFFFF0000u);
        f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xFFFF0000u);
    }
    static __device__ __forceinline__ uint32_t two(float lo, float hi) {
        __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);  // round to nearest even
        return *reinterpret_cast<uint32_t*>(&h);
    }
    static __device__ __forceinline__ uint4 pack(const float (&f)[8]) {
        return make_uint4(two(f[0], f[1]), two(f[2], f[3]), two(f[4], f[5]), two(f[6], f[7]));
    }
    static __device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
    static __device__ __forceinline__ __nv_bfloat16 from_float(float x) { return __float2bfloat16_rn(x); }
};

__device__ __forceinline__ uint4 ld_stream16(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream16(uint4* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// ---- bulk asynchronous copies (the 1-D form of the tensor memory accelerator) -----------
// One elected thread moves a whole contiguous slab between global and shared memory; the
// other threads spend no instructions on staging.  Source, destination and size must be
// multiples of 16 bytes.  Loads signal an mbarrier in shared memory; stores are tracked by
// bulk async-groups.  No multicast and no cluster: every copy is local to the block.
__device__ __forceinline__ uint32_t smem_addr(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbarrier_init(uint64_t* bar, uint32_t arrivals) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(arrivals) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
// Initialisation of many barriers: each without a fence, then one fence_mbarrier_init() by every
// initialising thread before the block-wide barrier that precedes their first use.
__device__ __forceinline__ void mbarrier_init_nofence(uint64_t* bar, uint32_t arrivals) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(arrivals) : "memory");
}
__device__ __forceinline__ void fence_mbarrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbarrier_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbarrier_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
// Waits for the phase with the given parity to complete.  The wait is bounded: if the
// bytes never arrive the caller gets `false` instead of a hang.
__device__ __forceinline__ bool mbarrier_wait(uint64_t* bar, uint32_t parity) {
    const uint32_t addr = smem_addr(bar);
    // each try may sleep up to the hint and a failed try backs off 64 ns: the wait gives up after
    // somewhere between ~0.07 s and ~1.1 s, far beyond any copy's latency, far short of a hang
    constexpr uint32_t kSuspendHintNs = 1000;
    for (uint32_t tries = 0; tries < (1u << 20); ++tries) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(addr), "r"(parity), "r"(kSuspendHintNs) : "memory");
        if (done) return true;
        __nanosleep(64);  // a failed try returns early on this part: back off instead of spinning
    }
    return false;
}
// One look at the barrier, without waiting: has the phase with the given parity completed?
__device__ __forceinline__ bool mbarrier_test(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return done != 0;
}
// The same wait for blocks in which several warps wait on one another's barriers: it also gives up
// (at once) when `*abort_flag` is set, and sets it when it gives up itself, so that one wait that
// runs out ends every other wait of the block instead of each running out in turn.
__device__ __forceinline__ bool mbarrier_wait(uint64_t* bar, uint32_t parity, int* abort_flag) {
    const uint32_t addr = smem_addr(bar);
    // (no suspend hint and no sleep between tries: the wait sits between a tile's landing and the first
    // instruction that uses it, and a hinted try followed by a 64 ns sleep measured 0.1 us per launch slower)
    for (uint32_t tries = 0; tries < (1u << 24); ++tries) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
        if (*reinterpret_cast<volatile int*>(abort_flag)) return false;
    }
    *reinterpret_cast<volatile int*>(abort_flag) = 1;
    return false;
}
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(smem_dst)), "l"(__cvta_generic_to_global(gmem_src)), "r"(bytes),
                 "r"(smem_addr(bar)) : "memory");
}
// Asks L2 to fetch a contiguous range (16-byte aligned, a multiple of 16 bytes); nothing waits for it.
__device__ __forceinline__ void bulk_prefetch_l2(const void* gmem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(__cvta_generic_to_global(gmem_src)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_store(void* gmem_dst, const void* smem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(__cvta_generic_to_global(gmem_dst)), "r"(smem_addr(smem_src)), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// Shared memory written by ordinary stores becomes visible to the copy engine.
__device__ __forceinline__ void fence_async_shared() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// All bulk stores of this thread have finished READING shared memory (it may be reused).
__device__ __forceinline__ void bulk_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

// ---- byte ranges that do not start or end on a 16-byte boundary ---------------------------
// A tile of a dense tensor starts wherever its first row does: for row pitches that are not a
// multiple of 16 bytes (A = 18 in bf16: 36 bytes) most tiles start and end inside a 16-byte
// granule, which a bulk copy cannot do.  Loads are therefore widened to the enclosing granules:
// the copy also brings the up to 15 bytes before the range and the up to 15 bytes after it (the
// tensor's own neighbouring rows) into the padding of the shared-memory slab, and the range
// itself lands at the same offset inside its granule as in global memory.  Only where the tensor
// ENDS inside the last granule is that granule fetched by ordinary loads instead.
struct WideRange {
    long long first;  // byte offset (in the tensor) of the first granule
    uint32_t span;    // bytes a bulk copy may move from there: a multiple of 16, possibly 0
    uint32_t tail;    // bytes after the span that belong to the tensor's last, partial granule (0..15)
};
__device__ __forceinline__ WideRange widen_range(long long byte0, uint32_t bytes, long long tensor_bytes) {
    WideRange w;
    const uint32_t m = (uint32_t)byte0 & 15u;
    w.first = byte0 - m;
    w.span = (m + bytes + 15u) & ~15u;
    w.tail = 0;
    if (w.first + (long long)w.span > tensor_bytes) {
        w.span -= 16u;
        w.tail = (uint32_t)(tensor_bytes - (w.first + (long long)w.span));
    }
    return w;
}
// Asks L2 for the granules of a byte range of a tensor whose base is 16-byte aligned (one request to the copy
// engine; nothing waits for it).  Ordinary per-line prefetch instructions were tried instead and slowed the
// launches down by half.
__device__ __forceinline__ void prefetch_range_l2(const void* base, long long byte0, uint32_t bytes, long long tensor_bytes) {
    const WideRange w = widen_range(byte0, bytes, tensor_bytes);
    if (w.span) bulk_prefetch_l2(static_cast<const unsigned char*>(base) + w.first, w.span);
}

// Run by a whole warp: sends `bytes` bytes of shared memory at `src` to global memory at `dst`, where src and
// dst agree modulo 16.  The whole granules in between leave by one bulk store (lane 0); the up to 15 bytes before
// the first whole granule and after the last one leave by byte stores, a lane each (a granule shared with a
// neighbouring range is written by both neighbours, each its own bytes).  `wrote`: the bytes were written by
// ordinary stores of this warp's threads, so they are fenced towards the copy engine first.  Lane 0 learns
// whether a bulk store was issued (its group is committed; see bulk_store_wait_read).
__device__ __forceinline__ bool warp_send_bytes(unsigned char* dst, const unsigned char* src, uint32_t bytes, bool wrote) {
    const uint32_t lane = threadIdx.x & 31u;
    if ((((uint32_t)reinterpret_cast<uintptr_t>(dst) | bytes) & 15u) == 0u) {  // whole granules only: the usual case
        if (wrote) fence_async_shared();
        __syncwarp();
        if (lane == 0 && bytes) {
            bulk_store(dst, src, bytes);
            return true;
        }
        return false;
    }
    uint32_t head = (16u - ((uint32_t)reinterpret_cast<uintptr_t>(dst) & 15u)) & 15u;
    if (head > bytes) head = bytes;
    const uint32_t body = (bytes - head) & ~15u;
    const uint32_t tail = bytes - head - body;
    if (wrote) fence_async_shared();
    __syncwarp();
    if (lane < head) dst[lane] = src[lane];
    if (lane >= 16u && lane - 16u < tail) dst[head + body + lane - 16u] = src[head + body + lane - 16u];
    if (lane == 0 && body) {
        bulk_store(dst + head, src + head, body);
        return true;
    }
    return false;
}

__device__ __forceinline__ float exp2_fast(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float log2_fast(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_fast(float x) {
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Sum of one value over the warp, in every lane (fixed order).
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
    return x;
}
// Sums of four values over the warp in one butterfly of six shuffles: lanes 0-7 return the
// total of `a`, lanes 8-15 of `b`, lanes 16-23 of `c`, lanes 24-31 of `d` (fixed order).
__device__ __forceinline__ float warp_sum4(float a, float b, float c, float d) {
    const int lane = threadIdx.x & 31;
    const bool hi16 = (lane & 16) != 0, hi8 = (lane & 8) != 0;
    float k0 = hi16 ? c : a, k1 = hi16 ? d : b;
    const float s0 = hi16 ? a : c, s1 = hi16 ? b : d;
    k0 += __shfl_xor_sync(0xffffffffu, s0, 16);
    k1 += __shfl_xor_sync(0xffffffffu, s1, 16);
    float x = hi8 ? k1 : k0;
    const float y = hi8 ? k0 : k1;
    x += __shfl_xor_sync(0xffffffffu, y, 8);
    x += __shfl_xor_sync(0xffffffffu, x, 4);
    x += __shfl_xor_sync(0xffffffffu, x, 2);
    x += __shfl_xor_sync(0xffffffffu, x, 1);
    return x;
}

// Walks (row, col) positions of a dense [rows, W] slab in steps of a fixed element count.
struct RowCol {
    int r, c;
    __device__ __forceinline__ void init(int e, int W) { r = e / W; c = e - r * W; }
    __device__ __forceinline__ void advance(int dq, int dr, int W) {
        r += dq; c += dr;
        if (c >= W) { c -= W; ++r; }
    }
};

// Stage `nelem` consecutive elements of `src`, starting at element `base`, into shared
// rows of stride `Ws` floats (element e of the slab lands at [e / W][e % W]).
template <typename ST, int NT>
__device__ __forceinline__ void stage_slab(float* __restrict__ dst, const ST* __restrict__ src,
                                           long long base, int nelem, int W, int Ws) {
    constexpr int VE = Pack<ST>::kElems;
    const int tid = threadIdx.x;
    int done = 0;
    if ((base % VE) == 0) {
        const int nvec = nelem / VE;
        const uint4* s4 = reinterpret_cast<const uint4*>(src + base);
        const int dq = (NT * VE) / W, dr = (NT * VE) % W;
        RowCol rc; rc.init(tid * VE, W);
        int v = tid;
        constexpr int U = 4;
        for (; v + (U - 1) * NT < nvec; v += U * NT) {
            uint4 x[U];
#pragma unroll
            for (int u = 0; u < U; ++u) x[u] = ld_stream16(s4 + v + u * NT);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float f[VE];
                Pack<ST>::unpack(x[u], f);
                int rr = rc.r, cc = rc.c;
#pragma unroll
                for (int j = 0; j < VE; ++j) {
                    dst[rr * Ws + cc] = f[j];
                    if (++cc == W) { cc = 0; ++rr; }
                }
                rc.advance(dq, dr, W);
            }
        }
        for (; v < nvec; v += NT) {
            uint4 x = ld_stream16(s4 + v);
            float f[VE];
            Pack<ST>::unpack(x, f);
            int rr = rc.r, cc = rc.c;
#pragma unroll
            for (int j = 0; j < VE; ++j) {
                dst[rr * Ws + cc] = f[j];
                if (++cc == W) { cc = 0; ++rr; }
            }
            rc.advance(dq, dr, W);
        }
        done = nvec * VE;
    }
    if (done + tid < nelem) {  // unaligned slab, or the last few elements of an aligned one
        const int dq = NT / W, dr = NT % W;
        RowCol rc; rc.init(done + tid, W);
        for (int e = done + tid; e < nelem; e += NT) {
            dst[rc.r * Ws + rc.c] = Pack<ST>::to_float(src[base + e]);
            rc.advance(dq, dr, W);
        }
    }
}

// The reverse of stage_slab: write the shared rows back to a dense global slab.
template <typename ST, int NT>
__device__ __forceinline__ void unstage_slab(ST* __restrict__ dst, const float* __restrict__ src,
                                             long long base, int nelem, int W, int Ws) {
    constexpr int VE = Pack<ST>::kElems;
    const int tid = threadIdx.x;
    int done = 0;
    if ((base % VE) == 0) {
        const int nvec = nelem / VE;
        uint4* d4 = reinterpret_cast<uint4*>(dst + base);
        const int dq = (NT * VE) / W, dr = (NT * VE) % W;
        RowCol rc; rc.init(tid * VE, W);
        for (int v = tid; v < nvec; v += NT) {
            float f[VE];
            int rr = rc.r, cc = rc.c;
#pragma unroll
            for (int j = 0; j < VE; ++j) {
                f[j] = src[rr * Ws + cc];
                if (++cc == W) { cc = 0; ++rr; }
            }
            st_stream16(d4 + v, Pack<ST>::pack(f));
            rc.advance(dq, dr, W);
        }
        done = nvec * VE;
    }
    if (done + tid < nelem) {
        const int dq = NT / W, dr = NT % W;
        RowCol rc; rc.init(done + tid, W);
        for (int e = done + tid; e < nelem; e += NT) {
            dst[base + e] = Pack<ST>::from_float(src[rc.r * Ws + rc.c]);
            rc.advance(dq, dr, W);
        }
    }
}

// ---- backward recursion as a suffix scan of affine maps ----------------------------------
// Each thread i holds the map f_i(x) = a*x + b of its time step
// (A_i = delta_i + (lambda gamma_i c_i) A_{i+1}).  Returns A_i = f_i(f_{i+1}(... f_{NT-1}(carry))).
// Affine maps compose associatively, so the recursion is a scan: shuffles inside a warp,
// one shared-memory hop across warps.  Contains one __syncthreads().
// `next` receives A_{i+1}, the value the thread's own map was applied to (the carry for the last row).
template <int NT>
__device__ __forceinline__ float suffix_affine_scan(float a, float b, float carry, float2* warp_agg, float& next) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const float a2 = __shfl_down_sync(0xffffffffu, a, off);
        const float b2 = __shfl_down_sync(0xffffffffu, b, off);
        if (lane + off < 32) {
            b = fmaf(a, b2, b);
            a = a * a2;
        }
    }
    if (lane == 0) warp_agg[warp] = make_float2(a, b);
    __syncthreads();
    float x = carry;
#pragma unroll 1
    for (int w = NT / 32 - 1; w > warp; --w) {
        const float2 g = warp_agg[w];
        x = fmaf(g.x, x, g.y);
    }
    const float result = fmaf(a, x, b);
    const float below = __shfl_down_sync(0xffffffffu, result, 1);
    next = (lane == 31) ? x : below;
    return result;
}

// The same scan inside a group of NT threads that synchronises on named barrier `bar_id`
// (trajectories never continue past a tile here, so there is no carry).
template <int NT>
__device__ __forceinline__ float suffix_affine_scan_group(float a, float b, float2* warp_agg, float& next, int bar_id) {
    const int lane = threadIdx.x & 31, warp = (threadIdx.x & (NT - 1)) >> 5;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const float a2 = __shfl_down_sync(0xffffffffu, a, off);
        const float b2 = __shfl_down_sync(0xffffffffu, b, off);
        if (lane + off < 32) {
            b = fmaf(a, b2, b);
            a = a * a2;
        }
    }
    if (lane == 0) warp_agg[warp] = make_float2(a, b);
    asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "n"(NT) : "memory");
    float x = 0.0f;
#pragma unroll
    for (int w = NT / 32 - 1; w > 0; --w) {
        const float2 g = warp_agg[w];
        if (w > warp) x = fmaf(g.x, x, g.y);
    }
    const float result = fmaf(a, x, b);
    const float below = __shfl_down_sync(0xffffffffu, result, 1);
    next = (lane == 31) ? x : below;
    return result;
}

// The same scan with R rows per thread: a group of NTH threads covers NTH * R consecutive steps, warp w the steps
// [32 R w, 32 R (w + 1)), lane l of it the steps 32 R w + 32 i + l for i < R (a lane's rows are 32 apart, which
// keeps its accesses to rows of shared memory on the banks a single row per lane would use).  a[i], b[i] are the
// rows' maps; res[i] receives A of row i, next[i] the value row i's map was applied to (0 after the last step).
template <int NTH, int R>
__device__ __forceinline__ void suffix_affine_scan_rows(float (&a)[R], float (&b)[R], float2* warp_agg, float (&res)[R],
                                                        float (&next)[R], int bar_id) {
    const int lane = threadIdx.x & 31, warp = (threadIdx.x & (NTH - 1)) >> 5;
#pragma unroll
    for (int i = 0; i < R; ++i) {
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const float a2 = __shfl_down_sync(0xffffffffu, a[i], off);
            const float b2 = __shfl_down_sync(0xffffffffu, b[i], off);
            if (lane + off < 32) {
                b[i] = fmaf(a[i], b2, b[i]);
                a[i] = a[i] * a2;
            }
        }
    }
    // inside the warp: the maps of the later sub-segments follow those of the earlier ones
#pragma unroll
    for (int i = R - 2; i >= 0; --i) {
        const float ta = __shfl_sync(0xffffffffu, a[i + 1], 0), tb = __shfl_sync(0xffffffffu, b[i + 1], 0);
        b[i] = fmaf(a[i], tb, b[i]);
        a[i] = a[i] * ta;
    }
    float x = 0.0f;
    if constexpr (NTH > 32) {
        if (lane == 0) warp_agg[warp] = make_float2(a[0], b[0]);
        asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "n"(NTH) : "memory");
#pragma unroll
        for (int w = NTH / 32 - 1; w > 0; --w) {
            const float2 g = warp_agg[w];
            if (w > warp) x = fmaf(g.x, x, g.y);
        }
    }
#pragma unroll
    for (int i = 0; i < R; ++i) res[i] = fmaf(a[i], x, b[i]);
#pragma unroll
    for (int i = 0; i < R; ++i) {
        const float below = __shfl_down_sync(0xffffffffu, res[i], 1);
        float first_after = x;  // what follows this sub-segment's last row
        if (i + 1 < R) first_after = __shfl_sync(0xffffffffu, res[i + 1], 0);
        next[i] = (lane == 31) ? first_after : below;
    }
}

// The scan as maps, for tiles that do not know yet what enters their last step: (ma, mb) is the
// composition of the maps of this thread's step and all later steps of the tile, (la, lb) that of
// all steps after this thread's warp (the identity for the last warp).  Thread 0's (ma, mb) is the
// tile's aggregate.
template <int NT>
__device__ __forceinline__ void suffix_affine_maps_group(float a, float b, float2* warp_agg, float& ma, float& mb,
                                                         float& la, float& lb, int bar_id) {
    const int lane = threadIdx.x & 31, warp = (threadIdx.x & (NT - 1)) >> 5;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const float a2 = __shfl_down_sync(0xffffffffu, a, off);
        const float b2 = __shfl_down_sync(0xffffffffu, b, off);
        if (lane + off < 32) {
            b = fmaf(a, b2, b);
            a = a * a2;
        }
    }
    if (lane == 0) warp_agg[warp] = make_float2(a, b);
    asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "n"(NT) : "memory");
    la = 1.0f;
    lb = 0.0f;
#pragma unroll
    for (int w = NT / 32 - 1; w > 0; --w) {
        const float2 g = warp_agg[w];
        if (w > warp) {  // (la, lb) <- g o (la, lb)
            lb = fmaf(g.x, lb, g.y);
            la = g.x * la;
        }
    }
    ma = a * la;
    mb = fmaf(a, lb, b);
}

__device__ __forceinline__ void publish_tagged(unsigned long long* slot, float value, unsigned int tag);

// A tile's aggregate map, published as two (value, launch tag) pairs (see publish_tagged).
__device__ __forceinline__ void publish_tile_aggregate(unsigned long long* slot, float a, float b, unsigned int tag) {
    publish_tagged(slot, a, tag);
    publish_tagged(slot + 1, b, tag);
}

// The two slots of the aggregate of the tile `j` places later in this tile's trajectory (they lie j * stride
// before `mine`), as they are right now.  The values are not looked at here, so the load can be issued long before
// it is needed.
__device__ __forceinline__ void load_aggregate(const unsigned long long* mine, long long stride, int j,
                                               unsigned long long& va, unsigned long long& vb) {
    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(va), "=l"(vb) : "l"(mine - (long long)j * stride) : "memory");
}

// Run by one warp: `mine` points at this tile's pair of slots; tile j (1 = the nearest later tile ... r = the
// trajectory's last) has its slots at mine - j * stride.  Reads their aggregates (a lane each, 32 at a time,
// waiting -- bounded -- until a pair carries this launch's tag), composes them in time order and returns the
// composition applied to 0: the value that enters this tile's last step.  `peeked` / (pa, pb): lane l brings along
// what load_aggregate found earlier for tile r - l; it counts if it carries the tag.
__device__ __forceinline__ float compose_later_aggregates(const unsigned long long* mine, long long stride, int r,
                                                          unsigned int tag, int* abort_flag, bool peeked,
                                                          unsigned long long pa, unsigned long long pb) {
    const int lane = threadIdx.x & 31;
    // the value flows from tile r down to tile 1: x <- agg_j(x).  Lanes take j = r - lane, r - lane - 32, ...:
    // chunk by chunk from the far end, lane 0 holding the map that is applied first.
    float x = 0.0f;
    for (int base = r; base > 0; base -= 32) {
        const int j = base - lane;
        float a = 1.0f, b = 0.0f;  // identity for lanes beyond the chunk
        if (j > 0) {
            unsigned long long va = pa, vb = pb;
            bool ok = peeked && base == r && ((unsigned int)(va >> 32) == tag) && ((unsigned int)(vb >> 32) == tag);
            for (int tries = 0; tries < (1 << 22) && !ok; ++tries) {
                load_aggregate(mine, stride, j, va, vb);
                ok = ((unsigned int)(va >> 32) == tag) && ((unsigned int)(vb >> 32) == tag);
                if (!ok && *reinterpret_cast<volatile int*>(abort_flag)) break;
            }
            if (!ok) *reinterpret_cast<volatile int*>(abort_flag) = 1;
            a = __uint_as_float((unsigned int)va);
            b = __uint_as_float((unsigned int)vb);
        }
        // compose over the warp: lane l ends up with map_{l+31} o ... o map_l; lane 0's is the chunk's
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const float a2 = __shfl_down_sync(0xffffffffu, a, off);
            const float b2 = __shfl_down_sync(0xffffffffu, b, off);
            if (lane + off < 32) {  // (a, b) <- (a2, b2) o (a, b): the higher lane's map is applied later
                b = fmaf(a2, b, b2);
                a = a2 * a;
            }
        }
        const float ca = __shfl_sync(0xffffffffu, a, 0), cb = __shfl_sync(0xffffffffu, b, 0);
        x = fmaf(ca, x, cb);
    }
    return x;
}

// Scalars of the loss that the kernels need; filled on the host.
struct LossScalars {
    float rho_bar, c_bar, clip_lo, clip_hi;
    float vf_coef, ent_coef, kl_coef, lambda_, log_rho_tw;
    float inv_M;
    int is_source, ratio_mode, objective;
    double steps_total;  // M: the steps the means are taken over (this call's, or the whole batch's when it is split)
};

// Per-step quantities once the three log-probabilities are known.
struct StepIn {
    float l_theta, l_target, l_worker;  // may all be shifted by one common amount ...
    float l_shift = 0.0f;               // ... which is this: l_theta + l_shift is the true log-probability
    float reward, discount, value, value_next;
    bool last_step;  // t == T-1: the trace stops, V_{t+1} is the bootstrap value
    float rho = 0.0f;       // truncated importance weight of the step (set by recursion_map)
    float adv_next = 0.0f;  // A_{t+1} (set from the scan)
};

// Truncated importance weights and the affine map of the advantage recursion
// (Section 2.2; Section 3.1).  Returns whether exp(x) exceeded rho_bar.
// exp of a log-probability difference.  Arguments are a few units at most, where the
// multiply-then-exp2 form stays within ~3e-7 relative of the correctly rounded result.
__device__ __forceinline__ float exp_of_logratio(float x) { return exp2_fast(x * 1.4426950408889634f); }

__device__ __forceinline__ bool recursion_map(StepIn& s, const LossScalars& k, float& a, float& b) {
    const float x = (k.is_source == 1 ? s.l_theta : s.l_target) - s.l_worker;
    const float w = (k.is_source == 2) ? 1.0f : exp_of_logratio(x);  // 2: plain GAE, no importance weights
    const float rho = fminf(k.rho_bar, w);
    s.rho = rho;
    const float c = fminf(k.c_bar, w);
    b = rho * (s.reward + s.discount * s.value_next - s.value);
    a = s.last_step ? 0.0f : k.lambda_ * s.discount * c;
    return w > k.rho_bar;
}

// Ratio of Section 4.1 and the eps-clipped surrogate of Appendix E.  Returns the weight
// adv * R of the policy-gradient term (0 where the clip removes it).
__device__ __forceinline__ float surrogate(const StepIn& s, const LossScalars& k, float adv,
                                           float& surr, float& ratio, bool& clipped) {
    if (k.objective == 1) {
        // IMPALA's actor update (Section 2.2): weight rho_t (r_t + gamma_t v_{t+1} - V_t) on
        // grad log pi_theta, v the V-trace target V + A (the bootstrap value after the last step)
        const float v_next = s.value_next + (s.last_step ? 0.0f : s.adv_next);
        const float w = s.rho * (s.reward + s.discount * v_next - s.value);
        surr = w * (s.l_theta + s.l_shift);
        ratio = s.rho;
        clipped = false;
        return w;
    }
    float d;
    if (k.ratio_mode == 1) d = s.l_target;
    else if (k.ratio_mode == 2) d = s.l_worker;
    else d = fmaxf(s.l_target, s.l_worker - k.log_rho_tw);
    const float R = exp_of_logratio(s.l_theta - d);
    const float Rc = fminf(fmaxf(R, k.clip_lo), k.clip_hi);
    surr = fminf(R * adv, Rc * adv);
    clipped = (adv > 0.0f && R > k.clip_hi) || (adv < 0.0f && R < k.clip_lo);
    ratio = R;
    return clipped ? 0.0f : adv * R;
}

// The two functions above for the default configuration (importance weights pi_target / pi_worker,
// ratio R3, clipped surrogate), without the run-time switches.
__device__ __forceinline__ bool recursion_map_plain(StepIn& s, const LossScalars& k, float& a, float& b) {
    const float w = exp_of_logratio(s.l_target - s.l_worker);
    const float rho = fminf(k.rho_bar, w);
    s.rho = rho;
    const float c = fminf(k.c_bar, w);
    b = rho * (s.reward + s.discount * s.value_next - s.value);
    a = s.last_step ? 0.0f : k.lambda_ * s.discount * c;
    return w > k.rho_bar;
}
__device__ __forceinline__ float surrogate_plain(const StepIn& s, const LossScalars& k, float adv, float& surr,
                                                 float& ratio, bool& clipped) {
    const float d = fmaxf(s.l_target, s.l_worker - k.log_rho_tw);
    const float R = exp_of_logratio(s.l_theta - d);
    const float Rc = fminf(fmaxf(R, k.clip_lo), k.clip_hi);
    surr = fminf(R * adv, Rc * adv);
    clipped = (adv > 0.0f && R > k.clip_hi) || (adv < 0.0f && R < k.clip_lo);
    ratio = R;
    return clipped ? 0.0f : adv * R;
}

// Sum the kNumSums per-thread values over the block (fixed order) and add them to `acc`,
// which only thread 0 keeps.  `red` is [NT/32][8] shared floats.  The caller must place a
// __syncthreads() between the write phase and the read phase: call stage 1, sync, stage 2.
template <int NT>
__device__ __forceinline__ void block_sums_stage1(float (&v)[kNumSums], float (*red)[8]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int j = 0; j < kNumSums; ++j) {
        float x = v[j];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
        if (lane == 0) red[warp][j] = x;
    }
}
template <int NT>
__device__ __forceinline__ void block_sums_stage2(float (&acc)[kNumSums], float (*red)[8]) {
    if (threadIdx.x == 0) {
#pragma unroll
        for (int j = 0; j < kNumSums; ++j) {
            float x = 0.0f;
            for (int w = 0; w < NT / 32; ++w) x += red[w][j];
            acc[j] += x;
        }
    }
}

// Last step of every loss kernel: publish this block's sums, and let the block that
// finishes last add all blocks' sums in index order (fp64) and write the eight loss terms.
// `counter` must be 0 on entry to the kernel and is 0 again on exit.
template <int NT>
__device__ __forceinline__ void finish_loss_terms(const float (&acc)[kNumSums], float* partials,
                                                  unsigned int* counter, float* loss_terms,
                                                  const LossScalars& k, double M) {
    __shared__ bool is_last;
    __shared__ double dred[NT / 32][kNumSums];
    if (threadIdx.x == 0) {
#pragma unroll
        for (int j = 0; j < kNumSums; ++j) partials[(size_t)blockIdx.x * 8 + j] = acc[j];
        __threadfence();
        const unsigned int ticket = atomicAdd(counter, 1u);
        is_last = (ticket == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    double s[kNumSums];
#pragma unroll
    for (int j = 0; j < kNumSums; ++j) s[j] = 0.0;
    for (unsigned int blk = threadIdx.x; blk < gridDim.x; blk += NT) {
        const float4 p0 = __ldcg(reinterpret_cast<const float4*>(partials + (size_t)blk * 8));
        const float4 p1 = __ldcg(reinterpret_cast<const float4*>(partials + (size_t)blk * 8 + 4));
        s[0] += p0.x; s[1] += p0.y; s[2] += p0.z; s[3] += p0.w;
        s[4] += p1.x; s[5] += p1.y; s[6] += p1.z;
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int j = 0; j < kNumSums; ++j) {
        double x = s[j];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
        if (lane == 0) dred[warp][j] = x;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double t[kNumSums];
#pragma unroll
        for (int j = 0; j < kNumSums; ++j) {
            double x = 0.0;
            for (int w = 0; w < NT / 32; ++w) x += dred[w][j];
            t[j] = x / M;
        }
        const double l_pi = -t[0], l_v = t[1], ent = t[2], kl = t[3];
        loss_terms[0] = (float)(l_pi + (double)k.vf_coef * l_v - (double)k.ent_coef * ent +
                                (double)k.kl_coef * kl);
        loss_terms[1] = (float)l_pi;
        loss_terms[2] = (float)l_v;
        loss_terms[3] = (float)ent;
        loss_terms[4] = (float)kl;
        loss_terms[5] = (float)t[4];
        loss_terms[6] = (float)t[5];
        loss_terms[7] = (float)t[6];
        *counter = 0u;
    }
}

// ---- early publication of a block's sums ---------------------------------------------------
// Thread 0 calls this as soon as its block's last sums are final, long before the block's
// stores are done: the fence and the counter's round trip then overlap the rest of the
// block's work instead of extending it.  Returns the block's ticket (0-based arrival order).
__device__ __forceinline__ unsigned int publish_block_sums(const float (&acc)[kNumSums], float* partials,
                                                           unsigned int* counter) {
    float4* row = reinterpret_cast<float4*>(partials + (size_t)blockIdx.x * 8);
    row[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
    row[1] = make_float4(acc[4], acc[5], acc[6], 0.0f);
    // one acq_rel atomic: releases this block's row and, for the block that draws the last ticket,
    // acquires every other block's (their atomics on the counter form the release sequence)
    unsigned int ticket;
    asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(ticket) : "l"(counter) : "memory");
    return ticket;
}
// Run by every thread of the block that drew the last ticket: add all blocks' sums in index
// order (fp64), write the eight loss terms, and leave the counter at 0 for the next launch.
template <int NT>
__device__ __noinline__ void reduce_published_sums(const float* partials, unsigned int* counter, float* loss_terms,
                                                      float vf_coef, float ent_coef, float kl_coef, double M) {
    __shared__ double dred[NT / 32][kNumSums];
    // thread 0 acquired the rows with its ticket and a block barrier lies between that and here;
    // the loads below go to L2 (ld.cg), so no further fence is needed
    double s[kNumSums];
#pragma unroll
    for (int j = 0; j < kNumSums; ++j) s[j] = 0.0;
    // rows in batches of eight per thread, all loads of a batch in flight together
    constexpr int kBatch = 8;
    for (unsigned int first = threadIdx.x; first < gridDim.x; first += NT * kBatch) {
        float4 p0[kBatch], p1[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const unsigned int blk = first + u * NT;
            if (blk < gridDim.x) {
                p0[u] = __ldcg(reinterpret_cast<const float4*>(partials + (size_t)blk * 8));
                p1[u] = __ldcg(reinterpret_cast<const float4*>(partials + (size_t)blk * 8 + 4));
            } else {
                p0[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                p1[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            s[0] += p0[u].x; s[1] += p0[u].y; s[2] += p0[u].z; s[3] += p0[u].w;
            s[4] += p1[u].x; s[5] += p1[u].y; s[6] += p1[u].z;
        }
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int j = 0; j < kNumSums; ++j) {
        double x = s[j];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
        if (lane == 0) dred[warp][j] = x;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const double inv_m = 1.0 / M;
        double t[kNumSums];
#pragma unroll
        for (int j = 0; j < kNumSums; ++j) {
            double x = 0.0;
            for (int w = 0; w < NT / 32; ++w) x += dred[w][j];
            t[j] = x * inv_m;
        }
        const double l_pi = -t[0], l_v = t[1], ent = t[2], kl = t[3];
        loss_terms[0] = (float)(l_pi + (double)vf_coef * l_v - (double)ent_coef * ent +
                                (double)kl_coef * kl);
        loss_terms[1] = (float)l_pi;
        loss_terms[2] = (float)l_v;
        loss_terms[3] = (float)ent;
        loss_terms[4] = (float)kl;
        loss_terms[5] = (float)t[4];
        loss_terms[6] = (float)t[5];
        loss_terms[7] = (float)t[6];
        *counter = 0u;
    }
}

// ---- sums published as tagged rows (persistent kernel) --------------------------------------
// Every launch that uses a workspace has a number, kept in the workspace's third counter word: the
// launch's tag is that word + 1 (never 0, which is what a cleared workspace holds), and the launch's
// collecting group stores the tag back as its last act.  A group's row is eight (value, tag) pairs,
// each written by ONE aligned 8-byte store, which the memory model makes indivisible: a reader that
// sees this launch's tag in a pair sees this launch's value beside it.  So rows need no fence, no
// atomic counter and no "last block" -- the collecting group simply reads every row until all its
// pairs carry the tag (a bounded wait), and adds them in index order.
__device__ __forceinline__ unsigned int launch_tag(const unsigned int* counter_words) {
    unsigned int n;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(n) : "l"(counter_words + 2) : "memory");
    return n + 1u == 0u ? 1u : n + 1u;
}
__device__ __forceinline__ void publish_tagged(unsigned long long* slot, float value, unsigned int tag) {
    const unsigned long long v = ((unsigned long long)tag << 32) | (unsigned long long)__float_as_uint(value);
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(slot), "l"(v) : "memory");
}

// The block's row of sums.  Every consumer warp, once its sums are final, leaves them in its row of shared memory
// -- [surrogate, value, entropy, kl, clipped, truncated, ratio, 0] -- and draws a ticket from a counter in shared
// memory; the producer warp draws one too, after it has left this launch's tag there.  Whoever draws the last
// ticket adds all rows in index order (so the result does not depend on who that is) and publishes the block's row
// of (value, tag) pairs.  A pair is one 8-byte store, so whoever reads the tag of this launch reads this launch's
// value with it: no fence, no round trip.  The tickets are acquire-release operations on one word: the last
// drawer sees every row and the tag.  (Before, the producer warp polled one barrier per group and published: its
// row left 0.35-0.5 us after the last group's sums were final.)
template <int C, int WPG>
__device__ __forceinline__ void draw_ticket_and_publish(unsigned int* tickets, const unsigned int* tag_s,
                                                        float (*red)[WPG][8], unsigned long long* tagged_rows) {
    const int lane = threadIdx.x & 31;
    unsigned int t = 0;
    __syncwarp();
    if (lane == 0)
        asm volatile("atom.acq_rel.cta.shared::cta.add.u32 %0, [%1], 1;" : "=r"(t) : "r"(smem_addr(tickets)) : "memory");
    __syncwarp();
    t = __shfl_sync(0xffffffffu, t, 0);
    if (t == (unsigned int)(C * WPG) && lane < 8) {  // C * WPG consumer warps and the producer warp: the last of C * WPG + 1
        float y = 0.0f;
#pragma unroll
        for (int c = 0; c < C; ++c) {
            float yc = 0.0f;
#pragma unroll
            for (int w = 0; w < WPG; ++w) yc += red[c][w][lane];
            y = (c == 0) ? yc : y + yc;
        }
        publish_tagged(tagged_rows + (size_t)blockIdx.x * 8 + lane, y, *reinterpret_cast<const volatile unsigned int*>(tag_s));
    }
}
// A consumer warp's part (called by every thread of the warp): a butterfly into the warp's row, then the ticket.
template <int C, int WPG>
__device__ __forceinline__ void hand_over_warp_sums(float t_surr, float t_val, float t_ent, float t_ratio, float t_kl,
                                                    bool want_kl, int n_clip, int n_trunc, float* warp_row,
                                                    unsigned int* tickets, const unsigned int* tag_s,
                                                    float (*red)[WPG][8], unsigned long long* tagged_rows) {
    const int lane = threadIdx.x & 31;
    const float x = warp_sum4(t_surr, t_val, t_ent, t_ratio);
    const float xk = want_kl ? warp_sum(t_kl) : 0.0f;
    if ((lane & 7) == 0) warp_row[lane == 24 ? 6 : (lane >> 3)] = x;
    if (lane == 0) {
        warp_row[3] = xk;
        warp_row[4] = (float)n_clip;
        warp_row[5] = (float)n_trunc;
        warp_row[7] = 0.0f;
    }
    draw_ticket_and_publish<C, WPG>(tickets, tag_s, red, tagged_rows);
}

// Run by the NT threads of one group (`gtid` in the group, named barrier `bar_id`): waits for `nrows`
// tagged rows, adds them, writes the eight loss terms and advances the workspace's launch number.
// Thread t owns column t % 8 of rows t / 8, t / 8 + NT / 8, ...: a row is read by eight neighbouring
// lanes (64 contiguous bytes) and all of a thread's loads are in flight together, so a grid's worth of rows
// costs one trip to L2.  The sum is a fixed fp32 tree (each thread its rows in index order, then lanes,
// then warps) -- the rows are fp32 sums over whole tiles already.  Returns false if a row never showed up.
template <int NT>
__device__ __noinline__ bool reduce_tagged_rows(const unsigned long long* rows, int nrows, unsigned int tag,
                                                  unsigned int* counter_words, float* loss_terms, float vf_coef,
                                                  float ent_coef, float kl_coef, double M, int gtid, int bar_id,
                                                  int* abort_flag) {
    __shared__ float fred[NT / 32][8];
    constexpr int kStride = NT / 8, kU = 10;
    const int col = gtid & 7, rc = gtid >> 3;
    const double inv_m = 1.0 / M;  // (a long division: done while the rows are still on their way)
    float acc = 0.0f;
    bool missing = false;
    for (int base = rc; base < nrows && !missing; base += kStride * kU) {
        unsigned long long v[kU];
        unsigned int have = 0;
#pragma unroll
        for (int u = 0; u < kU; ++u)
            if (base + kStride * u >= nrows) have |= 1u << u;  // beyond the last row: nothing to wait for
        for (int tries = 0; tries < (1 << 22) && have != (1u << kU) - 1u; ++tries) {
#pragma unroll
            for (int u = 0; u < kU; ++u)
                if (!(have & (1u << u)))
                    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];"
                                 : "=l"(v[u]) : "l"(rows + (size_t)(base + kStride * u) * 8 + col) : "memory");
#pragma unroll
            for (int u = 0; u < kU; ++u)
                if (!(have & (1u << u)) && (unsigned int)(v[u] >> 32) == tag) have |= 1u << u;
            if (have != (1u << kU) - 1u && *reinterpret_cast<volatile int*>(abort_flag)) break;
        }
        if (have != (1u << kU) - 1u) missing = true;
#pragma unroll
        for (int u = 0; u < kU; ++u)
            if (base + kStride * u < nrows) acc += __uint_as_float((unsigned int)v[u]);
    }
    if (missing) *reinterpret_cast<volatile int*>(abort_flag) = 1;  // read back below, after the group's barrier
    const int lane = gtid & 31, warp = gtid >> 5;
    acc += __shfl_xor_sync(0xffffffffu, acc, 8);
    acc += __shfl_xor_sync(0xffffffffu, acc, 16);
    if (lane < 8) fred[warp][lane] = acc;
    asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "n"(NT) : "memory");
    // the last steps sit between the slowest block's row and the end of the launch: a lane per column
    if (gtid < 8) {
        float x = 0.0f;
#pragma unroll
        for (int w = 0; w < NT / 32; ++w) x += fred[w][gtid];
        const double t = (double)x * inv_m;  // columns: surrogate, value, entropy, kl, clipped, truncated, ratio
        const double t1 = __shfl_sync(0xffu, t, 1), t2 = __shfl_sync(0xffu, t, 2), t3 = __shfl_sync(0xffu, t, 3);
        if (gtid == 0) {
            loss_terms[0] = (float)(-t + (double)vf_coef * t1 - (double)ent_coef * t2 + (double)kl_coef * t3);
            counter_words[2] = tag;
        }
        if (gtid < kNumSums) loss_terms[gtid + 1] = (float)(gtid == 0 ? -t : t);
    }
    return *reinterpret_cast<volatile int*>(abort_flag) == 0;
}

}  // namespace dev
}  // namespace impact
