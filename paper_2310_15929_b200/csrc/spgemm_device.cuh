// Device and host helpers shared by the GEMM translation units: kernel parameters, barrier / bulk-copy / tcgen05 wrappers,
// descriptors, the tensor-map encoder.  Everything here has internal linkage.
#pragma once

#include "esp_common.cuh"

#include <cuda.h>

#include <cstdio>
#include <cstdlib>

namespace esp {
namespace {

constexpr uint32_t kSpinLimit = 1u << 22;

// Host-side caches of what a repeated call would otherwise redo (a decode call is a few microseconds of GPU time: the
// host must not take longer).  All thread-local: no lock on the call path.
//
// The opt-in shared-memory size of a kernel sticks to the function: it is raised once per kernel, device and size.
inline cudaError_t ensure_dynamic_smem(const void *kern, int bytes) {
    struct Entry { const void *kern; int dev, bytes; };
    thread_local Entry cache[96];
    thread_local int n = 0;
    int dev = 0;
    cudaGetDevice(&dev);
    for (int i = 0; i < n; ++i)
        if (cache[i].kern == kern && cache[i].dev == dev) {
            if (cache[i].bytes >= bytes) return cudaSuccess;
            const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
            if (e == cudaSuccess) cache[i].bytes = bytes;
            return e;
        }
    const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess && n < 96) cache[n++] = Entry{kern, dev, bytes};
    return e;
}
inline bool log_plans() {
    static const bool on = getenv("ESP_LOG") != nullptr;
    return on;
}

struct GemmParams {
    const __half *X;
    long ldx;
    int M, K, N;
    int x_channel_major;
    const uint8_t *packed;
    const int32_t *perm;
    void *Y;
    long ldy;
    int out_f32;
    int k_tiles;             // ceil(K / 128)
    int k_tiles_per_split;
    const uint8_t *ximg;     // tiled pair kernel: permuted X as shared-memory images (written by xtile_kernel)
    const uint32_t *xflags;  // one word per image: 1 once it is complete
    const __half *bias;      // [N] added to every token row before the activation, or NULL
    int act;                 // ESP_ACT_*
    int raster_panel;        // pair kernel: token tiles per panel of the cluster -> tile map (0 / 1 = row by row)
};

// Up to ESP_MAX_GROUP independent products in one launch of the streaming kernel: the feature tiles of the problems
// follow each other along grid.x (problem i owns tiles [ft_start[i], ft_start[i + 1])); M, K and the launch shape are common.
struct GemmGroup {
    int count;
    int ft_start[ESP_MAX_GROUP + 1];
    GemmParams p[ESP_MAX_GROUP];
};

// Bias and activation on the finished fp32 sum of one output element (never on a K-slice's partial sum).  The bias of a
// feature is fetched once per thread (epilogue_bias) and applied to all of that feature's tokens (epilogue_apply).
__device__ __forceinline__ float epilogue_bias(const GemmParams &p, long feature) {
    float b = 0.f;
    if (p.bias != nullptr && feature < p.N) {
        // volatile: the fp16 overload of __ldg is a plain (non-volatile) asm statement, which the compiler may execute
        // ahead of the null test above; with bias == NULL that read address 2 * feature and faulted
        unsigned short h;
        asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(h) : "l"(p.bias + feature));
        b = __half2float(__ushort_as_half(h));
    }
    return b;
}
__device__ __forceinline__ float epilogue_apply(float acc, float bias, int act) {
    acc += bias;
    return act == ESP_ACT_RELU ? fmaxf(acc, 0.f) : acc;
}
__device__ __forceinline__ float epilogue_value(const GemmParams &p, float acc, long feature) {
    return epilogue_apply(acc, epilogue_bias(p, feature), p.act);
}

// ---------------------------------------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls (or when another thread of the CTA gave up), records
// ESP_ERR_TIMEOUT in the device status word and lets the caller fall through to the common exit.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 128) {
            if (*abort_flag) return false;
            __nanosleep(64);
        }
    }
    *abort_flag = 1;
    atomicExch(&g_device_status, (int)ESP_ERR_TIMEOUT);
    return false;
}

__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// shared memory (128 rows x 16 bytes, rows 16 bytes apart) -> 4 tensor-memory columns of all 128 lanes
__device__ __forceinline__ void tc_copy_128x128b(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::1.128x128b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
// D[tmem] (+)= A_sparse[smem] * B[smem], fp16 inputs, K = 32 channels (16 stored values per row of A)
__device__ __forceinline__ void tc_mma_sparse_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t e_tmem,
                                                  uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.sp.cta_group::1.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(e_tmem), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tmem_load_16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float ld_dsmem_f32(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}

// Shared-memory matrix descriptor of the tensor-core instructions (address, leading / stride byte
// offsets in 16-byte units, descriptor version 1, swizzle mode in the top bits).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)layout << 61;
    return d;
}
constexpr uint32_t kLayoutNone = 0, kLayoutSw128 = 2;

// Instruction descriptor, kind::f16: sparse flag (bit 2), fp32 accumulator (bits 4-5 = 1), fp16 A and B
// (formats 0), A K-major, B major as given (bit 16), N >> 3 (bits 17-22), M >> 4 (bits 24-28).
__host__ __device__ constexpr uint32_t instr_desc_sparse_f16(int mma_m, int mma_n, int b_mn_major) {
    return (1u << 2) | (1u << 4) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(mma_n >> 3) << 17) |
           ((uint32_t)(mma_m >> 4) << 24);
}

__host__ __device__ constexpr int tmem_cols_for(int bn) { return bn + 8 <= 32 ? 32 : bn + 8 <= 64 ? 64 : bn + 8 <= 128 ? 128 : bn + 8 <= 256 ? 256 : 512; }

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_arrive_noinc(uint32_t bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    return remote;
}
__device__ __forceinline__ void st_remote_f32(uint32_t remote_addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote_addr), "f"(v) : "memory");
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t remote_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}
__device__ __forceinline__ void fence_cluster() { asm volatile("fence.acq_rel.cluster;" ::: "memory"); }
// Bounded wait with cluster-scope acquire (the arrivals come from other CTAs of the cluster).
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
        if (i > 128) {
            if (*abort_flag) return false;
            __nanosleep(64);
        }
    }
    *abort_flag = 1;
    atomicExch(&g_device_status, (int)ESP_ERR_TIMEOUT);
    return false;
}

// Bounded wait for an image flag (set by a CTA of the tiling pass that is resident before this kernel can start).
__device__ __forceinline__ bool xflag_wait(const uint32_t *flag, volatile int *abort_flag) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        uint32_t v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
        if (v == 1u) return true;
        if (i > 8) {
            if (*abort_flag) return false;
            __nanosleep(128);
        }
    }
    *abort_flag = 1;
    atomicExch(&g_device_status, (int)ESP_ERR_TIMEOUT);
    return false;
}

constexpr int kMaxStages = 12;
constexpr int kPermRing = 16;        // stages of permutation entries kept ahead in shared memory

// Asynchronous remote stores: the data lands in the target CTA's shared memory and its byte count completes on the
// target's mbarrier, so the receiver needs no fence and the sender no separate arrive.
__device__ __forceinline__ void st_async_b32(uint32_t remote_addr, uint32_t v, uint32_t remote_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];" ::"r"(remote_addr), "r"(v),
                 "r"(remote_bar)
                 : "memory");
}
__device__ __forceinline__ void st_async_v2(uint32_t remote_addr, uint32_t a, uint32_t b, uint32_t remote_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.b32 [%0], {%1, %2}, [%3];" ::"r"(remote_addr),
                 "r"(a), "r"(b), "r"(remote_bar)
                 : "memory");
}
__device__ __forceinline__ void st_async_v4(uint32_t remote_addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d,
                                            uint32_t remote_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(remote_addr),
                 "r"(a), "r"(b), "r"(c), "r"(d), "r"(remote_bar)
                 : "memory");
}
__device__ __forceinline__ float4 ld_dsmem_v4(uint32_t local_addr, uint32_t rank) {
    float4 v;
    const uint32_t remote = map_to_rank(local_addr, rank);
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(remote) : "memory");
    return v;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
inline esp_status_t tensor_map_encoder(EncodeTiledFn *out) {
    static EncodeTiledFn encode = nullptr;
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn)
            return ESP_ERR_CUDA;
        encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    *out = encode;
    return ESP_OK;
}

}  // namespace
}  // namespace esp
