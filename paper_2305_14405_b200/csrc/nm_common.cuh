// Shared device/host pieces of the NeuralMatrix B200 library: the context, the
// device-resident PWL table and its evaluation primitive, and raw sm_100a PTX
// wrappers (mbarrier, TMA, tcgen05) with bounded waits.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/nm_b200.h"

// ---------------------------------------------------------------- tables ------

// One PWL table as kernels see it (Section 3.2: k and b pre-stored, indexed by
// segment number).  kb[s] = (k_s, b_s).
struct NmTable {
    int32_t n;
    float inv_h;  // (float)(n / (x_max - x_min))
    float off;    // (float)(-x_min * n / (x_max - x_min))
    float x_min, x_max;
    int32_t loaded;
    int32_t pad[2];
    float2 kb[NM_MAX_SEGMENTS];
};

struct NmProfRecord {
    cudaEvent_t start, stop;
    int kind;
    double work;
};
#define NM_PROF_MAX 8192

struct nm_ctx {
    int device;
    NmTable* d_tables;         // NM_NUM_SLOTS tables in device memory
    NmTable h_tables[NM_NUM_SLOTS];
    int* d_status;             // device status word (nm_status)
    int sm_count;
    int64_t launches;
    void* encode_tiled;        // cuTensorMapEncodeTiled, resolved at create
    int profiling;             // nonzero: bracket every launch with events
    int prof_count;            // records in use
    int prof_created;          // event pairs created so far (kept for reuse)
    NmProfRecord* prof;        // NM_PROF_MAX records, host memory
    int pdl;                   // launch kernels with programmatic stream serialization (prologue overlap)
    int attn_resident;         // algo 0 prefers the attention kernel with the score block resident in TMEM
    void* static_ws;           // device address of the library's fixed scratch array on this device (or null)
    void* d_pool_w;            // 64 x 64 matrix (1/HW on the diagonal) of the average pool run as a GEMM; 8 KB
    int pool_w_hw, pool_w_dtype;   // what d_pool_w currently holds (0 = nothing)
};

// Brackets one kernel launch with events when profiling is on; counts the launch always.
struct NmLaunchScope {
    nm_ctx* ctx;
    cudaStream_t st;
    NmProfRecord* rec;
    NmLaunchScope(nm_ctx* c, int kind, double work, cudaStream_t s) : ctx(c), st(s), rec(nullptr)
    {
        ctx->launches++;
        if (!ctx->profiling || ctx->prof_count >= NM_PROF_MAX) return;
        NmProfRecord* r = &ctx->prof[ctx->prof_count];
        if (ctx->prof_count >= ctx->prof_created) {
            if (cudaEventCreate(&r->start) != cudaSuccess || cudaEventCreate(&r->stop) != cudaSuccess) return;
            ctx->prof_created = ctx->prof_count + 1;
        }
        r->kind = kind;
        r->work = work;
        ctx->prof_count++;
        rec = r;
        cudaEventRecord(r->start, st);
    }
    ~NmLaunchScope()
    {
        if (rec) cudaEventRecord(rec->stop, st);
    }
};

// Segment number of x: one fp32 fused multiply-add, floor, clamp to [0, n-1];
// inputs outside the range land in the end segments (Section 3.2.1), NaN in 0.
__device__ __forceinline__ int nm_pwl_index(float x, float inv_h, float off, float nm1)
{
    float u = __fmaf_rn(x, inv_h, off);
    u = fminf(fmaxf(u, 0.0f), nm1);
    return __float2int_rd(u);
}

// Per-lane replicated table in shared memory: entry s of lane l lives at
// rep[s * 32 + l], so a warp's 32 lookups with arbitrary s never collide on a bank pair.
__device__ __forceinline__ void nm_table_replicate(float2* rep, const NmTable* __restrict__ t, int n,
                                                   int tid, int nthreads)
{
    for (int i = tid; i < n * 32; i += nthreads) rep[i] = t->kb[i >> 5];
}

__device__ __forceinline__ float nm_pwl_eval_rep(const float2* rep, int lane, float x, float inv_h,
                                                 float off, float nm1, int* idx_out = nullptr)
{
    int s = nm_pwl_index(x, inv_h, off, nm1);
    if (idx_out) *idx_out = s;
    float2 kb = rep[s * 32 + lane];
    return __fmaf_rn(kb.x, x, kb.y);
}

// ---------------------------------------------------------------- dtypes ------

template <typename T> struct NmType;
template <> struct NmType<float> {
    static __device__ __forceinline__ float to_f(float v) { return v; }
    static __device__ __forceinline__ float from_f(float v) { return v; }
};
template <> struct NmType<__nv_bfloat16> {
    static __device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
    static __device__ __forceinline__ __nv_bfloat16 from_f(float v) { return __float2bfloat16_rn(v); }
};
template <> struct NmType<__half> {
    static __device__ __forceinline__ float to_f(__half v) { return __half2float(v); }
    static __device__ __forceinline__ __half from_f(float v) { return __float2half_rn(v); }
};

// q = clamp(rint(y * inv_scale), -127, 127), ties to even.  Clamped first and rounded in the conversion: the same
// integer for every input (the bounds are integers), one instruction fewer; NaN gives -127 either way.
__device__ __forceinline__ int8_t nm_quant_i8(float y, float inv_scale)
{
    const float v = fminf(fmaxf(y * inv_scale, -127.0f), 127.0f);
    return (int8_t)__float2int_rn(v);
}
// Four such codes packed into one word (byte 0 = a).  The lower bound is applied in fp32, the upper one by the
// saturating pack instruction: d = (c << 16) | (sat8(a) << 8) | sat8(b).
__device__ __forceinline__ uint32_t nm_quant_i8x4(float a, float b, float c, float d, float inv_scale)
{
    const int ia = __float2int_rn(fmaxf(a * inv_scale, -127.0f)), ib = __float2int_rn(fmaxf(b * inv_scale, -127.0f));
    const int ic = __float2int_rn(fmaxf(c * inv_scale, -127.0f)), id = __float2int_rn(fmaxf(d * inv_scale, -127.0f));
    uint32_t hi, w;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(id), "r"(ic), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(ib), "r"(ia), "r"(hi));
    return w;
}

// ---------------------------------------------------------------- PTX ---------

#define NM_WAIT_LIMIT_CYCLES (4000000000LL)  // ~2 s at 2 GHz: every device wait gives up after this

__device__ __forceinline__ uint32_t nm_smem_u32(const void* p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void nm_mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(nm_smem_u32(bar)), "r"(count));
}

__device__ __forceinline__ void nm_mbar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(nm_smem_u32(bar)), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void nm_mbar_arrive(uint64_t* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(nm_smem_u32(bar)) : "memory");
}

__device__ __forceinline__ bool nm_mbar_try_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(nm_smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Non-blocking test of an mbarrier phase (try_wait may suspend the thread for a while when the
// phase is not complete; a loop that polls several barriers wants an immediate answer).
__device__ __forceinline__ bool nm_mbar_test_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(nm_smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait on an mbarrier phase.  Gives up when another thread of the CTA has
// already given up (*abort_flag != 0) or after NM_WAIT_LIMIT_CYCLES; on expiry it
// records NM_ERR_TIMEOUT in the global status word, raises the CTA's abort flag
// and returns false.  The caller then skips its remaining work and falls through
// to the common teardown (no trap, no endless spin).
__device__ __forceinline__ bool nm_mbar_wait_limit(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                                   int* status, long long limit_cycles)
{
    if (nm_mbar_try_wait(bar, parity)) return true;
    long long t0 = clock64();
    uint32_t spins = 0;
    while (true) {
        if (nm_mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63u) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > limit_cycles) {
                *abort_flag = 1;
                atomicExch(status, (int)NM_ERR_TIMEOUT);
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool nm_mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                             int* status)
{
    return nm_mbar_wait_limit(bar, parity, abort_flag, status, NM_WAIT_LIMIT_CYCLES);
}

// The same bounded wait for warps that are NOT on the critical issue path (epilogue and
// softmax warps waiting for the tensor core): between polls the thread sleeps, so that a
// waiting warp does not take issue slots from the single thread that feeds the tensor core
// on the same scheduler.
template <unsigned SLEEP_NS = 40>
__device__ __forceinline__ bool nm_mbar_wait_relaxed(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                                     int* status)
{
    if (nm_mbar_try_wait(bar, parity)) return true;
    long long t0 = clock64();
    uint32_t spins = 0;
    while (true) {
        __nanosleep(SLEEP_NS);
        if (nm_mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63u) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > NM_WAIT_LIMIT_CYCLES) {
                *abort_flag = 1;
                atomicExch(status, (int)NM_ERR_TIMEOUT);
                return false;
            }
        }
    }
}

__device__ __forceinline__ void nm_fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void nm_fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// TMA: 2-D tiled load global -> shared, completion counted on an mbarrier.  c0 is
// the innermost (contiguous) coordinate and must be a multiple of 16 bytes.
__device__ __forceinline__ void nm_tma_load_2d(void* smem_dst, const CUtensorMap* tmap, int c0, int c1,
                                               uint64_t* bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(nm_smem_u32(smem_dst)), "l"(tmap), "r"(nm_smem_u32(bar)), "r"(c0), "r"(c1)
        : "memory");
}

__device__ __forceinline__ void nm_tma_load_3d(void* smem_dst, const CUtensorMap* tmap, int c0, int c1, int c2,
                                               uint64_t* bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(nm_smem_u32(smem_dst)), "l"(tmap), "r"(nm_smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

// 4-D tiled load (c0 innermost; NHWC activations as {channel, x, y, image}).  Coordinates beyond the tensor
// read the fill value (zero), which is how a convolution's border padding is produced.
__device__ __forceinline__ void nm_tma_load_4d(void* smem_dst, const CUtensorMap* tmap, int c0, int c1, int c2, int c3,
                                               uint64_t* bar)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(nm_smem_u32(smem_dst)), "l"(tmap), "r"(nm_smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}

// 4-D tiled store shared -> global as one bulk group; parts of the box beyond the tensor's extents are
// not written.  No coordinate may be negative.
__device__ __forceinline__ void nm_tma_store_4d(const CUtensorMap* tmap, const void* smem_src, int c0, int c1, int c2,
                                                int c3)
{
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(tmap),
                 "r"(nm_smem_u32(smem_src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

// TMA: 2-D tiled store shared -> global as one bulk group; parts of the box beyond the
// tensor's extents are not written.  c0 (innermost) must be a multiple of 16 bytes.
__device__ __forceinline__ void nm_tma_store_2d(const CUtensorMap* tmap, const void* smem_src, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(tmap),
                 "r"(nm_smem_u32(smem_src)), "r"(c0), "r"(c1)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// All earlier bulk stores of this thread have finished READING shared memory (the
// staging buffer may be overwritten; the global writes may still be in flight).
__device__ __forceinline__ void nm_tma_store_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

// PWL lookup for hot loops.  `rep_lane` is the shared::cta byte address of this lane's
// column of a 32-way replicated table (entry s of lane l at rep + (s*32 + l)*8).  The segment
// number is floor(clamp(fma(x, inv_h, off), 0, n-1)): the floor is taken by adding 1.5*2^23
// with round-toward-minus-infinity, which leaves floor(u) in the low mantissa bits (exact for
// 0 <= u < 2^22), and the table address is formed from those bits with one shift-add.
__device__ __forceinline__ float nm_pwl_fast(uint32_t rep_lane, float x, float inv_h, float off, float nm1,
                                             int* idx_out = nullptr)
{
    float u = __fmaf_rn(x, inv_h, off);
    u = fminf(fmaxf(u, 0.0f), nm1);
    const uint32_t bits = __float_as_uint(__fadd_rd(u, 12582912.0f));   // 0x4B400000 + floor(u)
    if (idx_out) *idx_out = (int)(bits - 0x4B400000u);
    // (bits << 8) = 0x40000000 + s*256 (mod 2^32); the constant is folded into the base
    const uint32_t addr = (bits << 8) + (rep_lane - 0x40000000u);
    float k, b;
    asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(k), "=f"(b) : "r"(addr));   // the table is read-only here
    return __fmaf_rn(k, x, b);
}

// Two values at once with the packed fp32 instructions (fma.rn.f32x2, add.rm.f32x2: each half is the same
// correctly rounded operation as the scalar form, so the results are those of nm_pwl_fast bit for bit).
__device__ __forceinline__ uint64_t nm_pack2(float a, float b)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void nm_unpack2(uint64_t v, float& a, float& b)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ void nm_pwl_fast2(uint32_t rep_lane, float& x0, float& x1, uint64_t inv_h2, uint64_t off2,
                                             float nm1)
{
    uint64_t u2;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(u2) : "l"(nm_pack2(x0, x1)), "l"(inv_h2), "l"(off2));
    float u0, u1;
    nm_unpack2(u2, u0, u1);
    u0 = fminf(fmaxf(u0, 0.0f), nm1);
    u1 = fminf(fmaxf(u1, 0.0f), nm1);
    uint64_t b2;
    asm("add.rm.f32x2 %0, %1, %2;" : "=l"(b2) : "l"(nm_pack2(u0, u1)), "l"(nm_pack2(12582912.0f, 12582912.0f)));
    float f0, f1;
    nm_unpack2(b2, f0, f1);
    const uint32_t a0 = (__float_as_uint(f0) << 8) + (rep_lane - 0x40000000u);
    const uint32_t a1 = (__float_as_uint(f1) << 8) + (rep_lane - 0x40000000u);
    float k0, c0, k1, c1;
    asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(k0), "=f"(c0) : "r"(a0));
    asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(k1), "=f"(c1) : "r"(a1));
    x0 = __fmaf_rn(k0, x0, c0);
    x1 = __fmaf_rn(k1, x1, c1);
}

__device__ __forceinline__ void nm_prefetch_tmap(const CUtensorMap* tmap)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(tmap) : "memory");
}

// Programmatic dependent launch: a kernel launched with the programmatic-stream-serialization
// attribute may start while its predecessor in the stream is still running; it must not touch
// memory the predecessor produces before nm_grid_dependency_wait() returns (which waits for the
// predecessor to complete and flush).  nm_grid_launch_dependents() lets the successor's CTAs be
// scheduled as soon as resources free up, so that its set-up overlaps this kernel's tail.
// Both are no-ops for a kernel launched without the attribute.
__device__ __forceinline__ void nm_grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void nm_grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- tcgen05 ------------------------------------------------------------------

__device__ __forceinline__ void nm_tmem_alloc(uint32_t* smem_slot, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(nm_smem_u32(smem_slot)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void nm_tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void nm_tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void nm_tc_fence_before()
{
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void nm_tc_fence_after()
{
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// All tcgen05.mma issued so far by this thread arrive (once) on `bar` when done.
__device__ __forceinline__ void nm_tc_commit(uint64_t* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                     nm_smem_u32(bar))
                 : "memory");
}

// One lane of a converged warp (always the same one for a full mask).  A warp that runs its loop
// with all lanes and issues the single-thread tcgen05 instructions under this predicate keeps its
// addresses, descriptors and counters warp-uniform, which the compiler can hold in uniform registers.
__device__ __forceinline__ bool nm_elect_one()
{
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}

// D[tmem] (+)= A[smem desc] * B[smem desc]; kind::f16 covers bf16 and fp16 inputs.
__device__ __forceinline__ void nm_mma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                           uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void nm_mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// ---- thread-block clusters and two-CTA tensor-core groups (cta_group::2) ----------

__device__ __forceinline__ uint32_t nm_cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the object at shared::cta address `addr` in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t nm_mapa(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// Arrival on a barrier that may live in the peer CTA.  Default (CTA-scope) release: what the arrival
// orders here are tcgen05 operations, which tcgen05.fence::before_thread_sync has already ordered; a
// cluster-scope release would in addition wait for every earlier global write of the thread.
__device__ __forceinline__ void nm_mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void nm_cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ bool nm_mbar_try_wait_cluster(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(nm_smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait, cluster-scope acquire (the arrivals come from the peer CTA as well).
__device__ __forceinline__ bool nm_mbar_wait_cluster(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                                     int* status)
{
    if (nm_mbar_try_wait_cluster(bar, parity)) return true;
    long long t0 = clock64();
    uint32_t spins = 0;
    while (true) {
        if (nm_mbar_try_wait_cluster(bar, parity)) return true;
        if ((++spins & 63u) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > NM_WAIT_LIMIT_CYCLES) {
                *abort_flag = 1;
                atomicExch(status, (int)NM_ERR_TIMEOUT);
                return false;
            }
        }
    }
}
// TMA load whose completion is counted on an mbarrier that may live in the peer CTA of a
// two-CTA group (`bar_cluster_addr` is a shared::cluster address).  Each CTA fetches its own
// operand slice into its own shared memory.
__device__ __forceinline__ void nm_tma_load_2d_2cta(void* smem_dst, const CUtensorMap* tmap, int c0, int c1,
                                                    uint32_t bar_cluster_addr)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(nm_smem_u32(smem_dst)), "l"(tmap), "r"(bar_cluster_addr), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void nm_tma_load_4d_2cta(void* smem_dst, const CUtensorMap* tmap, int c0, int c1, int c2,
                                                    int c3, uint32_t bar_cluster_addr)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(nm_smem_u32(smem_dst)), "l"(tmap), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void nm_tmem_alloc2(uint32_t* smem_slot, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(nm_smem_u32(smem_slot)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void nm_tmem_relinquish2()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void nm_tmem_dealloc2(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// Commit of a two-CTA group: arrives once on the barrier at the same shared-memory offset
// in every CTA named by `cta_mask`.
__device__ __forceinline__ void nm_tc_commit2(uint64_t* bar, uint16_t cta_mask)
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
            nm_smem_u32(bar)),
        "h"(cta_mask)
        : "memory");
}
// One MMA over both CTAs of the pair: M = 256 (128 rows of A and of D per CTA), B split
// along N between the two CTAs' shared memories.  Issued by the leader CTA only.
__device__ __forceinline__ void nm_mma_f16_2cta(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void nm_mma_i8_2cta(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Shared-memory operand descriptor, 128-byte swizzle, rows of 128 bytes, groups of
// 8 rows 1024 bytes apart.  Valid for a K-major operand whose K extent per tile is
// 128 bytes, and for an MN-major operand whose MN extent is 128 bytes (then the
// 8-row groups run along K).
__device__ __forceinline__ uint64_t nm_smem_desc_sw128(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);       // start address
    d |= (uint64_t)1 << 16;                             // leading byte offset (unused with swizzle)
    d |= (uint64_t)(1024 >> 4) << 32;                   // stride byte offset: 8 rows * 128 B
    d |= (uint64_t)1 << 46;                             // descriptor version (sm_100)
    d |= (uint64_t)2 << 61;                             // SWIZZLE_128B
    return d;
}

// Instruction descriptor: D format (1 = f32, 2 = s32), A/B format (f16 kinds:
// 0 = f16, 1 = bf16; i8 kind: 1 = signed), major-ness (0 = K-major), N>>3, M>>4.
__host__ __device__ constexpr uint32_t nm_idesc(uint32_t c_fmt, uint32_t ab_fmt, uint32_t a_mn_major,
                                                uint32_t b_mn_major, uint32_t M, uint32_t N)
{
    return (c_fmt << 4) | (ab_fmt << 7) | (ab_fmt << 10) | (a_mn_major << 15) | (b_mn_major << 16) |
           ((N >> 3) << 17) | ((M >> 4) << 24);
}

// Tensor-memory reads: 32 lanes x 32 (or 16) consecutive 32-bit columns into registers; thread l of the
// warp receives row (lane base + l).
// Load and wait in one statement: the registers are valid when it ends.  (While a tcgen05.ld is in flight
// its destination registers do not hold the data yet, and a compiler that sees them as ordinary values may
// copy or spill them before the wait -- a tied in/out operand on a separate wait statement is itself
// materialised as such a copy -- so the two are never separated.)
__device__ __forceinline__ void nm_tmem_ld32_sync(uint32_t taddr, uint32_t* r)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void nm_tmem_ld16_sync(uint32_t taddr, uint32_t* r)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}

// ---------------------------------------------------------------- host --------

#define NM_CUDA_TRY(expr)                         \
    do {                                          \
        cudaError_t _e = (expr);                  \
        if (_e != cudaSuccess) return NM_ERR_CUDA; \
    } while (0)

static inline bool nm_aligned16(const void* p) { return (((uintptr_t)p) & 15u) == 0; }
static inline size_t nm_dtype_size(nm_dtype t)
{
    switch (t) {
    case NM_F32: return 4;
    case NM_BF16: return 2;
    case NM_F16: return 2;
    case NM_I8: return 1;
    }
    return 0;
}

// kernels implemented in the other translation units
nm_status nm_launch_pwl_apply(nm_ctx* ctx, int slot, const void* x, void* y, int64_t count, nm_dtype dtype,
                              int32_t* idx_out, cudaStream_t st);
nm_status nm_launch_layernorm(nm_ctx* ctx, const void* x, const float* gamma, const float* beta, void* y,
                              int64_t rows, int32_t H, float eps, int32_t slot, int32_t slot2, nm_dtype dtype,
                              cudaStream_t st, int8_t* q = nullptr, float q_inv_scale = 0.f);
// slot2 != NM_SLOT_NONE: sqrt in slot, 1/x in slot2; q != nullptr: also the int8 codes of the stored output
nm_status nm_launch_wait_selftest(nm_ctx* ctx, long long limit_cycles, cudaStream_t st);
nm_status nm_launch_quantize(nm_ctx* ctx, const void* x, nm_dtype dtype, int64_t count, float inv_scale,
                             int8_t* q, cudaStream_t st);
nm_status nm_launch_linear_simt(nm_ctx* ctx, const nm_linear_desc* d, cudaStream_t st);
nm_status nm_launch_linear_tc(nm_ctx* ctx, const nm_linear_desc* d, cudaStream_t st);
bool nm_linear_tc_supported(const nm_linear_desc* d);
nm_status nm_launch_attention_simt(nm_ctx* ctx, const nm_attn_desc* d, cudaStream_t st);
nm_status nm_launch_attention_tc(nm_ctx* ctx, const nm_attn_desc* d, cudaStream_t st);
bool nm_attention_tc_supported(const nm_attn_desc* d);
// out_q != nullptr: the output is written as int8 codes (of the value rounded to the storage type) to out_q
// [B*L, heads*d] instead of d->out
nm_status nm_launch_attention_stream(nm_ctx* ctx, const nm_attn_desc* d, cudaStream_t st, int8_t* out_q = nullptr,
                                     float q_inv_scale = 0.f);
bool nm_attention_stream_supported(const nm_attn_desc* d);
nm_status nm_launch_attention_i8(nm_ctx* ctx, const nm_attn_i8_desc* d, cudaStream_t st);
// Implicit-GEMM convolution on the tensor-core kernel.  The A operand is described as a 4-D view
// {inner, x, y, image} of the activation (dims in elements, strides in bytes); K-block
// kb = (ky*taps_x + kx)*cblocks + cb reads the 64 inner elements cb*64.. at x = ox*sw - pw + kx,
// y = oy*sh - ph + ky for every output pixel (oy, ox) of the tile; W is [Cout, Ktot] with row pitch ldw.
struct NmConvTc {
    nm_dtype dtype;
    const void* a_base;
    uint64_t a_dim[4];
    uint64_t a_stride[3];
    int sw, sh, pw, ph;
    int taps_y, taps_x, cblocks;
    const void* w;
    int64_t ldw, Ktot;
    int N, Ho, Wo, Cout;
    const float* bias;
    const void* residual;
    int slot, res_first;
    void* out;
    int algo;
    int depthwise;  // pooling as a GEMM: 64-channel column tile nt reads channel block nt; w is one constant 64 x 64 matrix
    double flops;   // 2 * pixels * Cout * (taps * Cin) of the convolution itself, for the launch records
};
nm_status nm_launch_conv_tc(nm_ctx* ctx, const NmConvTc* c, cudaStream_t st);
// zero-padded copies that let a few-channel first layer run as an implicit GEMM: x [N,H,W,Cin] -> xp [N,Hp,Wp,8]
// (border of `pad` pixels, channels Cin..7 zero) and w [Cout,kh,kw,Cin] -> wp [Cout,kh,8,8]
nm_status nm_launch_pad_input(nm_ctx* ctx, const void* x, void* xp, nm_dtype dt, int Nb, int H, int W, int Cin, int pad,
                              int Hp, int Wp, cudaStream_t st);
nm_status nm_launch_pad_weight(nm_ctx* ctx, const void* w, void* wp, nm_dtype dt, int Cout, int kh, int kw, int Cin,
                               cudaStream_t st);
nm_status nm_launch_im2col(nm_ctx* ctx, const void* x, void* A, nm_dtype dt, int Nb, int H, int W, int Cin, int kh,
                           int kw, int stride, int pad, int Ho, int Wo, int Kpad, cudaStream_t st);
nm_status nm_launch_pad_rows(nm_ctx* ctx, const void* w, void* wp, nm_dtype dt, int rows, int K, int Kpad,
                             cudaStream_t st);
nm_status nm_launch_maxpool(nm_ctx* ctx, const void* x, void* y, nm_dtype dt, int Nb, int H, int W, int C, int ks,
                            int stride, int pad, int Ho, int Wo, cudaStream_t st, int relu_slot = NM_SLOT_NONE);
nm_status nm_launch_avgpool(nm_ctx* ctx, const void* x, void* y, nm_dtype dt, int Nb, int HW, int C, cudaStream_t st);
// fills the 64 x 64 matrix `w` with `value` on the diagonal and zero elsewhere
nm_status nm_launch_fill_diag(nm_ctx* ctx, void* w, nm_dtype dt, float value, cudaStream_t st);
