// INT8 attention with PWL softmax: both matrix products on the int8 tensor-core path (tcgen05 kind::i8,
// int32 accumulators in tensor memory), strict fp32 in between.
//
// Section 5 of the paper evaluates whole INT8 networks; it fixes no scheme, and the reading taken here
// (stated in the header of nm_attention_pwl_i8) keeps every integer exact and every fp32 step a single
// correctly rounded operation, so that the result is defined bit for bit: per query row
//     acc_j = <q, k_j>                      int32 on the tensor cores
//     m     = max_j acc_j                   on the integers (the scale is positive)
//     x_j   = fma((float)acc_j, sc, -((float)m * sc)),   sc = (s_q * s_k) * scale
//     e_j   = PWL_exp(x_j)                  fp32 index contract, fma(k, x, b)
//     p_j   = clamp(rint(e_j * 127), -127, 127)          int8 code, scale 1/127
//     sigma = (float)(sum_j p_j) / 127      the row sum of the codes, an exact integer sum
//     o_c   = sum_j p_j * v_jc              int32 on the tensor cores
//     out_c = ((float)o_c * (s_v / 127)) * PWL_recip(sigma)
// The structure is the streaming kernel's (attention_stream.cu) with one softmax group per CTA, persistent
// CTAs walking over tiles and the P codes handed to P V through tensor memory: Q K^T is
// computed twice, a first sweep for the final row maximum (here an integer maximum), a second for the
// exponentials; one control warp issues TMA and MMA, four softmax warps own one tensor-memory lane quarter
// each.  int8 differences: a head's 64 channels are 64 bytes, half of the 128-byte swizzle span, so tiles are
// loaded 128 bytes wide (the head and its neighbour) and the MMAs address the head's half of each row; the
// P codes of a chunk are 16 tensor-memory columns (four codes per column); an MMA covers 32 bytes of K.
#include <string.h>

#include "nm_common.cuh"

namespace {

constexpr int BQ = 128;    // query rows per CTA
constexpr int HD = 64;     // head dimension
constexpr int CK = 64;     // keys per chunk
constexpr int ROWB = 128;  // bytes per tile row
constexpr int STAGE = CK * ROWB;      // 8 KB
constexpr int PBUF = BQ * ROWB;       // 16 KB

struct I8Args {
    int B, L, heads;
    float sc;        // (s_q * s_k) * scale
    float c1;        // s_v * (1/127)
    const NmTable* t_exp;
    const NmTable* t_rcp;
    void* out;       // [B*L, heads*64] of OutT
    int* status;
    int n_exp;
    int32_t* acc_dump;    // [B, heads, L, L] or null
    int8_t* p_dump;       // [B, heads, L, L] or null
    int32_t* oacc_dump;   // [B*L, heads*64] or null
};

template <typename OutT> __device__ __forceinline__ OutT out_cast(float v);
template <> __device__ __forceinline__ float out_cast<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 out_cast<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// 8 packed words (32 one-byte codes) of this thread's row into 8 consecutive tensor-memory columns
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* r)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), "r"(r[0]),
                 "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
__device__ __forceinline__ void tmem_st_wait()
{
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
// D (+)= A B on kind::i8 with the A operand in tensor memory: row m of A in lane m, bytes 4c .. 4c + 3 of the row in
// column c (32 codes = 8 columns per instruction)
__device__ __forceinline__ void mma_i8_a_tmem(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                              uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

template <typename OutT, bool CLAMP_HI>
__global__ void __launch_bounds__(160, 3)
attention_i8_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const I8Args a)
{
    constexpr uint32_t IDESC_QK = nm_idesc(2, 1, 0, 0, BQ, CK);        // S chunk: 128 x 64, int32
    constexpr uint32_t IDESC_QK1 = nm_idesc(2, 1, 0, 0, BQ, 2 * CK);   // sweep 1: 128 x 128
    constexpr uint32_t IDESC_PV = nm_idesc(2, 1, 0, 1, BQ, HD);        // O: 128 x 64, V MN-major
    constexpr uint32_t TMEM_COLS = 128;   // [S | O]; sweep 1 writes 128 keys over both
    constexpr uint32_t O_OFF = 64;
    // the P tile's codes go through 16 columns of a second tensor-memory allocation (32, the smallest) and are
    // the A operand of P V from there: no stores to shared memory, no reads of the tile by the tensor core
    constexpr uint32_t P_COLS = 32;

    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_q, bar_drain;
    __shared__ uint64_t bar_k_full[2], bar_k1_full[2], bar_v_full, bar_s_full, bar_p_empty;
    __shared__ uint32_t tmem_slot, tmem_slot_p;
    __shared__ int abort_flag;

    const int L = a.L;
    const int half = L / CK;          // 64-key chunks of sweep 2
    const int n128 = L / (2 * CK);    // 128-key chunks of sweep 1
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* q_s = base;                       // 16 KB
    uint8_t* k_st = q_s + BQ * ROWB;           // 2 x 8 KB
    uint8_t* v_st = k_st + 2 * STAGE;          // 8 KB
    uint8_t* p_s = v_st + STAGE;               // 16 KB
    float2* rep = reinterpret_cast<float2*>(p_s + PBUF);   // (n_exp + 1) x 16 copies

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Persistent CTAs: a CTA walks over the (batch, head, 128-query block) tiles blockIdx.x, blockIdx.x + gridDim.x,
    // ...; barriers, tensor memory and the table are set up once, barrier phases are running counts, and the control
    // warp fetches the next tile's Q, first K chunks and first V chunk while the softmax warps finish the current one.
    const int blocks_per_seq = L / BQ;
    const int n_tiles = a.B * a.heads * blocks_per_seq;
    struct Tile { int qb, g, b, x0; uint32_t hsel; };
    auto tile_of = [=](int t) {
        Tile r;
        r.qb = t % blocks_per_seq;
        r.g = (t / blocks_per_seq) % a.heads;
        r.b = t / (blocks_per_seq * a.heads);
        r.x0 = (r.g & ~1) * HD;                 // tiles are loaded 128 bytes wide: the head and its neighbour
        r.hsel = (uint32_t)(r.g & 1) * 4u;      // the head's 64-byte half of a row, in 16-byte descriptor units
        return r;
    };

    if (threadIdx.x == 0) {
        abort_flag = 0;
        nm_prefetch_tmap(&tmQ);
        nm_prefetch_tmap(&tmK);
        nm_prefetch_tmap(&tmV);
        nm_mbar_init(&bar_q, 1);
        nm_mbar_init(&bar_drain, 1);
        nm_mbar_init(&bar_k_full[0], 1);
        nm_mbar_init(&bar_k_full[1], 1);
        nm_mbar_init(&bar_k1_full[0], 1);
        nm_mbar_init(&bar_k1_full[1], 1);
        nm_mbar_init(&bar_v_full, 1);
        nm_mbar_init(&bar_s_full, 1);
        nm_mbar_init(&bar_p_empty, 1);
        nm_fence_barrier_init();
        // first copies before the rest of the set-up: Q, the first two 128-key chunks of sweep 1 (stage 0 =
        // the two K stages, stage 1 = the P tile, unused in sweep 1) and the first V chunk
        nm_grid_dependency_wait();
        if ((int)blockIdx.x < n_tiles) {
            const Tile t = tile_of((int)blockIdx.x);
            nm_mbar_expect_tx(&bar_q, BQ * ROWB);
            nm_tma_load_3d(q_s, &tmQ, t.x0, t.qb * BQ, t.b, &bar_q);
            for (int st = 0; st < 2 && st < n128; ++st) {
                uint8_t* dst = st == 0 ? k_st : p_s;
                nm_mbar_expect_tx(&bar_k1_full[st], 2 * STAGE);
                nm_tma_load_3d(dst, &tmK, t.x0, st * 2 * CK, t.b, &bar_k1_full[st]);
                nm_tma_load_3d(dst + STAGE, &tmK, t.x0, st * 2 * CK + CK, t.b, &bar_k1_full[st]);
            }
            nm_mbar_expect_tx(&bar_v_full, STAGE);
            nm_tma_load_3d(v_st, &tmV, t.x0, 0, t.b, &bar_v_full);
        }
    }
    if (warp == 0) {
        nm_tmem_alloc(&tmem_slot, TMEM_COLS);
        nm_tmem_alloc(&tmem_slot_p, P_COLS);
        nm_tmem_relinquish();
    } else {
        // 16-way replicated exp table (a 64-bit warp load is served half a warp at a time); one extra entry
        // (a copy of the last) lets input 0 of a table whose range ends at 0 go unclamped
        const int ne = a.n_exp;
        for (int i = threadIdx.x - 32; i < (ne + 1) * 16; i += 128) rep[i] = a.t_exp->kb[min(i >> 4, ne - 1)];
    }
    nm_tc_fence_before();
    __syncthreads();
    nm_tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    const uint32_t tmem_p = tmem_slot_p;
    volatile int* abortp = &abort_flag;
    nm_grid_launch_dependents();
    nm_grid_dependency_wait();

    if (warp == 0) {
        // ------------------------------------------------ control warp (all lanes run, one elected lane issues)
        const uint32_t bar_sc = 2, bar_pr = 3, bar_oc = 4;
        auto wait = [&](uint64_t* bar, uint32_t parity) {
            return __all_sync(0xffffffffu, nm_mbar_wait_relaxed<20>(bar, parity, abortp, a.status)) != 0;
        };
        bool ok = true;
        // completions consumed so far on each barrier (they run on from tile to tile)
        uint32_t q_cnt = 0, k1_cnt0 = 0, k1_cnt1 = 0, k_cnt0 = 0, k_cnt1 = 0, v_cnt = 0, pv_cnt = 0;
        for (int tile = (int)blockIdx.x, ti = 0; tile < n_tiles; tile += (int)gridDim.x, ++ti) {
            const Tile t = tile_of(tile);
            const int b = t.b, x0 = t.x0;
            const uint32_t hsel = t.hsel;
            const bool more = tile + (int)gridDim.x < n_tiles;
            if (ok && !wait(&bar_q, q_cnt & 1u)) ok = false;
            ++q_cnt;
            // the previous tile's epilogue has read O out of tensor memory (sweep 1 writes over [S | O])
            if (ti > 0) asm volatile("bar.sync %0, %1;" ::"r"(bar_oc), "n"(160) : "memory");
            const uint64_t qdesc = nm_smem_desc_sw128(nm_smem_u32(q_s)) + hsel;
            // ---- sweep 1: [S | O] = Q K^T for 128 keys at a time
            auto issue_qk1 = [&](int i) {
                const uint32_t par = ((i & 1) ? k1_cnt1 : k1_cnt0) & 1u;
                if (i & 1) ++k1_cnt1; else ++k1_cnt0;
                if (!ok) return;
                if (!wait(&bar_k1_full[i & 1], par)) { ok = false; return; }
                nm_tc_fence_after();
                const uint64_t kdesc = nm_smem_desc_sw128(nm_smem_u32((i & 1) ? p_s : k_st)) + hsel;
                if (nm_elect_one()) {
#pragma unroll
                    for (int k = 0; k < 2; ++k) nm_mma_i8(tmem_base, qdesc + 2 * k, kdesc + 2 * k, IDESC_QK1, k != 0);
                    nm_tc_commit(&bar_s_full);
                }
                __syncwarp();
            };
            if (n128 > 0) issue_qk1(0);
            for (int i = 0; i < n128; ++i) {
                asm volatile("bar.sync %0, %1;" ::"r"(bar_sc), "n"(160) : "memory");   // S-consumed(i)
                if (i + 1 < n128) issue_qk1(i + 1);
                if (ok && i + 2 < n128 && nm_elect_one()) {
                    uint8_t* dst = (i & 1) ? p_s : k_st;
                    const int key0 = (i + 2) * 2 * CK;
                    nm_mbar_expect_tx(&bar_k1_full[i & 1], 2 * STAGE);
                    nm_tma_load_3d(dst, &tmK, x0, key0, b, &bar_k1_full[i & 1]);
                    nm_tma_load_3d(dst + STAGE, &tmK, x0, key0 + CK, b, &bar_k1_full[i & 1]);
                }
                __syncwarp();
            }
            // ---- sweep 2: 64 keys at a time
            auto load_k = [&](int j) {
                if (ok && nm_elect_one()) {
                    nm_mbar_expect_tx(&bar_k_full[j & 1], STAGE);
                    nm_tma_load_3d(k_st + (size_t)(j & 1) * STAGE, &tmK, x0, j * CK, b, &bar_k_full[j & 1]);
                }
                __syncwarp();
            };
            auto issue_qk = [&](int j) {
                const uint32_t par = ((j & 1) ? k_cnt1 : k_cnt0) & 1u;
                if (j & 1) ++k_cnt1; else ++k_cnt0;
                if (!ok) return;
                if (!wait(&bar_k_full[j & 1], par)) { ok = false; return; }
                nm_tc_fence_after();
                const uint64_t kdesc = nm_smem_desc_sw128(nm_smem_u32(k_st + (size_t)(j & 1) * STAGE)) + hsel;
                if (nm_elect_one()) {
#pragma unroll
                    for (int k = 0; k < 2; ++k) nm_mma_i8(tmem_base, qdesc + 2 * k, kdesc + 2 * k, IDESC_QK, k != 0);
                    nm_tc_commit(&bar_s_full);
                }
                __syncwarp();
            };
            load_k(0);
            if (half > 1) load_k(1);
            issue_qk(0);
            for (int j = 0; j < half; ++j) {
                asm volatile("bar.sync %0, %1;" ::"r"(bar_sc), "n"(160) : "memory");   // S-consumed(j)
                if (j + 1 < half) issue_qk(j + 1);
                if (j + 2 < half) load_k(j + 2);
                // Last chunk: every Q K^T of the tile has completed, so Q, the K stages and the P tile (which only
                // sweep 1 uses, as a K stage) take the next tile's first loads now.
                if (j + 1 == half && more && ok && nm_elect_one()) {
                    const Tile nt = tile_of(tile + (int)gridDim.x);
                    nm_mbar_expect_tx(&bar_q, BQ * ROWB);
                    nm_tma_load_3d(q_s, &tmQ, nt.x0, nt.qb * BQ, nt.b, &bar_q);
                    for (int st = 0; st < 2 && st < n128; ++st) {
                        uint8_t* dst = st == 0 ? k_st : p_s;
                        nm_mbar_expect_tx(&bar_k1_full[st], 2 * STAGE);
                        nm_tma_load_3d(dst, &tmK, nt.x0, st * 2 * CK, nt.b, &bar_k1_full[st]);
                        nm_tma_load_3d(dst + STAGE, &tmK, nt.x0, st * 2 * CK + CK, nt.b, &bar_k1_full[st]);
                    }
                }
                __syncwarp();
                asm volatile("bar.sync %0, %1;" ::"r"(bar_pr), "n"(160) : "memory");   // P-ready(j)
                if (ok && !wait(&bar_v_full, v_cnt & 1u)) ok = false;
                ++v_cnt;
                if (ok) {
                    nm_tc_fence_after();
                    const uint32_t v_addr = nm_smem_u32(v_st);
                    if (nm_elect_one()) {
#pragma unroll
                        for (int k = 0; k < 2; ++k)   // keys 32k..32k+31: 8 columns of P; four groups of 8 V rows
                            mma_i8_a_tmem(tmem_base + O_OFF, tmem_p + (uint32_t)(8 * k),
                                          nm_smem_desc_sw128(v_addr + (uint32_t)(32 * k * ROWB)) + hsel, IDESC_PV, (j | k) != 0);
                        nm_tc_commit(&bar_p_empty);
                    }
                    __syncwarp();
                }
                const uint32_t pv_par = pv_cnt & 1u;   // parity of this P V's completion
                ++pv_cnt;
                // the V stage is free once this P V has completed: it takes the next chunk's V, or after the last
                // chunk the next tile's first one
                if (ok && (j + 1 < half || more)) {
                    if (!wait(&bar_p_empty, pv_par)) ok = false;
                    if (ok && nm_elect_one()) {
                        nm_mbar_expect_tx(&bar_v_full, STAGE);
                        if (j + 1 < half) {
                            nm_tma_load_3d(v_st, &tmV, x0, (j + 1) * CK, b, &bar_v_full);
                        } else {
                            const Tile nt = tile_of(tile + (int)gridDim.x);
                            nm_tma_load_3d(v_st, &tmV, nt.x0, 0, nt.b, &bar_v_full);
                        }
                    }
                    __syncwarp();
                }
            }
        }
        if (!ok) {
            if (nm_elect_one()) {
                nm_tc_commit(&bar_drain);
                long long t0 = clock64();
                while (!nm_mbar_try_wait(&bar_drain, 0) && clock64() - t0 < 200000000LL) {}
                while (clock64() - t0 < 4000000LL) {}
            }
            __syncwarp();
        }
    } else {
        // ------------------------------------------------ softmax warps: one row per thread
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const uint32_t bar_sc = 2, bar_pr = 3, bar_oc = 4;
        const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
        const float inv_h = a.t_exp->inv_h, off = a.t_exp->off, nm1 = (float)(a.n_exp - 1);
        const uint32_t rep_lane = nm_smem_u32(rep) + (uint32_t)(lane & 15) * 8u - 0xA0000000u;
        const uint32_t p_row = tmem_p + ((uint32_t)(q * 32) << 16);   // this warp's lane quarter of the P columns
        const float sc = a.sc;
        const uint64_t sc2 = nm_pack2(sc, sc), inv_h2 = nm_pack2(inv_h, inv_h), off2 = nm_pack2(off, off);
        const uint64_t magic2 = nm_pack2(12582912.0f, 12582912.0f);
        int ok = 1;
        auto wait_all = [&](uint64_t* bar, uint32_t par) {
            if (!ok) return;
            const bool done = nm_mbar_try_wait(bar, par);
            if (!__all_sync(0xffffffffu, done)) {
                int w = 1;
                if (lane == 0) w = nm_mbar_wait_relaxed(bar, par, abortp, a.status) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, w, 0);
                if (ok) (void)nm_mbar_try_wait(bar, par);
            }
        };
        uint32_t s_cnt = 0, pv_base = 0;   // completions consumed so far: score products, P V products
        for (int tile = (int)blockIdx.x; tile < n_tiles; tile += (int)gridDim.x) {
            const Tile t = tile_of(tile);
            const int qb = t.qb, g = t.g, b = t.b;
            const bool more = tile + (int)gridDim.x < n_tiles;
            const size_t srow = (((size_t)b * a.heads + g) * L + (size_t)qb * BQ + row) * (size_t)L;   // row of the dumps
            // ---- sweep 1: the row maximum, on the integers
            int m = INT_MIN;
#pragma unroll 1
            for (int i = 0; i < n128; ++i) {
                wait_all(&bar_s_full, s_cnt & 1u);
                ++s_cnt;
                if (ok) {
                    nm_tc_fence_after();
#pragma unroll
                    for (int hh = 0; hh < 4; ++hh) {
                        uint32_t r[32];
                        nm_tmem_ld32_sync(t_row + (uint32_t)(hh * 32), r);
                        if (hh == 3) {
                            nm_tc_fence_before();
                            asm volatile("bar.arrive %0, %1;" ::"r"(bar_sc), "n"(160) : "memory");
                        }
                        int m0 = INT_MIN, m1 = INT_MIN;
#pragma unroll
                        for (int k = 0; k < 32; k += 2) {
                            m0 = max(m0, (int)r[k]);
                            m1 = max(m1, (int)r[k + 1]);
                        }
                        m = max(m, max(m0, m1));
                    }
                } else {
                    asm volatile("bar.arrive %0, %1;" ::"r"(bar_sc), "n"(160) : "memory");
                }
            }
            const float neg = -((float)m * sc);
            const uint64_t neg2 = nm_pack2(neg, neg);
            int isum = 0;
            // ---- sweep 2: exponentials, codes, the integer row sum, P tiles
#pragma unroll 1
            for (int j = 0; j < half; ++j) {
                wait_all(&bar_s_full, s_cnt & 1u);
                ++s_cnt;
                if (ok) nm_tc_fence_after();
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    uint32_t r[32];
                    if (ok) nm_tmem_ld32_sync(t_row + (uint32_t)(hh * 32), r);
                    if (hh == 1) {
                        nm_tc_fence_before();
                        asm volatile("bar.arrive %0, %1;" ::"r"(bar_sc), "n"(160) : "memory");
                    }
                    uint32_t pk[8];   // the half's 32 codes
                    if (ok) {
#pragma unroll
                        for (int w = 0; w < 8; ++w) {
                            float e[4];
#pragma unroll
                            for (int k = 0; k < 4; k += 2) {
                                // two scores at a time on the packed fp32 instructions: each half is the same correctly
                                // rounded operation as the scalar form
                                uint64_t x2, u2, b2;
                                asm("fma.rn.f32x2 %0, %1, %2, %3;"
                                    : "=l"(x2)
                                    : "l"(nm_pack2((float)(int)r[w * 4 + k], (float)(int)r[w * 4 + k + 1])), "l"(sc2), "l"(neg2));
                                asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(u2) : "l"(x2), "l"(inv_h2), "l"(off2));
                                float x0, x1, u0, u1;
                                nm_unpack2(x2, x0, x1);
                                nm_unpack2(u2, u0, u1);
                                u0 = fmaxf(u0, 0.0f);
                                u1 = fmaxf(u1, 0.0f);
                                if (CLAMP_HI) {
                                    u0 = fminf(u0, nm1);
                                    u1 = fminf(u1, nm1);
                                }
                                asm("add.rm.f32x2 %0, %1, %2;" : "=l"(b2) : "l"(nm_pack2(u0, u1)), "l"(magic2));
                                float f0, f1;
                                nm_unpack2(b2, f0, f1);
                                float k0, c0, k1, c1;
                                asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(k0), "=f"(c0) : "r"((__float_as_uint(f0) << 7) + rep_lane));
                                asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(k1), "=f"(c1) : "r"((__float_as_uint(f1) << 7) + rep_lane));
                                e[k] = __fmaf_rn(k0, x0, c0);
                                e[k + 1] = __fmaf_rn(k1, x1, c1);
                            }
                            pk[w] = nm_quant_i8x4(e[0], e[1], e[2], e[3], 127.0f);
                            isum = __dp4a((int)pk[w], 0x01010101, isum);
                        }
                        if (a.acc_dump) {
#pragma unroll
                            for (int k = 0; k < 32; k += 4)
                                *reinterpret_cast<int4*>(a.acc_dump + srow + (size_t)j * CK + hh * 32 + k) =
                                    make_int4((int)r[k], (int)r[k + 1], (int)r[k + 2], (int)r[k + 3]);
                        }
                        if (a.p_dump) {
                            *reinterpret_cast<uint4*>(a.p_dump + srow + (size_t)j * CK + hh * 32) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                            *reinterpret_cast<uint4*>(a.p_dump + srow + (size_t)j * CK + hh * 32 + 16) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                        }
                    }
                    // the stores wait until P V of the previous chunk has read the columns
                    if (hh == 0 && j >= 1) wait_all(&bar_p_empty, (pv_base + (uint32_t)(j - 1)) & 1u);
                    if (ok) {
                        if (hh == 0 && j >= 1) nm_tc_fence_after();   // ordered after the P V that read the columns
                        tmem_st8(p_row + (uint32_t)(hh * 8), pk);     // keys 32 hh .. 32 hh + 31 of this thread's row
                    }
                }
                tmem_st_wait();          // the P columns are written
                nm_tc_fence_before();
                asm volatile("bar.arrive %0, %1;" ::"r"(bar_pr), "n"(160) : "memory");
            }
            // ---- sigma from the integer sum, r = PWL_recip(sigma), out = ((float)o * c1) * r
            const float sigma = (float)isum * (1.0f / 127.0f);
            const int sr = nm_pwl_index(sigma, a.t_rcp->inv_h, a.t_rcp->off, (float)(a.t_rcp->n - 1));
            const float2 kbr = a.t_rcp->kb[sr];
            const float rinv = __fmaf_rn(kbr.x, sigma, kbr.y);
            wait_all(&bar_p_empty, (pv_base + (uint32_t)(half - 1)) & 1u);
            pv_base += (uint32_t)half;
            if (ok) nm_tc_fence_after();
            const size_t orow = ((size_t)b * L + (size_t)qb * BQ + row) * ((size_t)a.heads * HD) + (size_t)g * HD;
            OutT* op = reinterpret_cast<OutT*>(a.out) + orow;
            const uint32_t o_addr = t_row + O_OFF;
#pragma unroll
            for (int jj = 0; jj < HD / 16; ++jj) {
                uint32_t r0[16];
                if (ok) nm_tmem_ld16_sync(o_addr + (uint32_t)(jj * 16), r0);
                if (jj == HD / 16 - 1 && more) {
                    // all of O is in registers: the control warp may start the next tile's sweep 1 over [S | O]
                    nm_tc_fence_before();
                    asm volatile("bar.arrive %0, %1;" ::"r"(bar_oc), "n"(160) : "memory");
                }
                if (ok) {
                    OutT v[16];
#pragma unroll
                    for (int k = 0; k < 16; ++k) v[k] = out_cast<OutT>(((float)(int)r0[k] * a.c1) * rinv);
                    if (a.oacc_dump) {
#pragma unroll
                        for (int k = 0; k < 16; k += 4)
                            *reinterpret_cast<int4*>(a.oacc_dump + orow + jj * 16 + k) =
                                make_int4((int)r0[k], (int)r0[k + 1], (int)r0[k + 2], (int)r0[k + 3]);
                    }
                    const uint4* src = reinterpret_cast<const uint4*>(v);
                    uint4* dst = reinterpret_cast<uint4*>(op + jj * 16);
#pragma unroll
                    for (int k = 0; k < (int)(16 * sizeof(OutT) / 16); ++k) dst[k] = src[k];
                }
            }
        }
    }

    nm_tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        nm_tc_fence_after();
        nm_tmem_dealloc(tmem_base, TMEM_COLS);
        nm_tmem_dealloc(tmem_p, P_COLS);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [B][L][heads*64] bytes with token pitch stride_t and batch pitch stride_b; box 128 bytes x rows x 1
nm_status make_map(nm_ctx* ctx, CUtensorMap* m, const void* ptr, const nm_attn_i8_desc* d, int rows)
{
    cuuint64_t gdim[3] = {(cuuint64_t)d->heads * HD, (cuuint64_t)d->L, (cuuint64_t)d->B};
    cuuint64_t gstr[2] = {(cuuint64_t)d->stride_t, (cuuint64_t)d->stride_b};
    cuuint32_t box[3] = {(cuuint32_t)ROWB, (cuuint32_t)rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = ((EncodeTiledFn)ctx->encode_tiled)(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(ptr), gdim, gstr,
                                                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? NM_OK : NM_ERR_CUDA;
}

template <typename OutT, bool CLAMP_HI>
nm_status launch(nm_ctx* ctx, const nm_attn_i8_desc* d, cudaStream_t st)
{
    I8Args a;
    memset(&a, 0, sizeof(a));
    a.B = d->B; a.L = d->L; a.heads = d->heads;
    a.sc = (d->s_q * d->s_k) * d->scale;
    a.c1 = d->s_v * (1.0f / 127.0f);
    a.t_exp = ctx->d_tables + d->exp_slot;
    a.t_rcp = ctx->d_tables + d->recip_slot;
    a.out = d->out;
    a.status = ctx->d_status;
    a.n_exp = ctx->h_tables[d->exp_slot].n;
    a.acc_dump = d->acc_dump; a.p_dump = d->p_dump; a.oacc_dump = d->oacc_dump;
    const size_t smem = (size_t)BQ * ROWB + 3 * (size_t)STAGE + (size_t)PBUF + (size_t)(a.n_exp + 1) * 16 * sizeof(float2) + 1024;
    CUtensorMap tmQ, tmK, tmV;
    nm_status s;
    if ((s = make_map(ctx, &tmQ, d->Q, d, BQ)) != NM_OK) return s;
    if ((s = make_map(ctx, &tmK, d->K, d, CK)) != NM_OK) return s;
    if ((s = make_map(ctx, &tmV, d->V, d, CK)) != NM_OK) return s;
    auto kern = attention_i8_kernel<OutT, CLAMP_HI>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return NM_ERR_CUDA;
    const int64_t tiles = (int64_t)d->B * d->heads * (d->L / BQ);
    if (tiles > 0x7fffffffLL) return NM_ERR_SHAPE;
    // persistent: one resident wave of CTAs, each walking over tiles; three per SM by the launch bounds and by
    // tensor memory (3 x 160 of 512 columns), fewer if the exp table makes the shared memory larger
    int64_t per_sm = 233472 / (int64_t)(smem + 1024 + 1536);
    if (per_sm > 3) per_sm = 3;
    if (per_sm < 1) per_sm = 1;
    int64_t grid = (int64_t)ctx->sm_count * per_sm;
    if (grid > tiles) grid = tiles;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(160);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = ctx->pdl ? 1 : 0;
    NmLaunchScope scope(ctx, NM_KERNEL_ATTENTION_TC, 4.0 * (double)d->B * d->heads * (double)d->L * d->L * HD, st);
    if (cudaLaunchKernelEx(&cfg, kern, tmQ, tmK, tmV, a) != cudaSuccess) return NM_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

}  // namespace

nm_status nm_launch_attention_i8(nm_ctx* ctx, const nm_attn_i8_desc* d, cudaStream_t st)
{
    const bool clamp_hi = ctx->h_tables[d->exp_slot].x_max < 0.0f;
    if (d->out_dtype == NM_F32)
        return clamp_hi ? launch<float, true>(ctx, d, st) : launch<float, false>(ctx, d, st);
    return clamp_hi ? launch<__nv_bfloat16, true>(ctx, d, st) : launch<__nv_bfloat16, false>(ctx, d, st);
}
