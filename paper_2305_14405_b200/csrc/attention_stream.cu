// Fused attention with PWL softmax, streaming variant: several CTAs per SM.
//
// Same function as attention_tc.cu (Section 3.1: attention is a linear operator; Section 3.2.2:
// exp and 1/x as PWL tables), per query row
//     s_j = scale*<q,k_j>;  m = max_j s_j;  e_j = PWL_exp(s_j - m);  sigma = sum_j e_j;
//     o = PWL_recip(sigma) * sum_j e_j v_j
// with m the FINAL row maximum (a PWL exponential is not multiplicative, so there is no
// running-maximum rescaling).  Instead of keeping the whole 128 x L score block in tensor memory,
// this kernel computes Q K^T TWICE: a first sweep over the keys only for the row maximum, a second
// sweep for the exponentials.  The tensor pipe is idle most of the time in this ALU-bound kernel, so
// the second Q K^T is free, and the footprint drops to 128 tensor-memory columns and ~50 KB of
// shared memory per softmax group (plus Q and the table): three CTAs fit on an SM and one
// CTA's loads, MMAs and hand-offs overlap the others' arithmetic.  Any L that is a multiple of 128.
//
// CTAs are persistent: one resident wave (three per SM) walks over the (batch, head, 128-query block) tiles.
// Barriers, tensor memory and the replicated table are set up once per CTA; every mbarrier's phase is a running
// count carried from tile to tile; after a tile's last Q K^T the control warp already fetches the next tile's Q
// and first K chunks, after its last P V the next first V chunk, and the next tile's first product starts as
// soon as the softmax warps have read the accumulator out of tensor memory.
//
// The 16-bit P tile of the one-group form never touches shared memory: the softmax warps write it to 32 further
// tensor-memory columns (tcgen05.st) and P V takes its A operand from there; the shared-memory pipe, which the
// table lookups load most, loses the tile's stores and the tensor core's reads of it.
//
// A group is one control warp and four softmax warps, an independent pipeline that owns 128
// tensor-memory columns [S_g | O_g], two K stages, a V stage and a P tile.  A CTA has NG = 1 or 2
// groups (template parameter; only NG = 1 is built, see nm_launch_attention_stream); with two, the groups split
// the keys: in sweep 1 group g takes the
// 128-key chunks g, g+NG, ... (scores over all 128 columns, K staged in its two K stages and,
// alternately, in its P tile); in sweep 2 the 64-key chunks g, g+NG, ... (scores in S_g, accumulator
// O_g); row maxima and sums are exchanged through shared memory and the accumulators summed in the
// epilogue.
//
//   warps 0..NG-1     control warp of group g: TMA loads (the group's K chunks through two stages, its V
//                     chunks through one) and the tcgen05.mma for S_g = Q K_c^T and O_g += P_c V_c (V as
//                     an MN-major operand).  It sleeps in a named barrier (bar.sync) that the group's
//                     softmax warps signal with bar.arrive, so hand-offs cost no polling.
//   warps NG..5NG-1   softmax, one per tensor-memory lane quarter and group: tcgen05.ld, row maximum
//                     (sweep 1); PWL exp, row sum, bf16 P tile in the swizzled K-major layout (sweep 2);
//                     PWL reciprocal, scaling, store (optionally as int8 codes for the int8 encoder).
#include <string.h>

#include "nm_common.cuh"

namespace {

constexpr int BQ = 128;    // query rows per CTA
constexpr int HD = 64;     // head dimension
constexpr int CK = 64;     // keys per chunk
constexpr int ROWB = 128;  // bytes per tile row (64 x 16-bit)
constexpr int STAGE = CK * ROWB;      // 8 KB
constexpr int PBUF = BQ * ROWB;       // 16 KB

struct SArgs {
    int B, L, heads;
    float scale;
    const NmTable* t_exp;
    const NmTable* t_rcp;
    void* out;
    int* status;
    int n_exp;
    int8_t* out_q;       // when set: the output goes out as int8 codes (of the value rounded to T) instead
    float q_inv_scale;
};

template <typename T> struct AT;
template <> struct AT<__nv_bfloat16> {
    static constexpr uint32_t fmt = 1;
    static __device__ __forceinline__ float round(float a) { return __bfloat162float(__float2bfloat16_rn(a)); }
    static __device__ __forceinline__ uint32_t pack(float a, float b)
    {
        __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
        return *reinterpret_cast<uint32_t*>(&h);
    }
};
template <> struct AT<__half> {
    static constexpr uint32_t fmt = 0;
    static __device__ __forceinline__ float round(float a) { return __half2float(__float2half_rn(a)); }
    static __device__ __forceinline__ uint32_t pack(float a, float b)
    {
        __half2 h = __floats2half2_rn(a, b);
        return *reinterpret_cast<uint32_t*>(&h);
    }
};

// 16 packed words of this thread's row into 16 consecutive tensor-memory columns (the mirror of the 16-column read)
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r)
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait()
{
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
// D (+)= A B with the A operand in tensor memory: row m of A in lane m, elements 2c and 2c + 1 of the row in the
// low and high half of column c (16 elements = 8 columns per instruction)
__device__ __forceinline__ void mma_f16_a_tmem(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ float max3f(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// A tile is one (batch, head, 128-query block); tile index = (b * heads + g) * blocks_per_seq + qb.
struct Tile { int qb, g, b; };
struct TileGeom { int blocks_per_seq, heads; };
__device__ __forceinline__ Tile tile_decode(const TileGeom& gm, int t)
{
    Tile r;
    r.qb = t % gm.blocks_per_seq;
    r.g = (t / gm.blocks_per_seq) % gm.heads;
    r.b = t / (gm.blocks_per_seq * gm.heads);
    return r;
}
// What the first loads of a tile need: tensor maps, staging buffers, their barriers.
struct LoadCtx {
    const CUtensorMap *tmQ, *tmK, *tmV;
    uint8_t *q_s, *k_st, *p_s, *v_st;
    uint64_t *bar_q, *bar_k1_full, *bar_v_full;   // bar_k1_full: [group][2]
    int n128;
};
// Q and each group's first two 128-key chunks of sweep 1 (stage 0 = the group's two K stages, stage 1 = its P
// tile).  One thread; the buffers must be free.
template <int NG>
__device__ __forceinline__ void load_tile_head(const LoadCtx& c, const Tile& t)
{
    nm_mbar_expect_tx(c.bar_q, BQ * ROWB);
    nm_tma_load_3d(c.q_s, c.tmQ, t.g * HD, t.qb * BQ, t.b, c.bar_q);
#pragma unroll
    for (int gi = 0; gi < NG; ++gi) {
#pragma unroll
        for (int st = 0; st < 2; ++st) {
            const int c128 = gi + NG * st;
            if (c128 >= c.n128) break;
            uint8_t* dst = st == 0 ? c.k_st + (size_t)gi * 2 * STAGE : c.p_s + (size_t)gi * PBUF;
            uint64_t* bar = c.bar_k1_full + gi * 2 + st;
            nm_mbar_expect_tx(bar, 2 * STAGE);
            nm_tma_load_3d(dst, c.tmK, t.g * HD, c128 * 2 * CK, t.b, bar);
            nm_tma_load_3d(dst + STAGE, c.tmK, t.g * HD, c128 * 2 * CK + CK, t.b, bar);
        }
    }
}
// The group's first V chunk of a tile (one thread; the V stage must be free).
__device__ __forceinline__ void load_first_v(const LoadCtx& c, const Tile& t, int gi)
{
    nm_mbar_expect_tx(c.bar_v_full + gi, STAGE);
    nm_tma_load_3d(c.v_st + (size_t)gi * STAGE, c.tmV, t.g * HD, gi * CK, t.b, c.bar_v_full + gi);
}

// NG = softmax groups per CTA: 2 (320 threads, 256 tensor-memory columns, two CTAs per SM) or
// 1 (160 threads, 128 columns, three CTAs per SM: more tiles in flight per SM, fewer warps per tile).
template <typename T, bool CLAMP_HI, int NG>
__global__ void __launch_bounds__(160 * NG, NG == 1 ? 3 : 2)
attention_stream_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                        const __grid_constant__ CUtensorMap tmV, const SArgs a)
{
    constexpr uint32_t IDESC_QK = nm_idesc(1, AT<T>::fmt, 0, 0, BQ, CK);   // S chunk: 128 x 64
    constexpr uint32_t IDESC_PV = nm_idesc(1, AT<T>::fmt, 0, 1, BQ, HD);   // O: 128 x 64, V MN-major
    constexpr uint32_t IDESC_QK1 = nm_idesc(1, AT<T>::fmt, 0, 0, BQ, 2 * CK);   // sweep 1: 128 x 128
    constexpr uint32_t TMEM_COLS = 128 * NG;   // S0 | O0 (| S1 | O1); sweep 1 writes 128 keys over [S_g | O_g]
    constexpr int NSOFT = 128 * NG;            // softmax threads
    constexpr uint32_t GRP_COLS = 128;    // tensor-memory columns of a group
    constexpr uint32_t O_OFF = 64;        // O_g within the group's columns
    // One group per CTA: the 16-bit P tile goes through tensor memory (a second allocation of 32 columns: 64 keys,
    // two per column) and is the A operand of P V from there; three CTAs hold 3 x (128 + 32) of the SM's 512
    // columns.  That takes the P tile's stores, its reads by the tensor core and the proxy fence off the shared-
    // memory pipe, which the table lookups load most.  With two groups the columns do not suffice (2 CTAs x 320).
    constexpr bool PT = NG == 1;
    constexpr uint32_t P_COLS = 32;

    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_q, bar_drain[NG];
    __shared__ uint64_t bar_k_full[NG][2], bar_k1_full[NG][2], bar_v_full[NG], bar_s_full[NG], bar_p_empty[NG];
    __shared__ uint32_t tmem_slot, tmem_slot_p;
    __shared__ int abort_flag;
    __shared__ float s_red[NG][BQ];

    const int L = a.L;
    const int n = L / CK;      // chunks (even: L is a multiple of 128)
    const int half = n / NG;   // chunks per group in sweep 2: group g takes g, g+NG, ...
    const int n128 = L / (2 * CK);   // 128-key chunks of sweep 1: group g takes g, g+NG, ...
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* q_s = base;                       // 16 KB
    uint8_t* k_st = q_s + BQ * ROWB;           // [group][2] x 8 KB
    uint8_t* v_st = k_st + NG * 2 * STAGE;     // [group] x 8 KB
    uint8_t* p_s = v_st + NG * STAGE;          // [group] x 16 KB
    float2* rep = reinterpret_cast<float2*>(p_s + NG * PBUF);   // (n_exp + 1) x 16 copies

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // A CTA walks over the (batch, head, 128-query block) tiles blockIdx.x, blockIdx.x + gridDim.x, ...: barriers,
    // tensor memory and the replicated table are set up once, and the control warp fetches the next tile's Q,
    // first K chunks and first V chunk while the softmax warps finish the current one.
    const int blocks_per_seq = L / BQ;
    const int n_tiles = a.B * a.heads * blocks_per_seq;
    const TileGeom geom = {blocks_per_seq, a.heads};
    auto tile_of = [geom](int t) { return tile_decode(geom, t); };
    LoadCtx lc;
    lc.tmQ = &tmQ; lc.tmK = &tmK; lc.tmV = &tmV;
    lc.q_s = q_s; lc.k_st = k_st; lc.p_s = p_s; lc.v_st = v_st;
    lc.bar_q = &bar_q; lc.bar_k1_full = &bar_k1_full[0][0]; lc.bar_v_full = &bar_v_full[0];
    lc.n128 = n128;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        nm_prefetch_tmap(&tmQ);
        nm_prefetch_tmap(&tmK);
        nm_prefetch_tmap(&tmV);
        nm_mbar_init(&bar_q, 1);
        for (int i = 0; i < NG; ++i) {
            nm_mbar_init(&bar_drain[i], 1);
            nm_mbar_init(&bar_k_full[i][0], 1);
            nm_mbar_init(&bar_k_full[i][1], 1);
            nm_mbar_init(&bar_k1_full[i][0], 1);
            nm_mbar_init(&bar_k1_full[i][1], 1);
            nm_mbar_init(&bar_v_full[i], 1);
            nm_mbar_init(&bar_s_full[i], 1);
            nm_mbar_init(&bar_p_empty[i], 1);
        }
        nm_fence_barrier_init();
        // The first copies go out before the rest of the set-up (tensor-memory allocation, table
        // replication, block barrier), so that their latency overlaps it: Q, each group's first two
        // 128-key chunks of sweep 1 (stage 0 = the group's two K stages, stage 1 = its P tile, which
        // sweep 1 does not use otherwise) and its first V chunk.
        nm_grid_dependency_wait();   // Q, K, V come from the previous kernel
        if ((int)blockIdx.x < n_tiles) {
            const Tile t0 = tile_of((int)blockIdx.x);
            load_tile_head<NG>(lc, t0);
            for (int gi = 0; gi < NG; ++gi) load_first_v(lc, t0, gi);
        }
    }
    if (warp == NG - 1) {
        nm_tmem_alloc(&tmem_slot, TMEM_COLS);
        if constexpr (PT) nm_tmem_alloc(&tmem_slot_p, P_COLS);
        nm_tmem_relinquish();
    }
    if (warp >= NG) {
        // 16-way replicated exp table: entry s, copy c at rep[s*16 + c].  A 64-bit warp load is served
        // half a warp at a time, so 16 copies already make arbitrary lookups conflict-free.  One extra
        // entry (a copy of the last) lets input 0 of a table whose range ends at 0 go unclamped.
        const int ne = a.n_exp;
        for (int i = threadIdx.x - 32 * NG; i < (ne + 1) * 16; i += NSOFT) rep[i] = a.t_exp->kb[min(i >> 4, ne - 1)];
    }
    nm_tc_fence_before();
    __syncthreads();
    nm_tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    const uint32_t tmem_p = PT ? tmem_slot_p : 0u;
    volatile int* abortp = &abort_flag;
    nm_grid_launch_dependents();   // the next kernel may start its set-up
    nm_grid_dependency_wait();     // Q, K, V come from the previous kernel

    if (warp < NG) {
        // ------------------------------------------------ control warp of group `warp`
        // Runs with all 32 lanes (barrier tests, counters and descriptors stay warp-uniform); one
        // elected lane issues the TMA and tcgen05 instructions.  It sleeps in a named barrier until
        // its group's four softmax warps have arrived there, so signalling costs no polling:
        //   S-consumed(i): chunk i's scores are in registers -> K stage i & 1 is free (load the chunk
        //                  after next into it) and S is free (issue Q K^T for the next chunk);
        //   P-ready(j):    the bf16 P tile of the j-th chunk of sweep 2 is in shared memory -> O += P V.
        const int gi = NG == 1 ? 0 : warp;
        const uint32_t bar_sc = 2 + 2 * gi, bar_pr = 3 + 2 * gi, bar_oc = 6 + gi;
        const int cnt1 = (n128 - gi + NG - 1) / NG;   // the group's 128-key chunks in sweep 1
        uint8_t* my_k = k_st + (size_t)gi * 2 * STAGE;
        uint8_t* my_v = v_st + (size_t)gi * STAGE;
        uint8_t* my_p = p_s + (size_t)gi * PBUF;
        const uint32_t my_tmem = tmem_base + (uint32_t)gi * GRP_COLS;
        auto wait = [&](uint64_t* bar, uint32_t parity) {
            return __all_sync(0xffffffffu, nm_mbar_wait_relaxed<20>(bar, parity, abortp, a.status)) != 0;
        };
        bool ok = true;
        const uint64_t qdesc = nm_smem_desc_sw128(nm_smem_u32(q_s));
        // completions consumed so far on each barrier (they run on from tile to tile)
        uint32_t q_cnt = 0, k1_cnt0 = 0, k1_cnt1 = 0, k_cnt0 = 0, k_cnt1 = 0, v_cnt = 0, pv_cnt = 0;
        for (int tile = (int)blockIdx.x, ti = 0; tile < n_tiles; tile += (int)gridDim.x, ++ti) {
            const Tile t = tile_of(tile);
            const int g = t.g, b = t.b;
            const bool more = tile + (int)gridDim.x < n_tiles;
            if (ok && !wait(&bar_q, q_cnt & 1u)) ok = false;
            ++q_cnt;
            // the previous tile's epilogue has read O out of tensor memory (sweep 1 writes over [S_g | O_g])
            if (ti > 0) asm volatile("bar.sync %0, %1;" ::"r"(bar_oc), "n"(160) : "memory");
            // ---- sweep 1: [S_g | O_g] = Q K^T for 128 keys at a time; K stage i & 1 (0: the two K stages
            // taken together, 1: the P tile)
            auto issue_qk1 = [&](int i) {
                const uint32_t par = ((i & 1) ? k1_cnt1 : k1_cnt0) & 1u;
                if (i & 1) ++k1_cnt1; else ++k1_cnt0;
                if (!ok) return;
                if (!wait(&bar_k1_full[gi][i & 1], par)) { ok = false; return; }
                nm_tc_fence_after();
                const uint64_t kdesc = nm_smem_desc_sw128(nm_smem_u32((i & 1) ? my_p : my_k));
                if (nm_elect_one()) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) nm_mma_f16(my_tmem, qdesc + 2 * k, kdesc + 2 * k, IDESC_QK1, k != 0);
                    nm_tc_commit(&bar_s_full[gi]);
                }
                __syncwarp();
            };
            if (cnt1 > 0) issue_qk1(0);
            for (int i = 0; i < cnt1; ++i) {
                asm volatile("bar.sync %0, %1;" ::"r"(bar_sc), "n"(160) : "memory");   // S-consumed: chunk i is in registers
                if (i + 1 < cnt1) issue_qk1(i + 1);
                if (ok && i + 2 < cnt1 && nm_elect_one()) {   // its MMAs are complete: the stage takes the chunk after next
                    uint8_t* dst = (i & 1) ? my_p : my_k;
                    const int key0 = (gi + NG * (i + 2)) * 2 * CK;
                    nm_mbar_expect_tx(&bar_k1_full[gi][i & 1], 2 * STAGE);
                    nm_tma_load_3d(dst, &tmK, g * HD, key0, b, &bar_k1_full[gi][i & 1]);
                    nm_tma_load_3d(dst + STAGE, &tmK, g * HD, key0 + CK, b, &bar_k1_full[gi][i & 1]);
                }
                __syncwarp();
            }
            // ---- sweep 2: the group's j-th chunk is the 64 keys of chunk g + NG*j; K stage j & 1
            auto load_k = [&](int j) {
                if (ok && nm_elect_one()) {
                    nm_mbar_expect_tx(&bar_k_full[gi][j & 1], STAGE);
                    nm_tma_load_3d(my_k + (size_t)(j & 1) * STAGE, &tmK, g * HD, (gi + NG * j) * CK, b, &bar_k_full[gi][j & 1]);
                }
                __syncwarp();
            };
            auto issue_qk = [&](int j) {   // S_g = Q K^T
                const uint32_t par = ((j & 1) ? k_cnt1 : k_cnt0) & 1u;
                if (j & 1) ++k_cnt1; else ++k_cnt0;
                if (!ok) return;
                if (!wait(&bar_k_full[gi][j & 1], par)) { ok = false; return; }
                nm_tc_fence_after();
                const uint64_t kdesc = nm_smem_desc_sw128(nm_smem_u32(my_k + (size_t)(j & 1) * STAGE));
                if (nm_elect_one()) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) nm_mma_f16(my_tmem, qdesc + 2 * k, kdesc + 2 * k, IDESC_QK, k != 0);
                    nm_tc_commit(&bar_s_full[gi]);
                }
                __syncwarp();
            };
            load_k(0);   // every MMA of sweep 1 has completed: the K stages are free
            if (half > 1) load_k(1);
            issue_qk(0);
            for (int j = 0; j < half; ++j) {
                asm volatile("bar.sync %0, %1;" ::"r"(bar_sc), "n"(160) : "memory");   // S-consumed(j)
                if (j + 1 < half) issue_qk(j + 1);
                if (j + 2 < half) load_k(j + 2);
                if constexpr (NG == 1) {
                    // Last chunk: every Q K^T of the tile has completed, so Q, the K stages and the P tile (which
                    // only sweep 1 uses when P goes through tensor memory) take the next tile's first loads now.
                    if (j + 1 == half && more && ok && nm_elect_one()) load_tile_head<NG>(lc, tile_of(tile + (int)gridDim.x));
                    __syncwarp();
                }
                asm volatile("bar.sync %0, %1;" ::"r"(bar_pr), "n"(160) : "memory");   // P-ready(j)
                if (ok && !wait(&bar_v_full[gi], v_cnt & 1u)) ok = false;
                ++v_cnt;
                if (ok) {
                    nm_tc_fence_after();
                    const uint64_t pdesc = nm_smem_desc_sw128(nm_smem_u32(my_p));
                    const uint32_t v_addr = nm_smem_u32(my_v);
                    if (nm_elect_one()) {
#pragma unroll
                        for (int k = 0; k < 4; ++k) {   // V rows (keys) 16k..16k+15: two groups of 8 rows, 1024 bytes apart
                            const uint64_t vdesc = nm_smem_desc_sw128(v_addr + (uint32_t)(16 * k * ROWB));
                            if constexpr (PT) mma_f16_a_tmem(my_tmem + O_OFF, tmem_p + (uint32_t)(8 * k), vdesc, IDESC_PV, (j | k) != 0);
                            else nm_mma_f16(my_tmem + O_OFF, pdesc + 2 * k, vdesc, IDESC_PV, (j | k) != 0);
                        }
                        nm_tc_commit(&bar_p_empty[gi]);
                    }
                    __syncwarp();
                }
                const uint32_t pv_par = pv_cnt & 1u;   // parity of this P V's completion
                ++pv_cnt;
                // the V stage is free once this P V has completed (nothing else to do until then): it takes the
                // next chunk's V, or after the last chunk the next tile's first one
                const bool next_v = j + 1 < half || (NG == 1 && more);
                if (ok && next_v) {
                    if (!wait(&bar_p_empty[gi], pv_par)) ok = false;
                    if (ok && nm_elect_one()) {
                        if (j + 1 < half) {
                            nm_mbar_expect_tx(&bar_v_full[gi], STAGE);
                            nm_tma_load_3d(my_v, &tmV, g * HD, (gi + NG * (j + 1)) * CK, b, &bar_v_full[gi]);
                        } else {
                            load_first_v(lc, tile_of(tile + (int)gridDim.x), gi);
                        }
                    }
                    __syncwarp();
                }
            }
        }
        if (!ok) {   // after an abort: let copies land and MMAs retire (bounded) before teardown
            if (nm_elect_one()) {
                nm_tc_commit(&bar_drain[gi]);
                long long t0 = clock64();
                while (!nm_mbar_try_wait(&bar_drain[gi], 0) && clock64() - t0 < 200000000LL) {}
                while (clock64() - t0 < 4000000LL) {}
            }
            __syncwarp();
        }
    } else {
        // ------------------------------------------------ softmax warps
        // Warps 2-5 (group 0) take the even chunks, warps 6-9 (group 1) the odd ones; group g owns S
        // buffer g, P buffer g and accumulator O_g, so the two groups form two independent pipelines.
        // A warp never blocks on its group: it signals the control warp with bar.arrive.
        const int q = warp & 3;
        const int g2 = NG == 1 ? 0 : (warp - NG) >> 2;
        const int row = q * 32 + lane;
        const uint32_t bar_sc = 2 + 2 * g2, bar_pr = 3 + 2 * g2, bar_oc = 6 + g2;
        const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)g2 * GRP_COLS;
        const int cnt1 = (n128 - g2 + NG - 1) / NG;   // the group's 128-key chunks in sweep 1
        const float inv_h = a.t_exp->inv_h, off = a.t_exp->off, nm1 = (float)(a.n_exp - 1);
        // this lane's copy of the replicated table, with the constant of the index trick folded in:
        // (bits << 7) = 0xA0000000 + s*128 (mod 2^32) for bits = 0x4B400000 + s
        const uint32_t rep_lane = nm_smem_u32(rep) + (uint32_t)(lane & 15) * 8u - 0xA0000000u;
        const uint64_t scale2 = nm_pack2(a.scale, a.scale), inv_h2 = nm_pack2(inv_h, inv_h), off2 = nm_pack2(off, off);
        const uint64_t magic2 = nm_pack2(12582912.0f, 12582912.0f);
        const uint32_t prow = nm_smem_u32(p_s) + (uint32_t)(g2 * PBUF + row * ROWB);
        const uint32_t p_row = tmem_p + ((uint32_t)(q * 32) << 16);   // this warp's lane quarter of the P columns
        int ok = 1;
        // All lanes test the barrier; only when it is not yet complete does lane 0 poll (with sleeps).
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
        // completions consumed so far: S products of this group, P V products of every group (the same count)
        uint32_t s_cnt = 0, pv_base = 0;
        for (int tile = (int)blockIdx.x; tile < n_tiles; tile += (int)gridDim.x) {
            const Tile t = tile_of(tile);
            const int qb = t.qb, g = t.g, b = t.b;
            const bool more = tile + (int)gridDim.x < n_tiles;
            // ---- sweep 1: the final row maximum
            float m = -INFINITY;
#pragma unroll 1
            for (int i = 0; i < cnt1; ++i) {
                wait_all(&bar_s_full[g2], s_cnt & 1u);
                ++s_cnt;
                if (ok) {
                    nm_tc_fence_after();
#pragma unroll
                    for (int hh = 0; hh < 4; ++hh) {   // 128 keys: the scores span [S_g | O_g]
                        uint32_t r[32];
                        nm_tmem_ld32_sync(t_row + (uint32_t)(hh * 32), r);
                        if (hh == 3) {   // all of it is in registers: the control warp may overwrite S
                            nm_tc_fence_before();
                            asm volatile("bar.arrive %0, %1;" ::"r"(bar_sc), "n"(160) : "memory");
                        }
                        float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
                        for (int k = 0; k < 32; k += 4) {
                            m0 = max3f(m0, __uint_as_float(r[k]), __uint_as_float(r[k + 1]));
                            m1 = max3f(m1, __uint_as_float(r[k + 2]), __uint_as_float(r[k + 3]));
                        }
                        m = max3f(m, m0, m1);
                    }
                } else {
                    asm volatile("bar.arrive %0, %1;" ::"r"(bar_sc), "n"(160) : "memory");
                }
            }
            if constexpr (NG == 2) {   // the two groups saw different keys of the row
                s_red[g2][row] = m;
                asm volatile("bar.sync 1, %0;" ::"n"(NSOFT) : "memory");
                m = fmaxf(s_red[0][row], s_red[1][row]);
                asm volatile("bar.sync 1, %0;" ::"n"(NSOFT) : "memory");
            }
            const float neg_ms = -(m * a.scale);
            const uint64_t neg_ms2 = nm_pack2(neg_ms, neg_ms);
            float sum0 = 0.f, sum1 = 0.f, sum2 = 0.f, sum3 = 0.f;
            // ---- sweep 2: e = PWL_exp(s - m), row sum, P tiles
#pragma unroll 1
            for (int j = 0; j < half; ++j) {
                wait_all(&bar_s_full[g2], s_cnt & 1u);
                ++s_cnt;
                if (ok) nm_tc_fence_after();
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    uint32_t r[32];
                    if (ok) {
                        nm_tmem_ld32_sync(t_row + (uint32_t)(hh * 32), r);
                    }
                    if (hh == 1) {
                        nm_tc_fence_before();
                        asm volatile("bar.arrive %0, %1;" ::"r"(bar_sc), "n"(160) : "memory");
                    }
                    uint32_t pk[16];   // the half's 32 exponentials, packed to 16 bits
                    if (ok) {
#pragma unroll
                        for (int jj = 0; jj < 4; ++jj) {   // 8 keys = one 16-byte chunk of the P row
                            float e[8];
#pragma unroll
                            for (int k = 0; k < 8; k += 2) {
                                // two scores at a time on the packed fp32 instructions: each half is the same correctly
                                // rounded operation as the scalar form
                                uint64_t x2, u2, b2;
                                asm("fma.rn.f32x2 %0, %1, %2, %3;"
                                    : "=l"(x2)
                                    : "l"(nm_pack2(__uint_as_float(r[jj * 8 + k]), __uint_as_float(r[jj * 8 + k + 1]))), "l"(scale2),
                                      "l"(neg_ms2));
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
                                // floor(u) sits in the low mantissa bits after a round-down add of 1.5 * 2^23
                                asm("add.rm.f32x2 %0, %1, %2;" : "=l"(b2) : "l"(nm_pack2(u0, u1)), "l"(magic2));
                                float f0, f1;
                                nm_unpack2(b2, f0, f1);
                                float k0, c0, k1, c1;
                                asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(k0), "=f"(c0) : "r"((__float_as_uint(f0) << 7) + rep_lane));
                                asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(k1), "=f"(c1) : "r"((__float_as_uint(f1) << 7) + rep_lane));
                                e[k] = __fmaf_rn(k0, x0, c0);
                                e[k + 1] = __fmaf_rn(k1, x1, c1);
                            }
                            sum0 += e[0] + e[4];
                            sum1 += e[1] + e[5];
                            sum2 += e[2] + e[6];
                            sum3 += e[3] + e[7];
#pragma unroll
                            for (int k = 0; k < 4; ++k) pk[jj * 4 + k] = AT<T>::pack(e[2 * k], e[2 * k + 1]);
                        }
                    }
                    // The stores wait until P V of the group's previous chunk has read the tile; that MMA was
                    // issued just before this chunk began, so the first half's arithmetic runs ahead of it.
                    if (hh == 0 && j >= 1) {
                        wait_all(&bar_p_empty[g2], (pv_base + (uint32_t)(j - 1)) & 1u);
                    }
                    if (ok) {
                        if constexpr (PT) {
                            if (hh == 0 && j >= 1) nm_tc_fence_after();   // ordered after the P V that read the columns
                            tmem_st16(p_row + (uint32_t)(hh * 16), pk);   // keys 32 hh .. 32 hh + 31 of this thread's row
                        } else {
#pragma unroll
                            for (int jj = 0; jj < 4; ++jj) {
                                // chunk index is XORed with the row (128-byte swizzle of the K-major P tile)
                                const uint32_t addr = prow + (uint32_t)(((hh * 4 + jj) ^ (row & 7)) << 4);
                                asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(pk[jj * 4]), "r"(pk[jj * 4 + 1]),
                                             "r"(pk[jj * 4 + 2]), "r"(pk[jj * 4 + 3])
                                             : "memory");
                            }
                        }
                    }
                }
                if constexpr (PT) {
                    tmem_st_wait();          // the P columns are written
                    nm_tc_fence_before();
                } else {
                    nm_fence_proxy_async();   // generic-proxy writes of P become visible to the tensor core
                }
                asm volatile("bar.arrive %0, %1;" ::"r"(bar_pr), "n"(160) : "memory");
            }
            float sum = (sum0 + sum1) + (sum2 + sum3);
            if constexpr (NG == 2) {
                s_red[g2][row] = sum;
                asm volatile("bar.sync 1, %0;" ::"n"(NSOFT) : "memory");
                sum = s_red[0][row] + s_red[1][row];
            }
            // ---- r = PWL_recip(sigma), then (O_0 + O_1) * r; each group stores 32 of the 64 channels
            const int sr = nm_pwl_index(sum, a.t_rcp->inv_h, a.t_rcp->off, (float)(a.t_rcp->n - 1));
            const float2 kbr = a.t_rcp->kb[sr];
            const float rinv = __fmaf_rn(kbr.x, sum, kbr.y);
#pragma unroll
            for (int gg = 0; gg < NG; ++gg)   // the last P V of every group has completed
                wait_all(&bar_p_empty[gg], (pv_base + (uint32_t)(half - 1)) & 1u);
            pv_base += (uint32_t)half;
            constexpr int CH = HD / NG;   // channels this warp stores
            if (ok) nm_tc_fence_after();
            T* orow = reinterpret_cast<T*>(a.out) + ((size_t)b * L + (size_t)qb * BQ + row) * ((size_t)a.heads * HD) +
                      (size_t)g * HD + g2 * CH;
            const uint32_t o_addr = tmem_base + ((uint32_t)(q * 32) << 16) + O_OFF + (uint32_t)(g2 * CH);
#pragma unroll
            for (int jj = 0; jj < CH / 16; ++jj) {   // 16 channels at a time, summed over the groups' accumulators
                uint32_t r0[16], r1[16];
                if (ok) {
                    nm_tmem_ld16_sync(o_addr + (uint32_t)(jj * 16), r0);
                    if constexpr (NG == 2) nm_tmem_ld16_sync(o_addr + GRP_COLS + (uint32_t)(jj * 16), r1);
                }
                if (jj == CH / 16 - 1 && more) {
                    // all of O is in registers: the control warp may start the next tile's sweep 1 over [S_g | O_g]
                    nm_tc_fence_before();
                    asm volatile("bar.arrive %0, %1;" ::"r"(bar_oc), "n"(160) : "memory");
                }
                if (ok) {
                    float v[16];
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        float x = __uint_as_float(r0[k]);
                        if constexpr (NG == 2) x += __uint_as_float(r1[k]);
                        v[k] = x * rinv;
                    }
                    if (a.out_q) {
                        int8_t code[16];
#pragma unroll
                        for (int k = 0; k < 16; ++k) code[k] = nm_quant_i8(AT<T>::round(v[k]), a.q_inv_scale);
                        int8_t* qrow = a.out_q + ((size_t)b * L + (size_t)qb * BQ + row) * ((size_t)a.heads * HD) +
                                       (size_t)g * HD + g2 * CH;
                        reinterpret_cast<uint4*>(qrow)[jj] = *reinterpret_cast<const uint4*>(code);
                    } else {
                        uint32_t w[8];
#pragma unroll
                        for (int k = 0; k < 8; ++k) w[k] = AT<T>::pack(v[2 * k], v[2 * k + 1]);
                        reinterpret_cast<uint4*>(orow)[2 * jj] = make_uint4(w[0], w[1], w[2], w[3]);
                        reinterpret_cast<uint4*>(orow)[2 * jj + 1] = make_uint4(w[4], w[5], w[6], w[7]);
                    }
                }
            }
        }
    }

    nm_tc_fence_before();
    __syncthreads();
    if (warp == NG - 1) {
        __syncwarp();
        nm_tc_fence_after();
        nm_tmem_dealloc(tmem_base, TMEM_COLS);
        if constexpr (PT) nm_tmem_dealloc(tmem_p, P_COLS);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [B][L][heads*64] view with token pitch stride_t and batch pitch stride_b (elements); box 64 x rows x 1.
nm_status make_map(nm_ctx* ctx, CUtensorMap* m, const void* ptr, nm_dtype dt, const nm_attn_desc* d, int rows)
{
    CUtensorMapDataType t = dt == NM_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
    cuuint64_t gdim[3] = {(cuuint64_t)d->heads * HD, (cuuint64_t)d->L, (cuuint64_t)d->B};
    cuuint64_t gstr[2] = {(cuuint64_t)d->stride_t * 2, (cuuint64_t)d->stride_b * 2};
    cuuint32_t box[3] = {HD, (cuuint32_t)rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = ((EncodeTiledFn)ctx->encode_tiled)(m, t, 3, const_cast<void*>(ptr), gdim, gstr, box, estr,
                                                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? NM_OK : NM_ERR_CUDA;
}

template <typename T, bool CLAMP_HI, int NG>
nm_status launch(nm_ctx* ctx, const nm_attn_desc* d, cudaStream_t st, int8_t* out_q, float q_inv_scale)
{
    SArgs a;
    a.B = d->B; a.L = d->L; a.heads = d->heads; a.scale = d->scale;
    a.t_exp = ctx->d_tables + d->exp_slot;
    a.t_rcp = ctx->d_tables + d->recip_slot;
    a.out = d->out;
    a.status = ctx->d_status;
    a.n_exp = ctx->h_tables[d->exp_slot].n;
    a.out_q = out_q;
    a.q_inv_scale = q_inv_scale;
    const size_t smem = (size_t)BQ * ROWB + NG * (3 * (size_t)STAGE + (size_t)PBUF) + (size_t)(a.n_exp + 1) * 16 * sizeof(float2) + 1024;
    if (smem > 227 * 1024 - 2048) return NM_ERR_UNSUPPORTED;   // an exp table too large to replicate
    CUtensorMap tmQ, tmK, tmV;
    nm_status s;
    if ((s = make_map(ctx, &tmQ, d->Q, d->dtype, d, BQ)) != NM_OK) return s;
    if ((s = make_map(ctx, &tmK, d->K, d->dtype, d, CK)) != NM_OK) return s;
    if ((s = make_map(ctx, &tmV, d->V, d->dtype, d, CK)) != NM_OK) return s;
    auto kern = attention_stream_kernel<T, CLAMP_HI, NG>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return NM_ERR_CUDA;
    const int64_t tiles = (int64_t)d->B * d->heads * (d->L / BQ);
    if (tiles > 0x7fffffffLL) return NM_ERR_SHAPE;
    int64_t grid = tiles;
    if (NG == 1) {
        // persistent: one resident wave of CTAs, each walking over tiles.  Three CTAs per SM by the launch bounds
        // (registers) and by tensor memory (3 x 160 of 512 columns); fewer if the exp table makes the shared
        // memory larger (233472 bytes per SM, 1 KB reserved per CTA).
        int64_t per_sm = 233472 / (int64_t)(smem + 1024 + 1536);
        if (per_sm > 3) per_sm = 3;
        if (per_sm < 1) per_sm = 1;
        const int64_t cap = (int64_t)ctx->sm_count * per_sm;
        if (grid > cap) grid = cap;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(160 * NG);
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

bool nm_attention_stream_supported(const nm_attn_desc* d)
{
    if (d->dtype != NM_BF16 && d->dtype != NM_F16) return false;
    if (d->d != HD) return false;
    if (d->L % 128 != 0 || d->L < 128) return false;
    if ((d->stride_t * 2) % 16 != 0 || (d->stride_b * 2) % 16 != 0) return false;
    return true;
}

nm_status nm_launch_attention_stream(nm_ctx* ctx, const nm_attn_desc* d, cudaStream_t st, int8_t* out_q,
                                     float q_inv_scale)
{
    if (!nm_attention_stream_supported(d)) return NM_ERR_UNSUPPORTED;
    // the softmax input is never positive: a table whose range reaches 0 needs no upper clamp
    const bool clamp_hi = ctx->h_tables[d->exp_slot].x_max < 0.0f;
    // One softmax group per CTA: three persistent CTAs per SM with P through tensor memory.  (The kernel text
    // still carries the two-group form, NG = 2, which splits the keys of a tile between two pipelines of one
    // CTA; it measured slower at every length from 128 to 2048 once P left shared memory, and is not built.)
    if (d->dtype == NM_BF16)
        return clamp_hi ? launch<__nv_bfloat16, true, 1>(ctx, d, st, out_q, q_inv_scale) : launch<__nv_bfloat16, false, 1>(ctx, d, st, out_q, q_inv_scale);
    return clamp_hi ? launch<__half, true, 1>(ctx, d, st, out_q, q_inv_scale) : launch<__half, false, 1>(ctx, d, st, out_q, q_inv_scale);
}
