// Host side of the tensor-core linear operator: tile selection, tensor maps and launch of
// linear_tc_kernel (linear_tc_kernel.cuh) for matrices in memory.
#include "linear_tc_kernel.cuh"

using namespace nm_tc;

namespace {

template <typename InT, typename OutT, bool TWO, int BN>
nm_status launch(nm_ctx* ctx, const nm_linear_desc* d, cudaStream_t st)
{
    constexpr int B_ROWS = TWO ? BN / 2 : BN;
    constexpr int TILE_M = TWO ? 2 * BM : BM;
    TcArgs a;
    memset(&a, 0, sizeof(a));
    a.M = d->M; a.N = d->N; a.K = d->K;
    a.bias = d->bias;
    a.has_res = d->residual ? 1 : 0;
    a.res_first = d->res_first;
    a.tab = d->slot == NM_SLOT_NONE ? nullptr : ctx->d_tables + d->slot;
    a.n_seg = d->slot == NM_SLOT_NONE ? 0 : ctx->h_tables[d->slot].n;
    a.a_scale = d->a_scale; a.w_scale = d->w_scale; a.inv_out_scale = d->inv_out_scale;
    a.acc_dump = d->acc_dump; a.idx_dump = d->idx_dump;
    a.status = ctx->d_status;
    const int bk = ROW_BYTES / (int)sizeof(InT);
    const int64_t m_tiles = (d->M + TILE_M - 1) / TILE_M;
    a.num_n_tiles = (int)((d->N + BN - 1) / BN);
    if (m_tiles * a.num_n_tiles > 0x7fffffffLL) return NM_ERR_SHAPE;
    a.num_tiles = (int)(m_tiles * a.num_n_tiles);
    a.num_k_blocks = (int)((d->K + bk - 1) / bk);
    size_t smem = 0;
    if (!plan_smem<InT, TWO, BN>(&a, d->bias || TcIn<InT>::is_int, &smem)) return NM_ERR_UNSUPPORTED;

    CUtensorMap tmA, tmW, tmO, tmR;
    nm_status s = make_tmap(ctx, &tmA, d->A, d->in_dtype, d->M, d->K, d->lda, BM);
    if (s != NM_OK) return s;
    s = make_tmap(ctx, &tmW, d->W, d->in_dtype, d->N, d->K, d->ldw, B_ROWS);
    if (s != NM_OK) return s;
    s = make_tmap(ctx, &tmO, d->out, d->out_dtype, d->M, d->N, d->ldo, 32);
    if (s != NM_OK) return s;
    if (d->residual) s = make_tmap(ctx, &tmR, d->residual, d->out_dtype, d->M, d->N, d->ldr, 32);
    else tmR = tmO;
    if (s != NM_OK) return s;
    return launch_kernel<InT, OutT, TWO, BN, false>(ctx, tmA, tmW, tmO, tmR, a, smem,
                                                    2.0 * (double)d->M * (double)d->N * (double)d->K, st);
}

template <typename InT, typename OutT, int BN>
nm_status launch_two(nm_ctx* ctx, const nm_linear_desc* d, cudaStream_t st)
{
    // algo 3 forces the one-CTA tile; otherwise problems with at least one 256-row tile use CTA pairs
    if (d->algo != 3 && d->M >= 256) return launch<InT, OutT, true, BN>(ctx, d, st);
    return launch<InT, OutT, false, BN>(ctx, d, st);
}

template <typename InT, typename OutT>
nm_status launch_sel(nm_ctx* ctx, const nm_linear_desc* d, cudaStream_t st)
{
    // narrow layers get a narrow tile (built for the 16-bit types)
    if constexpr (!TcIn<InT>::is_int) {
        if (d->N <= 64) return launch_two<InT, OutT, 64>(ctx, d, st);
        if (d->N <= 128) return launch_two<InT, OutT, 128>(ctx, d, st);
    }
    return launch_two<InT, OutT, 256>(ctx, d, st);
}

}  // namespace

bool nm_linear_tc_supported(const nm_linear_desc* d)
{
    if (d->in_dtype == NM_F32) return false;
    const size_t es = nm_dtype_size(d->in_dtype);
    if (d->M < 1 || d->N < 8 || d->K < 1) return false;
    if ((d->K * es) % 16 != 0) return false;  // TMA: global extents and pitches in 16-byte units
    if (d->N % 4 != 0) return false;          // vector loads of bias / scales, vector dumps
    if (d->in_dtype == NM_I8) return d->out_dtype == NM_BF16 || d->out_dtype == NM_F32 || d->out_dtype == NM_I8;
    return d->out_dtype == d->in_dtype;
}

nm_status nm_launch_linear_tc(nm_ctx* ctx, const nm_linear_desc* d, cudaStream_t st)
{
    if (!nm_linear_tc_supported(d)) return NM_ERR_UNSUPPORTED;
    switch (d->in_dtype) {
    case NM_BF16: return launch_sel<__nv_bfloat16, __nv_bfloat16>(ctx, d, st);
    case NM_F16: return launch_sel<__half, __half>(ctx, d, st);
    case NM_I8:
        if (d->out_dtype == NM_BF16) return launch_sel<int8_t, __nv_bfloat16>(ctx, d, st);
        if (d->out_dtype == NM_F32) return launch_sel<int8_t, float>(ctx, d, st);
        return launch_sel<int8_t, int8_t>(ctx, d, st);
    default: return NM_ERR_UNSUPPORTED;
    }
}
