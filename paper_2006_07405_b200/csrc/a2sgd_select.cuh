// Kernel selection: maps the run-time shape of a call (mode, worker count, access width, ...) to
// one instantiation of the kernel templates.  Like the kernel headers it is compiled once per
// kernel variant into the namespace A2SGD_NS (after a2sgd_kernels.cuh and a2sgd_segments.cuh), and
// each variant exports its choices as one a2sgd_kernel_table.
namespace A2SGD_NS {

const void *select_encode(bool ef, bool mask, int vw)
{
#define A2_PICK(EF, MASK)                                                               \
    (vw == 8 ? (const void *)k_encode_vec<EF, MASK, 8>                                  \
             : vw == 4 ? (const void *)k_encode_vec<EF, MASK, 4> : (const void *)k_encode_scalar<EF, MASK>)
    if (ef) return mask ? A2_PICK(true, true) : A2_PICK(true, false);
    return mask ? A2_PICK(false, true) : A2_PICK(false, false);
#undef A2_PICK
}

template <bool EF, bool STORE, int VW, bool MOM>
const void *select_decode_shared_p(uint32_t P)
{
    switch (P) {
    case 1: return (const void *)k_decode_shared_vec<EF, STORE, 1, VW, 0, MOM>;
    case 2: return (const void *)k_decode_shared_vec<EF, STORE, 2, VW, 0, MOM>;
    case 4: return (const void *)k_decode_shared_vec<EF, STORE, 4, VW, 0, MOM>;
    case 8: return (const void *)k_decode_shared_vec<EF, STORE, 8, VW, 0, MOM>;
    default: return (const void *)k_decode_shared_vec<EF, STORE, 0, VW, 0, MOM>;
    }
}

template <bool MOM>
const void *select_decode_shared_m(bool ef, bool store, uint32_t P, int vw)
{
    if (vw == 8) {
        if (ef) return select_decode_shared_p<true, true, 8, MOM>(P);
        return store ? select_decode_shared_p<false, true, 8, MOM>(P) : select_decode_shared_p<false, false, 8, MOM>(P);
    }
    if (ef) return select_decode_shared_p<true, true, 4, MOM>(P);
    return store ? select_decode_shared_p<false, true, 4, MOM>(P) : select_decode_shared_p<false, false, 4, MOM>(P);
}

const void *select_decode_shared(bool ef, bool store, uint32_t P, int vw, bool mom)
{
    return mom ? select_decode_shared_m<true>(ef, store, P, vw) : select_decode_shared_m<false>(ef, store, P, vw);
}

template <bool MOM>
const void *select_decode_repl_m(bool ef, bool store, int vw)
{
    if (vw == 8) {
        if (ef) return (const void *)k_decode_repl_vec<true, true, 8, 0, MOM>;
        return store ? (const void *)k_decode_repl_vec<false, true, 8, 0, MOM>
                     : (const void *)k_decode_repl_vec<false, false, 8, 0, MOM>;
    }
    if (ef) return (const void *)k_decode_repl_vec<true, true, 4, 0, MOM>;
    return store ? (const void *)k_decode_repl_vec<false, true, 4, 0, MOM>
                 : (const void *)k_decode_repl_vec<false, false, 4, 0, MOM>;
}

const void *select_decode_repl(bool ef, bool store, int vw, bool mom)
{
    return mom ? select_decode_repl_m<true>(ef, store, vw) : select_decode_repl_m<false>(ef, store, vw);
}

const void *select_decode_scalar(bool ef, bool store, bool mom)
{
    if (mom) {
        if (ef) return (const void *)k_decode_scalar<true, true, 0, true>;
        return store ? (const void *)k_decode_scalar<false, true, 0, true> : (const void *)k_decode_scalar<false, false, 0, true>;
    }
    if (ef) return (const void *)k_decode_scalar<true, true>;
    return store ? (const void *)k_decode_scalar<false, true> : (const void *)k_decode_scalar<false, false>;
}

// 16-bit gradient rows (GT = 1 bfloat16, 2 half): 8-element (128-bit) vectors or scalar accesses
template <bool EF, bool STORE, int GT>
const void *select_decode_shared_lowp_p(uint32_t P)
{
    switch (P) {
    case 1: return (const void *)k_decode_shared_vec<EF, STORE, 1, 8, GT>;
    case 2: return (const void *)k_decode_shared_vec<EF, STORE, 2, 8, GT>;
    case 4: return (const void *)k_decode_shared_vec<EF, STORE, 4, 8, GT>;
    case 8: return (const void *)k_decode_shared_vec<EF, STORE, 8, 8, GT>;
    default: return (const void *)k_decode_shared_vec<EF, STORE, 0, 8, GT>;
    }
}

template <int GT>
const void *select_encode_lowp(bool ef, int vw)
{
    if (vw == 8) return ef ? (const void *)k_encode_vec<true, false, 8, GT> : (const void *)k_encode_vec<false, false, 8, GT>;
    return ef ? (const void *)k_encode_scalar<true, false, GT> : (const void *)k_encode_scalar<false, false, GT>;
}

template <int GT>
const void *select_decode_lowp(bool ef, bool store, bool shared, uint32_t P, int vw)
{
    if (vw == 8 && shared) {
        if (ef) return select_decode_shared_lowp_p<true, true, GT>(P);
        return store ? select_decode_shared_lowp_p<false, true, GT>(P) : select_decode_shared_lowp_p<false, false, GT>(P);
    }
    if (vw == 8) {
        if (ef) return (const void *)k_decode_repl_vec<true, true, 8, GT>;
        return store ? (const void *)k_decode_repl_vec<false, true, 8, GT> : (const void *)k_decode_repl_vec<false, false, 8, GT>;
    }
    if (ef) return (const void *)k_decode_scalar<true, true, GT>;
    return store ? (const void *)k_decode_scalar<false, true, GT> : (const void *)k_decode_scalar<false, false, GT>;
}

template <int VW, bool REPL>
const void *select_dense_p(uint32_t P)
{
    switch (P) {
    case 1: return (const void *)k_dense_sync_vec<1, VW, REPL>;
    case 2: return (const void *)k_dense_sync_vec<2, VW, REPL>;
    case 4: return (const void *)k_dense_sync_vec<4, VW, REPL>;
    case 8: return (const void *)k_dense_sync_vec<8, VW, REPL>;
    default: return (const void *)k_dense_sync_vec<0, VW, REPL>;
    }
}

const void *select_dense(uint32_t P, int vw, bool repl)
{
    if (vw == 8) return repl ? select_dense_p<8, true>(P) : select_dense_p<8, false>(P);
    if (vw == 4) return repl ? select_dense_p<4, true>(P) : select_dense_p<4, false>(P);
    return (const void *)k_dense_sync_scalar;
}

template <bool EF, bool STORE, bool SHARED>
const void *select_coop_p(uint32_t P)
{
    switch (P) {
    case 1: return (const void *)k_step_coop<EF, STORE, 1, SHARED>;
    case 2: return (const void *)k_step_coop<EF, STORE, 2, SHARED>;
    case 4: return (const void *)k_step_coop<EF, STORE, 4, SHARED>;
    case 8: return (const void *)k_step_coop<EF, STORE, 8, SHARED>;
    default: return nullptr;
    }
}

template <bool EF, bool STORE, bool SHARED>
const void *select_coop_l2_p(uint32_t P)
{
    switch (P) {
    case 1: return (const void *)k_step_coop_l2<EF, STORE, 1, SHARED>;
    case 2: return (const void *)k_step_coop_l2<EF, STORE, 2, SHARED>;
    case 4: return (const void *)k_step_coop_l2<EF, STORE, 4, SHARED>;
    case 8: return (const void *)k_step_coop_l2<EF, STORE, 8, SHARED>;
    default: return nullptr;
    }
}

const void *select_coop_l2(bool ef, bool store, bool shared, uint32_t P)
{
    if (ef) return shared ? select_coop_l2_p<true, true, true>(P) : select_coop_l2_p<true, true, false>(P);
    if (store) return shared ? select_coop_l2_p<false, true, true>(P) : select_coop_l2_p<false, true, false>(P);
    return shared ? select_coop_l2_p<false, false, true>(P) : select_coop_l2_p<false, false, false>(P);
}

const void *select_coop(bool ef, bool store, bool shared, uint32_t P)
{
    if (ef) return shared ? select_coop_p<true, true, true>(P) : select_coop_p<true, true, false>(P);
    if (store) return shared ? select_coop_p<false, true, true>(P) : select_coop_p<false, true, false>(P);
    return shared ? select_coop_p<false, false, true>(P) : select_coop_p<false, false, false>(P);
}

template <bool REPL>
const void *select_decode_deferred(uint32_t P)
{
    switch (P) {
    case 1: return (const void *)k_decode_deferred<1, REPL>;
    case 2: return (const void *)k_decode_deferred<2, REPL>;
    case 4: return (const void *)k_decode_deferred<4, REPL>;
    case 8: return (const void *)k_decode_deferred<8, REPL>;
    default: return (const void *)k_decode_deferred<0, REPL>;
    }
}

template <bool EF, bool STORE, bool PER_TENSOR>
const void *select_decode_segments_p(uint32_t P)
{
    switch (P) {
    case 1: return (const void *)k_decode_segments<EF, STORE, 1, PER_TENSOR>;
    case 2: return (const void *)k_decode_segments<EF, STORE, 2, PER_TENSOR>;
    case 4: return (const void *)k_decode_segments<EF, STORE, 4, PER_TENSOR>;
    case 8: return (const void *)k_decode_segments<EF, STORE, 8, PER_TENSOR>;
    default: return (const void *)k_decode_segments<EF, STORE, 0, PER_TENSOR>;
    }
}

inline const void *table_encode_deferred(bool holds_v)
{
    return holds_v ? (const void *)k_encode_vec<true, true, 8, 0, 2> : (const void *)k_encode_vec<true, true, 8, 0, 1>;
}
inline const void *table_encode_lowp(int gt, bool ef, int vw)
{
    return gt == 1 ? select_encode_lowp<1>(ef, vw) : select_encode_lowp<2>(ef, vw);
}
inline const void *table_encode_segments(bool ef, bool per_tensor)
{
    if (per_tensor) return ef ? (const void *)k_encode_segments<true, true> : (const void *)k_encode_segments<false, true>;
    return ef ? (const void *)k_encode_segments<true, false> : (const void *)k_encode_segments<false, false>;
}
inline const void *table_decode_lowp(int gt, bool ef, bool store, bool shared, uint32_t P, int vw)
{
    return gt == 1 ? select_decode_lowp<1>(ef, store, shared, P, vw) : select_decode_lowp<2>(ef, store, shared, P, vw);
}
inline const void *table_decode_deferred(bool repl, uint32_t P)
{
    return repl ? select_decode_deferred<true>(P) : select_decode_deferred<false>(P);
}
template <bool PER_TENSOR>
const void *table_decode_segments_m(bool ef, bool store, uint32_t P)
{
    return ef ? select_decode_segments_p<true, true, PER_TENSOR>(P)
              : store ? select_decode_segments_p<false, true, PER_TENSOR>(P)
                      : select_decode_segments_p<false, false, PER_TENSOR>(P);
}
inline const void *table_decode_segments(bool ef, bool store, uint32_t P, bool per_tensor)
{
    return per_tensor ? table_decode_segments_m<true>(ef, store, P) : table_decode_segments_m<false>(ef, store, P);
}

inline a2sgd_kernel_table kernel_table()
{
    a2sgd_kernel_table t{};
    t.encode = select_encode;
    t.encode_deferred = table_encode_deferred;
    t.encode_lowp = table_encode_lowp;
    t.encode_segments = table_encode_segments;
    t.decode_shared = select_decode_shared;
    t.decode_repl = select_decode_repl;
    t.decode_scalar = select_decode_scalar;
    t.decode_lowp = table_decode_lowp;
    t.decode_deferred = table_decode_deferred;
    t.decode_segments = table_decode_segments;
    t.dense = select_dense;
    t.coop = select_coop;
    t.coop_l2 = select_coop_l2;
    t.global_average = (const void *)k_global_average;
    t.global_average_from_sums = (const void *)k_global_average_from_sums;
    t.materialize_err = (const void *)k_materialize_err;
    t.fold_jobs = (const void *)k_fold_jobs;
    t.fold_segments = (const void *)k_fold_segments;
    return t;
}

} // namespace A2SGD_NS
