// What the root receives from each of its f+1 children (Algorithm "reduce_root": "receive from any child (data,
// failure information)"): the value, whether anything arrived, the failed bit (third scheme of section "Failure
// information") and the size of the list of failed processes (second scheme). The batch kernels evaluate only the
// child the root selects; this kernel plays every child's subtree, dead nodes included: a node that does not send
// delivers nothing, its parent sets the failed bit and notes it. General shapes, level by level through a
// per-block slice of the workspace (values, then per-node presence / failed bit / list size).
#include "ftc_device.cuh"
#include "ftc_kernels.h"

namespace ftc {

template <typename T, int OP>
__global__ void __launch_bounds__(256) candidates_kernel(Params p, T* cand, uint32_t* info) {
    extern __shared__ uint32_t smem[];
    Ctx* cx = reinterpret_cast<Ctx*>(smem);
    uint32_t* pf = smem + sizeof(Ctx) / 4;
    uint32_t* inc = pf + p.W + 1;          // bit v: the value of v reaches the member of its group below child s
    uint32_t* snd = inc + p.W + 1;         // bit v: v performs its tree send
    const uint32_t tid = threadIdx.x, nt = blockDim.x;
    const size_t slice = (size_t)p.Gmax * p.kbytes + (size_t)p.Gmax * 12;
    char* wsb = reinterpret_cast<char*>(p.ws) + (size_t)blockIdx.x * ((slice + 15) & ~(size_t)15);
    T* val = reinterpret_cast<T*>(wsb);
    uint32_t* pres = reinterpret_cast<uint32_t*>(wsb + (size_t)p.Gmax * p.kbytes);
    uint32_t* fbit = pres + p.Gmax;
    uint32_t* nfl = fbit + p.Gmax;

    for (uint64_t s = blockIdx.x; s < p.S; s += gridDim.x) {
        decode_scenario(p, s, cx, pf, inc);
        T* cand_s = cand + s * (uint64_t)p.m * p.k;
        uint32_t* info_s = info + s * (uint64_t)p.m * 2;
        const uint32_t code = cx->code;
        if (code == FTC_ST_BAD_ROOT || code == FTC_ST_PRECONDITION_INOP_ROOT) {    // no attempt is played
            for (uint32_t u = tid; u < p.m * p.k; u += nt) cand_s[u] = T(0);
            for (uint32_t u = tid; u < p.m; u += nt) { info_s[2 * u] = 2; info_s[2 * u + 1] = 0; }
            __syncthreads();
            continue;
        }
        uint32_t root = cx->root, base = cx->base;
        if (code == FTC_ST_NO_LIVE_ROOT_CANDIDATE) {                                // the last attempt, toward a dead root
            const uint32_t first = p.root >= 0 ? (uint32_t)p.root : p.roots[s];
            root = (first + p.f) % p.P; base = p.f * p.Ratt;
        }
        const T* in_s = reinterpret_cast<const T*>(p.in) + s * (size_t)p.P * p.k;
        // the root's up-correction sends to the members of its (short, last) group happen in rounds 0, 1, ...
        const uint32_t troot = local_round(fail_round(p, cx, pf, root), base);
        // who sends up the tree (independent of the child looked at)
        for (uint32_t w = tid; w < p.W; w += nt) {
            uint32_t word = ~pf[w];
            if (w == p.W - 1 && (p.P & 31)) word &= (1u << (p.P & 31)) - 1u;
            snd[w] = word;
        }
        if (tid == 0) snd[p.W] = 0;
        __syncthreads();
        if (tid == 0 && root != 0) {               // renumbered bit `root` is process 0
            const uint32_t b0 = snd[0] & 1u;
            if (b0) snd[root >> 5] |= 1u << (root & 31); else snd[root >> 5] &= ~(1u << (root & 31));
        }
        __syncthreads();
        if (tid < p.max_inop && cx->iv[tid] != FTC_INOP_UNUSED) {
            const uint32_t v = renumber(cx->iv[tid], root);
            if (v) {
                const uint32_t d = 1 + heap_level(p.arity, (v - 1) / p.m), t = local_round(cx->ir[tid], base);
                if (!(p.f + p.H - d < t)) atomicAnd(&snd[v >> 5], ~(1u << (v & 31)));
            }
        }
        __syncthreads();

        for (uint32_t sc = 0; sc < p.m; ++sc) {
            // arrival mask for the members of subtree sc
            for (uint32_t w = tid; w < p.W; w += nt) {
                uint32_t word = ~pf[w];
                if (w == p.W - 1 && (p.P & 31)) word &= (1u << (p.P & 31)) - 1u;
                inc[w] = word;
            }
            if (tid == 0) inc[p.W] = 0;
            __syncthreads();
            if (tid == 0 && root != 0) {
                const uint32_t b0 = inc[0] & 1u;
                inc[0] |= 1u;
                if (b0) inc[root >> 5] |= 1u << (root & 31); else inc[root >> 5] &= ~(1u << (root & 31));
            }
            __syncthreads();
            if (tid < p.max_inop && cx->iv[tid] != FTC_INOP_UNUSED) {
                const uint32_t v = renumber(cx->iv[tid], root);
                if (v) {
                    const uint32_t j = (v - 1) / p.m, sv = (v - 1) % p.m, t = local_round(cx->ir[tid], base);
                    const bool has_member = j < p.q || sc < p.r;
                    if (has_member && sv != sc && !(partner_slot(p, j, sv, sc) < t)) atomicAnd(&inc[v >> 5], ~(1u << (v & 31)));
                }
            }
            __syncthreads();
            const uint32_t G = p.q + (sc < p.r ? 1u : 0u);
            // one node: its group's fold as member sc holds it (own input, then what arrived, in the partner order),
            // then its children in ascending order; a child that sent nothing sets the failed bit
            auto node = [&](uint32_t j, uint32_t e) {
                const uint32_t v = j * p.m + sc + 1;
                if (!test_bit(snd, v)) { if (e == 0) { pres[j] = 0; fbit[j] = 0; nfl[j] = 0; } return; }
                const uint32_t mj = j < p.q ? p.m : p.r, vbase = j * p.m + 1;
                const uint32_t mask = extract_bits(inc, vbase, mj);
                T acc = in_s[(size_t)renumber(v, root) * p.k + e];
                // the root's up-correction send to member sc of its group is its send number sc (descending: r-1-sc)
                const bool from_root = j == p.q && (p.pdesc ? p.r - 1 - sc : sc) < troot;
                if (from_root && !p.pdesc) acc = Comb<T, OP>::f(acc, in_s[(size_t)root * p.k + e]);
                for (uint32_t i = 0; i < mj; ++i) {
                    const uint32_t sp = p.pdesc ? mj - 1 - i : i;
                    if (sp != sc && ((mask >> sp) & 1u)) acc = Comb<T, OP>::f(acc, in_s[(size_t)renumber(vbase + sp, root) * p.k + e]);
                }
                if (from_root && p.pdesc) acc = Comb<T, OP>::f(acc, in_s[(size_t)root * p.k + e]);
                uint32_t fb = 0, nf = mj - __popc(mask) + ((j == p.q && !from_root) ? 1u : 0u);   // partners whose message did not arrive
                auto child = [&](uint64_t c) {
                    if (pres[c]) { acc = Comb<T, OP>::f(acc, val[(size_t)c * p.k + e]); fb |= fbit[c]; nf += nfl[c]; }
                    else { fb = 1; nf += 1; }
                };
                if (p.arity == 1) { for (uint64_t bit = 1; (j == 0 || bit < (j & (0u - j))) && j + bit < G; bit <<= 1) child(j + bit); }
                else for (uint64_t c = (uint64_t)p.arity * j + 1; c <= (uint64_t)p.arity * j + p.arity && c < G; ++c) child(c);
                val[(size_t)j * p.k + e] = acc;
                if (e == 0) { pres[j] = 1; fbit[j] = fb; nfl[j] = nf; }
            };
            if (p.arity == 1) {
                // binomial subtrees: a level's nodes are those with that many set bits
                for (int lvl = (int)p.H - 1; lvl >= 0; --lvl) {
                    for (uint32_t u = tid; u < G * p.k; u += nt)
                        if (__popc(u / p.k) == lvl) node(u / p.k, u % p.k);
                    __syncthreads();
                }
            } else {
                for (int lvl = (int)heap_level(p.arity, G - 1); lvl >= 0; --lvl) {
                    const uint32_t lo = (uint32_t)heap_level_start(p.arity, lvl);
                    const uint32_t hi = (uint32_t)min(heap_level_start(p.arity, lvl + 1), (uint64_t)G);
                    for (uint32_t u = tid; u < (hi - lo) * p.k; u += nt) node(lo + u / p.k, u % p.k);
                    __syncthreads();
                }
            }
            for (uint32_t e = tid; e < p.k; e += nt) cand_s[(size_t)sc * p.k + e] = pres[0] ? val[e] : T(0);
            if (tid == 0) { info_s[2 * sc] = pres[0] ? fbit[0] : 2u; info_s[2 * sc + 1] = pres[0] ? nfl[0] : 0u; }
            __syncthreads();
        }
    }
}

size_t candidates_slice_bytes(const Params& p) {
    const size_t slice = (size_t)p.Gmax * p.kbytes + (size_t)p.Gmax * 12;
    return (slice + 15) & ~(size_t)15;
}

template <typename T, int OP>
static cudaError_t launch_candidates_t(const Params& p, void* cand, uint32_t* info, int sm_count, cudaStream_t st) {
    const size_t smem = sizeof(Ctx) + 3 * (size_t)(p.W + 1) * 4;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(candidates_kernel<T, OP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    candidates_kernel<T, OP><<<generic_grid(p, sm_count), 256, smem, st>>>(p, static_cast<T*>(cand), info);
    return cudaGetLastError();
}

cudaError_t launch_candidates(const Params& p, int tsel, void* cand, uint32_t* info, int sm_count, cudaStream_t st) {
    switch (tsel) {
    case TS_U32_SUM: return launch_candidates_t<uint32_t, OP_SUM>(p, cand, info, sm_count, st);
    case TS_I32_MAX: return launch_candidates_t<int32_t, OP_MAX>(p, cand, info, sm_count, st);
    case TS_U32_XOR: return launch_candidates_t<uint32_t, OP_XOR>(p, cand, info, sm_count, st);
    case TS_U64_SUM: return launch_candidates_t<unsigned long long, OP_SUM>(p, cand, info, sm_count, st);
    case TS_I64_MAX: return launch_candidates_t<long long, OP_MAX>(p, cand, info, sm_count, st);
    case TS_U64_MAX: return launch_candidates_t<unsigned long long, OP_MAX>(p, cand, info, sm_count, st);
    case TS_U64_XOR: return launch_candidates_t<unsigned long long, OP_XOR>(p, cand, info, sm_count, st);
    case TS_F32_SUM: return launch_candidates_t<float, OP_SUM>(p, cand, info, sm_count, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace ftc
