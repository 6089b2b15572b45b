// Message accounting (theorem on the number of messages of a reduce, theorem on the messages of an allreduce,
// section "Properties"): how many up-correction, tree, tree-down and correction messages a scenario's
// processes send, over every attempt that is played and in the last one. No input value is read: which
// message is sent depends on the failure pattern only.
//
// Counting rule: a failure-free attempt sends the closed-form numbers; every process with a failure round t
// on the attempt's clock takes away exactly the sends it no longer performs ("a process that fails sends no
// more messages than one that does not"), and in the broadcast every process the tree no longer reaches takes
// away the sends it would have made as a holder of the value.
#include "ftc_device.cuh"
#include "ftc_kernels.h"

namespace ftc {

// Partners of renumbered process v in its up-correction group: f in a full group; in the short last group the
// r members see r-1 others plus the root, and the root sees the r members (none when there is no short group).
__device__ __forceinline__ uint32_t n_partners(const Params& p, uint32_t v) {
    if (v == 0) return p.r;
    return (v - 1) / p.m < p.q ? p.f : p.r;
}
__device__ __forceinline__ uint32_t depth_of(const Params& p, uint32_t v) { return v ? 1u + heap_level(p.arity, (v - 1) / p.m) : 0u; }

// What a process with failure round t (on the attempt's clock, t != kNever) does not send in the reduce of an
// attempt: up-correction sends i >= t, and its tree send when that lies in a round >= t.
__device__ __forceinline__ void reduce_loss(const Params& p, uint32_t v, uint32_t t, uint32_t& uc, uint32_t& tree) {
    const uint32_t np = n_partners(p, v);
    uc += np - min(np, t);
    if (v && t <= p.f + p.H - depth_of(p, v)) tree += 1;
}

constexpr int kMsgThreads = 128;

__global__ void __launch_bounds__(kMsgThreads) messages_kernel(Params p, unsigned long long* out) {
    extern __shared__ __align__(16) uint32_t smem[];
    Ctx* cx = reinterpret_cast<Ctx*>(smem);
    uint32_t* pf = smem + sizeof(Ctx) / 4;
    uint32_t* inc = pf + p.W + 1;
    uint32_t* unr = inc + p.W + 1;
    __shared__ uint32_t lost_uc[FTC_MAX_F + 1], lost_tree[FTC_MAX_F + 1];   // per attempt
    __shared__ uint32_t n_unreached, lost_corr;

    const uint32_t tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, wid = tid >> 5, nw = nt >> 5;
    const unsigned long long uc0 = (unsigned long long)p.f * p.m * p.q + (unsigned long long)(p.r + 1) * p.r;

    for (uint64_t s = blockIdx.x; s < p.S; s += gridDim.x) {
        decode_scenario(p, s, cx, pf, inc);
        unsigned long long* o = out + s * FTC_MSG_WORDS;
        const uint32_t code = cx->code;
        // attempts that are played: none for an invalid root or a violated precondition; one for a reduce
        const uint32_t A = (code == FTC_ST_BAD_ROOT || code == FTC_ST_PRECONDITION_INOP_ROOT) ? 0u
                           : (p.is_allreduce ? cx->attempts : 1u);
        if (A == 0) {
            if (tid < FTC_MSG_WORDS) o[tid] = 0;
            __syncthreads();
            continue;
        }
        const uint32_t first_root = p.root >= 0 ? (uint32_t)p.root : p.roots[s];
        if (tid <= FTC_MAX_F) { lost_uc[tid] = 0; lost_tree[tid] = 0; }
        if (tid == 0) { n_unreached = 0; lost_corr = 0; }
        __syncthreads();

        // ---- reduce part of every attempt: closed form minus what the failed processes do not send ----
        const bool my_slot = tid < p.max_inop && cx->iv[tid] != FTC_INOP_UNUSED && ((cx->ifirst >> tid) & 1u);
        for (uint32_t a = 0; a < A; ++a) {
            const uint32_t root = (first_root + a) % p.P, base = a * p.Ratt;
            uint32_t uc = 0, tree = 0;
            for (uint32_t w = tid; w < p.W; w += nt) {
                uint32_t word = pf[w];
                while (word) {
                    const uint32_t b = __ffs(word) - 1; word &= word - 1;
                    reduce_loss(p, renumber((w << 5) + b, root), 0u, uc, tree);
                }
            }
            if (my_slot) {
                const uint32_t t = local_round(cx->ir[tid], base);
                if (t != kNever) reduce_loss(p, renumber(cx->iv[tid], root), t, uc, tree);
            }
            uc = __reduce_add_sync(0xFFFFFFFFu, uc); tree = __reduce_add_sync(0xFFFFFFFFu, tree);
            if (lane == 0 && uc) atomicAdd(&lost_uc[a], uc);
            if (lane == 0 && tree) atomicAdd(&lost_tree[a], tree);
        }

        // ---- broadcast of the attempt that stands (a root that is alive and found a failure-free subtree) ----
        const bool bcast = p.is_allreduce && code == FTC_ST_OK;
        if (bcast) {
            const uint32_t root = cx->root, base = cx->base;
            for (uint32_t w = tid; w <= p.W; w += nt) unr[w] = 0;
            __syncthreads();
            // a process that does not pass the value on cuts off everything below it: bit v of unr = the tree-down
            // phase sends no message to renumbered process v
            auto mark_below = [&](uint32_t v) {
                const uint32_t sv = (v - 1) % p.m;
                mark_descendants(p.arity, p.m, unr, (v - 1) / p.m, sv, p.q + (sv < p.r ? 1u : 0u), lane);
            };
            const uint32_t nwords_round = (p.W + 31) & ~31u;
            for (uint32_t w0 = wid * 32; w0 < nwords_round; w0 += nw * 32) {
                const uint32_t w = w0 + lane;
                const uint32_t word = w < p.W ? pf[w] : 0u;
                uint32_t pend = __ballot_sync(0xFFFFFFFFu, word != 0);
                while (pend) {
                    const uint32_t src = __ffs(pend) - 1; pend &= pend - 1;
                    uint32_t ww = __shfl_sync(0xFFFFFFFFu, word, src);
                    const uint32_t wbase = (w0 + src) << 5;
                    while (ww) {
                        const uint32_t b = __ffs(ww) - 1; ww &= ww - 1;
                        const uint32_t v = renumber(wbase + b, root);
                        if (v) mark_below(v);
                    }
                }
            }
            if (wid == 0) {
                for (uint32_t i = 0; i < p.max_inop; ++i) {
                    if (cx->iv[i] == FTC_INOP_UNUSED || !((cx->ifirst >> i) & 1u)) continue;
                    const uint32_t v = renumber(cx->iv[i], root), t = local_round(cx->ir[i], base);
                    // the tree-down send of a process at depth d is round f+H+d of the attempt
                    if (v && t <= p.Rred + depth_of(p, v)) mark_below(v);
                }
            }
            __syncthreads();
            // correction sends that are not made: all of an unreached process, and of a reached process that
            // has a failure round those scheduled in rounds >= it (correction iteration i is round f+2H+i)
            const uint32_t rowq0 = p.q * p.m + 1;            // first member of the short last group
            uint32_t n = 0, loss = 0;
            for (uint32_t w = tid; w < p.W; w += nt) {
                const uint32_t word = unr[w];
                uint32_t in_short = 0;
                if (((w + 1) << 5) > rowq0) in_short = (w << 5) >= rowq0 ? word : (word & ~((1u << (rowq0 & 31)) - 1u));
                const uint32_t nq = __popc(in_short), nall = __popc(word);
                n += nall; loss += (nall - nq) * p.f + nq * p.r;
                uint32_t dead = pf[w];
                while (dead) {
                    const uint32_t b = __ffs(dead) - 1; dead &= dead - 1;
                    const uint32_t v = renumber((w << 5) + b, root);
                    if (v && !test_bit(unr, v)) loss += n_partners(p, v);
                }
            }
            if (my_slot) {
                const uint32_t v = renumber(cx->iv[tid], root), t = local_round(cx->ir[tid], base);
                if (v && t != kNever && !test_bit(unr, v)) {
                    const uint32_t np = n_partners(p, v);
                    // it holds the value only if it was still alive when it sent up the tree
                    const uint32_t sent = t > p.f + p.H - depth_of(p, v) ? min(np, t > p.Rred + p.H ? t - (p.Rred + p.H) : 0u) : 0u;
                    loss += np - sent;
                }
            }
            n = __reduce_add_sync(0xFFFFFFFFu, n); loss = __reduce_add_sync(0xFFFFFFFFu, loss);
            if (lane == 0 && n) atomicAdd(&n_unreached, n);
            if (lane == 0 && loss) atomicAdd(&lost_corr, loss);
        }
        __syncthreads();
        if (tid == 0) {
            unsigned long long all_uc = 0, all_tree = 0;
            for (uint32_t a = 0; a < A; ++a) { all_uc += uc0 - lost_uc[a]; all_tree += (p.P - 1) - lost_tree[a]; }
            const unsigned long long bt = bcast ? (p.P - 1) - n_unreached : 0ull, corr = bcast ? uc0 - lost_corr : 0ull;
            o[0] = all_uc; o[1] = all_tree; o[2] = bt; o[3] = corr;
            o[4] = uc0 - lost_uc[A - 1]; o[5] = (p.P - 1) - lost_tree[A - 1]; o[6] = bt; o[7] = corr;
        }
        __syncthreads();
    }
}

// The list of failed processes that reaches the root with the value it delivers (first scheme of section "Failure
// information"): every process appends the ids of those it could not receive a value from, in the up-correction
// phase and in the tree phase, and the lists travel up the tree with the values. The child the root selects has no
// failed process in its subtree, so its list holds exactly the up-correction partners whose message did not reach
// the subtree's member of their group; when that subtree holds no member of the root's own (short, last) group the
// root adds those it noted itself. Group by group that is the complement of the arrival mask the decode builds.
// Output: the list as a bitmask over the caller's process ids, and its size.
__global__ void __launch_bounds__(kMsgThreads) failed_list_kernel(Params p, uint32_t* failed, uint32_t* nfail) {
    extern __shared__ __align__(16) uint32_t smem[];
    Ctx* cx = reinterpret_cast<Ctx*>(smem);
    uint32_t* pf = smem + sizeof(Ctx) / 4;
    uint32_t* inc = pf + p.W + 1;
    __shared__ uint32_t total;
    const uint32_t tid = threadIdx.x, nt = blockDim.x, lane = tid & 31;
    for (uint64_t s = blockIdx.x; s < p.S; s += gridDim.x) {
        decode_scenario(p, s, cx, pf, inc);
        if (tid == 0) total = 0;
        __syncthreads();
        const bool ok = cx->code == FTC_ST_OK;
        const uint32_t root = cx->root;
        // bit `root` of the renumbered mask belongs to process 0, bit 0 to the root (which delivers, so it is alive)
        const uint32_t b0 = ok && root != 0 ? ((~inc[root >> 5]) >> (root & 31)) & 1u : 0u;
        uint32_t cnt = 0;
        for (uint32_t w = tid; w < p.W; w += nt) {
            uint32_t word = 0;
            if (ok) {
                word = ~inc[w];
                if (w == p.W - 1 && (p.P & 31)) word &= (1u << (p.P & 31)) - 1u;
                if (w == 0) word &= ~1u;
                cnt += __popc(word);
                if (root != 0) {
                    if (w == (root >> 5)) word &= ~(1u << (root & 31));
                    if (w == 0) word |= b0;
                }
            }
            failed[s * p.W + w] = word;
        }
        cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
        if (lane == 0 && cnt) atomicAdd(&total, cnt);
        __syncthreads();
        if (tid == 0) nfail[s] = total;
        __syncthreads();
    }
}

cudaError_t launch_failed_list(const Params& p, uint32_t* failed, uint32_t* nfail, int sm_count, cudaStream_t st) {
    const size_t smem = sizeof(Ctx) + 2 * (size_t)(p.W + 1) * 4;
    cudaError_t e = cudaFuncSetAttribute(failed_list_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const uint64_t cap = (uint64_t)sm_count * 8;
    const uint32_t grid = (uint32_t)(p.S < cap ? p.S : cap);
    failed_list_kernel<<<grid, kMsgThreads, smem, st>>>(p, failed, nfail);
    return cudaGetLastError();
}

size_t messages_smem_bytes(const Params& p) { return sizeof(Ctx) + 3 * (size_t)(p.W + 1) * 4; }

cudaError_t launch_messages(const Params& p, unsigned long long* out, int sm_count, cudaStream_t st) {
    const size_t smem = messages_smem_bytes(p);
    cudaError_t e = cudaFuncSetAttribute(messages_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const uint64_t cap = (uint64_t)sm_count * 8;
    const uint32_t grid = (uint32_t)(p.S < cap ? p.S : cap);
    messages_kernel<<<grid, kMsgThreads, smem, st>>>(p, out);
    return cudaGetLastError();
}

}  // namespace ftc
