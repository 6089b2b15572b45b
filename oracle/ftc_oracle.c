/*
 * ftc_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, literal CPU simulation of the correction-based fault-tolerant
 * reduce and allreduce of Kuettler & Haertig, "Fault-tolerant Reduce and
 * Allreduce operations based on correction".  Every logical process is a small
 * state machine that executes its own program (send, receive, combine) and
 * exchanges explicit messages with the others; a cooperative scheduler sweeps
 * over the processes until all have finished.  Nothing is blocked, fused,
 * reordered or derived in closed form: the result is whatever the messages
 * produce.  It shares no code, header, table or helper with the CUDA library
 * and must only be used by tests, the smoke check and the CPU-baseline timing.
 *
 * Passages followed (section / algorithm names of the paper):
 *   - failure model (section "Failures"): a failed process stops sending; a
 *     send to a failed process completes silently.
 *   - root renumbering (section "Reduce", first paragraph): the root swaps
 *     numbers with process 0.
 *   - up-correction groups and Algorithm "Up-correction": group number
 *     floor((p-1)/(f+1)); the root joins the last group iff that group has
 *     fewer than f+1 members; every member sends its ORIGINAL value to every
 *     other member and folds what it receives into its data.
 *   - Algorithms "reduce_root", "reduce_non_root", "reduce": tree phase over
 *     an I(f)-tree with the interleaved numbering (process a lies in the
 *     subtree of root child k iff (a-1) mod (f+1) = k-1), single failed bit
 *     as failure information (third scheme of section "Failure information").
 *   - Algorithm "Allreduce": reduce to root candidate r, broadcast from r,
 *     next candidate if r had failed before the operation.
 *
 * Readings where the paper is silent (the same ones the documentation lists):
 *   - group partners are visited in ascending (renumbered) rank, skipping self,
 *     the root first in the short last group (on request: the reverse order);
 *   - below each root child the subtree is a heap on the local index
 *     j = floor((v-1)/(f+1)): binary by default (children 2j+1 and 2j+2), or
 *     a-ary on request (children a*j+1 .. a*j+a), or a binomial tree (parent of
 *     j = j without its lowest set bit), children received in ascending order;
 *     the paper asks only for f+1 root children whose subtree sizes differ by
 *     at most one, which the interleaved numbering gives for any such shape;
 *   - the root examines its children in ascending order and takes the first
 *     message that arrived with the failed bit clear;
 *   - a "failure round" t of a process means: it performs exactly those of
 *     its sends that are scheduled in rounds < t.  Up-correction iteration i
 *     is round i (rounds 0..f-1), the tree send of a node at depth d is round
 *     f+H-d, H = depth of the deepest node (binary: 1+floor(log2(ceil((n-1)/(f+1))))).  A broadcast adds H rounds
 *     of tree-down sends (a node at depth d sends to all its children in
 *     round d of the broadcast) and f rounds of correction.  An allreduce
 *     attempt therefore has 2(f+H) rounds and attempt a starts at a*2(f+H);
 *   - the broadcast (not defined in this paper) is assembled from the paper's
 *     own pieces: the value travels down the same tree, then every process
 *     that got it from the tree sends it to the other members of its
 *     up-correction group.  It only copies the root's value.
 *   - root candidates of the allreduce are first_root, first_root+1, ...
 *     (mod n), f+1 of them; the loop stops at the first candidate that had
 *     not failed before the operation.
 *
 * Parity pins live in tests/ (worked example of the paper, message-count
 * theorem, brute-force reductions over every failure set on small n,
 * scheduler-order independence).  Unpinned by the paper: the fp32 combine
 * order, the broadcast's round and message counts, and which of several
 * correct results is chosen under in-operation failures; those rest on the
 * readings above ("parity unpinned" for these three).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_NEVER INT64_MAX

enum { DT_I32 = 0, DT_I64 = 1, DT_U64 = 2, DT_F32 = 3 };
enum { OP_SUM = 0, OP_MAX = 1, OP_XOR = 2 };
enum { ST_OK = 0, ST_ROOT_FAILED = 1, ST_NO_CLEAN_SUBTREE = 2, ST_NO_LIVE_ROOT_CANDIDATE = 3,
       ST_PRECONDITION_INOP_ROOT = 4 };
enum { SLOT_NOT_YET = 0, SLOT_SENT = 1, SLOT_SKIPPED = 2 };
enum { PH_UC = 0, PH_TREE_RECV, PH_TREE_SEND, PH_ROOT_SELECT, PH_BC_RECV, PH_BC_SEND, PH_CORR, PH_DONE, PH_DEAD };

typedef struct {
    uint32_t P, f, k;
    uint32_t dtype;
    uint32_t op;
    uint32_t max_inop;   /* in-operation failure slots per scenario */
    uint32_t sweep;      /* scheduler order: 0 descending rank, 1 ascending, >=2 seeded shuffle */
    uint32_t track_sets; /* carry a P-bit contribution set with every value (instrumentation) */
    uint32_t partners_descending; /* 1: group partners are visited in descending rank, the root last (default: ascending, root first) */
    uint32_t arity;      /* shape below the root's children: 0 or 2 = binary heap, a >= 2 = a-ary heap, 1 = binomial tree */
} orc_cfg_t;

typedef struct { uint32_t victim, round; } orc_inop_t;

/* Every pointer may be NULL. Indices named "physical" are the caller's process ids. */
typedef struct {
    void*     result;     /* [k] value at the root (reduce) / value every holder has (allreduce) */
    uint32_t* status;     /* [4] code | subtree<<8 | attempts<<16 ; |C| ; in-op included mask ; holders */
    void*     cand;       /* [f+1][k] what each root child delivered in the last attempt */
    uint32_t* cand_flag;  /* [f+1] 0 delivered clean, 1 delivered with failed bit, 2 nothing delivered */
    uint32_t* holders;    /* [ceil(P/32)] physical ids that deliver the allreduce value */
    void*     expanded;   /* [P][k] value per physical process, zeros for non-holders */
    uint64_t* msgs;       /* [8] all attempts: upcorr, tree, bcast-tree, bcast-corr; last attempt: same four */
    uint32_t* contrib;    /* [ceil(P/32)] physical ids whose input is in the result (needs track_sets) */
    uint32_t* sends;      /* [P] messages sent by each physical process over all attempts */
    uint32_t* events;     /* [P] bit0 init called, bit1 deliver called, bit2 deliver called twice */
    void*     uc_values;  /* [P][k] data of each physical process after up-correction (last attempt) */
    void*     tree_values;/* [P][k] payload of each physical process' tree message (zeros if unsent) */
    uint32_t* tree_sent;  /* [P] 1 if the tree message was sent, with bit1 = its failed bit */
    uint32_t* tree_sets;  /* [P][ceil(P/32)] contribution set of each tree message (needs track_sets) */
    uint32_t* cand_nfail; /* [f+1] size of the failed-process list each root child delivered (0 if nothing) */
    uint32_t* nfail;      /* [1] size of the root's final list of failed processes */
    uint32_t* failed;     /* [ceil(P/32)] that list, physical ids (needs track_sets) */
} orc_out_t;

typedef struct {
    const orc_cfg_t* cfg;
    uint32_t P, f, k, m, esz, W;
    uint32_t arity;     /* children per node below the root's children */
    uint32_t q, r, H, Rred, Ratt;
    int is_allreduce;
    uint32_t root;      /* physical id of the current root */
    int64_t base;       /* first round of the current attempt */
    /* per virtual rank */
    unsigned char* x;      /* [P][k] original input ("senddata") */
    unsigned char* data;   /* [P][k] */
    unsigned char* tdata;  /* [P][k] tree message payload */
    unsigned char* hval;   /* [P][k] broadcast value held */
    unsigned char* ucval;  /* [P][k] data right after up-correction */
    uint8_t *failbit, *tfail, *tree_state, *bct_state, *hold, *tree_holder;
    uint8_t *uc_state, *corr_state; /* [P][f] */
    uint8_t *phase, *sub;
    uint32_t *idx;
    uint32_t *cnt, *tcnt, *imask, *timask, *imask0;
    uint32_t *nf, *tnf;     /* size of the list of known failed processes (second failure-information scheme) */
    uint32_t *fl, *tfl;     /* the list itself as a P-bit set per process / per tree message, when tracking (first scheme) */
    uint32_t *set, *tset;  /* [P][W] when tracking */
    int64_t* fail_round;   /* per virtual rank, global clock */
    uint8_t *inited, *delivered;
    uint32_t* nsent;       /* per virtual rank, this attempt */
    uint64_t msgs_attempt[4];
    /* root outcome of the attempt */
    uint32_t st_code, st_subtree;
} sim_t;


/* ---- renumbering: the root swaps numbers with process 0 ---- */
static uint32_t v2p(const sim_t* s, uint32_t v) { return v == 0 ? s->root : (v == s->root ? 0 : v); }

/* ---- the reduction function: dst <- dst (op) src, accumulator on the left ---- */
static void combine(const sim_t* s, void* dst, const void* src) {
    uint32_t k = s->k, i;
    switch (s->cfg->dtype) {
    case DT_I32: {
        uint32_t* d = (uint32_t*)dst; const uint32_t* c = (const uint32_t*)src;
        for (i = 0; i < k; ++i) {
            if (s->cfg->op == OP_SUM) d[i] = d[i] + c[i];            /* wraps mod 2^32 */
            else if (s->cfg->op == OP_MAX) d[i] = ((int32_t)d[i] >= (int32_t)c[i]) ? d[i] : c[i];
            else d[i] = d[i] ^ c[i];
        }
    } break;
    case DT_I64: {
        uint64_t* d = (uint64_t*)dst; const uint64_t* c = (const uint64_t*)src;
        for (i = 0; i < k; ++i) {
            if (s->cfg->op == OP_SUM) d[i] = d[i] + c[i];
            else if (s->cfg->op == OP_MAX) d[i] = ((int64_t)d[i] >= (int64_t)c[i]) ? d[i] : c[i];
            else d[i] = d[i] ^ c[i];
        }
    } break;
    case DT_U64: {
        uint64_t* d = (uint64_t*)dst; const uint64_t* c = (const uint64_t*)src;
        for (i = 0; i < k; ++i) {
            if (s->cfg->op == OP_SUM) d[i] = d[i] + c[i];
            else if (s->cfg->op == OP_MAX) d[i] = (d[i] >= c[i]) ? d[i] : c[i];
            else d[i] = d[i] ^ c[i];
        }
    } break;
    default: {
        float* d = (float*)dst; const float* c = (const float*)src;
        for (i = 0; i < k; ++i) { volatile float t = d[i] + c[i]; d[i] = t; } /* one fp32 rounding per add */
    } break;
    }
}

static void merge_contrib(sim_t* s, uint32_t* cnt, uint32_t* imask, uint32_t* set,
                          uint32_t ocnt, uint32_t oimask, const uint32_t* oset, int* overlap) {
    *cnt += ocnt;
    if (*imask & oimask) *overlap = 1;
    *imask |= oimask;
    if (s->cfg->track_sets) {
        for (uint32_t w = 0; w < s->W; ++w) { if (set[w] & oset[w]) *overlap = 1; set[w] |= oset[w]; }
    }
}

/* the unmodified input of process u carries exactly u's own contribution */
static void merge_single(sim_t* s, uint32_t v, uint32_t u, int* overlap) {
    s->cnt[v] += 1;
    if (s->imask[v] & s->imask0[u]) *overlap = 1;
    s->imask[v] |= s->imask0[u];
    if (s->set) {
        uint32_t* w = s->set + (size_t)v * s->W + (u >> 5);
        if (*w & (1u << (u & 31))) *overlap = 1;
        *w |= 1u << (u & 31);
    }
}

/* process v could not receive a value from u: append u to v's list of failed processes */
static void note_failed(sim_t* s, uint32_t v, uint32_t u) {
    s->nf[v] += 1;
    if (s->fl) s->fl[(size_t)v * s->W + (u >> 5)] |= 1u << (u & 31);
}
/* v takes over the list that came with a message */
static void take_list(sim_t* s, uint32_t v, uint32_t n, const uint32_t* list) {
    s->nf[v] += n;
    if (s->fl) for (uint32_t w = 0; w < s->W; ++w) s->fl[(size_t)v * s->W + w] |= list[w];
}

/* ---- topology in renumbered ranks ---- */
static uint32_t row_of(const sim_t* s, uint32_t v) { return (v - 1) / s->m; }      /* group number */
static uint32_t sub_of(const sim_t* s, uint32_t v) { return (v - 1) % s->m; }      /* root child index */
static uint32_t rank_of(const sim_t* s, uint32_t j, uint32_t sidx) { return j * s->m + sidx + 1; }
/* level of local index j in an a-ary heap: level l holds the a^l indices after those of the levels above */
static uint32_t heap_level(uint32_t arity, uint32_t j) {
    if (arity == 1) { uint32_t l = 0; for (; j; j &= j - 1) ++l; return l; }   /* binomial tree: depth = number of set bits */
    uint32_t l = 0; uint64_t start = 0, width = 1;
    while (j >= start + width) { start += width; width *= arity; ++l; }
    return l;
}
/* deepest level among the local indices 0..G-1 */
static uint32_t deepest_level(uint32_t arity, uint32_t G) {
    if (arity != 1) return heap_level(arity, G - 1);
    uint32_t best = 0;
    for (uint32_t j = 0; j < G; ++j) { uint32_t l = heap_level(1, j); if (l > best) best = l; }
    return best;
}
static uint32_t depth_of(const sim_t* s, uint32_t v) { return v == 0 ? 0 : 1 + heap_level(s->arity, row_of(s, v)); }

/* members of the up-correction group of v in the order v visits them (ascending rank with the root first, or the
   reverse), v excluded; returns their number */
static uint32_t partners_ascending(const sim_t* s, uint32_t v, uint32_t* out) {
    uint32_t n = 0, lo, hi, u;
    if (v == 0) {
        if (s->r == 0) return 0;                       /* root belongs to no group */
        lo = s->q * s->m + 1; hi = s->P - 1;           /* last, short group */
        for (u = lo; u <= hi; ++u) out[n++] = u;
        return n;
    }
    uint32_t j = row_of(s, v);
    lo = j * s->m + 1; hi = lo + s->m - 1; if (hi > s->P - 1) hi = s->P - 1;
    if (j == s->q) out[n++] = 0;                        /* short last group: the root is a member, rank 0 first */
    for (u = lo; u <= hi; ++u) if (u != v) out[n++] = u;
    return n;
}
static uint32_t partners(const sim_t* s, uint32_t v, uint32_t* out) {
    uint32_t n = partners_ascending(s, v, out);
    if (s->cfg->partners_descending)
        for (uint32_t i = 0; i + 1 < n - i; ++i) { uint32_t t = out[i]; out[i] = out[n - 1 - i]; out[n - 1 - i] = t; }
    return n;
}
static uint32_t partner_index(const sim_t* s, uint32_t u, uint32_t v) {
    uint32_t buf[64], n = partners(s, u, buf), i;
    for (i = 0; i < n; ++i) if (buf[i] == v) return i;
    return 0xFFFFFFFFu;
}
/* tree children of v; the root's children are ranks 1..f+1 */
static uint32_t children(const sim_t* s, uint32_t v, uint32_t* out) {
    uint32_t n = 0;
    if (v == 0) { for (uint32_t c = 1; c <= s->m && c < s->P; ++c) out[n++] = c; return n; }
    uint32_t j = row_of(s, v), sidx = sub_of(s, v);
    if (s->arity == 1) {
        /* binomial tree on the local index: the parent of j is j without its lowest set bit, so the children of j
           are j + 2^i for every 2^i below that bit (all powers of two for j = 0), in ascending order */
        for (uint64_t bit = 1; (j == 0 || bit < (j & (0u - j))) && (j + bit) * s->m + sidx + 1 < s->P; bit <<= 1)
            out[n++] = rank_of(s, (uint32_t)(j + bit), sidx);
        return n;
    }
    for (uint32_t c = 1; c <= s->arity; ++c) {
        uint64_t jc = (uint64_t)s->arity * j + c;                 /* heap children of j: a*j+1 .. a*j+a */
        if (jc * s->m + sidx + 1 < s->P) out[n++] = rank_of(s, (uint32_t)jc, sidx);
    }
    return n;
}
static uint32_t parent_of(const sim_t* s, uint32_t v) {
    uint32_t j = row_of(s, v);
    if (s->arity == 1) return j == 0 ? 0 : rank_of(s, j & (j - 1), sub_of(s, v));
    return j == 0 ? 0 : rank_of(s, (j - 1) / s->arity, sub_of(s, v));
}

/* A send scheduled in round `round` happens iff the sender's failure round is later. */
static int can_send(const sim_t* s, uint32_t v, int64_t round) { return round < s->fail_round[v]; }

static void die(sim_t* s, uint32_t v) {
    for (uint32_t i = 0; i < s->f; ++i) {
        if (s->uc_state[(size_t)v * s->f + i] == SLOT_NOT_YET) s->uc_state[(size_t)v * s->f + i] = SLOT_SKIPPED;
        if (s->corr_state[(size_t)v * s->f + i] == SLOT_NOT_YET) s->corr_state[(size_t)v * s->f + i] = SLOT_SKIPPED;
    }
    if (s->tree_state[v] == SLOT_NOT_YET) s->tree_state[v] = SLOT_SKIPPED;
    if (s->bct_state[v] == SLOT_NOT_YET) s->bct_state[v] = SLOT_SKIPPED;
    s->phase[v] = PH_DEAD;
}

static void deliver(sim_t* s, uint32_t v) {
    if (s->delivered[v]) s->delivered[v] = 2; else s->delivered[v] = 1;
}

/* Run process v until it blocks, finishes or dies. Returns 1 if it made progress. */
static int advance(sim_t* s, uint32_t v, int* overlap) {
    int progress = 0;
    uint32_t pb[64], cb[64];
    size_t kb = (size_t)s->k * s->esz;
    for (;;) {
        switch (s->phase[v]) {
        case PH_DONE: case PH_DEAD: return progress;
        case PH_UC: {
            uint32_t np = partners(s, v, pb);
            if (s->idx[v] >= np) {
                memcpy(s->ucval + v * kb, s->data + v * kb, kb);
                s->idx[v] = 0; s->sub[v] = 0;
                s->phase[v] = (v == 0) ? PH_ROOT_SELECT : PH_TREE_RECV;
                progress = 1; break;
            }
            uint32_t i = s->idx[v], u = pb[i];
            if (s->sub[v] == 0) {           /* send (senddata) to p */
                if (!can_send(s, v, s->base + i)) { die(s, v); return 1; }
                s->uc_state[(size_t)v * s->f + i] = SLOT_SENT;
                s->msgs_attempt[0]++; s->nsent[v]++;
                s->sub[v] = 1; progress = 1;
            }
            /* receive (data) from p */
            uint32_t iu = partner_index(s, u, v);
            uint8_t st = s->uc_state[(size_t)u * s->f + iu];
            if (st == SLOT_NOT_YET) return progress;
            if (st == SLOT_SENT) {
                combine(s, s->data + v * kb, s->x + u * kb);   /* payload is p's unmodified input */
                merge_single(s, v, u, overlap);
            } else note_failed(s, v, u);   /* p has failed: noted in the list; the failed bit is not touched in this phase */
            s->idx[v]++; s->sub[v] = 0; progress = 1;
        } break;
        case PH_TREE_RECV: {
            uint32_t nc = children(s, v, cb);
            if (s->idx[v] >= nc) { s->phase[v] = PH_TREE_SEND; progress = 1; break; }
            uint32_t c = cb[s->idx[v]];
            uint8_t st = s->tree_state[c];
            if (st == SLOT_NOT_YET) return progress;
            if (st == SLOT_SENT) {
                combine(s, s->data + v * kb, s->tdata + c * kb);
                s->failbit[v] |= s->tfail[c];
                merge_contrib(s, &s->cnt[v], &s->imask[v], s->set ? s->set + (size_t)v * s->W : NULL,
                              s->tcnt[c], s->timask[c], s->tset ? s->tset + (size_t)c * s->W : NULL, overlap);
                take_list(s, v, s->tnf[c], s->tfl ? s->tfl + (size_t)c * s->W : NULL);
            } else {
                s->failbit[v] = 1;          /* no value from this child: set the failed bit */
                note_failed(s, v, c);
            }
            s->idx[v]++; progress = 1;
        } break;
        case PH_TREE_SEND: {
            int64_t round = s->base + s->f + s->H - depth_of(s, v);
            if (!can_send(s, v, round)) { die(s, v); return 1; }
            memcpy(s->tdata + v * kb, s->data + v * kb, kb);
            s->tfail[v] = s->failbit[v]; s->tcnt[v] = s->cnt[v]; s->timask[v] = s->imask[v]; s->tnf[v] = s->nf[v];
            if (s->tfl) memcpy(s->tfl + (size_t)v * s->W, s->fl + (size_t)v * s->W, (size_t)s->W * 4);
            if (s->tset) memcpy(s->tset + (size_t)v * s->W, s->set + (size_t)v * s->W, (size_t)s->W * 4);
            s->tree_state[v] = SLOT_SENT;
            s->msgs_attempt[1]++; s->nsent[v]++;
            if (!s->is_allreduce) deliver(s, v);   /* deliver_reduce after sending to the parent */
            s->idx[v] = 0; s->sub[v] = 0;
            s->phase[v] = s->is_allreduce ? PH_BC_RECV : PH_DONE;
            progress = 1;
        } break;
        case PH_ROOT_SELECT: {
            /* Is the root still alive when the last tree messages arrive? */
            if (!(s->base + (int64_t)s->Rred <= s->fail_round[v])) {
                s->st_code = ST_ROOT_FAILED; die(s, v); return 1;
            }
            uint32_t nc = children(s, v, cb);
            int chosen = -1;
            while (s->idx[v] < nc) {
                uint32_t c = cb[s->idx[v]];
                uint8_t st = s->tree_state[c];
                if (st == SLOT_NOT_YET) return progress;
                progress = 1;
                if (st == SLOT_SKIPPED || s->tfail[c]) { s->idx[v]++; continue; }
                chosen = (int)s->idx[v]; break;
            }
            if (chosen < 0) {
                s->st_code = ST_NO_CLEAN_SUBTREE; s->st_subtree = 0xFF;
                if (s->is_allreduce) { s->bct_state[v] = SLOT_SKIPPED; s->phase[v] = PH_CORR; s->idx[v] = 0; s->sub[v] = 0; }
                else s->phase[v] = PH_DONE;
                break;
            }
            uint32_t c = cb[chosen];
            if ((uint32_t)chosen < s->r) {
                /* this subtree holds a member of the root's group, hence the root's value already */
                memcpy(s->data + v * kb, s->tdata + c * kb, kb);
                s->cnt[v] = s->tcnt[c]; s->imask[v] = s->timask[c];
                if (s->set) memcpy(s->set + (size_t)v * s->W, s->tset + (size_t)c * s->W, (size_t)s->W * 4);
                s->nf[v] = s->tnf[c];       /* and its list of failed processes is the complete one */
                if (s->fl) memcpy(s->fl + (size_t)v * s->W, s->tfl + (size_t)c * s->W, (size_t)s->W * 4);
            } else {
                combine(s, s->data + v * kb, s->tdata + c * kb);   /* root's data on the left */
                merge_contrib(s, &s->cnt[v], &s->imask[v], s->set ? s->set + (size_t)v * s->W : NULL,
                              s->tcnt[c], s->timask[c], s->tset ? s->tset + (size_t)c * s->W : NULL, overlap);
                take_list(s, v, s->tnf[c], s->tfl ? s->tfl + (size_t)c * s->W : NULL);
            }
            s->st_code = ST_OK; s->st_subtree = (uint32_t)chosen;
            if (!s->is_allreduce) { deliver(s, v); s->phase[v] = PH_DONE; }
            else {
                memcpy(s->hval + v * kb, s->data + v * kb, kb);
                s->hold[v] = 1; s->tree_holder[v] = 1;
                s->phase[v] = PH_BC_SEND;
            }
            progress = 1;
        } break;
        case PH_BC_RECV: {
            uint32_t par = parent_of(s, v);
            uint8_t st = s->bct_state[par];
            if (st == SLOT_NOT_YET) return progress;
            if (st == SLOT_SENT) {
                memcpy(s->hval + v * kb, s->hval + par * kb, kb);
                s->hold[v] = 1; s->tree_holder[v] = 1;
            }
            s->phase[v] = PH_BC_SEND; progress = 1;
        } break;
        case PH_BC_SEND: {
            uint32_t nc = children(s, v, cb);
            if (!s->tree_holder[v] || nc == 0) { s->bct_state[v] = SLOT_SKIPPED; }   /* nothing to pass on, or nobody below */
            else {
                int64_t round = s->base + s->Rred + depth_of(s, v);
                if (!can_send(s, v, round)) { die(s, v); return 1; }
                s->bct_state[v] = SLOT_SENT;
                s->msgs_attempt[2] += nc; s->nsent[v] += nc;
            }
            s->idx[v] = 0; s->sub[v] = 0; s->phase[v] = PH_CORR; progress = 1;
        } break;
        case PH_CORR: {
            uint32_t np = partners(s, v, pb);
            if (s->idx[v] >= np) {
                /* end of the attempt: deliver if still alive and holding the value */
                if (s->base + (int64_t)s->Ratt <= s->fail_round[v]) { if (s->hold[v]) deliver(s, v); s->phase[v] = PH_DONE; }
                else die(s, v);
                return 1;
            }
            uint32_t i = s->idx[v], u = pb[i];
            if (s->sub[v] == 0) {
                if (s->tree_holder[v]) {
                    int64_t round = s->base + s->Rred + s->H + i;
                    if (!can_send(s, v, round)) { die(s, v); return 1; }
                    s->corr_state[(size_t)v * s->f + i] = SLOT_SENT;
                    s->msgs_attempt[3]++; s->nsent[v]++;
                } else s->corr_state[(size_t)v * s->f + i] = SLOT_SKIPPED;
                s->sub[v] = 1; progress = 1;
            }
            uint32_t iu = partner_index(s, u, v);
            uint8_t st = s->corr_state[(size_t)u * s->f + iu];
            if (st == SLOT_NOT_YET) return progress;
            if (st == SLOT_SENT && !s->hold[v]) { memcpy(s->hval + v * kb, s->hval + u * kb, kb); s->hold[v] = 1; }
            s->idx[v]++; s->sub[v] = 0; progress = 1;
        } break;
        }
    }
}

static uint64_t mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull; z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull; return z ^ (z >> 31);
}

/* Plays one attempt (reduce, plus broadcast for an allreduce) toward `root`. Returns 0, or -1 on deadlock. */
static int play_attempt(sim_t* s, const void* in, const int64_t* fail_round_phys, const uint32_t* imask_phys,
                        uint32_t root, int64_t base, uint32_t* order, int* overlap) {
    uint32_t P = s->P, f = s->f, v;
    size_t kb = (size_t)s->k * s->esz;
    s->root = root; s->base = base;
    s->st_code = ST_ROOT_FAILED; s->st_subtree = 0xFF;
    memset(s->msgs_attempt, 0, sizeof s->msgs_attempt);
    for (v = 0; v < P; ++v) {
        uint32_t p = v2p(s, v);
        memcpy(s->x + v * kb, (const unsigned char*)in + p * kb, kb);
        memcpy(s->data + v * kb, s->x + v * kb, kb);
        memset(s->tdata + v * kb, 0, kb); memset(s->hval + v * kb, 0, kb); memset(s->ucval + v * kb, 0, kb);
        s->fail_round[v] = fail_round_phys[p];
        s->failbit[v] = 0; s->tfail[v] = 0; s->tree_state[v] = SLOT_NOT_YET; s->bct_state[v] = SLOT_NOT_YET;
        s->hold[v] = 0; s->tree_holder[v] = 0;
        for (uint32_t i = 0; i < f; ++i) { s->uc_state[(size_t)v * f + i] = SLOT_NOT_YET; s->corr_state[(size_t)v * f + i] = SLOT_NOT_YET; }
        s->phase[v] = PH_UC; s->idx[v] = 0; s->sub[v] = 0;
        s->cnt[v] = 1; s->tcnt[v] = 0; s->timask[v] = 0; s->nf[v] = 0; s->tnf[v] = 0;
        if (s->fl) { memset(s->fl + (size_t)v * s->W, 0, (size_t)s->W * 4); memset(s->tfl + (size_t)v * s->W, 0, (size_t)s->W * 4); }
        s->imask[v] = imask_phys[p]; s->imask0[v] = imask_phys[p];
        if (s->set) { memset(s->set + (size_t)v * s->W, 0, (size_t)s->W * 4); s->set[(size_t)v * s->W + (v >> 5)] = 1u << (v & 31);
                      memset(s->tset + (size_t)v * s->W, 0, (size_t)s->W * 4); }
        s->nsent[v] = 0; s->delivered[v] = 0;
        if (s->fail_round[v] <= base) { s->inited[v] = 0; die(s, v); }   /* failed before this attempt began */
        else s->inited[v] = 1;                                          /* init_(all)reduce */
    }
    for (;;) {
        int progress = 0, pending = 0;
        for (uint32_t t = 0; t < P; ++t) {
            v = order[t];
            progress |= advance(s, v, overlap);
        }
        for (v = 0; v < P; ++v) if (s->phase[v] != PH_DONE && s->phase[v] != PH_DEAD) { pending = 1; break; }
        if (!pending) return 0;
        if (!progress) return -1;
    }
}

/*
 * One scenario. `root` is the reduce root, or the first root candidate of an allreduce.
 * Returns 0; -1 invalid arguments; -2 out of memory; -3 scheduler deadlock; -4 a value was combined twice.
 */
int ftc_oracle_run(const orc_cfg_t* cfg, int is_allreduce, const void* in, const uint32_t* prefail,
                   const orc_inop_t* inop, uint32_t root, const orc_out_t* out) {
    if (!cfg || !in || !prefail || !out) return -1;
    uint32_t P = cfg->P, f = cfg->f, k = cfg->k;
    if (k == 0 || P < f + 2 || f + 1 > 60 || root >= P || cfg->max_inop > 32) return -1;
    if (cfg->arity > 32) return -1;
    if (cfg->dtype > DT_F32 || cfg->op > OP_XOR) return -1;
    if (cfg->dtype == DT_F32 && cfg->op != OP_SUM) return -1;
    sim_t S; memset(&S, 0, sizeof S);
    sim_t* s = &S;
    s->cfg = cfg; s->P = P; s->f = f; s->k = k; s->m = f + 1;
    s->esz = (cfg->dtype == DT_I32 || cfg->dtype == DT_F32) ? 4 : 8;
    s->W = (P + 31) / 32;
    s->q = (P - 1) / s->m; s->r = (P - 1) % s->m;
    s->arity = cfg->arity ? cfg->arity : 2;
    s->H = 1 + deepest_level(s->arity, s->q + (s->r ? 1 : 0));      /* depth of the deepest node of the largest subtree */
    s->Rred = f + s->H; s->Ratt = 2 * s->Rred;
    s->is_allreduce = is_allreduce;
    size_t kb = (size_t)k * s->esz, fz = f ? f : 1;
    s->x = malloc(P * kb); s->data = malloc(P * kb); s->tdata = malloc(P * kb); s->hval = malloc(P * kb); s->ucval = calloc(P, kb);
    s->failbit = malloc(P); s->tfail = malloc(P); s->tree_state = malloc(P); s->bct_state = malloc(P);
    s->hold = malloc(P); s->tree_holder = malloc(P);
    s->uc_state = malloc(P * fz); s->corr_state = malloc(P * fz);
    s->phase = malloc(P); s->sub = malloc(P); s->idx = malloc(P * 4);
    s->cnt = malloc(P * 4); s->tcnt = malloc(P * 4); s->imask = malloc(P * 4); s->imask0 = malloc(P * 4); s->timask = malloc(P * 4);
    s->nf = malloc(P * 4); s->tnf = malloc(P * 4);
    s->fail_round = malloc(P * 8); s->inited = malloc(P); s->delivered = malloc(P); s->nsent = malloc(P * 4);
    int64_t* frp = malloc(P * 8); uint32_t* imp = calloc(P, 4); uint32_t* order = malloc(P * 4);
    uint32_t* sends_tot = calloc(P, 4); uint8_t* ev = calloc(P, 1);
    if (cfg->track_sets) { s->set = malloc((size_t)P * s->W * 4); s->tset = malloc((size_t)P * s->W * 4);
                           s->fl = malloc((size_t)P * s->W * 4); s->tfl = malloc((size_t)P * s->W * 4); }
    int rc = 0;
    if (!s->x || !s->data || !s->tdata || !s->hval || !s->failbit || !s->tfail || !s->tree_state || !s->bct_state ||
        !s->hold || !s->tree_holder || !s->uc_state || !s->corr_state || !s->phase || !s->sub || !s->idx || !s->cnt ||
        !s->tcnt || !s->imask || !s->imask0 || !s->ucval || !s->timask || !s->fail_round || !s->inited || !s->delivered || !s->nsent || !frp ||
        !imp || !order || !sends_tot || !ev || !s->nf || !s->tnf ||
        (cfg->track_sets && (!s->set || !s->tset || !s->fl || !s->tfl))) { rc = -2; goto done; }

    /* failure rounds on the global clock: 0 = failed before the operation */
    for (uint32_t p = 0; p < P; ++p) frp[p] = ((prefail[p >> 5] >> (p & 31)) & 1) ? 0 : ORC_NEVER;
    for (uint32_t i = 0; i < cfg->max_inop && inop; ++i) {
        uint32_t vic = inop[i].victim;
        if (vic == 0xFFFFFFFFu) continue;
        if (vic >= P) { rc = -1; goto done; }
        if ((int64_t)inop[i].round < frp[vic]) frp[vic] = inop[i].round;
    }
    for (uint32_t i = 0; i < cfg->max_inop && inop; ++i) {
        uint32_t vic = inop[i].victim;
        if (vic == 0xFFFFFFFFu) continue;
        if (frp[vic] > 0) imp[vic] |= 1u << i;          /* slot bits of processes that fail during the operation */
    }
    /* scheduler order */
    for (uint32_t t = 0; t < P; ++t) order[t] = (cfg->sweep == 1) ? t : P - 1 - t;
    if (cfg->sweep >= 2) {
        for (uint32_t t = 0; t < P; ++t) order[t] = t;
        uint64_t z = cfg->sweep;
        for (uint32_t t = P - 1; t > 0; --t) { z = mix64(z); uint32_t u = (uint32_t)(z % (t + 1)); uint32_t tmp = order[t]; order[t] = order[u]; order[u] = tmp; }
    }

    uint64_t msgs_all[4] = {0, 0, 0, 0};
    uint32_t attempts = 0, code = ST_OK, subtree = 0xFF;
    int overlap = 0, have_result = 0;

    if (is_allreduce) {
        /* candidates must be known never to fail during the operation */
        for (uint32_t a = 0; a <= f; ++a) {
            uint32_t c = (root + a) % P;
            if (frp[c] != 0 && frp[c] != ORC_NEVER) { code = ST_PRECONDITION_INOP_ROOT; break; }
        }
    }
    if (code == ST_OK) {
        uint32_t max_attempts = is_allreduce ? f + 1 : 1;
        code = is_allreduce ? ST_NO_LIVE_ROOT_CANDIDATE : ST_ROOT_FAILED;
        for (uint32_t a = 0; a < max_attempts; ++a) {
            uint32_t c = (root + a) % P;
            if (play_attempt(s, in, frp, imp, c, (int64_t)a * s->Ratt, order, &overlap) != 0) { rc = -3; goto done; }
            attempts = a + 1;
            for (int i = 0; i < 4; ++i) msgs_all[i] += s->msgs_attempt[i];
            for (uint32_t v = 0; v < P; ++v) {
                uint32_t p = v2p(s, v);
                sends_tot[p] += s->nsent[v];
                if (s->inited[v]) ev[p] |= 1;
                if (s->delivered[v]) ev[p] |= (ev[p] & 2) ? 4 : 2;
                if (s->delivered[v] == 2) ev[p] |= 4;
            }
            if (!is_allreduce) { code = s->st_code; subtree = s->st_subtree; have_result = (code == ST_OK); break; }
            if (frp[c] != 0) {       /* the candidate had not failed before the operation: the attempt stands */
                code = s->st_code; subtree = s->st_subtree; have_result = (code == ST_OK); break;
            }
        }
    }
    if (overlap) { rc = -4; goto done; }

    /* ---- outputs (translate renumbered ranks back to physical ids) ---- */
    uint32_t W = s->W, nhold = 0;
    if (out->result) { memset(out->result, 0, kb); if (have_result) memcpy(out->result, s->data, kb); }
    if (out->holders) memset(out->holders, 0, (size_t)W * 4);
    if (out->expanded) memset(out->expanded, 0, P * kb);
    if (have_result && is_allreduce) {
        for (uint32_t v = 0; v < P; ++v) {
            if (s->phase[v] == PH_DONE && s->hold[v]) {
                uint32_t p = v2p(s, v); ++nhold;
                if (out->holders) out->holders[p >> 5] |= 1u << (p & 31);
                if (out->expanded) memcpy((unsigned char*)out->expanded + p * kb, s->hval + v * kb, kb);
            }
        }
    }
    if (out->status) {
        out->status[0] = code | (subtree << 8) | (attempts << 16);
        out->status[1] = have_result ? s->cnt[0] : 0;
        out->status[2] = have_result ? s->imask[0] : 0;
        out->status[3] = nhold;
    }
    if (out->msgs) { for (int i = 0; i < 4; ++i) { out->msgs[i] = msgs_all[i]; out->msgs[4 + i] = attempts ? s->msgs_attempt[i] : 0; } }
    if (out->sends) memcpy(out->sends, sends_tot, P * 4);
    if (out->events) for (uint32_t p = 0; p < P; ++p) out->events[p] = ev[p];
    if (out->nfail) out->nfail[0] = have_result ? s->nf[0] : 0;
    if (out->failed) {
        memset(out->failed, 0, (size_t)W * 4);
        if (have_result && s->fl) for (uint32_t v = 0; v < P; ++v)
            if ((s->fl[v >> 5] >> (v & 31)) & 1) { uint32_t p = v2p(s, v); out->failed[p >> 5] |= 1u << (p & 31); }
    }
    if (out->contrib) {
        memset(out->contrib, 0, (size_t)W * 4);
        if (have_result && s->set) for (uint32_t v = 0; v < P; ++v)
            if ((s->set[v >> 5] >> (v & 31)) & 1) { uint32_t p = v2p(s, v); out->contrib[p >> 5] |= 1u << (p & 31); }
    }
    if (attempts) {
        uint32_t cb[64], nc = children(s, 0, cb);
        for (uint32_t i = 0; i < nc; ++i) {
            uint32_t c = cb[i];
            if (out->cand) memcpy((unsigned char*)out->cand + i * kb, s->tdata + c * kb, kb);
            if (out->cand_flag) out->cand_flag[i] = s->tree_state[c] != SLOT_SENT ? 2 : (s->tfail[c] ? 1 : 0);
            if (out->cand_nfail) out->cand_nfail[i] = s->tree_state[c] == SLOT_SENT ? s->tnf[c] : 0;
        }
        for (uint32_t v = 0; v < P; ++v) {
            uint32_t p = v2p(s, v);
            if (out->tree_values) memcpy((unsigned char*)out->tree_values + p * kb, s->tdata + v * kb, kb);
            if (out->uc_values) memcpy((unsigned char*)out->uc_values + p * kb, s->ucval + v * kb, kb);
            if (out->tree_sent) out->tree_sent[p] = (s->tree_state[v] == SLOT_SENT ? 1u : 0u) | ((uint32_t)s->tfail[v] << 1);
            if (out->tree_sets && s->tset) {
                uint32_t* dst = out->tree_sets + (size_t)p * W; memset(dst, 0, (size_t)W * 4);
                for (uint32_t u = 0; u < P; ++u)
                    if ((s->tset[(size_t)v * W + (u >> 5)] >> (u & 31)) & 1) { uint32_t pu = v2p(s, u); dst[pu >> 5] |= 1u << (pu & 31); }
            }
        }
    }
done:
    free(s->x); free(s->data); free(s->tdata); free(s->hval); free(s->failbit); free(s->tfail); free(s->tree_state);
    free(s->bct_state); free(s->hold); free(s->tree_holder); free(s->uc_state); free(s->corr_state); free(s->phase);
    free(s->sub); free(s->idx); free(s->cnt); free(s->tcnt); free(s->imask); free(s->imask0); free(s->ucval); free(s->timask); free(s->fail_round);
    free(s->inited); free(s->delivered); free(s->nsent); free(frp); free(imp); free(order); free(sends_tot); free(ev);
    free(s->set); free(s->tset); free(s->nf); free(s->tnf); free(s->fl); free(s->tfl);
    return rc;
}

/*
 * Batch form with host pointers: scenarios one after the other.
 * in [S][P][k]; prefail [S][ceil(P/32)]; inop [S][max_inop] or NULL; roots [S] or NULL (then `root` is used);
 * result [S][k]; status [S][4].
 */
int ftc_oracle_batch(const orc_cfg_t* cfg, int is_allreduce, uint64_t S, const void* in, const uint32_t* prefail,
                     const orc_inop_t* inop, const uint32_t* roots, uint32_t root, void* result, uint32_t* status) {
    if (!cfg) return -1;
    uint32_t esz = (cfg->dtype == DT_I32 || cfg->dtype == DT_F32) ? 4 : 8;
    size_t W = (cfg->P + 31) / 32, kb = (size_t)cfg->k * esz, pb = (size_t)cfg->P * kb;
    for (uint64_t i = 0; i < S; ++i) {
        orc_out_t o; memset(&o, 0, sizeof o);
        o.result = (unsigned char*)result + i * kb; o.status = status + i * 4;
        int rc = ftc_oracle_run(cfg, is_allreduce, (const unsigned char*)in + i * pb, prefail + i * W,
                                inop ? inop + i * cfg->max_inop : NULL, roots ? roots[i] : root, &o);
        if (rc) return rc;
    }
    return 0;
}

/* Schedule constants under the readings above: q, r, H, rounds of a reduce, rounds of an allreduce attempt. */
int ftc_oracle_schedule(uint32_t P, uint32_t f, uint32_t arity, uint32_t* out5) {
    if (P < f + 2) return -1;
    uint32_t m = f + 1, q = (P - 1) / m, r = (P - 1) % m, H = 1 + deepest_level(arity ? arity : 2, q + (r ? 1 : 0));
    out5[0] = q; out5[1] = r; out5[2] = H; out5[3] = f + H; out5[4] = 2 * (f + H);
    return 0;
}
