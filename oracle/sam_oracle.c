/*
 * CPU oracle for suffix-automaton speculative drafting and greedy verification.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, by-eye-checkable
 * statement of what the draft+verify path computes.  It shares no code with the
 * CUDA library and must never be called from the product path; only tests, the
 * smoke check and the benchmark's CPU-baseline leg use it.
 *
 * What it follows:
 *   - Section 5.4.2 ("Algorithm design"): all substrings of the context are
 *     indexed in a suffix automaton; after verification the decoder follows
 *     automaton transitions from the current verified suffix and retrieves a
 *     continuation of a specified length; the longest verified prefix of the
 *     proposal is committed and a mismatch falls back to the model's own token.
 *   - Section 5.4.3: the automaton is built incrementally, token by token, in
 *     time linear in the context length.  The paper gives no further detail, so
 *     the construction is the classical online one (Blumer et al. 1985): every
 *     new position creates one state; a split creates a clone that copies the
 *     transitions, suffix link and first end-position of the state it splits.
 *   - Algorithm 3, step 3 (speculative decoding loop): FollowTransitions, emit,
 *     validate, commit matched prefix, fall back on mismatch.
 *
 * Readings where the paper is silent (all repeated in the design notes):
 *   - states are numbered in creation order: root 0, then for each position the
 *     new state, then its clone if one is made;
 *   - the continuation is read after the FIRST occurrence of the matched suffix
 *     (firstpos = smallest end position), stops before a separator token or the
 *     corpus end, and is empty when fewer than min_match tokens are matched;
 *   - verification is greedy: row argmax with the lowest index winning ties,
 *     -0 and +0 equal, a NaN never replaces the running maximum.
 *
 * Pins (tests, CPU only): substring counts and membership against brute force,
 * first-occurrence positions against naive search, closed forms for a^N and
 * all-distinct corpora, the extremal families a b^(N-1) and a b^(N-2) c, a
 * hand-derived worked example, longest-suffix/draft against a naive scan,
 * argmax against planted unique maxima and library argmax on tie-free rows,
 * accept against a direct prefix compare.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t len;       /* length of the longest string of the state */
    int32_t link;      /* suffix link, -1 for the root */
    int32_t firstpos;  /* smallest end position (index of last token) of the state's strings */
    int32_t n, cap;    /* transitions, kept sorted ascending by token */
    int32_t *tok;
    int32_t *dst;
} ostate;

typedef struct {
    ostate *st;
    int64_t n_states, cap_states;
    int64_t n_edges;
    int64_t n_tokens;  /* corpus positions indexed so far */
    int32_t last;
} osam;

/* ---- transitions of one state: sorted small arrays, binary search ---------- */
static int32_t edge_slot(const ostate *s, int32_t c) /* first slot with tok >= c */
{
    int32_t lo = 0, hi = s->n;
    while (lo < hi) {
        int32_t mid = lo + (hi - lo) / 2;
        if (s->tok[mid] < c) lo = mid + 1; else hi = mid;
    }
    return lo;
}

static int32_t edge_get(const ostate *s, int32_t c) /* destination or -1 */
{
    int32_t k = edge_slot(s, c);
    return (k < s->n && s->tok[k] == c) ? s->dst[k] : -1;
}

static int edge_set(osam *a, int32_t s_id, int32_t c, int32_t d) /* insert or overwrite */
{
    ostate *s = &a->st[s_id];
    int32_t k = edge_slot(s, c);
    if (k < s->n && s->tok[k] == c) { s->dst[k] = d; return 0; }
    if (s->n == s->cap) {
        int32_t nc = s->cap ? s->cap * 2 : 2;
        int32_t *t = (int32_t *)realloc(s->tok, sizeof(int32_t) * (size_t)nc);
        if (!t) return -1;
        s->tok = t;
        int32_t *d2 = (int32_t *)realloc(s->dst, sizeof(int32_t) * (size_t)nc);
        if (!d2) return -1;
        s->dst = d2;
        s->cap = nc;
    }
    memmove(s->tok + k + 1, s->tok + k, sizeof(int32_t) * (size_t)(s->n - k));
    memmove(s->dst + k + 1, s->dst + k, sizeof(int32_t) * (size_t)(s->n - k));
    s->tok[k] = c;
    s->dst[k] = d;
    s->n++;
    a->n_edges++;
    return 0;
}

static int32_t new_state(osam *a)
{
    if (a->n_states == a->cap_states) {
        int64_t nc = a->cap_states * 2;
        ostate *t = (ostate *)realloc(a->st, sizeof(ostate) * (size_t)nc);
        if (!t) return -1;
        a->st = t;
        a->cap_states = nc;
    }
    ostate *s = &a->st[a->n_states];
    memset(s, 0, sizeof(*s));
    return (int32_t)a->n_states++;
}

/* ---- construction (Section 5.4.3: incremental, one token at a time) -------- */
static int extend(osam *a, int32_t c, int32_t i)
{
    int32_t cur = new_state(a);
    if (cur < 0) return -1;
    a->st[cur].len = a->st[a->last].len + 1;
    a->st[cur].firstpos = i;
    int32_t p = a->last;
    while (p != -1 && edge_get(&a->st[p], c) == -1) {
        if (edge_set(a, p, c, cur)) return -1;
        p = a->st[p].link;
    }
    if (p == -1) {
        a->st[cur].link = 0;
    } else {
        int32_t q = edge_get(&a->st[p], c);
        if (a->st[p].len + 1 == a->st[q].len) {
            a->st[cur].link = q;
        } else {
            int32_t clone = new_state(a);
            if (clone < 0) return -1;
            ostate *sq = &a->st[q];
            a->st[clone].len = a->st[p].len + 1;
            a->st[clone].link = sq->link;
            a->st[clone].firstpos = sq->firstpos;
            for (int32_t k = 0; k < sq->n; k++) {
                if (edge_set(a, clone, a->st[q].tok[k], a->st[q].dst[k])) return -1;
            }
            while (p != -1 && edge_get(&a->st[p], c) == q) {
                if (edge_set(a, p, c, clone)) return -1;
                p = a->st[p].link;
            }
            a->st[q].link = clone;
            a->st[cur].link = clone;
        }
    }
    a->last = cur;
    return 0;
}

void oracle_sam_free(osam *a)
{
    if (!a) return;
    for (int64_t s = 0; s < a->n_states; s++) { free(a->st[s].tok); free(a->st[s].dst); }
    free(a->st);
    free(a);
}

/* Appends tokens[0..n) to the indexed text (Section 5.4.2: verified tokens are inserted into the
 * automaton so that the index stays consistent with the growing context; Section 5.4.3: the
 * construction is incremental, so appending is just more steps of it).  Returns 0, or -1 when out
 * of memory. */
int oracle_sam_extend(osam *a, const int32_t *tokens, int64_t n)
{
    for (int64_t i = 0; i < n; i++) {
        if (extend(a, tokens[i], (int32_t)a->n_tokens)) return -1;
        a->n_tokens++;
    }
    return 0;
}

/* Builds the automaton of corpus[0..n). Separators are ordinary symbols here. */
osam *oracle_sam_build(const int32_t *corpus, int64_t n)
{
    osam *a = (osam *)calloc(1, sizeof(osam));
    if (!a) return NULL;
    a->cap_states = 16;
    a->st = (ostate *)malloc(sizeof(ostate) * (size_t)a->cap_states);
    if (!a->st) { free(a); return NULL; }
    int32_t root = new_state(a);
    a->st[root].len = 0;
    a->st[root].link = -1;
    a->st[root].firstpos = -1;
    a->last = root;
    if (oracle_sam_extend(a, corpus, n)) { oracle_sam_free(a); return NULL; }
    return a;
}

/* A stream's pair (state, matched_len) taken before the automaton grew still names a string that
 * occurs in the text, but a split may have moved that string into a new state: the state of a
 * string of length L is the one with len(link(s)) < L <= len(s).  Climb suffix links until that
 * holds again (the paper is silent on this; it follows from what the states of a suffix automaton
 * are). */
int32_t oracle_renormalize(const osam *a, int32_t state, int32_t matched_len)
{
    int32_t s = state;
    if (s < 0 || s >= a->n_states) return state;   /* not a state of this automaton: left alone */
    while (s != 0 && matched_len <= a->st[a->st[s].link].len) s = a->st[s].link;
    return s;
}

int64_t oracle_sam_states(const osam *a) { return a->n_states; }
int64_t oracle_sam_edges(const osam *a) { return a->n_edges; }

/* Flat arrays: len/link/firstpos [S]; row_ptr [S+1]; edge_tok/edge_dst [E], rows ascending by token. */
void oracle_sam_export(const osam *a, int32_t *len, int32_t *link, int32_t *firstpos,
                       int64_t *row_ptr, int32_t *edge_tok, int32_t *edge_dst)
{
    int64_t e = 0;
    for (int64_t s = 0; s < a->n_states; s++) {
        const ostate *st = &a->st[s];
        len[s] = st->len;
        link[s] = st->link;
        firstpos[s] = st->firstpos;
        row_ptr[s] = e;
        for (int32_t k = 0; k < st->n; k++) { edge_tok[e] = st->tok[k]; edge_dst[e] = st->dst[k]; e++; }
    }
    row_ptr[a->n_states] = e;
}

/* ---- walk (Algorithm 3, FollowTransitions over the newly verified tokens) -- */
/* One stream: consume n tokens from (state, matched_len). On a miss follow the
 * suffix link and shorten the match to that state's length; at the root a miss
 * resets the match to zero. */
void oracle_walk(const osam *a, int32_t *state, int32_t *matched_len,
                 const int32_t *tokens, int32_t n)
{
    int32_t s = *state, L = *matched_len;
    for (int32_t t = 0; t < n; t++) {
        int32_t c = tokens[t];
        for (;;) {
            int32_t d = edge_get(&a->st[s], c);
            if (d != -1) { s = d; L = L + 1; break; }
            if (s == 0) { L = 0; break; }
            s = a->st[s].link;
            L = a->st[s].len;
        }
    }
    *state = s;
    *matched_len = L;
}

static int is_separator(int32_t tok, const int32_t *seps, int32_t n_sep)
{
    for (int32_t k = 0; k < n_sep; k++) if (seps[k] == tok) return 1;
    return 0;
}

/* ---- draft (Section 5.4.2: continuation of a specified length) ------------- */
/* Writes drafts[0..K) (unused slots -1) and returns n_draft. */
int32_t oracle_draft(const osam *a, const int32_t *corpus, int64_t n,
                     const int32_t *seps, int32_t n_sep,
                     int32_t state, int32_t matched_len, int32_t K, int32_t min_match,
                     int32_t *drafts)
{
    int32_t nd = 0;
    for (int32_t j = 0; j < K; j++) drafts[j] = -1;
    if (matched_len < min_match) return 0;
    int64_t p = (int64_t)a->st[state].firstpos + 1;
    for (int32_t j = 0; j < K; j++) {
        if (p + j >= n) break;
        if (is_separator(corpus[p + j], seps, n_sep)) break;
        drafts[j] = corpus[p + j];
        nd++;
    }
    return nd;
}

/* ---- greedy verification (Algorithm 3: validate, commit matched prefix) ---- */
static float bf16_to_float(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* Index of the maximum of V bf16 values; only a strictly greater value replaces
 * the running maximum, so the lowest index wins among equal maxima. */
int32_t oracle_argmax_row(const uint16_t *row, int32_t V)
{
    int32_t idx = 0;
    float best = bf16_to_float(row[0]);
    for (int32_t v = 1; v < V; v++) {
        float x = bf16_to_float(row[v]);
        if (x > best) { best = x; idx = v; }
    }
    return idx;
}

/* Longest prefix of the draft that equals the model's greedy choice, then the
 * model's own token at the first mismatch (or after a full accept).
 * accepted has K+1 slots (unused -1); returns n_accepted in [1, n_draft+1]. */
int32_t oracle_accept(const int32_t *drafts, int32_t n_draft, const int32_t *argmax_row,
                      int32_t K, int32_t *accepted)
{
    int32_t a = 0;
    for (int32_t j = 0; j <= K; j++) accepted[j] = -1;
    while (a < n_draft && drafts[a] == argmax_row[a]) { accepted[a] = drafts[a]; a++; }
    accepted[a] = argmax_row[a];
    return a + 1;
}

/* ---- batch drivers: plain loops over streams / rows ------------------------ */
void oracle_draft_batch(const osam *a, const int32_t *corpus, int64_t n,
                        const int32_t *seps, int32_t n_sep, int32_t B,
                        int32_t *state, int32_t *matched_len,
                        const int32_t *new_tokens, int32_t ld, const int32_t *n_new,
                        int32_t K, int32_t min_match, int32_t *drafts, int32_t *n_draft,
                        int32_t threads)
{
    (void)threads;
#pragma omp parallel for num_threads(threads) schedule(static)
    for (int32_t b = 0; b < B; b++) {
        oracle_walk(a, &state[b], &matched_len[b], new_tokens + (int64_t)b * ld, n_new[b]);
        n_draft[b] = oracle_draft(a, corpus, n, seps, n_sep, state[b], matched_len[b],
                                  K, min_match, drafts + (int64_t)b * K);
    }
}

/* logits: [B*(K+1)] rows of V bf16, consecutive rows row_stride elements apart. */
void oracle_argmax_batch(const uint16_t *logits, int64_t row_stride, int64_t rows, int32_t V,
                         int32_t *argmax_out, int32_t threads)
{
    (void)threads;
#pragma omp parallel for num_threads(threads) schedule(static)
    for (int64_t r = 0; r < rows; r++)
        argmax_out[r] = oracle_argmax_row(logits + r * row_stride, V);
}

void oracle_accept_batch(int32_t B, int32_t K, const int32_t *drafts, const int32_t *n_draft,
                         const int32_t *argmax_out, int32_t *accepted, int32_t *n_accepted)
{
    for (int32_t b = 0; b < B; b++)
        n_accepted[b] = oracle_accept(drafts + (int64_t)b * K, n_draft[b],
                                      argmax_out + (int64_t)b * (K + 1), K,
                                      accepted + (int64_t)b * (K + 1));
}

/* One closed-loop step after the logits exist: argmax, accept, walk the accepted
 * tokens, emit the next draft (Algorithm 3, loop body). */
void oracle_step(const osam *a, const int32_t *corpus, int64_t n,
                 const int32_t *seps, int32_t n_sep,
                 const uint16_t *logits, int64_t row_stride, int32_t B, int32_t K, int32_t V,
                 const int32_t *drafts, const int32_t *n_draft,
                 int32_t *argmax_out, int32_t *accepted, int32_t *n_accepted,
                 int32_t *state, int32_t *matched_len, int32_t min_match,
                 int32_t *next_drafts, int32_t *next_n_draft, int32_t threads)
{
    oracle_argmax_batch(logits, row_stride, (int64_t)B * (K + 1), V, argmax_out, threads);
    oracle_accept_batch(B, K, drafts, n_draft, argmax_out, accepted, n_accepted);
    oracle_draft_batch(a, corpus, n, seps, n_sep, B, state, matched_len,
                       accepted, K + 1, n_accepted, K, min_match,
                       next_drafts, next_n_draft, threads);
}

/* ---- step with options and running statistics ------------------------------ */
/* Options of a step:
 *   ORACLE_NO_SPECULATION (Section 5.4.3 "Adaptive switch", Algorithm 3 step 4): speculation is off
 *     for this step - every stream verifies an empty proposal (plain decoding: one row, one committed
 *     token), the automaton walk still follows the committed token, and no new draft is emitted.
 *   ORACLE_SKIP_UNUSED_ROWS: only rows 0..n_draft[b] of stream b are looked at (row n_draft[b] gives
 *     the model's own token after a full accept); the rows beyond get index -1.
 * Statistics (Section 6.5): OTE = committed tokens / verification passes; SHR = accepted speculative
 * tokens / proposed speculative tokens over the steps with a non-empty proposal.
 * counters[0..5] += { passes, committed tokens, proposed draft tokens, accepted draft tokens,
 *                     non-empty proposals, rows looked at }. */
#define ORACLE_NO_SPECULATION   1
#define ORACLE_SKIP_UNUSED_ROWS 2

void oracle_step_ex(const osam *a, const int32_t *corpus, int64_t n,
                    const int32_t *seps, int32_t n_sep,
                    const uint16_t *logits, int64_t row_stride, int32_t B, int32_t K, int32_t V,
                    const int32_t *drafts, const int32_t *n_draft,
                    int32_t *argmax_out, int32_t *accepted, int32_t *n_accepted,
                    int32_t *state, int32_t *matched_len, int32_t min_match,
                    int32_t *next_drafts, int32_t *next_n_draft,
                    uint32_t flags, int64_t *counters)
{
    for (int32_t b = 0; b < B; b++) {
        int32_t nd = n_draft[b];
        if (nd < 0) nd = 0;
        if (nd > K) nd = K;
        if (flags & ORACLE_NO_SPECULATION) nd = 0;
        int32_t *am = argmax_out + (int64_t)b * (K + 1);
        int64_t rows = 0;
        for (int32_t j = 0; j <= K; j++) {
            if ((flags & ORACLE_SKIP_UNUSED_ROWS) && j > nd) { am[j] = -1; continue; }
            am[j] = oracle_argmax_row(logits + ((int64_t)b * (K + 1) + j) * row_stride, V);
            rows++;
        }
        int32_t *acc = accepted + (int64_t)b * (K + 1);
        n_accepted[b] = oracle_accept(drafts + (int64_t)b * K, nd, am, K, acc);
        oracle_walk(a, &state[b], &matched_len[b], acc, n_accepted[b]);
        int32_t *nx = next_drafts + (int64_t)b * K;
        if (flags & ORACLE_NO_SPECULATION) {
            for (int32_t j = 0; j < K; j++) nx[j] = -1;
            next_n_draft[b] = 0;
        } else {
            next_n_draft[b] = oracle_draft(a, corpus, n, seps, n_sep, state[b], matched_len[b], K, min_match, nx);
        }
        if (counters) {
            counters[0] += 1;
            counters[1] += n_accepted[b];
            counters[2] += nd;
            counters[3] += n_accepted[b] - 1;
            counters[4] += nd > 0;
            counters[5] += rows;
        }
    }
}

/* The adaptive switch (Section 5.4.3; Algorithm 3 step 4): speculation stays on unless the context
 * length or the batch size exceeds its threshold. */
int32_t oracle_speculation_enabled(int64_t context_len, int64_t batch_size,
                                   int64_t max_context_len, int64_t max_batch_size)
{
    return !(context_len > max_context_len || batch_size > max_batch_size);
}

/* The switch driven by the running statistics (Section 5.4.3: speculation is switched off "when its overhead
 * outweighs the gains"; Algorithm 3 step 4; Section 6.5 for OTE).  The paper leaves the rule to the deployment
 * ("empirically determined" thresholds).  Reading taken here: a verification pass over one row costs 1, a pass
 * over all K+1 rows costs cost_ratio (supplied by the caller from measurements), a pass over r rows lies on the
 * line between the two, 1 + (cost_ratio - 1)(r - 1)/K; plain decoding commits one token per unit of cost.
 * Speculation pays when the window of passes described by the counters committed more tokens than it cost:
 *      sum(committed) > sum over passes of [1 + (cost_ratio - 1)(rows - 1)/K]
 * With the counters of oracle_step_ex (committed - passes = accepted draft tokens) this is
 *      accepted * K > (cost_ratio - 1) * (rows - passes),
 * evaluated in double precision; when every pass reads all K+1 rows it is OTE > cost_ratio.
 * A window without passes says nothing: speculation stays on. */
int32_t oracle_speculation_pays(const int64_t *counters, int32_t K, double cost_ratio)
{
    const int64_t passes = counters[0], accepted = counters[3], rows = counters[5];
    if (passes <= 0) return 1;
    return (double)accepted * (double)K > (cost_ratio - 1.0) * (double)(rows - passes);
}
