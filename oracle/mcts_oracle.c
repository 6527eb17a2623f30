/* TEST INFRASTRUCTURE: a plain, sequential tree search (Sec. 3.4 "Search and self-play", Eq. 1;
 * Sec. 4.1 parallel leaves; App. D.2 search constants), one game at a time, against which the GPU
 * search driver is compared.  Only tests, the smoke check and the benchmark's CPU baseline may use it.
 *
 * Readings of the paper taken here (the paper gives the rule and the constants, not the bookkeeping):
 *  - statistics live on the edges: N(s,a), W(s,a), Q = W/N; N(s) of Eq. 1 is the sum of N(s,a) over
 *    the node's edges (the form in which max(1, N) matters);
 *  - an edge without visits takes Q = V(s) - 0.2, V(s) the mean of all values backed up through s
 *    (its own evaluation included) from the point of view of the player to move at s;
 *  - a backed-up value changes sign and is multiplied by the discount at every ply it climbs;
 *  - a reservation (parallel leaves) counts on its edges as one visit that lost: N + m visits,
 *    W - m value; it is removed when the traversal's result arrives.  A traversal that runs into a
 *    node still waiting for its evaluation is given up (its reservations are removed, its slot idles);
 *  - a new node's repetition count (the record's `repetitions` field, which the input planes show) is one
 *    more than that of the most recent earlier occurrence of the same position (pieces, side to move,
 *    castling rights, en-passant square) among its ancestors in the tree and the positions of the game
 *    before the root, as far back as its halfmove clock reaches; 0 if there is none.  The game's earlier
 *    positions are those the tree itself has seen as roots (played moves); the first root brings its own
 *    count in its record;
 *  - a node is terminal if the mover has no legal move (value -1 in check, else 0), if the halfmove
 *    clock has reached 100 or if the position has occurred twice before (value 0);
 *  - the root's evaluation is a step of its own before the counted simulations;
 *  - root noise, when the caller asks for it, replaces the priors of the root's edges by (1 - epsilon) P +
 *    epsilon * noise with noise values the caller has drawn; it is applied to the current root as it stands
 *    (a kept subtree's root included) and stays with those edges;
 *  - when a move is played (Sec. 3.3: the relevant subtree becomes the next root) the subtree under the
 *    root's edge of that action is kept with all its statistics and renumbered breadth-first (a node's
 *    children in the order of its edges), everything else is dropped; if that edge has no child yet the
 *    new tree is the bare successor position, waiting for its root evaluation.  Retaining only a share
 *    of the visits (the paper's 60 %) belongs to self-play's recipe and is not applied.
 * Every decision (the arg-max of Eq. 1) is taken in float32 with one rounding per operation, in the
 * order written below, ties to the lower action index.
 *
 * The evaluator is the deterministic stand-in described at synth_eval(): priors and value are pure
 * functions of the position and a seed, in arithmetic that rounds the same way everywhere. */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

int orc_legal_masks(const void *records, int stride, int n, int head, uint64_t *masks);
int orc_apply_moves(const void *records, int stride, int n, int head, const int32_t *actions, void *out);
int orc_in_check(const void *record);

#define MAX_STRIDE 784
#define MAX_DEPTH 128

typedef struct {
    uint64_t pieces[12];
    uint8_t stm, castling, ep_square, halfmove, repetitions, pad[3];
} Cur;

typedef struct { int action, child, n, m; float prior, w; } Edge;
typedef struct {
    int edge_begin, n_edges;      /* n_edges < 0: waiting for its evaluation */
    int terminal; float tvalue;
    int nvis; float wsum;         /* values backed up through the node, its own first */
    int nsum;                     /* sum over edges of N + m */
    int parent;                   /* -1 for the root */
    unsigned char rec[MAX_STRIDE];
} Node;
#define MAX_HISTORY 128

static uint64_t mix64(uint64_t x) {
    x ^= x >> 30; x *= 0xbf58476d1ce4e5b9ULL;
    x ^= x >> 27; x *= 0x94d049bb133111ebULL;
    x ^= x >> 31;
    return x;
}

/* Stand-in evaluator: key = hash of the twelve bitboards, side to move, castling rights and en-passant
 * square under `seed`.  Legal action a gets the integer weight 1 + r*r/64, r the top ten bits of
 * mix64(key + (a + 1) * 0x9e3779b97f4a7c15); its prior is weight / sum of weights (one float32 division).
 * The value is 0.75 * (t * 2^-23 - 1), t the top 24 bits of mix64(key ^ 0x5851f42d4c957f2d). */
static uint64_t position_key(const Cur *c, uint64_t seed) {
    uint64_t h = mix64(seed);
    for (int i = 0; i < 12; ++i) h = mix64(h ^ c->pieces[i]);
    return mix64(h ^ ((uint64_t)c->stm | (uint64_t)c->castling << 8 | (uint64_t)c->ep_square << 16));
}
static int synth_weight(uint64_t key, int action) {
    const int r = (int)(mix64(key + (uint64_t)(action + 1) * 0x9e3779b97f4a7c15ULL) >> 54);
    return 1 + r * r / 64;
}
static float synth_value(uint64_t key) {
    const int t = (int)(mix64(key ^ 0x5851f42d4c957f2dULL) >> 40);
    const float u = (float)t * 0x1p-23f - 1.0f;
    return u * 0.75f;
}

int orc_synth_eval(const void *record, int head, uint64_t seed, int32_t *actions, float *priors, float *value) {
    uint64_t mask[73];
    const int words = head == 0 ? 73 : 30;
    if (orc_legal_masks(record, 104, 1, head, mask) != 0) return -1;
    const uint64_t key = position_key((const Cur *)record, seed);
    int k = 0, sum = 0, w[256];
    for (int i = 0; i < words * 64 && k < 256; ++i)
        if (mask[i >> 6] >> (i & 63) & 1) { actions[k] = i; w[k] = synth_weight(key, i); sum += w[k]; ++k; }
    for (int i = 0; i < k; ++i) priors[i] = (float)w[i] / (float)sum;
    *value = synth_value(key);
    return k;
}

typedef struct {
    Node *nodes; Edge *edges;
    int n_nodes, n_edges, node_cap, edge_cap;
    int stride, head;
    float c_puct, fpu_reduction, discount;
    uint64_t seed;
    uint32_t flags;               /* 1: node pool full, 2: edge pool full, 4: depth limit */
    int root_submitted, idle;     /* idle: traversals given up (collisions, full pools) */
    Cur hist[MAX_HISTORY];        /* the game's positions before the root since the last irreversible move, oldest first */
    int hist_n;
} Tree;

static int same_position(const Cur *a, const Cur *b) {
    return memcmp(a->pieces, b->pieces, sizeof a->pieces) == 0 && a->stm == b->stm && a->castling == b->castling &&
           a->ep_square == b->ep_square;
}

/* Repetition count of position `c`, reached from node `parent`: one more than the count of its most recent earlier
 * occurrence within the last c->halfmove plies (ancestors first, then the game before the root), 0 without one. */
static int repetition_count(const Tree *t, int parent, const Cur *c) {
    int k = 1;
    for (int n = parent; n >= 0 && k <= c->halfmove; n = t->nodes[n].parent, ++k) {
        const Cur *p = (const Cur *)t->nodes[n].rec;
        if (same_position(p, c)) return p->repetitions < 255 ? p->repetitions + 1 : 255;
    }
    for (int i = t->hist_n - 1; i >= 0 && k <= c->halfmove; --i, ++k)
        if (same_position(&t->hist[i], c)) return t->hist[i].repetitions < 255 ? t->hist[i].repetitions + 1 : 255;
    return 0;
}

typedef struct { int kind, leaf, depth; int path_e[MAX_DEPTH], path_n[MAX_DEPTH]; } Slot;
enum { SLOT_NONE = 0, SLOT_EVAL = 1, SLOT_TERMINAL = 2 };

static void undo(Tree *t, Slot *s) {
    for (int d = 0; d < s->depth; ++d) { t->edges[s->path_e[d]].m -= 1; t->nodes[s->path_n[d]].nsum -= 1; }
    s->kind = SLOT_NONE;
    t->idle += 1;
}

static void descend(Tree *t, Slot *s) {
    int node = 0;
    s->depth = 0; s->kind = SLOT_NONE; s->leaf = -1;
    if (!t->root_submitted) {                 /* the root's own evaluation, once; the step's other slots idle */
        t->root_submitted = 1; s->kind = SLOT_EVAL; s->leaf = 0;
        return;
    }
    for (;;) {
        Node *nd = &t->nodes[node];
        if (nd->terminal) { s->kind = SLOT_TERMINAL; s->leaf = node; return; }
        if (nd->n_edges < 0) { undo(t, s); return; }
        if (s->depth == MAX_DEPTH) { t->flags |= 4; undo(t, s); return; }
        const float sqrt_n = sqrtf((float)(nd->nsum > 1 ? nd->nsum : 1));
        const float fpu = nd->wsum / (float)nd->nvis - t->fpu_reduction;
        int best = -1; float best_score = 0.0f;
        for (int i = 0; i < nd->n_edges; ++i) {
            const Edge *e = &t->edges[nd->edge_begin + i];
            const int n = e->n + e->m;
            const float q = n > 0 ? (e->w - (float)e->m) / (float)n : fpu;
            float u = t->c_puct * e->prior;
            u = u * sqrt_n;
            u = u / (float)(1 + n);
            const float score = q + u;
            if (best < 0 || score > best_score) { best = i; best_score = score; }
        }
        Edge *e = &t->edges[nd->edge_begin + best];
        e->m += 1; nd->nsum += 1;
        s->path_e[s->depth] = nd->edge_begin + best; s->path_n[s->depth] = node; s->depth += 1;
        if (e->child < 0) {
            if (t->n_nodes == t->node_cap) { t->flags |= 1; undo(t, s); return; }
            const int child = t->n_nodes++;
            Node *c = &t->nodes[child];
            memset(c, 0, sizeof *c);
            c->n_edges = -1;
            int32_t a = e->action;
            orc_apply_moves(nd->rec, t->stride, 1, t->head, &a, c->rec);
            c->parent = node;
            ((Cur *)c->rec)->repetitions = (uint8_t)repetition_count(t, node, (const Cur *)c->rec);
            e->child = child;
            s->kind = SLOT_EVAL; s->leaf = child;
            return;
        }
        node = e->child;
    }
}

static void finish(Tree *t, Slot *s) {
    if (s->kind == SLOT_NONE) return;
    Node *nd = &t->nodes[s->leaf];
    float v;
    if (s->kind == SLOT_EVAL) {
        int32_t actions[256]; float priors[256], value;
        const int k = orc_synth_eval(nd->rec, t->head, t->seed, actions, priors, &value);
        const Cur *c = (const Cur *)nd->rec;
        nd->nsum = 0;
        if (k == 0) { nd->terminal = 1; nd->tvalue = orc_in_check(nd->rec) ? -1.0f : 0.0f; nd->n_edges = 0; }
        else if (c->halfmove >= 100 || c->repetitions >= 2) { nd->terminal = 1; nd->tvalue = 0.0f; nd->n_edges = 0; }
        else if (t->n_edges + k > t->edge_cap) { t->flags |= 2; nd->terminal = 1; nd->tvalue = value; nd->n_edges = 0; }
        else {
            nd->edge_begin = t->n_edges; nd->n_edges = k; t->n_edges += k;
            for (int i = 0; i < k; ++i) {
                Edge *e = &t->edges[nd->edge_begin + i];
                e->action = actions[i]; e->prior = priors[i]; e->child = -1; e->n = 0; e->m = 0; e->w = 0.0f;
            }
        }
        v = nd->terminal ? nd->tvalue : value;
    } else {
        v = nd->tvalue;
    }
    nd->nvis += 1; nd->wsum += v;
    for (int d = s->depth - 1; d >= 0; --d) {
        v = -v * t->discount;
        Edge *e = &t->edges[s->path_e[d]];
        e->n += 1; e->w += v; e->m -= 1;
        Node *p = &t->nodes[s->path_n[d]];
        p->nvis += 1; p->wsum += v;
    }
}

static Tree *tree_new(const void *root_record, int stride, int head, float c_puct, float fpu_reduction, float discount,
                      uint64_t seed, int node_cap, int edge_cap) {
    Tree *t = (Tree *)calloc(1, sizeof(Tree));
    t->nodes = (Node *)calloc((size_t)node_cap, sizeof(Node));
    t->edges = (Edge *)calloc((size_t)edge_cap, sizeof(Edge));
    t->node_cap = node_cap; t->edge_cap = edge_cap; t->stride = stride; t->head = head;
    t->c_puct = c_puct; t->fpu_reduction = fpu_reduction; t->discount = discount; t->seed = seed;
    memcpy(t->nodes[0].rec, root_record, (size_t)stride);
    t->nodes[0].n_edges = -1;
    t->nodes[0].parent = -1;
    t->n_nodes = 1;
    return t;
}

static void tree_run(Tree *t, int simulations, int leaves) {
    Slot *slots = (Slot *)calloc((size_t)leaves, sizeof(Slot));
    const int steps = simulations + (t->root_submitted ? 0 : 1);      /* the root's own evaluation first */
    for (int step = 0; step < steps; ++step) {
        for (int j = 0; j < leaves; ++j) descend(t, &slots[j]);
        for (int j = 0; j < leaves; ++j) finish(t, &slots[j]);
    }
    free(slots);
}

/* The move `action` is played at the root.  Returns 0, or -1 if the root has no such edge (nothing changes). */
static int tree_advance(Tree *t, int action) {
    const Node *root = &t->nodes[0];
    int e0 = -1;
    for (int i = 0; i < root->n_edges; ++i)
        if (t->edges[root->edge_begin + i].action == action) e0 = root->edge_begin + i;
    if (e0 < 0) return -1;
    Node *nodes = (Node *)calloc((size_t)t->node_cap, sizeof(Node));
    Edge *edges = (Edge *)calloc((size_t)t->edge_cap, sizeof(Edge));
    int n_nodes = 1, n_edges = 0;
    if (t->edges[e0].child < 0) {
        int32_t a = action;
        orc_apply_moves(root->rec, t->stride, 1, t->head, &a, nodes[0].rec);
        ((Cur *)nodes[0].rec)->repetitions = (uint8_t)repetition_count(t, 0, (const Cur *)nodes[0].rec);
        nodes[0].n_edges = -1;
        nodes[0].parent = -1;
        t->root_submitted = 0;
    } else {
        int *old_of = (int *)calloc((size_t)t->node_cap, sizeof(int));
        old_of[0] = t->edges[e0].child;
        for (int i = 0; i < n_nodes; ++i) {                           /* breadth-first: new node i was old node old_of[i] */
            const int new_parent = nodes[i].parent;                   /* set when the node was queued */
            nodes[i] = t->nodes[old_of[i]];
            nodes[i].parent = i == 0 ? -1 : new_parent;
            const int begin = nodes[i].edge_begin;
            nodes[i].edge_begin = n_edges;
            for (int j = 0; j < nodes[i].n_edges; ++j) {
                Edge e = t->edges[begin + j];
                if (e.child >= 0) { old_of[n_nodes] = e.child; nodes[n_nodes].parent = i; e.child = n_nodes++; }
                edges[n_edges++] = e;
            }
        }
        free(old_of);
    }
    /* the old root joins the game's earlier positions, unless the move was irreversible (then nothing before it can recur) */
    if (((const Cur *)nodes[0].rec)->halfmove == 0) t->hist_n = 0;
    else {
        if (t->hist_n == MAX_HISTORY) { memmove(t->hist, t->hist + 1, sizeof(Cur) * (MAX_HISTORY - 1)); t->hist_n -= 1; }
        memcpy(&t->hist[t->hist_n++], root->rec, sizeof(Cur));
    }
    free(t->nodes); free(t->edges);
    t->nodes = nodes; t->edges = edges; t->n_nodes = n_nodes; t->n_edges = n_edges;
    return 0;
}

static int tree_read(const Tree *t, int32_t *root_actions, int32_t *root_visits, float *root_w, float *root_prior,
                     int32_t *counts, int32_t *node_nvis, float *node_wsum, void *root_record) {
    const Node *root = &t->nodes[0];
    const int k = root->n_edges > 0 ? root->n_edges : 0;
    for (int i = 0; i < k && i < 256; ++i) {
        const Edge *e = &t->edges[root->edge_begin + i];
        root_actions[i] = e->action; root_visits[i] = e->n; root_w[i] = e->w; root_prior[i] = e->prior;
    }
    counts[0] = t->n_nodes; counts[1] = t->n_edges; counts[2] = (int32_t)t->flags; counts[3] = t->idle;
    if (node_nvis && node_wsum)
        for (int i = 0; i < t->n_nodes; ++i) { node_nvis[i] = t->nodes[i].nvis; node_wsum[i] = t->nodes[i].wsum; }
    if (root_record) memcpy(root_record, root->rec, (size_t)t->stride);
    return k;
}

/* A search that lives across calls (moves played, subtrees kept). */
void *orc_mcts_new(const void *root_record, int stride, int head, float c_puct, float fpu_reduction, float discount,
                   uint64_t seed, int node_cap, int edge_cap) {
    if (stride > MAX_STRIDE || node_cap < 2 || edge_cap < 1) return NULL;
    return tree_new(root_record, stride, head, c_puct, fpu_reduction, discount, seed, node_cap, edge_cap);
}
int orc_mcts_run(void *tree, int simulations, int leaves) {
    if (!tree || leaves < 1 || leaves > 64) return -1;
    tree_run((Tree *)tree, simulations, leaves);
    return 0;
}
int orc_mcts_advance(void *tree, int action) { return tree ? tree_advance((Tree *)tree, action) : -1; }
int orc_mcts_read(const void *tree, int32_t *root_actions, int32_t *root_visits, float *root_w, float *root_prior,
                  int32_t *counts, int32_t *node_nvis, float *node_wsum, void *root_record) {
    return tree_read((const Tree *)tree, root_actions, root_visits, root_w, root_prior, counts, node_nvis, node_wsum, root_record);
}
/* Root noise (Sec. 3.4: noise added to the root prior makes games consider different continuations; App. D.2:
 * Dirichlet with epsilon 0.25, alpha 0.3).  The noise itself is drawn by the caller and passed in: the priors of
 * the root's edges become (1 - epsilon) * P + epsilon * noise[i], i the edge's place among the root's edges,
 * in float32 with one rounding per operation.  Returns the number of edges changed (0 if the root has not
 * been evaluated yet or has no moves). */
int orc_mcts_root_noise(void *tree, const float *noise, float epsilon) {
    Tree *t = (Tree *)tree;
    if (!t) return -1;
    const Node *root = &t->nodes[0];
    const float keep = 1.0f - epsilon;
    for (int i = 0; i < root->n_edges; ++i) {
        Edge *e = &t->edges[root->edge_begin + i];
        const float a = keep * e->prior;
        const float b = epsilon * noise[i];
        e->prior = a + b;
    }
    return root->n_edges > 0 ? root->n_edges : 0;
}

/* One node, for inspection: its record and its parent's index (-1 for the root).  Returns 0, -1 if there is no such node. */
int orc_mcts_node(const void *tree, int index, void *record_out, int32_t *parent_out) {
    const Tree *t = (const Tree *)tree;
    if (!t || index < 0 || index >= t->n_nodes) return -1;
    memcpy(record_out, t->nodes[index].rec, (size_t)t->stride);
    *parent_out = t->nodes[index].parent;
    return 0;
}
void orc_mcts_free(void *tree) {
    Tree *t = (Tree *)tree;
    if (!t) return;
    free(t->nodes); free(t->edges); free(t);
}

/* One search from `root_record`: the root's evaluation, then `simulations` steps of `leaves` traversals each
 * (all traversals of a step choose their paths before any of the step's results arrive).
 * Out: the root's edges (action, visits, value sum, prior; at most 256), the counts of nodes and edges,
 * per node (node_cap entries) its visit count and value sum, and the flags.  Returns the root's edge count. */
int orc_mcts_search(const void *root_record, int stride, int head, int simulations, int leaves,
                    float c_puct, float fpu_reduction, float discount, uint64_t seed, int node_cap, int edge_cap,
                    int32_t *root_actions, int32_t *root_visits, float *root_w, float *root_prior,
                    int32_t *counts /* n_nodes, n_edges, flags, idle */, int32_t *node_nvis, float *node_wsum) {
    if (stride > MAX_STRIDE || leaves < 1 || leaves > 64) return -1;
    Tree *t = tree_new(root_record, stride, head, c_puct, fpu_reduction, discount, seed, node_cap, edge_cap);
    tree_run(t, simulations, leaves);
    const int k = tree_read(t, root_actions, root_visits, root_w, root_prior, counts, node_nvis, node_wsum, NULL);
    orc_mcts_free(t);
    return k;
}
