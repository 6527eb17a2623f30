/*
 * az_search: batched tree search on top of the leaf evaluator (Sec. 3.4 "Search and self-play",
 * Eq. 1; Sec. 4.1 parallel leaves; Sec. 5.1 "Native ownership of the search loop": many games are
 * interleaved and share inference batches, two batches outstanding; App. D.2 constants: exploration
 * constant 1.5, reduced-parent first-play value with reduction 0.2, backup discount 0.99 per ply).
 *
 * The whole loop runs on the GPU: the trees of all games live in device memory, and one step of a
 * group of games is four launches on one stream -- select (one warp per game walks Eq. 1 down to
 * an edge without a child and builds the successor position), legal-move masks of the new
 * positions, the evaluation of that batch (az_evaluate_legal's kernels, or the stand-in evaluator),
 * expand-and-backup (one warp per game).  The host only queues launches; nothing is copied to or
 * from the host between az_search_set_roots and the read-out calls.  With two groups the steps of
 * one group overlap the evaluation of the other on a second stream.
 *
 * Conventions the paper leaves open, fixed here:
 *  - statistics sit on the edges: N(s,a), W(s,a), Q = W / N; N(s) of Eq. 1 is the sum of N(s,a)
 *    over the node's edges;
 *  - an edge without visits takes Q = V(s) - fpu_reduction, V(s) the mean of every value backed
 *    up through s (its own evaluation first), seen by the player to move at s;
 *  - a value changes sign and is multiplied by `discount` at every ply it is backed up;
 *  - a reservation (a traversal whose result is still outstanding; `leaves` > 1) counts on its
 *    edges as one lost visit: N + m visits, W - m value; a traversal that reaches a node still
 *    waiting for its evaluation is given up and its batch row idles;
 *  - a new node's repetition count (the `repetitions` field of its record, which the input planes
 *    show) is one more than that of the most recent earlier occurrence of the same position (pieces,
 *    side to move, castling rights, en-passant square; compared through a 64-bit hash) among its
 *    ancestors in the tree and the game's positions before the root, as far back as its halfmove
 *    clock reaches; 0 without one.  The game's earlier positions are the roots the search has seen
 *    (az_search_advance); the first root brings its own count in its record;
 *  - a node is terminal if the mover has no legal move (value -1 in check, else 0), if its
 *    halfmove clock has reached 100 or if its position has occurred twice before (value 0);
 *  - the root's evaluation is a step of its own, queued by az_search_set_roots' first run;
 *  - the arg-max of Eq. 1 is taken in float32 with one rounding per operation
 *    (Q + ((c * P) * sqrt(max(1, N))) / (1 + n)), ties to the lower action index;
 *  - with a network whose value head is (win, draw, loss) the scalar is win - loss (Sec. 3.3).
 *
 * Rows of a step that have nothing to evaluate (a traversal that ended in a known terminal node or was
 * given up) are evaluated all the same (the batch keeps its shape) and their results ignored; leaves
 * without a legal move go through the evaluator too, so the az_net's "a position had no legal move"
 * status bit (az_device_status bit 0) may be set by a search and means nothing there.
 *
 * Threading: one az_search is used by one host thread at a time; it uses the az_net's evaluation
 * workspace, so no other evaluation of that az_net may run during az_search_run.
 */
#ifndef AZ_SEARCH_H
#define AZ_SEARCH_H

#include "az_eval.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct az_search az_search;

#define AZ_SEARCH_EVAL_NET 0        /* leaves are evaluated by the az_net */
#define AZ_SEARCH_EVAL_STANDIN 1    /* deterministic stand-in (below): verifies the search itself */
#define AZ_SEARCH_MAX_LEAVES 16
#define AZ_SEARCH_MAX_DEPTH 128     /* a traversal that would go deeper is given up (flag 4) */

/* flags reported by az_search_tree (per game) */
#define AZ_SEARCH_FLAG_NODES_FULL 1u
#define AZ_SEARCH_FLAG_EDGES_FULL 2u   /* the node that found the pool full becomes a leaf worth its own evaluation */
#define AZ_SEARCH_FLAG_DEPTH 4u
#define AZ_SEARCH_FLAG_BAD_ACTION 8u   /* az_apply_moves: the action's origin square holds no piece of the mover */

typedef struct az_search_config {
    uint32_t games;          /* trees searched side by side (>= 1) */
    uint32_t leaves;         /* traversals per tree and step, 1..AZ_SEARCH_MAX_LEAVES (Sec. 4.1) */
    uint32_t groups;         /* 1 or 2: the games are split into groups whose steps overlap (Sec. 5.1: two outstanding batches) */
    uint32_t max_nodes;      /* per tree; a search of S steps opens at most 1 + S * leaves nodes */
    uint32_t max_edges;      /* per tree; about 35 per node in middlegame positions, 218 at most */
    uint32_t evaluator;      /* AZ_SEARCH_EVAL_* */
    uint32_t policy_head;    /* AZ_POLICY_*: the action list; must equal the az_net's when one is given */
    uint32_t position_bytes; /* 104, 784 or 128; must equal az_position_bytes() of the az_net when one is given */
    float c_puct;            /* 1.5 in self-play, 1.0 in evaluation matches (App. D.2, App. B.1) */
    float fpu_reduction;     /* 0.2 */
    float discount;          /* 0.99 */
    uint32_t reserved;
    uint64_t seed;           /* stand-in evaluator only */
} az_search_config;

/*
 * Successor positions: out record i is positions record i after the legal action actions_dev[i]
 * (a policy index of `policy_head`).  Same record layout in and out (stride 104, 784 or 128
 * bytes; out must not overlap positions): bitboards, side to move, castling rights (lost when the
 * king or a rook leaves its home square or a rook is captured there), en-passant square (behind a
 * pawn that advanced two ranks, else 64), halfmove clock (0 after a pawn move or a capture, else
 * one more, at most 255), repetitions 0.  784-byte records push the old position onto their
 * seven boards, 128-byte records push the move onto their eight (castling as the king's own move).
 * In the 73-plane and 1,858 lists a pawn reaching the last rank through a plain action becomes a
 * queen.  Legality is not checked beyond the origin square: an action whose origin holds no piece
 * of the mover leaves a copy of the record and ORs AZ_SEARCH_FLAG_BAD_ACTION into *status_dev
 * (status_dev may be NULL).  All pointers are device pointers, 8-byte aligned (actions 4).
 * Errors: BAD_ARG, CUDA.  batch == 0 is a no-op.
 */
int az_apply_moves(const void *positions_dev, size_t position_stride, int batch, int policy_head,
                   const int32_t *actions_dev, void *out_positions_dev, uint32_t *status_dev, void *cuda_stream);

/*
 * The stand-in evaluator by itself, in az_evaluate_legal's output form: priors over the legal
 * actions in ascending index order and one value per position.  With key = the position's hash
 * under `seed` (splitmix64 finaliser chained over the twelve bitboards, then side to move |
 * castling << 8 | en-passant square << 16), legal action a weighs 1 + r * r / 64, r the top ten
 * bits of mix(key + (a + 1) * 0x9e3779b97f4a7c15); prior = weight / sum (one float32 division);
 * value = 0.75 * (t * 2^-23 - 1), t the top 24 bits of mix(key ^ 0x5851f42d4c957f2d).
 */
int az_standin_evaluate(const void *positions_dev, size_t position_stride, const uint64_t *legal_masks_dev, int batch,
                        int policy_head, uint64_t seed, float *legal_policy_dev, int32_t *legal_counts_dev,
                        float *value_dev, void *cuda_stream);

/*
 * Allocates the trees and the per-group batch buffers on the current device (the az_net's device
 * when one is given).  net may be NULL with the stand-in evaluator.  games * leaves / groups (the
 * batch of one step) must not exceed the az_net's max_batch.
 * Errors: BAD_ARG, BAD_ARCH (config does not match the net), BATCH_TOO_LARGE, NOT_CALIBRATED, CUDA.
 */
int az_search_create(az_net *net, const az_search_config *config, az_search **out);
void az_search_destroy(az_search *search);

/* New searches: positions_host holds `games` root records; all trees are emptied. */
int az_search_set_roots(az_search *search, const void *positions_host);

/*
 * New searches in some of the games only (a game is over, the next one starts in its place; Sec. 5.1: an actor
 * keeps its games interleaved): games_host lists `count` game indices, positions_host holds their new root
 * records in the same order.  Those trees are emptied and their histories of earlier positions forgotten; the
 * other games are untouched.
 * Errors: BAD_ARG (an index out of range or listed twice, count above the number of games), BUSY, CUDA.
 * count == 0 is a no-op.
 */
int az_search_replace_roots(az_search *search, const int32_t *games_host, int count, const void *positions_host);

/*
 * Runs `simulations` more steps on every tree (the first call after az_search_set_roots runs the
 * roots' own evaluation first) and waits for them.  One step of a tree is `leaves` traversals
 * that all choose their paths before any of the step's results are backed up.
 * elapsed_ms_out (may be NULL): device time of the call, from CUDA events around the queued work.
 * Errors: BAD_ARG, CUDA, DEVICE_TIMEOUT (a bounded wait inside an evaluation kernel ran out).
 */
int az_search_run(az_search *search, int simulations, float *elapsed_ms_out);

/*
 * The same in two halves, for a host thread that has other work while the GPU searches (Sec. 3.3: the actor
 * interleaves games and submits batches without waiting): az_search_run_async queues the steps and returns;
 * az_search_wait blocks until they are done and reports like az_search_run.  Between the two every other
 * call on this az_search answers AZ_ERR_BUSY (az_search_destroy excepted, which waits); a second
 * az_search_run_async answers AZ_ERR_BUSY as well, az_search_wait without a pending run AZ_ERR_BAD_ARG.
 */
int az_search_run_async(az_search *search, int simulations);
int az_search_wait(az_search *search, float *elapsed_ms_out);

/*
 * Root statistics of one game, to host buffers of AZ_MAX_LEGAL entries each: the root's actions in
 * ascending order with their visit counts N, value sums W and priors P; *count_out their number.
 */
int az_search_root(az_search *search, int game, int32_t *actions_host, int32_t *visits_host, float *w_host,
                   float *prior_host, int32_t *count_out);

/*
 * The search's result for every game in one copy (Sec. 3.4: the distribution of root visits is the policy
 * target and decides the move): host buffers actions_host and visits_host of [games][AZ_MAX_LEGAL] int32 and
 * counts_host of [games] int32; row g holds counts[g] actions in ascending order with their visit counts;
 * the rows are copied whole, entries beyond counts[g] carry no meaning.
 */
int az_search_root_visits(az_search *search, int32_t *actions_host, int32_t *visits_host, int32_t *counts_host);

/*
 * A move is played in every game (Sec. 3.3: "the relevant subtree becomes the next root").  actions_host holds
 * one policy index per game, -1 for "no move in this game"; actions_host == NULL plays each game's most visited
 * root move (ties to the lower policy index).  The subtree under the played move is kept with all its
 * statistics and renumbered breadth-first (a node's children in the order of its edges); if that move has no
 * subtree yet the game's tree becomes the bare successor position and the next az_search_run starts with a step
 * in which such trees evaluate their roots while the others sit out.  A game whose root has no moves (the game
 * is over, or the root was never evaluated), whose action is -1 or is not a move of its root (flag
 * AZ_SEARCH_FLAG_BAD_ACTION) keeps its tree.  played_host (may be NULL) receives the action played per game,
 * -1 where none was.  Keeping only a share of the old visits (the paper's 60 %) is self-play's recipe and is
 * not applied.  The first call allocates a second set of tree pools (the kept subtrees are copied there).
 * Errors: BAD_ARG, BUSY, CUDA.
 */
int az_search_advance(az_search *search, const int32_t *actions_host, int32_t *played_host);

/*
 * Root noise (Sec. 3.4: "noise added to the root prior makes games consider different continuations"; App. D.2:
 * Dirichlet, epsilon 0.25, alpha 0.3).  The noise is the caller's (drawn on the host, any distribution):
 * noise_host is [games][AZ_MAX_LEGAL] float32, entry i of row g belonging to the i-th move of game g's current
 * root (ascending policy index); the priors of those edges become (1 - epsilon) P + epsilon * noise, in
 * float32 with one rounding per operation, and stay with the edges.  Applies to the root as it stands, a kept
 * subtree's root included; a root that has not been evaluated yet (run az_search_run(search, 0) first) or has
 * no moves is left alone.  changed_host (may be NULL) receives per game the number of edges changed.
 * Errors: BAD_ARG (epsilon outside [0, 1]), BUSY, CUDA.
 */
int az_search_root_noise(az_search *search, const float *noise_host, float epsilon, int32_t *changed_host);

/* The current root records of all games, to a host buffer of games * position_bytes. */
int az_search_root_positions(az_search *search, void *positions_host);

/*
 * One game's tree: counts_out[4] = nodes, edges, AZ_SEARCH_FLAG_* bits, traversals given up;
 * node_visits_host / node_value_sum_host (max_nodes entries each, may be NULL) receive per node, in
 * the order the nodes were opened, the number of values backed up through it and their sum.
 */
int az_search_tree(az_search *search, int game, int32_t *counts_out, int32_t *node_visits_host, float *node_value_sum_host);

/* Kernel launches az_search_run queues per step of one group (for launch accounting). */
int az_search_launches_per_step(const az_search *search);

#ifdef __cplusplus
}
#endif

#endif /* AZ_SEARCH_H */
