/*
 * mtpp.h -- C ABI of the slicing of topological orders into pipeline blocks, batched over a
 * population of orders.
 *
 * Source of the operation: the paper's section "Dynamic sharding of neural networks" (the I/O
 * cost io(S, T), the overflow cost, the block cost f(S) and the max-throughput partitioning
 * objective: minimise the largest block cost) and its section "Enhanced MTPP slicing of
 * topological order", Algorithm 1: a segment cost structure for (G, pi) and a dynamic programme
 * that cuts the order pi into at most k blocks.  The section "Biased random-key genetic
 * algorithm" evaluates a whole population of orders, each decoded from a vector of node
 * priorities; that population is the batch here: one CTA slices one order.
 *
 * Readings (the paper prints the overflow cost with mismatched units and leaves peak(S), the
 * "heuristic-based weighting" and heuristic_adjustment undefined).  All node attributes are
 * non-negative integers and every cost is kept multiplied by the bandwidth B, so results are
 * exact integers:
 *     F(S) = in(S) + B work(S) + max(0, sizeparam(S) + peak(S) - M) + peak(S) + out(S)
 *   in(S)   = sum of sizeout(u) over nodes u outside S with a consumer in S (each u once)
 *   out(S)  = sum of sizeout(u) over nodes u of S with a consumer outside S (each u once)
 *   peak(S) = the largest sizeout of a node of S;  work, sizeparam: sums over S
 *   no weighting, heuristic_adjustment = identity
 *   result = the best bottleneck over k' = 1 .. min(k, n) non-empty blocks; on equal bottlenecks
 *            the smaller k'; inside the dynamic programme the earlier cut wins.
 *
 * Conventions: status codes are bq_status (include/bq.h).  Pointers marked HOST are read during the
 * call; pointers marked DEVICE belong to the caller and are used on `cuda_stream`, on which the
 * calls enqueue and return without synchronising.  Nothing is allocated per call and no kernel
 * uses global scratch memory.  Limits: n <= 1024 nodes, k <= 16 blocks.
 */
#ifndef MTPP_H
#define MTPP_H

#include <stddef.h>
#include <stdint.h>

#include "bq.h"

#ifdef __cplusplus
extern "C" {
#endif

enum { MTPP_MAX_NODES = 1024, MTPP_MAX_BLOCKS = 16 };

/* Opaque: the device copy of a computation graph (predecessor and consumer lists, attributes). */
typedef struct mtpp_graph mtpp_graph;

/*
 * mtpp_graph_create -- checks and uploads a graph to the current device.
 *   n nodes 0..n-1 (1 <= n <= MTPP_MAX_NODES); m edges, edges_host = m pairs (u, v) (HOST): v
 *   consumes u's output; duplicates are dropped.  work_host, sizeparam_host, sizeout_host: n
 *   int64 each (HOST), all >= 0, each total below 2^40.
 * Errors: BQ_ERR_NULL; BQ_ERR_SIZE (n or m out of range, a node index out of range, a self loop, a
 * negative or too large attribute, or a cycle); BQ_ERR_CUDA.  Synchronises the device once.
 */
int mtpp_graph_create(int n, int m, const int32_t* edges_host, const int64_t* work_host, const int64_t* sizeparam_host,
                      const int64_t* sizeout_host, mtpp_graph** out);
int mtpp_graph_free(mtpp_graph* g);

/*
 * mtpp_decode_orders -- the map from priority vectors to topological orders (Kahn's algorithm,
 * always taking the ready node with the highest priority; equal priorities: the smaller node).
 *   keys: P x n floats (DEVICE, row-major; NaN is outside the contract); orders_out: P x n int32
 *   (DEVICE): row p lists the nodes in the order decoded from keys row p.
 */
int mtpp_decode_orders(const mtpp_graph* g, const float* keys, int P, int32_t* orders_out, void* cuda_stream);

/*
 * mtpp_slice_orders -- Algorithm 1 for every order of the population.
 *   orders: P x n int32 (DEVICE); k: most blocks (1 <= k <= MTPP_MAX_BLOCKS); B >= 1, M >= 0 with
 *   B * (total work) below 2^62.
 *   cost_out[p]   (int64, DEVICE): the smallest bottleneck F of order p;
 *   blocks_out[p] (int32, DEVICE): how many blocks reach it;
 *   cuts_out      (int32, DEVICE, P x k): the 1-based last position of each block in turn (the last
 *                 one is n), zero in the unused entries;
 *   status_out[p] (int32, DEVICE): 0, or 1 when row p is not a topological order of the graph (a
 *                 node twice or out of range, or a consumer placed before its producer): its other
 *                 outputs are then -1 / 0 and nothing is read out of bounds.
 */
int mtpp_slice_orders(const mtpp_graph* g, const int32_t* orders, int P, int k, int64_t B, int64_t M, int64_t* cost_out,
                      int32_t* blocks_out, int32_t* cuts_out, int32_t* status_out, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif
