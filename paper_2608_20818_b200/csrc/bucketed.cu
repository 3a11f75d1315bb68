// Host-side planning of the bucketed refresh (paper, Section 3.3; Algorithm 2
// lines 1-7; appendix "Idealized overlap model"): which matrices travel in
// which all-gather bucket, where each one sits inside a rank's segment, and
// the two-stage pipeline's makespan for given per-bucket times.  Integers and
// doubles only; nothing here touches a device.
#include "common.cuh"

using namespace prm;

extern "C" int prm_shard_rows(int64_t rows, int world, int rank, int64_t* row_start, int64_t* row_count) {
  if (rows < 1 || world < 1 || rank < 0 || rank >= world || !row_start || !row_count) return PRM_ERR_ARG;
  shard_rows(rows, world, rank, row_start, row_count);
  return PRM_OK;
}

extern "C" int prm_bucket_plan(const int64_t* shapes, int n_mats, int world, int64_t bucket_bytes,
                               int* bucket_of_mat, int64_t* offset_in_segment, int* n_buckets,
                               int64_t* segment_elems) {
  if (!shapes || n_mats < 1 || world < 1 || bucket_bytes < 1 || !bucket_of_mat || !offset_in_segment || !n_buckets ||
      !segment_elems)
    return PRM_ERR_ARG;
  for (int i = 0; i < n_mats; ++i)
    if (shapes[2 * i] < 1 || shapes[2 * i + 1] < 1) return PRM_ERR_SHAPE;
  // Walk order: matrices of one shape together (shape groups in order of first appearance, caller
  // order inside a group), so that a bucket holds matrices that NS5 can batch in one launch.
  std::vector<int> group(n_mats), order(n_mats);
  int n_groups = 0;
  for (int i = 0; i < n_mats; ++i) {
    int gi = -1;
    for (int k = 0; k < i && gi < 0; ++k)
      if (shapes[2 * k] == shapes[2 * i] && shapes[2 * k + 1] == shapes[2 * i + 1]) gi = group[k];
    group[i] = gi < 0 ? n_groups++ : gi;
    order[i] = i;
  }
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return group[a] < group[b]; });
  int bucket = 0;
  int64_t seg = 0;   // elements reserved so far in the current bucket's segment
  for (int k = 0; k < n_mats; ++k) {
    const int i = order[k];
    // chunk rows of every rank, rounded up to 8 elements so that every matrix starts 16-byte aligned
    const int64_t need = round_up(shard_chunk(shapes[2 * i], world) * shapes[2 * i + 1], 8);
    // gathered payload of the bucket: world segments of bf16
    if (seg > 0 && (seg + need) * 2 * world > bucket_bytes) {
      segment_elems[bucket] = seg;
      ++bucket;
      seg = 0;
    }
    bucket_of_mat[i] = bucket;
    offset_in_segment[i] = seg;
    seg += need;
  }
  segment_elems[bucket] = seg;
  *n_buckets = bucket + 1;
  return PRM_OK;
}

extern "C" int prm_pipeline_model(const double* a, const double* c, int n_buckets, double* t_pipe,
                                  double* t_comm_exposed) {
  if (!a || !c || n_buckets < 1) return PRM_ERR_ARG;
  double pipe = a[0], exposed = a[0];
  for (int l = 0; l + 1 < n_buckets; ++l) {
    pipe += std::max(c[l], a[l + 1]);
    exposed += std::max(0.0, a[l + 1] - c[l]);
  }
  pipe += c[n_buckets - 1];
  if (t_pipe) *t_pipe = pipe;
  if (t_comm_exposed) *t_comm_exposed = exposed;
  return PRM_OK;
}

// Whole matrices assigned to ranks (no optimizer collective at all: every
// matrix's update is independent of every other's, Algorithm 1 lines 4-10).
// Longest-processing-time greedy on the refresh cost: matrices in decreasing
// order of the NS5 flop the default schedule executes for them (ties: lower
// index first) go to the rank with the least load so far (ties: lower rank).
// cost_out[q] receives the load of rank q in flop (may be NULL).
extern "C" int prm_partition_matrices(const int64_t* shapes, int n_mats, int world, int* owner_of_mat,
                                      double* cost_out) {
  if (!shapes || n_mats < 1 || world < 1 || !owner_of_mat) return PRM_ERR_ARG;
  std::vector<double> cost(n_mats);
  std::vector<int> order(n_mats);
  for (int i = 0; i < n_mats; ++i) {
    const int64_t m = shapes[2 * i], n = shapes[2 * i + 1];
    if (m < 1 || n < 1) return PRM_ERR_SHAPE;
    cost[i] = ns5_schedule(std::min(m, n), std::max(m, n), 2, std::min(m, n) < kTinyRows).flop;
    order[i] = i;
  }
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return cost[a] > cost[b]; });
  std::vector<double> load(world, 0.0);
  for (int k = 0; k < n_mats; ++k) {
    int best = 0;
    for (int q = 1; q < world; ++q)
      if (load[q] < load[best]) best = q;
    owner_of_mat[order[k]] = best;
    load[best] += cost[order[k]];
  }
  if (cost_out)
    for (int q = 0; q < world; ++q) cost_out[q] = load[q];
  return PRM_OK;
}
