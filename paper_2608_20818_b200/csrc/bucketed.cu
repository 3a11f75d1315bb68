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
  int bucket = 0;
  int64_t seg = 0;   // elements reserved so far in the current bucket's segment
  for (int i = 0; i < n_mats; ++i) {
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
