"""KVReviver hot path for B200: the C-ABI library libkvr.so (hand-written sm_100a kernels) and
its ctypes binding.  `synth` draws the seeded synthetic workloads."""
from .binding import (  # noqa: F401
    KVR_ALL_LAYERS, KVR_BF16, KVR_DECODE_AUTO, KVR_DECODE_STAGED, KVR_DECODE_SPLIT, KVR_SCORE_AUTO, KVR_SCORE_MMA_SYNC, KVR_SCORE_TCGEN05, KVR_F16, KVR_MAX_B, KvrError, Sketch, kvr_compress, kvr_compress_host,
    kvr_accumulate_scores, kvr_accumulate_vague_scores, kvr_swap, kvr_decode_attention, kvr_decode_attention_host, kvr_demote, kvr_decode_attention_static, kvr_get_assignment, kvr_get_cells, kvr_get_scores,
    kvr_launch_count, kvr_measure_pipe_peaks, kvr_append, kvr_append_sizes, kvr_decode_attention_mq, kvr_sketch_set_wait_test, kvr_decode_attention_scored, kvr_layer_shape, kvr_reconstruct, kvr_sketch_create, kvr_sketch_destroy,
    kvr_last_decode_kernel, kvr_last_score_kernel, kvr_sketch_set_score_kernel, kvr_sketch_set_obs_window_causal, kvr_paper_storage_split, kvr_layer_budgets, kvr_sketch_set_combine, KVR_COMBINE_MEDIAN, KVR_COMBINE_MEAN, kvr_sketch_device_bytes, kvr_sketch_device_status, kvr_sketch_reset, kvr_sketch_set_decode_kernel, status_string,
)
