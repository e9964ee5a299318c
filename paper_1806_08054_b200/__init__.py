"""B200-native ECQ-SGD gradient codec: fused encode and decode-mean kernels.

``binding`` exposes the C ABI of ``include/ecq.h`` under the same names;
``workloads`` makes the seeded synthetic gradients; ``build`` compiles the
library in-tree for sm_100a.
"""
from . import workloads  # noqa: F401
from .binding import (  # noqa: F401
    ECQ_ERR_ARG, ECQ_ERR_NONFINITE, ECQ_ERR_TIMEOUT, ECQ_OK, EcqError, ecq_code_bits, ecq_code_histogram, ecq_entropy_bound_bits,
    ecq_codes_words, ecq_create, ecq_decode_mean, ecq_decode_mean_update, ecq_destroy, ecq_encode, ecq_encode_batch,
    ecq_launch_count, pointer_table, PointerTable,
    ecq_num_buckets, ecq_set_decode_plan, ecq_set_error_mode, ecq_set_norm, ecq_set_wait_limit, ECQ_WAIT_LIMIT_DEFAULT,
    ECQ_DECODE_AUTO, ECQ_DECODE_RING, ECQ_DECODE_WARP, ecq_status, ecq_step_host, ecq_step_static,
    ecq_step_host_workspace_bytes,
    ECQ_ERR_CAPACITY, ECQ_ERR_SYMBOL, ECQ_HUFFMAN_TABLE_BYTES, ecq_huffman_chunks, ecq_huffman_decode,
    ecq_huffman_encode, ecq_huffman_lengths, ecq_huffman_stream_bound, ecq_huffman_tables,
)
