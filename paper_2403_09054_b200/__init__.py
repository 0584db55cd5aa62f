"""B200-native Keyformer score-and-evict path: CUDA kernels behind a C ABI, plus this thin binding."""
from .binding import (Keyformer, KeyformerError, kf_config, make_config, kf_workspace_bytes, kf_strerror,
                      kf_decode_step_static, kf_static_step, KF_STATIC_SCRATCH_BYTES,
                      LIB, LIB_PATH, EXPORTS,
                      KF_OK, KF_EINVAL, KF_ENOSPC, KF_ESTATE, KF_ECUDA, KF_ETIMEOUT, KF_EBOUNDS,
                      KF_NOISE_GUMBEL, KF_NOISE_NONE, KF_NOISE_CONST, KF_NOISE_GAUSS, KF_BIAS_NONE, KF_BIAS_ALIBI, KF_PREFILL_TENSOR, KF_PREFILL_SIMT,
                      KF_POS_ORIGINAL, KF_POS_NEW, KF_DECODE_AUTO, KF_DECODE_CUDA_CORES, KF_DECODE_TENSOR)
