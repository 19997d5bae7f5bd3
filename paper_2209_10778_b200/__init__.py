"""Nested Forward-AD activation pass for B200 (sm_100a).

``binding`` mirrors the C interface of ``libnfad.so`` (see ``include/nfad.h``);
``workloads`` draws the seeded synthetic inputs; ``build`` compiles the library.
"""
from . import workloads  # noqa: F401
from .binding import (  # noqa: F401
    DTYPES, KINDS, LAYOUTS, NfadError, load,
    nfad_act_backward, nfad_act_forward, nfad_act_forward_infer, nfad_act_forward_strict,
    nfad_bias_act_backward, nfad_bias_act_backward_scratch_bytes, nfad_bias_act_forward, nfad_bias_act_forward_infer,
    nfad_cmp_conv_backward, nfad_cmp_recompute_backward, nfad_cmp_recompute_backward_noalloc,
    nfad_cmp_recompute_scratch_bytes,
    nfad_ew_op, nfad_host_step, nfad_host_step_workspace_bytes, nfad_probe_stream, nfad_saved_bytes_per_element, nfad_seq_backward, nfad_seq_forward,
    nfad_status_string, nfad_version,
)
