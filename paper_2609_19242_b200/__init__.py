"""BDLM block-diffusion attention (forward, backward, LSE merge) for B200 / sm_100a.

The compute lives in the C-ABI shared library built from `csrc/`; `binding` marshals
PyTorch device pointers into it.  `synth` makes seeded inputs.  Nothing here falls back
to a CPU or library implementation: if the shared library is missing, calls raise.
"""

def __getattr__(name):
    if name in ("bdlm_attn_fwd", "bdlm_attn_bwd", "bdlm_lse_merge", "bdlm_workspace_bytes",
                "bdlm_status_string", "bdlm_get_device_status", "lib", "BdlmError"):
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)
