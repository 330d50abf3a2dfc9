"""B200-native packed parallel verification for FREE (speculative sampling of Diffusion Transformers).

Thin Python binding over the C-ABI library `libfree_b200.so` (hand-written sm_100a CUDA).  Every
numerical step runs in that library; this package only marshals arguments.  PyTorch is used for device
memory and streams.  There is no CPU fallback: using any operation without the built library raises.
"""
from .schedule import linear_schedule, respaced_schedule        # noqa: F401


def __getattr__(name):
    # the binding loads the shared library on first use, so that `python -m paper_2511_20390_b200.build`
    # can run before the library exists
    if name in ("spec_verify", "spec_verify_fused", "spec_verify_host", "fit_lambda_profile", "drafter_loss", "Model", "DeviceSchedule", "lib", "FreeError",
                "op_linear", "op_ln_modulate", "op_attention", "selftest_bounded_wait", "split_range", "LIB_PATH"):
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)
