"""B200-native N-way Adasum combine (arXiv 2006.02924): hand-written sm_100a kernels behind a
C-ABI library, with a thin Python binding.

``workloads`` (synthetic inputs) imports without the native library; every compute entry point
lives in ``binding`` and raises if the library has not been built.  ``rvh`` runs the reduce with
one gradient per GPU over a torch.distributed group (recursive vector halving).
"""

_BINDING_NAMES = (
    "adasum_reduce", "adasum_reduce_ex", "adasum_reduce_delta", "adasum_sharded_gram", "adasum_sharded_apply", "adasum_reduce_sharded",
    "adasum_pair", "adasum_pair_noalloc", "adasum_workspace_bytes",
    "adasum_plan_info", "adasum_status_string", "adasum_last_error", "adasum_shutdown",
    "adasum_profile_enable", "adasum_profile_collect", "flags_radix", "AdasumError",
)


def __getattr__(name):
    if name in _BINDING_NAMES or name == "binding":
        import importlib

        binding = importlib.import_module(__name__ + ".binding")
        return binding if name == "binding" else getattr(binding, name)
    raise AttributeError(name)
