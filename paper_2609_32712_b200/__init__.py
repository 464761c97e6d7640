"""B200-native MassAlloc Attention (MALA) hot path: C-ABI library ``libmala.so`` + thin binding.

``paper_2609_32712_b200.mala``      -- ctypes binding of the C ABI declared in ``include/mala.h``
``paper_2609_32712_b200.autograd``  -- ``mala_attention``: the forward / backward pair as a ``torch.autograd`` function
``paper_2609_32712_b200.workloads`` -- seeded synthetic input generators (no method arithmetic)
"""
__version__ = "0.1.0"
