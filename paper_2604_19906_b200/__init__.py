"""B200-native batched spectral-element tensor-product operators (see ``ops``)."""
